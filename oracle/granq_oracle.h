/*
 * GranQ channel-wise activation fake-quantization: CPU oracle (TEST INFRASTRUCTURE).
 *
 * A plain, slow, single-threaded restatement of the paper's definitions, used only
 * to check the CUDA library and to serve as the timed CPU baseline.  It shares no
 * code with the CUDA path and must never be called from the product path.
 *
 * What it computes, group by group and element by element, in IEEE fp32 with
 * round-to-nearest-even and no fused multiply-add:
 *   activation decomposition + per-group range .......... Eq. 4, Algorithm 1 (range step)
 *   scale and zero-point ................................ Eq. 2 / Eq. 5
 *   integer mapping  x_q = round(x / s + z) ............. Eq. 1, Algorithm 1 (quantize step)
 *   dequantize / pre-scale  s * (x_q - z) ............... Eq. 6, Algorithm 1 (pre-scale step)
 *   straight-through-estimator backward ................. Section 2.1 (named only)
 *
 * Readings taken where the paper is silent (all listed again in the design notes):
 *   - rounding is round-half-to-even;
 *   - the rounded value is clamped to [0, 2^b - 1] before dequantization;
 *   - a degenerate range is floored: s = max(s, 1e-8);
 *   - the backward mask is 1 exactly where the clamp was inactive;
 *   - with a batch axis, one group is one channel over (n, h, w) (GROUP_CHANNEL);
 *     the per-sample reading of Eq. 4 is GROUP_SAMPLE_CHANNEL; the layer-wise
 *     baseline is GROUP_TENSOR.
 *
 * Every function is pinned by tests that do not call the oracle to produce the
 * expected value (hand-worked cases, closed forms, exact rational arithmetic,
 * invariants): no part is "parity unpinned".
 *
 * All pointers are host memory.  Tensors are contiguous row-major dims[4].
 * dtype 0 = fp32 (float), 1 = bf16 (uint16_t bit patterns, widened exactly on
 * read, narrowed round-to-nearest-even on write).
 */
#ifndef GRANQ_ORACLE_H
#define GRANQ_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { GRANQ_ORACLE_F32 = 0, GRANQ_ORACLE_BF16 = 1 };
enum { GRANQ_ORACLE_GROUP_CHANNEL = 0, GRANQ_ORACLE_GROUP_SAMPLE_CHANNEL = 1, GRANQ_ORACLE_GROUP_TENSOR = 2 };

/* Number of groups G for the given geometry; -1 on invalid arguments. */
int64_t granq_oracle_num_groups(const int64_t dims[4], int channel_axis, int group_mode);

/* Eq. 4: lo[g] = min, hi[g] = max over the members of group g (-0 canonicalised to +0).
 * Returns 0, or -1 on invalid arguments, or -2 if a non-finite input is met. */
int granq_oracle_range(const void* x, int dtype, const int64_t dims[4], int channel_axis,
                       int group_mode, float* lo, float* hi);

/* Eq. 2 / Eq. 5 for G groups. */
int granq_oracle_params(const float* lo, const float* hi, int64_t G, int bits, float* s, float* z);

/* Eq. 1 + clamp + Eq. 6 + STE mask with a GIVEN range (lo, hi per group).
 * gy/gx may both be NULL (forward only); codes, mask, s, z may be NULL. */
int granq_oracle_fakequant(const void* x, const void* gy, int dtype, const int64_t dims[4],
                           int channel_axis, int group_mode, int bits,
                           const float* lo, const float* hi,
                           void* y, void* gx, uint8_t* codes, uint8_t* mask, float* s, float* z);

/* Range from the tensor itself, then fakequant: the whole hot path. lo/hi are outputs. */
int granq_oracle_fused(const void* x, const void* gy, int dtype, const int64_t dims[4],
                       int channel_axis, int group_mode, int bits,
                       void* y, void* gx, float* lo, float* hi,
                       uint8_t* codes, uint8_t* mask, float* s, float* z);

/* Mask-carrying split of forward and backward (Section 2.1: the straight-through estimator
 * needs nothing of the forward pass but the mask).  The forward pass stores its STE mask
 * at one bit per element: bit e % 8 (least significant first) of byte e / 8, ceil(E / 8)
 * bytes, unused high bits of the last byte 0.  The backward pass then reads gy and the
 * packed mask instead of gy and x. */
int granq_oracle_pack_mask(const uint8_t* mask, int64_t E, uint8_t* packed);
int granq_oracle_bwd_packed(const void* gy, const uint8_t* packed, int dtype, int64_t E, void* gx);

/* Distortion statistics of a quantization, the quantities of Table 2 (Section 4.1): with X the
 * activations and Q their fake-quantized values, sums = { sum X^2, sum Q^2, sum X*Q, sum (X-Q)^2 }
 * in fp64, and from them the cosine similarity X.Q / (|X|_2 |Q|_2) and the relative error
 * |X - Q|_2 / |X|_2 (0 where a denominator vanishes). */
int granq_oracle_distortion_sums(const void* x, const void* q, int dtype, int64_t E, double sums[4]);
int granq_oracle_distortion(const double sums[4], double* cosine, double* rel_error);

/* Integer codes as a packed bit string: Eq. 1 yields b-bit integers, and it is those (with the
 * per-group scale and zero-point) that Eq. 6 and the accumulation of Algorithm 1 consume.  Element e
 * occupies bits [e*b, (e+1)*b) of a little-endian bit string of ceil(E*b / 8) bytes.
 * granq_oracle_dequant_packed() is Eq. 6 evaluated from that string: y = s * (code - z). */
int granq_oracle_pack_codes(const uint8_t* codes, int64_t E, int bits, uint8_t* packed);
int granq_oracle_dequant_packed(const uint8_t* packed, int dtype, const int64_t dims[4], int channel_axis,
                                int group_mode, int bits, const float* s, const float* z, void* y);

/* The accumulation over the pre-scaled activations, pointwise (1 x 1) case: Eq. 6 left-hand side and the
 * output step of Algorithm 1, y[n][o][p] = sum_c w[o][c] * A~[n][c][p] with A~ = s_c * (code - z_c) formed
 * first in fp32 (the pre-scale step), the sum in fp64 with c ascending.  dims = {N, C, P}; codes are
 * [N, C, P] (channels_last = 0) or [N, P, C] (1); y is [N, O, P] or [N, P, O].  The _inloop form is Eq. 3,
 * the conventional order with the scale inside the loop, all in fp64: the same real number. */
int granq_oracle_accumulate(const uint8_t* codes, const int64_t dims[3], int channels_last, const float* s,
                            const float* z, const float* w, int64_t O, double* y);
int granq_oracle_accumulate_inloop(const uint8_t* codes, const int64_t dims[3], int channels_last, const float* s,
                                   const float* z, const float* w, int64_t O, double* y);

#ifdef __cplusplus
}
#endif
#endif
