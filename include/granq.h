/*
 * granq.h - C ABI of the GranQ channel-wise activation fake-quantization library
 * for NVIDIA B200 (sm_100a).
 *
 * The library implements one data-parallel path of GranQ (arXiv 2503.18339):
 *   1. activation decomposition and per-group range ............ Eq. 4, Algorithm 1 (range step)
 *   2. scale and zero-point for b bits ........................... Eq. 2 / Eq. 5
 *   3. quantize -> clamp -> dequantize ("pre-scaling") ........... Eq. 1, Eq. 6, Algorithm 1
 *   4. straight-through-estimator backward ....................... Section 2.1
 * and, built on the same arithmetic: the forward / backward split that carries a 1-bit mask,
 * the distortion statistics of Table 2, all weight tensors of a model in one launch
 * (Section 5.1) and the integer codes as a packed bit string.
 *
 * Arithmetic (identical for every entry point), per group g with members x_i, in IEEE
 * fp32, round-to-nearest-even, no fused multiply-add:
 *     lo = min x_i, hi = max x_i                 (-0 reported as +0)
 *     s  = max((hi - lo) / (2^b - 1), 1e-8)      z = round(-lo / s)
 *     r  = round(x_i / s + z)                    code = clamp(r, 0, 2^b - 1)
 *     y_i  = s * (code - z)                      mask_i = (0 <= r <= 2^b - 1)
 *     gx_i = mask_i ? gy_i : 0
 * round() is round-half-to-even.  The clamp, the 1e-8 floor, the tie rule and the mask
 * are this library's reading of points the paper leaves open.
 *
 * Tensors.  Contiguous row-major dims[4] (NCHW for activations), element type fp32 or
 * bf16.  `channel_axis` (0..3) selects the channel dimension; with outer = product of the
 * dims before it, C = dims[channel_axis], inner = product of the dims after it:
 *     GRANQ_GROUP_CHANNEL        one group per channel, reduced over everything else
 *                                (batch included: "per channel at the batch level") G = C
 *     GRANQ_GROUP_SAMPLE_CHANNEL Eq. 4 applied to each sample: G = outer * C, group index
 *                                o * C + c
 *     GRANQ_GROUP_TENSOR         layer-wise baseline: G = 1
 * bf16 inputs are widened exactly, all arithmetic is fp32, y / gx are narrowed with
 * round-to-nearest-even; lo, hi, s, z are always fp32.
 *
 * Memory.  Unless a parameter is documented as HOST memory, every pointer is DEVICE
 * memory owned by the caller, valid until the stream has passed the call.  The library
 * never allocates or frees device memory and keeps no results between calls; scratch comes
 * from the caller's `workspace` (at least granq_workspace_bytes(), 256-byte aligned,
 * contents irrelevant on entry unless GRANQ_FLAG_WORKSPACE_ZEROED says otherwise, overwritten by
 * the call).  Outputs must not overlap
 * inputs.  Inputs must be finite (NaN / Inf give unspecified results, never a fault).
 *
 * Execution.  All work is enqueued on `cuda_stream` (a cudaStream_t passed as void*;
 * NULL = the default stream); no entry point synchronises with the host except
 * granq_fakequant_fused_host() (unless GRANQ_FLAG_HOST_ASYNC), granq_host_arena_status(),
 * granq_workspace_status() and granq_fakequant_weights() (which reads its host descriptor
 * array before it returns).  Results are bit-identical from run to run, except the last bits
 * of the distortion sums, whose fp64 atomics arrive in no fixed order.  The library keeps no
 * results and no per-call state; the only process-wide state is (a) the planner overrides set with
 * granq_tune() (all zero unless a test or a tuning run sets them; they never change results),
 * (b) memoised answers of pure functions of (geometry, device): occupancy per kernel and device,
 * the column-walk planner's wave cut, the device address of granq_range_noalloc()'s array.
 *
 * Errors.  Every function returning int returns a granq_status code.  Argument errors
 * (null required pointer, bits outside 1..8, non-positive dim, more than 2^40 elements,
 * bad enum, workspace too small or misaligned) are detected on the host before anything
 * is launched and leave all outputs untouched.  CUDA launch errors are returned as
 * GRANQ_ERR_CUDA.  The persistent plans of granq_fakequant_fused() contain bounded
 * device-side waits; should one run out (it cannot unless the GPU is preempted for
 * seconds) the kernel stops, outputs are unspecified, and granq_workspace_status()
 * reports GRANQ_ERR_TIMEOUT.
 */
#ifndef GRANQ_H
#define GRANQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum granq_status {
    GRANQ_OK = 0,
    GRANQ_ERR_INVALID_ARG = 1,
    GRANQ_ERR_UNSUPPORTED = 2,
    GRANQ_ERR_WORKSPACE = 3,
    GRANQ_ERR_CUDA = 4,
    GRANQ_ERR_TIMEOUT = 5
};

enum granq_dtype { GRANQ_F32 = 0, GRANQ_BF16 = 1 };

enum granq_group { GRANQ_GROUP_CHANNEL = 0, GRANQ_GROUP_SAMPLE_CHANNEL = 1, GRANQ_GROUP_TENSOR = 2 };

/* flags (bitwise or).  The plan-forcing flags exist so that every execution plan can be
 * checked and measured on the same input; results do not depend on the plan. */
enum granq_flags {
    GRANQ_FLAG_NONE = 0,
    GRANQ_FLAG_FORCE_TWO_PASS = 1u,  /* fused: range launch + quantize launch (x is read twice)      */
    GRANQ_FLAG_FORCE_NAIVE = 2u,     /* fused: host loop over channels, three launches per channel -
                                        the "conventional" scalar-loop scheme of Section 5.3.2       */
    GRANQ_FLAG_FORCE_STAGED = 4u,    /* fused: on-chip-staged persistent kernel or GRANQ_ERR_UNSUPPORTED */
    GRANQ_FLAG_FORCE_L2WAVE = 8u,    /* fused: L2-resident-wave persistent kernel or GRANQ_ERR_UNSUPPORTED */
    GRANQ_FLAG_FORCE_COLWALK = 16u,  /* fused: column-walk persistent kernel or GRANQ_ERR_UNSUPPORTED     */
    GRANQ_FLAG_WORKSPACE_ZEROED = 32u, /* fused: the caller guarantees that the whole workspace is zero on
                                        entry (cleared after allocation, or left by an earlier call with
                                        this flag that ended with status GRANQ_OK); the call then skips
                                        its own clearing step and leaves the workspace zero again on
                                        success.  After GRANQ_ERR_TIMEOUT clear it before the next use. */
    GRANQ_FLAG_HOST_ASYNC = 64u,      /* granq_fakequant_fused_host(): enqueue only, do not wait for the stream
                                        (host outputs are valid once the stream has passed the call; ask
                                        granq_host_arena_status() then).  Lets calls on two streams with two
                                        arenas overlap one call's uploads with the other's downloads.       */
    GRANQ_FLAG_FORCE_CLUSTER = 128u   /* fused: cluster-local kernel (a run of channels staged once in the shared
                                        memory of one thread-block cluster) or GRANQ_ERR_UNSUPPORTED        */
};

/* Human-readable name of a status code (static storage, never NULL). */
const char* granq_status_string(int status);

/* Number of groups G for a geometry, or -1 if the arguments are invalid. */
int64_t granq_num_groups(const int64_t dims[4], int channel_axis, int group);

/* Bytes of scratch every entry point that takes a workspace needs for this geometry
 * (0 if the arguments are invalid). */
size_t granq_workspace_bytes(int dtype, const int64_t dims[4], int channel_axis, int group);

/*
 * Eq. 4 / Algorithm 1 (range step): min_out[g], max_out[g] for g in [0, G).
 *   x          in   E elements of `dtype`
 *   min_out    out  G floats        max_out   out  G floats
 */
int granq_range(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group,
                float* min_out, float* max_out,
                void* workspace, size_t workspace_bytes, uint32_t flags, void* cuda_stream);

/*
 * granq_range() without a workspace (the paper has no counterpart: this exists for callers,
 * not for the method).  Some callers cannot allocate device memory where they need the range:
 * code running inside a framework's allocator callback or out-of-memory handler, a plugin that
 * is handed nothing but its input and output buffers, a latency-critical loop that must stay
 * out of the driver's allocator.  For them the min/max scratch is an array inside the library
 * itself, so the call allocates and frees nothing (no cudaMalloc / cudaFree, no allocating
 * library routine).
 *   - Limit: at most GRANQ_NOALLOC_MAX_GROUPS groups; more gives GRANQ_ERR_UNSUPPORTED and
 *     nothing is launched.  The array (256 KB) is resident on every GPU that loads the library,
 *     until the process exits.
 *   - The first call on a device looks up the array's device address (with that device
 *     current); make that first call before starting any stream capture.
 *   - Every call uses the same array: calls that overlap on the GPU (two streams, two host
 *     threads) race with each other.  Calls issued on one stream are safe; the array is
 *     cleared at the start of each call.
 * Arguments and results are those of granq_range() (x, min_out, max_out in DEVICE memory).
 */
#define GRANQ_NOALLOC_MAX_GROUPS 32768
int granq_range_noalloc(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group,
                        float* min_out, float* max_out, void* cuda_stream);

/*
 * Eq. 1 + clamp + Eq. 6 with a range supplied by the caller (for instance one measured on
 * another batch): y = s * (clamp(round(x / s + z)) - z), with s, z from Eq. 2 / Eq. 5.
 *   min_in, max_in  in   G floats each
 *   y               out  E elements of `dtype`
 *   codes_opt       out  E bytes, the integer codes (NULL to skip)
 *   scale_opt, zp_opt out G floats each (NULL to skip)
 */
int granq_fakequant_fwd(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group,
                        int bits, const float* min_in, const float* max_in,
                        void* y, uint8_t* codes_opt, float* scale_opt, float* zp_opt,
                        uint32_t flags, void* cuda_stream);

/*
 * Straight-through-estimator backward (Section 2.1): gx = gy where the forward clamp was
 * inactive for x, else 0.  The range, scale and zero-point are treated as constants.
 *   gy, x      in   E elements each       gx   out  E elements
 *   mask_opt   out  E bytes of 0/1 (NULL to skip)
 */
int granq_fakequant_bwd(const void* gy, const void* x, int dtype, const int64_t dims[4], int channel_axis,
                        int group, int bits, const float* min_in, const float* max_in,
                        void* gx, uint8_t* mask_opt, uint32_t flags, void* cuda_stream);

/*
 * The whole path in one call (Algorithm 1, range step through pre-scale step, plus the
 * backward): range of x itself -> scale / zero-point -> y, and gx when gy_opt is given.
 * The default plan stages a run of adjacent channels once in the shared memory of one thread-block
 * cluster where their group fits (x is then read from HBM exactly once); larger groups are processed
 * in waves of channel groups that stay in the L2 cache between the range pass and the quantize pass, so
 * x is read from HBM (about) once; channels-last geometries (channel_axis = 3, or planes of one element)
 * take a range launch and a quantize launch with one 16-byte unit column per thread.
 *   x                 in   E elements          gy_opt   in   E elements or NULL (forward only)
 *   y                 out  E elements          gx_opt   out  E elements (required iff gy_opt)
 *   min_out, max_out  out  G floats each (required)
 *   codes_opt, mask_opt    E bytes each or NULL;  scale_opt, zp_opt  G floats each or NULL
 */
int granq_fakequant_fused(const void* x, const void* gy_opt, int dtype, const int64_t dims[4],
                          int channel_axis, int group, int bits,
                          void* y, void* gx_opt, float* min_out, float* max_out,
                          uint8_t* codes_opt, uint8_t* mask_opt, float* scale_opt, float* zp_opt,
                          void* workspace, size_t workspace_bytes, uint32_t flags, void* cuda_stream);

/*
 * Mask-carrying split of forward and backward (Section 2.1: the straight-through estimator
 * needs nothing of the forward pass but where the clamp was inactive).  In training the
 * upstream gradient does not exist yet when the forward pass runs, so the forward pass
 * stores its mask at ONE BIT per element and the backward pass reads gy and that mask
 * instead of gy and x: 8.125 instead of 12 bytes per fp32 element.
 *
 * Packed mask layout: bit e % 32 of the 32-bit word e / 32 (on this little-endian target the
 * same as bit e % 8 of byte e / 8) is 1 iff 0 <= round(x_e / s + z) <= 2^b - 1.  The buffer
 * holds granq_packmask_bytes() = 4 * ceil(E / 32) bytes, 4-byte aligned, DEVICE memory; bits
 * beyond element E - 1 are written as 0.
 */
size_t granq_packmask_bytes(const int64_t dims[4]);

/* Eq. 1 + clamp + Eq. 6 with a supplied range, as granq_fakequant_fwd(), also writing the packed mask.
 *   x in E elements;  y out E elements;  packed_mask out;  scale_opt, zp_opt G floats or NULL */
int granq_fakequant_fwd_packmask(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group,
                                 int bits, const float* min_in, const float* max_in, void* y,
                                 uint32_t* packed_mask, float* scale_opt, float* zp_opt, uint32_t flags,
                                 void* cuda_stream);

/* STE backward from the packed mask alone: gx_e = gy_e where bit e is set, else +0.  Needs neither x
 * nor the range, hence no channel axis or grouping.
 *   gy in E elements;  packed_mask in;  gx out E elements (must not overlap gy) */
int granq_fakequant_bwd_packmask(const void* gy, const uint32_t* packed_mask, int dtype, const int64_t dims[4],
                                 void* gx, uint32_t flags, void* cuda_stream);

/* The forward half of the whole path in one call (Algorithm 1, range step through pre-scale step):
 * range of x itself -> scale / zero-point -> y and the packed mask.  Takes the cluster-local plan
 * where a run of channels that is whole bytes of mask fits one cluster, the column-walk plan when slabs
 * and waves are whole mask words, else a range pass followed by an elementwise pass
 * (GRANQ_FLAG_FORCE_TWO_PASS / GRANQ_FLAG_FORCE_COLWALK / GRANQ_FLAG_FORCE_CLUSTER select one;
 * GRANQ_FLAG_WORKSPACE_ZEROED as for granq_fakequant_fused()).
 *   min_out, max_out out G floats each (required);  scale_opt, zp_opt G floats or NULL */
int granq_fakequant_fused_fwd_packmask(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group,
                                       int bits, void* y, uint32_t* packed_mask, float* min_out, float* max_out,
                                       float* scale_opt, float* zp_opt, void* workspace, size_t workspace_bytes,
                                       uint32_t flags, void* cuda_stream);

/*
 * Distortion statistics of a quantization (Section 4.1, Table 2).  With X the activations and Q
 * their fake-quantized values the table reports the cosine similarity X.Q / (|X|_2 |Q|_2) and the
 * relative error |X - Q|_2 / |X|_2; both follow from four sums over all elements,
 *   sums_out = { sum X^2, sum Q^2, sum X*Q, sum (X-Q)^2 }      (4 doubles, DEVICE memory, 8-byte aligned)
 * which these calls write (they clear them first).  The terms of one 16-byte pack are summed in
 * fp32, everything else in fp64.
 *
 * granq_distortion():            the sums for an existing pair (x, q) of E elements each.
 * granq_fakequant_fused_stats(): the forward half of the whole path (range of x itself -> scale /
 *     zero-point -> y) that gathers the sums in the pass that writes y, for any grouping - so the
 *     layer-wise baseline (GRANQ_GROUP_TENSOR) and the channel-wise method can be compared on the
 *     same tensor as in Table 2.  Plans and flags as granq_fakequant_fused_fwd_packmask().
 */
int granq_distortion(const void* x, const void* q, int dtype, const int64_t dims[4], double* sums_out,
                     uint32_t flags, void* cuda_stream);
/* Host-only: Table 2's two statistics from the four sums (HOST memory, as copied back from sums_out):
 *   cosine = sum X*Q / (sqrt(sum X^2) * sqrt(sum Q^2)),   rel_error = sqrt(sum (X-Q)^2) / sqrt(sum X^2),
 * each 0 when its denominator is 0.  cosine_out / rel_error_out may be NULL. */
int granq_distortion_stats(const double sums[4], double* cosine_out, double* rel_error_out);
int granq_fakequant_fused_stats(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group,
                                int bits, void* y, float* min_out, float* max_out, float* scale_opt, float* zp_opt,
                                double* sums_out, void* workspace, size_t workspace_bytes, uint32_t flags,
                                void* cuda_stream);

/*
 * Channel-wise fake-quantization of many weight tensors in ONE launch (Section 5.1: all weights are
 * quantized per output channel; Eq. 1, 2, 4-6 per channel, STE backward when a gradient is given).
 * Tensor i is a contiguous [channels, group_elems] array of `dtype` (for a convolution weight
 * [C_out, C_in, k, k]: channels = C_out, group_elems = C_in * k * k); each leading index is one
 * group.  Results are those of granq_fakequant_fused() with channel_axis = 0 on every tensor.
 *   descs       HOST array of n_tensors descriptors (read before the call returns); the pointers
 *               inside are DEVICE memory: x in, y out, gy_opt / gx_opt both or neither,
 *               min_out / max_out `channels` floats each (required), scale_opt / zp_opt or NULL
 *   workspace   DEVICE scratch of granq_weights_workspace_bytes(n_tensors), 256-byte aligned
 * Limits: fewer than 2^31 groups in the batch and 2^31 elements per group.  The call stages the
 * descriptors through host memory it owns only until it returns, so it cannot be recorded into a CUDA
 * graph: on a capturing stream it returns GRANQ_ERR_UNSUPPORTED and enqueues nothing.
 */
typedef struct granq_weight_desc {
    const void* x;
    const void* gy_opt;
    void* y;
    void* gx_opt;
    float* min_out;
    float* max_out;
    float* scale_opt;
    float* zp_opt;
    int64_t channels;
    int64_t group_elems;
    int32_t bits;
    int32_t reserved;
} granq_weight_desc;
size_t granq_weights_workspace_bytes(int n_tensors);
int granq_fakequant_weights(const granq_weight_desc* descs, int n_tensors, int dtype, void* workspace,
                            size_t workspace_bytes, uint32_t flags, void* cuda_stream);

/*
 * The fused call (Algorithm 1, range step through pre-scale step, + STE backward) for a LIST of activation
 * tensors in one host call: a layer stack's tensors of one training step (the ResNet-20 mix has 19 of 1-17 MB
 * each, where the host's per-call cost, not the GPU, sets the pace).  Tensor i is processed exactly as
 * granq_fakequant_fused(descs[i].x, descs[i].gy_opt, dtype, descs[i].dims, channel_axis, group, descs[i].bits,
 * ..., NULL codes, NULL mask, ..., flags, cuda_stream) would, in order, on the same stream; the results are
 * bit for bit those of the single calls.
 *   descs       HOST array of n_tensors descriptors; pointers inside are DEVICE memory, owned by the caller;
 *               every tensor has its own workspace of granq_workspace_bytes() (they may not share one: the
 *               kernels of consecutive tensors overlap on the GPU)
 *   failed_opt  HOST int or NULL: receives the index of the tensor whose call failed (-1 if none)
 * Returns the first non-OK status; the tensors before the failing one have been enqueued, none after it.
 */
typedef struct granq_fused_desc {
    const void* x;
    const void* gy_opt;
    void* y;
    void* gx_opt;
    float* min_out;
    float* max_out;
    float* scale_opt;
    float* zp_opt;
    void* workspace;
    size_t workspace_bytes;
    int64_t dims[4];
    int32_t bits;
    int32_t reserved;
} granq_fused_desc;
int granq_fakequant_fused_batch(const granq_fused_desc* descs, int n_tensors, int dtype, int channel_axis, int group,
                                uint32_t flags, void* cuda_stream, int* failed_opt);

/*
 * Integer codes as a packed bit string (Eq. 1 yields b-bit integers; Eq. 6 and the accumulation of
 * Algorithm 1 consume them together with the per-group scale and zero-point).  Element e occupies bits
 * [e*b, (e+1)*b) of a little-endian bit string (bit k of the string = bit k % 32 of word k / 32);
 * the buffer holds granq_packed_codes_bytes() = 4 * ceil(E*b / 32) bytes, 4-byte aligned, DEVICE memory;
 * bits beyond the last element are written as 0.  An activation kept this way takes b/32 of its fp32 size.
 *
 * granq_quantize_packed():   Eq. 1 + clamp with a supplied range -> packed codes, scale and zero-point
 *                            (both required: they are what gives the codes a meaning); y_opt, when not
 *                            NULL, also receives the dequantized values as granq_fakequant_fwd() would.
 * granq_dequantize_packed(): Eq. 6, y = s * (code - z), from the packed codes; bit for bit the y of
 *                            granq_fakequant_fwd() for the same range.
 * granq_quantize_packed_fused(): the producer of the integer pipeline in one call (Algorithm 1, range step
 *                            through quantize step): range of x itself -> scale / zero-point -> packed codes; x is
 *                            read from HBM once where a single-read plan fits (cluster-local kernel, column
 *                            walk: groups of 8 codes must not straddle slabs and the tensor is a multiple of 32
 *                            elements), else a range pass, the parameters and an elementwise pass.  The codes
 *                            are bit for bit those of granq_range() + granq_quantize_packed().  workspace and
 *                            flags (GRANQ_FLAG_WORKSPACE_ZEROED, GRANQ_FLAG_FORCE_TWO_PASS / _COLWALK / _CLUSTER) as
 *                            for granq_fakequant_fused().
 */
size_t granq_packed_codes_bytes(const int64_t dims[4], int bits);
int granq_quantize_packed(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group, int bits,
                          const float* min_in, const float* max_in, uint32_t* packed_codes, void* y_opt,
                          float* scale_out, float* zp_out, uint32_t flags, void* cuda_stream);
int granq_dequantize_packed(const uint32_t* packed_codes, int dtype, const int64_t dims[4], int channel_axis,
                            int group, int bits, const float* scale_in, const float* zp_in, void* y, uint32_t flags,
                            void* cuda_stream);
int granq_quantize_packed_fused(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group, int bits,
                                uint32_t* packed_codes, float* min_out, float* max_out, float* scale_out, float* zp_out,
                                void* workspace, size_t workspace_bytes, uint32_t flags, void* cuda_stream);

/*
 * The accumulation over the integer codes, pointwise (1 x 1) case: Eq. 6 left-hand side and the output
 * step of Algorithm 1 (Eq. 3 is the order the paper contrasts it with),
 *     y[n][o][p] = sum_c w[o][c] * s_c * (code[n][c][p] - z_c)
 * evaluated as  sum_c (w[o][c] * s_c) * code  -  sum_c (w[o][c] * s_c) * z_c : the scale is folded into the
 * weights once, the sum runs over the integer codes on the tensor cores (bf16 operands - the codes are exact,
 * the scaled weights are split into two bf16 halves - with fp32 accumulation), the zero-points become one
 * bias per output channel.
 *   packed_codes  in   the codes as written by granq_quantize_packed() for a tensor of `dims`
 *                      (channel_axis 1: NCHW;  channel_axis 3: channels-last, N H W C), GRANQ_GROUP_CHANNEL
 *   scale, zp     in   C floats each (per-channel, as written by granq_quantize_packed())
 *   weights       in   fp32 [out_channels, C], row-major
 *   y             out  fp32, [N, out_channels, H, W] for channel_axis 1, [N, H, W, out_channels] for 3
 *   workspace          DEVICE scratch of granq_accumulate_workspace_bytes() (the two weight halves and the bias:
 *                      the codes are expanded to bf16 inside the contraction kernel and never exist as a matrix
 *                      in device memory), 256-byte aligned; its first word is a status word as described at
 *                      granq_workspace_status()
 *   flags              0, or GRANQ_FLAG_FORCE_TWO_PASS for the kernel with one pixel tile per CTA instead of the
 *                      persistent one (which is taken whenever the weight halves of all channels fit in shared
 *                      memory, and holds all of an SM's tensor memory while it runs)
 * Two launches on `cuda_stream` (weights, then expansion + contraction + epilogue) after a 4-byte clear of the
 * status word.
 * Result: within (2^-17 + C * 2^-22) * sum_c |w s_c| (code + |z_c|) + 2^-21 * (|bias| + |y|) of the exact sum
 * (the split of the scaled weights, fp32 accumulation of the C products of each half in any order, the sum of
 * the two halves, one rounding each of bias and y).
 * Limits: fewer than 2^31 pixels in the batch, C < 2^20, out_channels < 2^24; otherwise GRANQ_ERR_INVALID_ARG.
 */
size_t granq_accumulate_workspace_bytes(const int64_t dims[4], int channel_axis, int64_t out_channels);
int granq_accumulate_codes(const uint32_t* packed_codes, const int64_t dims[4], int channel_axis, int bits,
                           const float* scale, const float* zp, const float* weights, int64_t out_channels,
                           float* y, void* workspace, size_t workspace_bytes, uint32_t flags, void* cuda_stream);

/*
 * Status word the persistent plans leave in the workspace.  Synchronises `cuda_stream`, then
 * returns GRANQ_OK, GRANQ_ERR_TIMEOUT (a bounded device-side wait ran out), or
 * GRANQ_ERR_CUDA.  `workspace` is the pointer given to the preceding call.
 */
int granq_workspace_status(const void* workspace, void* cuda_stream);

/* Bytes of device memory granq_fakequant_fused_host() needs as its arena. */
size_t granq_host_arena_bytes(int dtype, const int64_t dims[4], int channel_axis, int group, int with_backward);

/*
 * granq_fakequant_fused() for tensors that live in HOST memory (pinned memory makes the
 * copies asynchronous and fast; pageable memory works).  x_host / gy_host_opt are copied
 * into `device_arena`, the fused path runs there, and y / gx / min / max (and scale / zp
 * when asked for) are copied back; the call returns after `cuda_stream` has drained, so
 * the host outputs are valid on return.
 *   x_host, gy_host_opt, y_host, gx_host_opt, min_host, max_host, scale_host_opt,
 *   zp_host_opt          HOST memory, sizes as for granq_fakequant_fused()
 *   device_arena         DEVICE memory, 256-byte aligned, >= granq_host_arena_bytes()
 */
int granq_fakequant_fused_host(const void* x_host, const void* gy_host_opt, int dtype, const int64_t dims[4],
                               int channel_axis, int group, int bits,
                               void* y_host, void* gx_host_opt, float* min_host, float* max_host,
                               float* scale_host_opt, float* zp_host_opt,
                               void* device_arena, size_t arena_bytes, uint32_t flags, void* cuda_stream);

/* For calls made with GRANQ_FLAG_HOST_ASYNC: synchronises `cuda_stream`, then reports the status word of
 * the workspace inside `device_arena` (same geometry arguments as the call), as granq_workspace_status(). */
int granq_host_arena_status(int dtype, const int64_t dims[4], int channel_axis, int group, int with_backward,
                            const void* device_arena, void* cuda_stream);

/*
 * Plan that granq_fakequant_fused() would take for this geometry and flags on the current
 * device: 0 = two-pass, 1 = naive per-channel loop, 2 = on-chip staged, 3 = L2-resident waves,
 * 4 = column walk, 5 = cluster-local, 6 = channels-last rows (range launch + quantize launch with one
 * 16-byte unit column per thread); negative = -status.
 * `launches_out` (HOST, may be NULL) receives the number of kernel launches of that plan.
 */
int granq_fused_plan(int dtype, const int64_t dims[4], int channel_axis, int group, int with_backward,
                     uint32_t flags, int* launches_out);

/*
 * Host-only query: how the staged plan would cut this tensor on a device with `sm_count`
 * SMs and `smem_bytes` of shared memory per CTA (no counterpart in the paper).
 * out = { CTAs, threads per CTA, buffers per CTA, shared-memory bytes per CTA,
 *         16-byte units per buffer, channels per wave, units per chunk, number of waves }.
 * Returns GRANQ_ERR_UNSUPPORTED when the geometry does not qualify for staging.
 */
int granq_staged_geometry(int dtype, const int64_t dims[4], int channel_axis, int group, int sm_count,
                          int smem_bytes, int64_t out[8]);

/*
 * Host-only query: how the cluster-local plan would cut this tensor (no counterpart in the paper).
 * out = { CTAs, threads per CTA, CTAs per cluster, shared-memory bytes per CTA, bytes of one staged
 *         tile, channels per run, staging (0 = plain loads, 1 = bulk copies for x, 2 = bulk copies
 *         for x and gy), 1 if gy is prefetched into the L2 }.
 * Returns GRANQ_ERR_UNSUPPORTED when the geometry does not qualify.
 */
int granq_cluster_geometry(int dtype, const int64_t dims[4], int channel_axis, int group, int with_backward,
                           int64_t out[8]);

/*
 * Device self-test (no counterpart in the paper).  The staged kernel divides by the
 * per-group scale with a product and two exact-residual corrections from the correctly
 * rounded reciprocal; this runs `pairs` generated (x, s) pairs, hard cases included,
 * through that sequence and through IEEE division and counts the pairs whose bits differ
 * (expected: 0).  `device_mismatches` is one 64-bit counter in DEVICE memory, written by
 * the call; read it after the stream has passed.
 */
int granq_selftest_division(uint64_t pairs, uint64_t seed, unsigned long long* device_mismatches,
                            void* cuda_stream);

/*
 * Planner overrides for tests and tuning (no counterpart in the paper).  Process-wide and
 * not thread-safe; value 0 restores the automatic choice.  They change how the staged plan
 * cuts a tensor into waves and chunks, never its results.
 */
enum granq_knob {
    GRANQ_KNOB_STAGED_DEPTH = 0,          /* shared-memory buffers per CTA (1..3)                  */
    GRANQ_KNOB_STAGED_MAX_BUF_UNITS = 1,  /* cap on 16-byte units per buffer (forces small waves)  */
    GRANQ_KNOB_STAGED_GRID = 2,           /* cap on the number of CTAs                             */
    GRANQ_KNOB_SPIN_LIMIT = 3,            /* iteration limit of the wait on a wave's arrival count */
    GRANQ_KNOB_TEST_EXTRA_ARRIVALS = 4,   /* test hook: a wave waits for this many arrivals more
                                             than the grid provides, so the bounded wait runs out
                                             and the call ends with GRANQ_ERR_TIMEOUT              */
    GRANQ_KNOB_STAGED_CTAS_PER_SM = 5,    /* CTAs that share one SM (1 or 2)                       */
    GRANQ_KNOB_L2_WAVE_KB = 6,            /* L2-wave plan: x bytes of one wave, in KiB             */
    GRANQ_KNOB_L2_UPL = 7,                /* L2-wave plan: 16-byte units per lane and step (2, 4)  */
    GRANQ_KNOB_L2_CTAS_PER_SM = 8,        /* L2-wave / column-walk plans: cap on resident CTAs per SM */
    GRANQ_KNOB_L2_LAG = 9,                /* column-walk plan: waves the range phase runs ahead (1..3) */
    GRANQ_KNOB_CLUSTER_TILE_KB = 10,      /* cluster plan: limit on the staged tile of one CTA, in KiB */
    GRANQ_KNOB_CLUSTER_CTAS = 11,         /* cluster plan: CTAs per cluster (1, 2, 4, 8)               */
    GRANQ_KNOB_CLUSTER_THREADS = 12,      /* cluster plan: threads per CTA (a multiple of 32, <= 512)  */
    GRANQ_KNOB_CLUSTER_LOAD = 13,         /* cluster plan: 1 = bulk copies for x, 2 = plain loads,
                                             3 = bulk copies for x and gy                              */
    GRANQ_KNOB_CLUSTER_PREFETCH = 14,     /* cluster plan: 1 = L2 prefetch of gy, 2 = none             */
    GRANQ_KNOB_CLUSTER_KMUL = 15,         /* cluster plan: multiplier of a run's minimal channel count */
    GRANQ_KNOB_CLUSTER_EARLY_LAUNCH = 16  /* cluster plan: 2 = launch without programmatic dependent launch */
};
int granq_tune(int knob, int value);

#ifdef __cplusplus
}
#endif
#endif /* GRANQ_H */
