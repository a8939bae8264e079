/*
 * GranQ CPU oracle (TEST INFRASTRUCTURE; see granq_oracle.h).
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -shared -fPIC
 * Everything is `float`: no double intermediates, no fused multiply-add, default
 * rounding mode (round-to-nearest-even).  Loops are the definitions written out.
 */
#include "granq_oracle.h"

#include <math.h>
#include <stddef.h>
#include <string.h>

/* ---- bf16 <-> fp32 (bit patterns) ------------------------------------------------ */

static float bf16_widen(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round-to-nearest-even on the 16 discarded mantissa bits; inputs are finite */
static uint16_t bf16_narrow(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

static float load_elem(const void* p, int dtype, int64_t i) {
    if (dtype == GRANQ_ORACLE_BF16) return bf16_widen(((const uint16_t*)p)[i]);
    return ((const float*)p)[i];
}

static void store_elem(void* p, int dtype, int64_t i, float v) {
    if (dtype == GRANQ_ORACLE_BF16) ((uint16_t*)p)[i] = bf16_narrow(v);
    else ((float*)p)[i] = v;
}

/* ---- geometry: activation decomposition (Eq. 4) ---------------------------------- */

typedef struct { int64_t outer, C, inner; } geom_t;

static int make_geom(const int64_t dims[4], int axis, int mode, geom_t* g) {
    if (!dims || axis < 0 || axis > 3 || mode < 0 || mode > 2) return -1;
    for (int d = 0; d < 4; ++d) if (dims[d] <= 0) return -1;
    g->outer = 1; g->inner = 1;
    for (int d = 0; d < axis; ++d) g->outer *= dims[d];
    for (int d = axis + 1; d < 4; ++d) g->inner *= dims[d];
    g->C = dims[axis];
    return 0;
}

/* group of the element at (o, c, *) */
static int64_t group_of(const geom_t* g, int mode, int64_t o, int64_t c) {
    if (mode == GRANQ_ORACLE_GROUP_CHANNEL) return c;
    if (mode == GRANQ_ORACLE_GROUP_SAMPLE_CHANNEL) return o * g->C + c;
    return 0;
}

int64_t granq_oracle_num_groups(const int64_t dims[4], int channel_axis, int group_mode) {
    geom_t g;
    if (make_geom(dims, channel_axis, group_mode, &g)) return -1;
    if (group_mode == GRANQ_ORACLE_GROUP_CHANNEL) return g.C;
    if (group_mode == GRANQ_ORACLE_GROUP_SAMPLE_CHANNEL) return g.outer * g.C;
    return 1;
}

/* ---- Eq. 4: per-group min / max --------------------------------------------------- */

int granq_oracle_range(const void* x, int dtype, const int64_t dims[4], int channel_axis,
                       int group_mode, float* lo, float* hi) {
    geom_t g;
    if (!x || !lo || !hi || make_geom(dims, channel_axis, group_mode, &g)) return -1;
    int64_t G = granq_oracle_num_groups(dims, channel_axis, group_mode);
    for (int64_t k = 0; k < G; ++k) { lo[k] = INFINITY; hi[k] = -INFINITY; }
    for (int64_t o = 0; o < g.outer; ++o)
        for (int64_t c = 0; c < g.C; ++c) {
            int64_t k = group_of(&g, group_mode, o, c);
            for (int64_t i = 0; i < g.inner; ++i) {
                float v = load_elem(x, dtype, (o * g.C + c) * g.inner + i);
                if (!isfinite(v)) return -2;
                if (v < lo[k]) lo[k] = v;
                if (v > hi[k]) hi[k] = v;
            }
        }
    for (int64_t k = 0; k < G; ++k) { lo[k] += 0.0f; hi[k] += 0.0f; } /* -0 -> +0 */
    return 0;
}

/* ---- Eq. 2 / Eq. 5: scale and zero-point ------------------------------------------ */

static void scale_zero(float lo, float hi, int bits, float* s_out, float* z_out) {
    float qmax = (float)((1 << bits) - 1);
    float s = (hi - lo) / qmax;      /* one subtract, one true division */
    if (!(s >= 1e-8f)) s = 1e-8f;    /* degenerate-range floor */
    float z = rintf((-lo) / s);      /* true division, round-half-to-even */
    *s_out = s;
    *z_out = z + 0.0f;               /* -0 -> +0 */
}

int granq_oracle_params(const float* lo, const float* hi, int64_t G, int bits, float* s, float* z) {
    if (!lo || !hi || !s || !z || G <= 0 || bits < 1 || bits > 8) return -1;
    for (int64_t k = 0; k < G; ++k) scale_zero(lo[k], hi[k], bits, &s[k], &z[k]);
    return 0;
}

/* ---- Eq. 1, clamp, Eq. 6, STE ------------------------------------------------------ */

int granq_oracle_fakequant(const void* x, const void* gy, int dtype, const int64_t dims[4],
                           int channel_axis, int group_mode, int bits,
                           const float* lo, const float* hi,
                           void* y, void* gx, uint8_t* codes, uint8_t* mask, float* s, float* z) {
    geom_t g;
    if (!x || !y || !lo || !hi || bits < 1 || bits > 8) return -1;
    if ((gy == NULL) != (gx == NULL)) return -1;
    if (make_geom(dims, channel_axis, group_mode, &g)) return -1;
    const float qmax = (float)((1 << bits) - 1);
    for (int64_t o = 0; o < g.outer; ++o)
        for (int64_t c = 0; c < g.C; ++c) {
            int64_t k = group_of(&g, group_mode, o, c);
            float sk, zk;
            scale_zero(lo[k], hi[k], bits, &sk, &zk);
            if (s) s[k] = sk;
            if (z) z[k] = zk;
            for (int64_t i = 0; i < g.inner; ++i) {
                int64_t e = (o * g.C + c) * g.inner + i;
                float v = load_elem(x, dtype, e);
                float t = v / sk;                  /* Eq. 1: true division          */
                float u = t + zk;                  /*        separate addition      */
                float r = rintf(u);                /*        round-half-to-even     */
                float q = r;                       /* clamp to [0, 2^b - 1]         */
                if (q < 0.0f) q = 0.0f;
                if (q > qmax) q = qmax;
                q += 0.0f;                         /* an integer code has no -0     */
                int inside = (r >= 0.0f) && (r <= qmax);   /* clamp inactive        */
                float d = q - zk;                  /* Eq. 6: subtract zero-point    */
                float yv = sk * d;                 /*        multiply by the scale  */
                store_elem(y, dtype, e, yv);
                if (codes) codes[e] = (uint8_t)q;
                if (mask) mask[e] = (uint8_t)inside;
                if (gx) {
                    float gv = load_elem(gy, dtype, e);
                    store_elem(gx, dtype, e, inside ? gv : 0.0f);  /* STE: pass or zero */
                }
            }
        }
    return 0;
}

int granq_oracle_fused(const void* x, const void* gy, int dtype, const int64_t dims[4],
                       int channel_axis, int group_mode, int bits,
                       void* y, void* gx, float* lo, float* hi,
                       uint8_t* codes, uint8_t* mask, float* s, float* z) {
    int rc = granq_oracle_range(x, dtype, dims, channel_axis, group_mode, lo, hi);
    if (rc) return rc;
    return granq_oracle_fakequant(x, gy, dtype, dims, channel_axis, group_mode, bits,
                                  lo, hi, y, gx, codes, mask, s, z);
}

/* ---- mask-carrying split of forward and backward (Section 2.1: the STE needs only the mask) ---- */

/* Bit e % 8 of byte e / 8 (least significant bit first) is mask[e] != 0; the unused high bits
 * of a last partial byte are 0. */
int granq_oracle_pack_mask(const uint8_t* mask, int64_t E, uint8_t* packed) {
    if (!mask || !packed || E < 0) return -1;
    for (int64_t b = 0; b < (E + 7) / 8; ++b) packed[b] = 0;
    for (int64_t e = 0; e < E; ++e)
        if (mask[e]) packed[e / 8] = (uint8_t)(packed[e / 8] | (1u << (e % 8)));
    return 0;
}

/* STE backward from the packed mask alone: gx[e] = gy[e] where bit e is set, else +0. */
int granq_oracle_bwd_packed(const void* gy, const uint8_t* packed, int dtype, int64_t E, void* gx) {
    if (!gy || !packed || !gx || E < 0) return -1;
    for (int64_t e = 0; e < E; ++e) {
        int bit = (packed[e / 8] >> (e % 8)) & 1;
        float gv = load_elem(gy, dtype, e);
        store_elem(gx, dtype, e, bit ? gv : 0.0f);
    }
    return 0;
}

/* ---- distortion statistics of a quantization (Section 4.1, Table 2) ---------------------------- */

/* sums[0] = sum x^2, sums[1] = sum q^2, sums[2] = sum x*q, sums[3] = sum (x - q)^2 over all E
 * elements, every term and every sum in fp64 (the products of two fp32 values are exact in fp64). */
int granq_oracle_distortion_sums(const void* x, const void* q, int dtype, int64_t E, double sums[4]) {
    if (!x || !q || !sums || E < 0) return -1;
    double sxx = 0.0, sqq = 0.0, sxq = 0.0, sdd = 0.0;
    for (int64_t e = 0; e < E; ++e) {
        double xv = (double)load_elem(x, dtype, e);
        double qv = (double)load_elem(q, dtype, e);
        double d = xv - qv;
        sxx += xv * xv;
        sqq += qv * qv;
        sxq += xv * qv;
        sdd += d * d;
    }
    sums[0] = sxx;
    sums[1] = sqq;
    sums[2] = sxq;
    sums[3] = sdd;
    return 0;
}

/* Table 2's two statistics from the sums: cosine similarity X.Q / (|X| |Q|) and relative error
 * |X - Q| / |X|; 0 where a denominator is 0. */
int granq_oracle_distortion(const double sums[4], double* cosine, double* rel_error) {
    if (!sums || !cosine || !rel_error) return -1;
    double den = sqrt(sums[0]) * sqrt(sums[1]);
    *cosine = den > 0.0 ? sums[2] / den : 0.0;
    *rel_error = sums[0] > 0.0 ? sqrt(sums[3]) / sqrt(sums[0]) : 0.0;
    return 0;
}

/* ---- integer codes as a packed bit string (Eq. 1 produces b-bit integers; Eq. 6 consumes them) ---- */

/* Element e occupies bits [e*b, (e+1)*b) of a little-endian bit string (bit k of the string is bit
 * k % 8 of byte k / 8); ceil(E*b / 8) bytes are written, unused high bits of the last byte 0. */
int granq_oracle_pack_codes(const uint8_t* codes, int64_t E, int bits, uint8_t* packed) {
    if (!codes || !packed || E < 0 || bits < 1 || bits > 8) return -1;
    for (int64_t k = 0; k < (E * bits + 7) / 8; ++k) packed[k] = 0;
    for (int64_t e = 0; e < E; ++e) {
        if (codes[e] >> bits) return -3;                    /* a code that does not fit b bits */
        for (int j = 0; j < bits; ++j) {
            int64_t k = e * bits + j;
            if ((codes[e] >> j) & 1) packed[k / 8] = (uint8_t)(packed[k / 8] | (1u << (k % 8)));
        }
    }
    return 0;
}

/* Eq. 6 from the packed codes: y[e] = s[g] * (code[e] - z[g]) with g the element's group. */
int granq_oracle_dequant_packed(const uint8_t* packed, int dtype, const int64_t dims[4], int channel_axis,
                                int group_mode, int bits, const float* s, const float* z, void* y) {
    geom_t g;
    if (!packed || !s || !z || !y || bits < 1 || bits > 8) return -1;
    if (make_geom(dims, channel_axis, group_mode, &g)) return -1;
    for (int64_t o = 0; o < g.outer; ++o)
        for (int64_t c = 0; c < g.C; ++c) {
            int64_t grp = group_of(&g, group_mode, o, c);
            for (int64_t i = 0; i < g.inner; ++i) {
                int64_t e = (o * g.C + c) * g.inner + i;
                unsigned code = 0;
                for (int j = 0; j < bits; ++j) {
                    int64_t k = e * bits + j;
                    code |= (unsigned)((packed[k / 8] >> (k % 8)) & 1) << j;
                }
                float d = (float)code - z[grp];
                store_elem(y, dtype, e, s[grp] * d);
            }
        }
    return 0;
}


/* ---- the accumulation over the pre-scaled activations (Eq. 6 left-hand side, Algorithm 1 output step) ---- */

/* Pointwise (1 x 1) case.  codes: the integer codes of Eq. 1, [N, C, P] (channels_last = 0: the paper's
 * C x (HW) matrix per sample) or [N, P, C] (channels_last = 1); s, z: per-channel scale and zero-point (Eq. 5);
 * w: fp32 [O, C]; y: fp64, [N, O, P] or [N, P, O].
 * Eq. 6 / Algorithm 1: the pre-scaled activation A~ = s_c * (code - z_c) is formed first, in fp32 exactly as
 * the pre-scale step forms it (one subtract, one multiply), then y = sum_c w[o][c] * A~[c], products and sum
 * in fp64, c ascending. */
int granq_oracle_accumulate(const uint8_t* codes, const int64_t dims[3], int channels_last, const float* s,
                            const float* z, const float* w, int64_t O, double* y) {
    if (!codes || !dims || !s || !z || !w || !y || O <= 0) return -1;
    const int64_t N = dims[0], C = dims[1], P = dims[2];
    if (N <= 0 || C <= 0 || P <= 0) return -1;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t o = 0; o < O; ++o)
            for (int64_t p = 0; p < P; ++p) {
                double acc = 0.0;
                for (int64_t c = 0; c < C; ++c) {
                    const uint8_t code = channels_last ? codes[(n * P + p) * C + c] : codes[(n * C + c) * P + p];
                    float d = (float)code - z[c];
                    float a = s[c] * d;                           /* the pre-scaled activation */
                    acc += (double)w[o * C + c] * (double)a;
                }
                if (channels_last) y[(n * P + p) * O + o] = acc;
                else y[(n * O + o) * P + p] = acc;
            }
    return 0;
}

/* Eq. 3, the conventional order the paper contrasts with: the per-channel scale is applied inside the
 * accumulation, y = sum_c w_c * s_c * (code_c - z_c), every operation in fp64.  The same real number as
 * Eq. 6 gives; only the order of the operations differs. */
int granq_oracle_accumulate_inloop(const uint8_t* codes, const int64_t dims[3], int channels_last, const float* s,
                                   const float* z, const float* w, int64_t O, double* y) {
    if (!codes || !dims || !s || !z || !w || !y || O <= 0) return -1;
    const int64_t N = dims[0], C = dims[1], P = dims[2];
    if (N <= 0 || C <= 0 || P <= 0) return -1;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t o = 0; o < O; ++o)
            for (int64_t p = 0; p < P; ++p) {
                double acc = 0.0;
                for (int64_t c = 0; c < C; ++c) {
                    const uint8_t code = channels_last ? codes[(n * P + p) * C + c] : codes[(n * C + c) * P + p];
                    acc += (double)w[o * C + c] * (double)s[c] * ((double)code - (double)z[c]);
                }
                if (channels_last) y[(n * P + p) * O + o] = acc;
                else y[(n * O + o) * P + p] = acc;
            }
    return 0;
}
