// Device-side building blocks shared by the GranQ kernels: ordered keys for min/max,
// the per-element quantizer arithmetic, 128-bit element packs, fast integer division and
// the warp-level run accumulator of the range reduction.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace granq {

// ---------------------------------------------------------------------------------------
// Ordered keys.  enc() maps a float to an unsigned integer with the same ordering, so an
// unsigned max over enc(x) is the float max and an unsigned max over ~enc(x) is the float
// min.  0 is the identity of both reductions (no finite float encodes to 0 or ~0).
// ---------------------------------------------------------------------------------------
__host__ __device__ __forceinline__ uint32_t enc_bits(uint32_t b) {
    return b ^ ((uint32_t)((int32_t)b >> 31) | 0x80000000u);
}
__device__ __forceinline__ uint32_t enc(float f) { return enc_bits(__float_as_uint(f)); }
__device__ __forceinline__ float dec(uint32_t k) {
    uint32_t b = (k & 0x80000000u) ? (k ^ 0x80000000u) : ~k;
    return __uint_as_float(b);
}
// key pair -> (lo, hi), with -0 canonicalised to +0
__device__ __forceinline__ void keys_to_range(uint32_t kmin, uint32_t kmax, float& lo, float& hi) {
    lo = __fadd_rn(dec(~kmin), 0.0f);
    hi = __fadd_rn(dec(kmax), 0.0f);
}

// ---------------------------------------------------------------------------------------
// Quantizer arithmetic (Eq. 1, 2, 5, 6).  Every operation is an explicitly rounded fp32
// intrinsic, so the compiler can neither contract multiply-adds nor replace the divisions.
// ---------------------------------------------------------------------------------------
struct QParam {
    float s, z;
};

__device__ __forceinline__ QParam make_qparam(float lo, float hi, float qmax) {
    QParam p;
    float s = __fdiv_rn(__fsub_rn(hi, lo), qmax);
    p.s = fmaxf(s, 1e-8f);
    p.z = __fadd_rn(rintf(__fdiv_rn(-lo, p.s)), 0.0f);
    return p;
}

// Given t = x / s: rounds u = t + z to the nearest integer (ties to even) and clamps it to
// [0, qmax].  The value is first clamped to [-1, qmax + 1]: rounding is monotone and the
// bounds are integers, so this changes neither the clamped code nor whether the clamp was
// active, and it makes the add/subtract of 1.5 * 2^23 an exact round-half-to-even
// (|u| < 2^22) that never yields -0.
__device__ __forceinline__ float quant_from_quotient(float t, float s, float z, float qmax, float& y, bool& inside) {
    const float kMagic = 12582912.0f;  // 1.5 * 2^23
    float u = __fadd_rn(t, z);
    float uc = fminf(fmaxf(u, -1.0f), __fadd_rn(qmax, 1.0f));
    float r = __fsub_rn(__fadd_rn(uc, kMagic), kMagic);
    float q = fminf(fmaxf(r, 0.0f), qmax);
    inside = (r == q);
    y = __fmul_rn(s, __fsub_rn(q, z));
    return q;
}

__device__ __forceinline__ float quant_one(float x, QParam p, float qmax, float& y, bool& inside) {
    return quant_from_quotient(__fdiv_rn(x, p.s), p.s, p.z, qmax, y, inside);
}

// Correctly rounded x / s from the correctly rounded reciprocal rcp = RN(1 / s): a product
// and two residual corrections, each residual x - q * s being exact in one fused
// multiply-add.  After the first correction q is a faithful rounding of x / s; a further
// correction of a faithful quotient with a correctly rounded reciprocal gives RN(x / s)
// (Markstein's division theorem), provided nothing over- or underflows on the way.
// div_is_safe() states the range for which that holds; groups outside it use __fdiv_rn.
__device__ __forceinline__ float div_by_scale(float x, float s, float rcp) {
    float q = __fmul_rn(x, rcp);
    float e = __fmaf_rn(-q, s, x);
    q = __fmaf_rn(e, rcp, q);
    e = __fmaf_rn(-q, s, x);
    return __fmaf_rn(e, rcp, q);
}
// s and every |x| of the group within [2^-60, 2^60] (x may also be tiny or zero: a quotient
// below 2^-120 cannot move u = x / s + z across a rounding boundary).
__device__ __forceinline__ bool div_is_safe(float s, float lo, float hi) {
    const float kBig = 1152921504606846976.0f;       // 2^60
    const float kSmall = 8.67361737988403547e-19f;   // 2^-60
    return s >= kSmall && s <= kBig && fmaxf(fabsf(lo), fabsf(hi)) <= kBig;
}

// ---------------------------------------------------------------------------------------
// 16-byte packs of elements.
// ---------------------------------------------------------------------------------------
template <typename T>
struct Pack;

template <>
struct Pack<float> {
    static constexpr int V = 4;
    uint4 raw;
    __device__ __forceinline__ float get(int i) const { return __uint_as_float((&raw.x)[i]); }
    __device__ __forceinline__ void set(int i, float v) { (&raw.x)[i] = __float_as_uint(v); }
    __device__ __forceinline__ void set_all(const float (&v)[4]) {
        raw = make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
    }
    // element i of g where bit i of `keep` is set, +0 elsewhere (the straight-through gradient)
    __device__ __forceinline__ void select(const Pack& g, uint32_t keep) {
        raw.x = (keep & 1u) ? g.raw.x : 0u;
        raw.y = (keep & 2u) ? g.raw.y : 0u;
        raw.z = (keep & 4u) ? g.raw.z : 0u;
        raw.w = (keep & 8u) ? g.raw.w : 0u;
    }
};

template <>
struct Pack<__nv_bfloat16> {
    static constexpr int V = 8;
    uint4 raw;
    __device__ __forceinline__ float get(int i) const {
        uint32_t w = (&raw.x)[i >> 1];
        uint32_t b = (i & 1) ? (w & 0xFFFF0000u) : (w << 16);
        return __uint_as_float(b);
    }
    __device__ __forceinline__ void set(int i, float v) {
        uint32_t h = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v));
        uint32_t& w = (&raw.x)[i >> 1];
        w = (i & 1) ? ((w & 0x0000FFFFu) | (h << 16)) : ((w & 0xFFFF0000u) | h);
    }
    // eight floats -> eight bf16 (round to nearest even), two per conversion instruction
    __device__ __forceinline__ void set_all(const float (&v)[8]) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);      // .x, the low half, = the first
            (&raw.x)[k] = *reinterpret_cast<const uint32_t*>(&h);
        }
    }
    // element i of g where bit i of `keep` is set, +0 elsewhere: on the raw halves, nothing is converted
    __device__ __forceinline__ void select(const Pack& g, uint32_t keep) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t m = ((keep >> (2 * k)) & 1u ? 0x0000FFFFu : 0u) | ((keep >> (2 * k + 1)) & 1u ? 0xFFFF0000u : 0u);
            (&raw.x)[k] = (&g.raw.x)[k] & m;
        }
    }
};

__device__ __forceinline__ float load_scalar(const float* p) { return __ldg(p); }
__device__ __forceinline__ float load_scalar(const __nv_bfloat16* p) {
    return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}
__device__ __forceinline__ void store_scalar(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_scalar(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// streaming 128-bit global accesses: data that is touched once should not displace anything
__device__ __forceinline__ uint4 ld_stream_16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream_16(void* p, uint4 v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// ---------------------------------------------------------------------------------------
// Division of n < 2^31 by a run-time constant d (1 <= d < 2^31): q = (n * M) >> (31 + l)
// with l = ceil(log2 d), M = floor(2^(31+l) / d) + 1.
// ---------------------------------------------------------------------------------------
struct FastDiv {
    uint32_t d, M, sh;
    __host__ __device__ __forceinline__ uint32_t div(uint32_t n) const {
        return (uint32_t)(((uint64_t)n * (uint64_t)M) >> sh);
    }
    __host__ __device__ __forceinline__ void divmod(uint32_t n, uint32_t& q, uint32_t& r) const {
        q = div(n);
        r = n - q * d;
    }
};

inline FastDiv make_fastdiv(uint32_t d) {
    FastDiv f;
    f.d = d;
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;
    f.M = (uint32_t)(((1ull << (31 + l)) / d) + 1ull);
    f.sh = 31 + l;
    return f;
}

constexpr uint32_t kNoGroup = 0xFFFFFFFFu;
constexpr uint32_t kFullMask = 0xFFFFFFFFu;

// ---------------------------------------------------------------------------------------
// Warp-level run accumulator for per-group min/max (Eq. 4).
// A warp walks memory in order, so the group of its elements changes rarely.  While all
// lanes see the same group the partial min/max stay in registers; a change of group (or
// a warp that straddles several groups) is resolved with warp reductions on the ordered
// keys and one pair of atomics per group.
// ---------------------------------------------------------------------------------------
struct WarpRun {
    uint32_t g, kmn, kmx;
};

__device__ __forceinline__ void run_flush(WarpRun& r, uint32_t* kmin, uint32_t* kmax) {
    if (r.g != kNoGroup) {
        uint32_t a = __reduce_max_sync(kFullMask, r.kmn);
        uint32_t b = __reduce_max_sync(kFullMask, r.kmx);
        if ((threadIdx.x & 31) == 0) {
            atomicMax(kmin + r.g, a);
            atomicMax(kmax + r.g, b);
        }
    }
    r.g = kNoGroup;
    r.kmn = 0;
    r.kmx = 0;
}

// must be called by all 32 lanes of a warp
__device__ __forceinline__ void run_add(WarpRun& r, bool valid, uint32_t g, uint32_t mn, uint32_t mx,
                                        uint32_t* kmin, uint32_t* kmax) {
    uint32_t pending = __ballot_sync(kFullMask, valid);
    if (!pending) return;
    const int lane = threadIdx.x & 31;
    uint32_t first = __shfl_sync(kFullMask, g, __ffs(pending) - 1);
    bool uniform = __all_sync(kFullMask, !valid || g == first);
    if (!valid) {
        mn = 0;
        mx = 0;
    }
    if (uniform) {
        if (first != r.g) {
            run_flush(r, kmin, kmax);
            r.g = first;
        }
        r.kmn = max(r.kmn, mn);
        r.kmx = max(r.kmx, mx);
        return;
    }
    run_flush(r, kmin, kmax);
    while (pending) {
        int src = __ffs(pending) - 1;
        uint32_t cur = __shfl_sync(kFullMask, g, src);
        bool mine = valid && g == cur;
        uint32_t a = __reduce_max_sync(kFullMask, mine ? mn : 0u);
        uint32_t b = __reduce_max_sync(kFullMask, mine ? mx : 0u);
        if (lane == src) {
            atomicMax(kmin + cur, a);
            atomicMax(kmax + cur, b);
        }
        pending &= ~__ballot_sync(kFullMask, mine);
    }
}

// ---------------------------------------------------------------------------------------
// Per-group parameters from the published min / max keys, and the arithmetic of one pack.
// ---------------------------------------------------------------------------------------
struct GroupParam {
    float s, z, r;   // scale, zero-point, RN(1 / s) or 0 when the group must use IEEE division
};

__device__ __forceinline__ GroupParam group_param_from_keys(const uint32_t* kmin, const uint32_t* kmax, uint32_t g,
                                                            float qmax, float& lo, float& hi) {
    keys_to_range(__ldcg(kmin + g), __ldcg(kmax + g), lo, hi);
    const QParam p = make_qparam(lo, hi, qmax);
    GroupParam gp;
    gp.s = p.s;
    gp.z = p.z;
    gp.r = div_is_safe(p.s, lo, hi) ? __frcp_rn(p.s) : 0.0f;
    return gp;
}

// The rounded value r = round(x / s + z) from ONE fused multiply-add, where that is provably the same integer.
// Only r enters the results (code = clamp(r), y = s * (code - z), mask = (r == code)); the quotient and the sum
// are intermediates.  With rcp = RN(1 / s), up = RN(x * rcp + z) lies within E = 2^-24 * (|x / s| + |up|) of the
// real number v = x / s + z, and so does the exactly rounded u = RN(RN(x / s) + z).  |x / s| <= |v| + |z|, and
// values beyond the clamp range [-1, qmax + 1] round to the same clamped integer either way, so inside it
// E <= 2^-24 * (|z| + 2 * 258) < M = 2^-23 * (|z| + 1024).  If up is farther than 2 M from every half-integer,
// v is farther than M from it, u lies on the same side, and round(u) = round(up).  tie_threshold() returns
// 0.5 - 2 M: an element whose distance |up - round(up)| reaches it takes the exact sequence instead (for
// |z| >= 2^21 the threshold is <= 0 and every element does).
__device__ __forceinline__ float tie_threshold(float z) {
    return __fmaf_rn(-2.384185791015625e-07f, __fadd_rn(fabsf(z), 1024.0f), 0.5f);      // 0.5 - 2^-22 * (|z| + 1024)
}

// Quantize one pack: elements [0, n1) belong to the group with parameters g1, the rest to
// g2 (n1 = V when the pack lies in one group).  EXTRAS = 1 also packs the codes and the mask
// (one byte per element); EXTRAS = 2 leaves the codes out and returns the mask as V bits in mb[0]
// (bit i: the clamp was inactive for element i), which is all the packed mask needs; EXTRAS = 3 returns
// only the codes, code_bits each (cb[h] = the four codes of half h as a string of 4 * code_bits bits; bytes for
// the default of 8), taken from the low mantissa bits of code + 2^23 instead of a float-to-integer conversion
// (packed-code output).  SELF: the range is that of the tensor itself, so x / s + z lies within
// [-1, qmax + 1] already (x in [lo, hi] gives RN(x / s) - round(RN(lo / s)) >= -1/2, and at most qmax plus a few
// units in the last place of hi / s < 2^33 above that) and the clamp before the rounding can go.
template <typename T, bool BWD, bool SPLIT, int EXTRAS, bool SELF = false>
__device__ __forceinline__ void quantize_pack(const Pack<T>& px, const Pack<T>& pg, const GroupParam& g1,
                                              const GroupParam& g2, int n1, float qmax, Pack<T>& py, Pack<T>& pgx,
                                              uint32_t (&cb)[Pack<T>::V / 4], uint32_t (&mb)[Pack<T>::V / 4],
                                              int code_bits = 8) {
    constexpr int V = Pack<T>::V;
    const float kMagic = 12582912.0f;  // 1.5 * 2^23
#pragma unroll
    for (int i = 0; i < V / 4; ++i) {
        cb[i] = 0;
        mb[i] = 0;
    }
    float yv[V];
    uint32_t keep = 0;                                          // bit i: the clamp was inactive for element i
    auto finish = [&](int i, float r, float s, float z) {      // r: the rounded value, within [-1, qmax + 1]
        const float q = fminf(fmaxf(r, 0.0f), qmax);
        const bool in = (r == q);
        yv[i] = __fmul_rn(s, __fsub_rn(q, z));
        if constexpr (BWD) {
            if constexpr (V == 4) pgx.set(i, in ? pg.get(i) : 0.0f);      // fp32: a select per element is all it takes
            else keep |= in ? (1u << i) : 0u;                              // bf16: on the raw halves, below
        }
        if constexpr (EXTRAS == 1) {
            cb[i / 4] |= (uint32_t)q << (8 * (i % 4));
            mb[i / 4] |= (in ? 1u : 0u) << (8 * (i % 4));
        } else if constexpr (EXTRAS == 2) {
            mb[0] |= in ? (1u << i) : 0u;
        } else if constexpr (EXTRAS == 3) {
            cb[i / 4] |= (__float_as_uint(__fadd_rn(q, 8388608.0f)) & 0xFFu) << ((i % 4) * code_bits);
        }
    };
    auto exact_round = [&](float t, float z) -> float {        // t = RN(x / s): the sequence as defined
        const float u = __fadd_rn(t, z);
        const float uc = fminf(fmaxf(u, -1.0f), __fadd_rn(qmax, 1.0f));
        return __fsub_rn(__fadd_rn(uc, kMagic), kMagic);
    };
    const bool fast = SPLIT ? (g1.r != 0.0f && g2.r != 0.0f) : (g1.r != 0.0f);
    if (fast) {
        const float thr1 = tie_threshold(g1.z), thr2 = SPLIT ? tie_threshold(g2.z) : thr1;
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const bool first = !SPLIT || i < n1;
            const float s = first ? g1.s : g2.s, z = first ? g1.z : g2.z, rc = first ? g1.r : g2.r;
            const float x = px.get(i);
            float up = __fmaf_rn(x, rc, z);
            if constexpr (!SELF) up = fminf(fmaxf(up, -1.0f), __fadd_rn(qmax, 1.0f));
            float r = __fsub_rn(__fadd_rn(up, kMagic), kMagic);
            if (!(fabsf(__fsub_rn(up, r)) < (first ? thr1 : thr2)))     // rare: too close to a tie for the shortcut
                r = exact_round(div_by_scale(x, s, rc), z);
            finish(i, r, s, z);
        }
    } else {
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const bool first = !SPLIT || i < n1;
            const float s = first ? g1.s : g2.s, z = first ? g1.z : g2.z;
            finish(i, exact_round(__fdiv_rn(px.get(i), s), z), s, z);
        }
    }
    py.set_all(yv);
    if constexpr (BWD && V != 4) pgx.select(pg, keep);
}

// Quantize one pack whose V elements belong to V different groups (channels-last rows), the range being the
// tensor's own: element i takes the parameters g[i].  Same arithmetic and shortcut as quantize_pack().
template <typename T, bool BWD, bool EXTRAS>
__device__ __forceinline__ void quantize_pack_each(const Pack<T>& px, const Pack<T>& pg,
                                                   const GroupParam (&g)[Pack<T>::V], float qmax, Pack<T>& py,
                                                   Pack<T>& pgx, uint32_t (&cb)[Pack<T>::V / 4],
                                                   uint32_t (&mb)[Pack<T>::V / 4]) {
    constexpr int V = Pack<T>::V;
    const float kMagic = 12582912.0f;  // 1.5 * 2^23
#pragma unroll
    for (int i = 0; i < V / 4; ++i) {
        cb[i] = 0;
        mb[i] = 0;
    }
    float yv[V];
    uint32_t keep = 0;
#pragma unroll
    for (int i = 0; i < V; ++i) {
        const float s = g[i].s, z = g[i].z, rc = g[i].r, x = px.get(i);
        float r;
        if (rc != 0.0f) {
            const float up = __fmaf_rn(x, rc, z);
            r = __fsub_rn(__fadd_rn(up, kMagic), kMagic);
            if (!(fabsf(__fsub_rn(up, r)) < tie_threshold(z))) {     // rare: too close to a tie for the shortcut
                const float u = __fadd_rn(div_by_scale(x, s, rc), z);
                const float uc = fminf(fmaxf(u, -1.0f), __fadd_rn(qmax, 1.0f));
                r = __fsub_rn(__fadd_rn(uc, kMagic), kMagic);
            }
        } else {
            const float u = __fadd_rn(__fdiv_rn(x, s), z);
            const float uc = fminf(fmaxf(u, -1.0f), __fadd_rn(qmax, 1.0f));
            r = __fsub_rn(__fadd_rn(uc, kMagic), kMagic);
        }
        const float q = fminf(fmaxf(r, 0.0f), qmax);
        const bool in = (r == q);
        yv[i] = __fmul_rn(s, __fsub_rn(q, z));
        if constexpr (BWD) {
            if constexpr (V == 4) pgx.set(i, in ? pg.get(i) : 0.0f);
            else keep |= in ? (1u << i) : 0u;
        }
        if constexpr (EXTRAS) {
            cb[i / 4] |= (uint32_t)q << (8 * (i % 4));
            mb[i / 4] |= (in ? 1u : 0u) << (8 * (i % 4));
        }
    }
    py.set_all(yv);
    if constexpr (BWD && V != 4) pgx.select(pg, keep);
}

// per-lane min / max of elements [first, last) of one pack
template <typename T>
__device__ __forceinline__ void pack_minmax(const Pack<T>& p, int first, int last, float& mn, float& mx) {
#pragma unroll
    for (int i = 0; i < Pack<T>::V; ++i) {
        if (i >= first && i < last) {
            float v = p.get(i);
            mn = fminf(mn, v);
            mx = fmaxf(mx, v);
        }
    }
}

// The V mask bits of one pack, from the mask bytes of quantize_pack<EXTRAS = 1> or the bits of <EXTRAS = 2>.
template <int V, int EXTRAS>
__device__ __forceinline__ uint32_t mask_bits_of(const uint32_t (&mb)[V / 4]) {
    if constexpr (EXTRAS == 2) {
        return mb[0];
    } else {
        uint32_t bits = 0;
#pragma unroll
        for (int i = 0; i < V; ++i) bits |= ((mb[i / 4] >> (8 * (i % 4))) & 1u) << i;
        return bits;
    }
}

// Store the packed mask one byte (8 elements) at a time: `bits` are the V mask bits of the pack that starts at
// element `first` (a multiple of V; for V = 4 the even lane of a pair holds the low half of a byte, and both
// lanes of the pair must call this together with neighbouring packs).
template <int V>
__device__ __forceinline__ void store_mask_byte(uint32_t* pmask, size_t first, uint32_t bits, uint32_t lane) {
    if constexpr (V == 4) {
        const uint32_t other = __shfl_xor_sync(3u << (lane & ~1u), bits, 1);
        if (!(lane & 1)) reinterpret_cast<uint8_t*>(pmask)[first >> 3] = (uint8_t)(bits | (other << 4));
    } else {
        static_assert(V == 8, "a pack is 4 or 8 elements");
        reinterpret_cast<uint8_t*>(pmask)[first >> 3] = (uint8_t)bits;
    }
}

// The codes of one pack as a string of V * b bits, from the half strings of quantize_pack<EXTRAS = 3>(.., code_bits).
template <int V>
__device__ __forceinline__ uint64_t code_string_of(const uint32_t (&cb)[V / 4], int code_bits) {
    uint64_t str = cb[0];
    if constexpr (V == 8) str |= (uint64_t)cb[1] << (4 * code_bits);
    return str;
}

// Store the packed codes 8 codes = b bytes at a time: `str` is the code string of the pack that starts at element
// `first` (a multiple of V); byte (first / 8) * b of the bit string is where the 8 codes of an aligned group of 8
// elements begin.  For V = 4 the even lane of a pair holds the first half and stores; both lanes of the pair must
// call this together with neighbouring packs.  The buffer is only known to be 4-byte aligned.
template <int V>
__device__ __forceinline__ void store_code_bytes(uint32_t* pcodes, size_t first, uint64_t str, int code_bits, uint32_t lane) {
    uint64_t eight = str;
    if constexpr (V == 4) {
        const uint32_t other = __shfl_xor_sync(3u << (lane & ~1u), (uint32_t)str, 1);
        if (lane & 1) return;
        eight |= (uint64_t)other << (4 * code_bits);
    }
    uint8_t* dst = reinterpret_cast<uint8_t*>(pcodes) + (first >> 3) * (size_t)code_bits;
    switch (code_bits) {
        case 8:
            reinterpret_cast<uint32_t*>(dst)[0] = (uint32_t)eight;
            reinterpret_cast<uint32_t*>(dst)[1] = (uint32_t)(eight >> 32);
            break;
        case 4: *reinterpret_cast<uint32_t*>(dst) = (uint32_t)eight; break;
        case 2: *reinterpret_cast<uint16_t*>(dst) = (uint16_t)eight; break;
        case 6:
            reinterpret_cast<uint16_t*>(dst)[0] = (uint16_t)eight;
            reinterpret_cast<uint16_t*>(dst)[1] = (uint16_t)(eight >> 16);
            reinterpret_cast<uint16_t*>(dst)[2] = (uint16_t)(eight >> 32);
            break;
        default:
            for (int t = 0; t < code_bits; ++t) dst[t] = (uint8_t)(eight >> (8 * t));
            break;
    }
}

// ---------------------------------------------------------------------------------------
// Distortion statistics of a quantization (Section 4.1, Table 2): sum x^2, sum q^2, sum x*q,
// sum (x - q)^2.  The terms of one pack are summed in fp32 (fused multiply-adds), everything
// beyond a pack in fp64, so a sum differs from the exact one by at most a few fp32 roundings
// of a pack-sized partial sum.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float as_stored(float v, const float*) { return v; }
__device__ __forceinline__ float as_stored(float v, const __nv_bfloat16*) {
    return __bfloat162float(__float2bfloat16_rn(v));
}

struct DistAcc {
    double xx, qq, xq, dd;
    __device__ __forceinline__ void reset() { xx = qq = xq = dd = 0.0; }
    __device__ __forceinline__ void add_one(float x, float q) {
        const float d = __fsub_rn(x, q);
        xx += (double)__fmul_rn(x, x);
        qq += (double)__fmul_rn(q, q);
        xq += (double)__fmul_rn(x, q);
        dd += (double)__fmul_rn(d, d);
    }
    template <typename T>
    __device__ __forceinline__ void add(const Pack<T>& px, const Pack<T>& pq) {
        float a = 0.0f, b = 0.0f, c = 0.0f, e = 0.0f;
#pragma unroll
        for (int i = 0; i < Pack<T>::V; ++i) {
            const float x = px.get(i), q = pq.get(i), d = __fsub_rn(x, q);
            a = __fmaf_rn(x, x, a);
            b = __fmaf_rn(q, q, b);
            c = __fmaf_rn(x, q, c);
            e = __fmaf_rn(d, d, e);
        }
        xx += (double)a;
        qq += (double)b;
        xq += (double)c;
        dd += (double)e;
    }
    // must be called by all 32 lanes of a warp: one atomic per warp and sum
    __device__ __forceinline__ void flush(double* out) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            xx += __shfl_xor_sync(kFullMask, xx, d);
            qq += __shfl_xor_sync(kFullMask, qq, d);
            xq += __shfl_xor_sync(kFullMask, xq, d);
            dd += __shfl_xor_sync(kFullMask, dd, d);
        }
        if ((threadIdx.x & 31) == 0) {
            atomicAdd(out + 0, xx);
            atomicAdd(out + 1, qq);
            atomicAdd(out + 2, xq);
            atomicAdd(out + 3, dd);
        }
    }
};

// 128-bit global accesses with an L2 eviction policy (createpolicy.fractional.L2::evict_*)
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint4 ld_hint_16(const void* p, uint64_t policy) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(policy)
                 : "memory");
    return v;
}
__device__ __forceinline__ void st_hint_16(void* p, uint4 v, uint64_t policy) {
    asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1,%2,%3,%4}, %5;" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w), "l"(policy)
                 : "memory");
}

}  // namespace granq
