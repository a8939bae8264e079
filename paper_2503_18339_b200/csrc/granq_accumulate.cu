// The accumulation over the integer codes, pointwise (1 x 1) case: Eq. 6 left-hand side and the
// output step of Algorithm 1,
//     y[n][o][p] = sum_c w[o][c] * s_c * (code[n][c][p] - z_c),
// regrouped so that the sum runs over the integer codes themselves (the paper's "pure integer-domain"
// accumulation; Eq. 3 is the contrast, with s_c inside the loop):
//     y = sum_c W'[o][c] * code[c]  -  bias[o],     W' = w * s (scale folded in ONCE, up front),
//                                                   bias[o] = sum_c W'[o][c] * z_c (a rank-one term).
// The first sum is a dense contraction and runs on the 5th-generation tensor cores:
//   - the codes (0 .. 255) are exact in bf16; W' is split into two bf16 matrices hi + lo (hi = the
//     rounding of W', lo = the rounding of the rest; what is left is below 2^-17 |W'|), so two
//     tcgen05.mma per K step accumulate into the same fp32 accumulator in tensor memory;
//   - the codes never exist as a matrix in HBM: the threads of a CTA read the packed bit string, expand the
//     codes of a tile (128 pixels x 64 channels) to bf16 and store them into shared memory in the layout the
//     tensor core reads (rows of 64 bf16, 128-byte swizzle), then make the stores visible to the asynchronous
//     proxy; the two weight halves come by TMA tile loads of this GPU's own memory (same swizzle, no
//     multicast); a ring of stages is handed back and forth through mbarriers;
//   - one elected thread issues the MMAs; the accumulator (128 pixels x BN output channels) lives in
//     tensor memory and is read back with tcgen05.ld for the epilogue, which subtracts the bias and
//     stores y in the layout of the input (NCHW or channels-last).
// Two launches: weights (W' hi / lo, bias), then expansion + contraction + epilogue in one kernel.  Every wait
// on an mbarrier is bounded; a wait that runs out records GRANQ_ERR_TIMEOUT in the workspace's status word,
// the CTA skips its remaining work, frees its tensor memory and returns.
#include "../../include/granq.h"

#include "granq_internal.h"

#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>

namespace granq {

namespace {

constexpr int kABm = 128;                 // pixels per tile (rows of the accumulator = tensor-memory lanes)
constexpr int kABk = 64;                  // channels per stage: 64 bf16 = one 128-byte swizzle row
constexpr int kAMaxStages = 4;         // the ring is as deep as the K blocks need, at most this
constexpr int kAThreads = 128;            // all four warps expand codes and run the epilogue; thread 0 loads the
                                          // weights, thread 32 issues the MMAs
constexpr uint32_t kASpin = 1u << 22;     // bounded mbarrier wait
constexpr uint32_t kATimeout = 5;         // GRANQ_ERR_TIMEOUT

__device__ __forceinline__ uint32_t a_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void a_mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a_smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void a_mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(a_smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool a_mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(a_smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void a_mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(a_smem_u32(bar)) : "memory");
}
// 2-d tile load of this GPU's own memory (no multicast): coordinates (x = innermost element, y = row)
__device__ __forceinline__ void a_tma_load_2d(void* dst_smem, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::
            "r"(a_smem_u32(dst_smem)),
        "l"(map), "r"(a_smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}
// K-major operand tile in shared memory, 128-byte swizzle: rows of 64 bf16, groups of 8 rows 1024 bytes apart
__device__ __forceinline__ uint64_t a_smem_desc(const void* tile) {
    uint64_t d = 0;
    d |= (uint64_t)((a_smem_u32(tile) >> 4) & 0x3FFF);      // start address, 16-byte units
    d |= (uint64_t)1 << 16;                                  // leading byte offset (unused with a swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;                        // stride byte offset: next group of 8 rows
    d |= (uint64_t)1 << 46;                                  // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                                  // 128-byte swizzle
    return d;
}
// bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n
__device__ __forceinline__ uint32_t a_instr_desc(uint32_t n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((uint32_t)(kABm >> 4) << 24);
}
__device__ __forceinline__ void a_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// the mbarrier gets one arrival when every MMA issued so far by this thread has completed
__device__ __forceinline__ void a_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(a_smem_u32(bar))
                 : "memory");
}

struct AArgs {
    float* y;
    const float* bias;
    uint32_t* status;
    const uint32_t* packed;   // the codes as a bit string, b bits each, in the storage order of the tensor
    int64_t nwords;           // 32-bit words of the bit string
    int64_t rows;             // pixels of the whole batch
    int64_t P;                // pixels of one sample
    int64_t C;                // input channels
    int64_t O;                // output channels
    int bits;
    int kblocks;              // ceil(C / 64)
    int stages;               // depth of the ring of operand stages
    uint32_t spin_limit;
};

// code e of a bit string of b-bit codes (element e in bits [e*b, (e+1)*b), little-endian words)
__device__ __forceinline__ uint32_t a_code_at(const uint32_t* __restrict__ packed, int64_t e, int bits) {
    const int64_t bit = e * bits;
    const int64_t word = bit >> 5;
    const int sh = (int)(bit & 31);
    uint32_t v = __ldg(packed + word) >> sh;
    if (sh + bits > 32) v |= __ldg(packed + word + 1) << (32 - sh);
    return v & ((1u << bits) - 1u);
}

// the `count` (1 .. 8) codes of elements e, e + 1, ... as one 64-bit string (code j in bits [j*b, (j+1)*b)),
// zero above them; reads at most three words, none beyond the end of the bit string
__device__ __forceinline__ uint64_t a_codes8(const uint32_t* __restrict__ packed, int64_t e, int bits, int count,
                                             int64_t nwords) {
    const int64_t bit = e * bits;
    const int64_t w = bit >> 5;
    const uint32_t sh = (uint32_t)(bit & 31);
    const uint32_t need = sh + (uint32_t)(count * bits);
    const uint32_t w0 = __ldg(packed + w);
    uint32_t w1 = 0, w2 = 0;
    if (need > 32 && w + 1 < nwords) w1 = __ldg(packed + w + 1);
    if (need > 64 && w + 2 < nwords) w2 = __ldg(packed + w + 2);
    const uint64_t v = ((uint64_t)__funnelshift_r(w1, w2, sh) << 32) | __funnelshift_r(w0, w1, sh);
    const int keep = count * bits;
    return keep >= 64 ? v : (v & ((1ull << keep) - 1ull));
}

// The same in two steps, so that the loads can be issued long before their words are needed: a_codes8_load() only
// loads (up to three words, none beyond the end of the bit string) and returns the shift; a_codes8_finish() lines
// the codes up at bit 0 and clears what lies above them.
__device__ __forceinline__ uint32_t a_codes8_load(const uint32_t* __restrict__ packed, uint64_t bit, uint32_t nbits,
                                                  int64_t nwords, uint32_t& w0, uint32_t& w1, uint32_t& w2) {
    const int64_t w = (int64_t)(bit >> 5);
    const uint32_t sh = (uint32_t)bit & 31u;
    const uint32_t need = sh + nbits;
    w0 = __ldg(packed + w);
    w1 = (need > 32 && w + 1 < nwords) ? __ldg(packed + w + 1) : 0u;
    w2 = (need > 64 && w + 2 < nwords) ? __ldg(packed + w + 2) : 0u;
    return sh;
}
__device__ __forceinline__ uint64_t a_codes8_finish(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t sh, int keep_bits) {
    const uint64_t v = ((uint64_t)__funnelshift_r(w1, w2, sh) << 32) | __funnelshift_r(w0, w1, sh);
    return keep_bits >= 64 ? v : (v & ((1ull << keep_bits) - 1ull));
}

// two codes -> two bf16 in one word (the first in the low half), exact.  Codes below 128: 0x4300 | code is the
// bf16 number 128 + code, and one packed subtraction of 128 gives the code; 8-bit codes go through fp32.
__device__ __forceinline__ uint32_t a_pair_bf16(uint32_t c0, uint32_t c1, bool wide) {
    if (!wide) {
        const uint32_t biased = c0 | (c1 << 16) | 0x43004300u, bias = 0x43004300u;
        const __nv_bfloat162 d = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&biased),
                                         *reinterpret_cast<const __nv_bfloat162*>(&bias));
        return *reinterpret_cast<const uint32_t*>(&d);
    }
    const float f0 = __fsub_rn(__uint_as_float(0x4B000000u | c0), 8388608.0f);
    const float f1 = __fsub_rn(__uint_as_float(0x4B000000u | c1), 8388608.0f);
    const __nv_bfloat162 d = __floats2bfloat162_rn(f0, f1);
    return *reinterpret_cast<const uint32_t*>(&d);
}

// 16 bytes of an operand row: chunk `chunk` (8 bf16) of row `row` of a K-major tile with the 128-byte swizzle
// (rows of 128 bytes; within each group of 8 rows chunk c of row r sits at position c ^ (r & 7))
__device__ __forceinline__ void a_store_chunk(unsigned char* tile, uint32_t row, uint32_t chunk, const uint32_t (&w)[4]) {
    *reinterpret_cast<uint4*>(tile + row * 128u + ((chunk ^ (row & 7u)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
}

// D[128 pixels x BN] = codes[128 x C] * (hi + lo)[BN x C]^T in tensor memory; y = D - bias.
// NHWC: the bit string is in channels-last order (and so is y), else in NCHW order.
template <int BN, bool NHWC>
__global__ void __launch_bounds__(kAThreads, BN == 64 ? 6 : 4)
accumulate_kernel(const __grid_constant__ CUtensorMap map_hi, const __grid_constant__ CUtensorMap map_lo, const AArgs a) {
    constexpr uint32_t kABytes = kABm * kABk * 2, kBBytes = BN * kABk * 2, kStageBytes = kABytes + 2 * kBBytes;
    extern __shared__ __align__(1024) unsigned char a_smem[];
    __shared__ __align__(8) uint64_t s_full[kAMaxStages], s_empty[kAMaxStages], s_done;
    __shared__ uint32_t s_tmem, s_abort;
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // 1024-byte aligned stage buffers (the swizzle pattern is a function of the address)
    unsigned char* stages = a_smem + ((1024u - (a_smem_u32(a_smem) & 1023u)) & 1023u);
    const int64_t row0 = (int64_t)blockIdx.x * kABm;
    const int col0 = (int)blockIdx.y * BN;

    if (tid == 0) {
        for (int s = 0; s < kAMaxStages; ++s) {
            a_mbar_init(&s_full[s], 1);
            a_mbar_init(&s_empty[s], 1);
        }
        a_mbar_init(&s_done, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {       // BN columns of tensor memory for the accumulator (a power of two >= 32)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(a_smem_u32(&s_tmem)),
                     "r"((uint32_t)BN)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;

    // bounded wait; false when it ran out or another thread of this CTA has given up
    auto wait = [&](uint64_t* bar, uint32_t parity) -> bool {
        for (uint32_t i = 0; i < a.spin_limit; ++i) {
            if (a_mbar_try_wait(bar, parity)) return true;
            if ((i & 1023u) == 1023u && *(volatile uint32_t*)&s_abort) return false;
        }
        atomicExch(a.status, kATimeout);
        *(volatile uint32_t*)&s_abort = 1;
        return false;
    };
    // the same for a whole warp: one lane polls (hundreds of threads polling one barrier word keep the shared-memory
    // atomic unit busy for a microsecond per hand-over), the shuffle hands the outcome and the ordering to the rest
    auto warp_wait = [&](uint64_t* bar, uint32_t parity) -> bool {
        uint32_t ok = 0;
        if (lane == 0) ok = wait(bar, parity) ? 1u : 0u;
        return __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
    };

    // ---- this thread's share of a tile of codes: 8 of its 1024 sixteen-byte chunks ----
    const int bits = a.bits;
    const bool wide = bits == 8;
    const uint32_t code_mask = (1u << bits) - 1u;
    const uint32_t cg = tid & 7;                 // which 8 of the stage's 64 channels
    // NCHW: rows 8 q .. 8 q + 7 (q = tid / 8), whose codes are consecutive in the bit string for each channel when
    // they lie in one sample
    const int64_t gp0 = row0 + 8 * (int64_t)(tid >> 3);
    const int64_t n0 = gp0 / a.P, p0 = gp0 - n0 * a.P;
    const bool together = (p0 + 7 < a.P) && (gp0 + 7 < a.rows);
    auto expand = [&](unsigned char* tile, int kb) {
        const int64_t c0 = (int64_t)kb * kABk + 8 * cg;
        if constexpr (NHWC) {
            const int count = (int)min((int64_t)8, a.C - c0);
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const uint32_t row = (tid >> 3) + 16u * r;
                const int64_t gp = row0 + row;
                uint64_t v = 0;
                if (gp < a.rows && count > 0) v = a_codes8(a.packed, gp * a.C + c0, bits, count, a.nwords);
                uint32_t w[4];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const uint32_t e0 = (uint32_t)v & code_mask;
                    v >>= bits;
                    const uint32_t e1 = (uint32_t)v & code_mask;
                    v >>= bits;
                    w[h] = a_pair_bf16(e0, e1, wide);
                }
                a_store_chunk(tile, row, cg, w);
            }
        } else {
            uint64_t v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int64_t c = c0 + i;
                v[i] = 0;
                if (c < a.C && gp0 < a.rows) {
                    if (together) {
                        v[i] = a_codes8(a.packed, (n0 * a.C + c) * a.P + p0, bits, 8, a.nwords);
                    } else {                                     // a sample boundary or the end of the batch inside
                        for (int j = 0; j < 8; ++j) {
                            const int64_t gp = gp0 + j;
                            if (gp < a.rows) {
                                const int64_t n = gp / a.P, p = gp - n * a.P;
                                v[i] |= (uint64_t)a_code_at(a.packed, (n * a.C + c) * a.P + p, bits) << (j * bits);
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint32_t w[4];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    w[h] = a_pair_bf16((uint32_t)v[2 * h] & code_mask, (uint32_t)v[2 * h + 1] & code_mask, wide);
                    v[2 * h] >>= bits;
                    v[2 * h + 1] >>= bits;
                }
                a_store_chunk(tile, 8u * (tid >> 3) + j, cg, w);
            }
        }
    };

    // ---- main loop over the K blocks: expand the codes, load the weights, multiply ----
    const uint32_t idesc = a_instr_desc(BN);
    bool ok = true;
    for (int kb = 0; kb < a.kblocks; ++kb) {
        const int s = kb % a.stages;
        if (kb >= a.stages) {            // the MMAs that read this stage have completed
            ok = __syncthreads_and(warp_wait(&s_empty[s], (uint32_t)((kb / a.stages - 1) & 1)) ? 1 : 0) != 0;
            if (!ok) break;
        }
        unsigned char* st = stages + (size_t)s * kStageBytes;
        if (tid == 0) {
            a_mbar_expect_tx(&s_full[s], 2 * kBBytes);
            a_tma_load_2d(st + kABytes, &map_hi, kb * kABk, col0, &s_full[s]);
            a_tma_load_2d(st + kABytes + kBBytes, &map_lo, kb * kABk, col0, &s_full[s]);
        }
        expand(st, kb);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the stores above, for the tensor core
        __syncthreads();
        if (tid == 32) {
            // per stage 4 K steps of 16, each against the hi and the lo half of the weights
            if (wait(&s_full[s], (uint32_t)((kb / a.stages) & 1))) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t dq = a_smem_desc(st), dh = a_smem_desc(st + kABytes), dl = a_smem_desc(st + kABytes + kBBytes);
#pragma unroll
                for (int k = 0; k < kABk / 16; ++k) {        // 16 bf16 = 32 bytes = 2 sixteen-byte units along K
                    a_mma(tmem, dq + 2 * k, dh + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    a_mma(tmem, dq + 2 * k, dl + 2 * k, idesc, 1u);
                }
                a_commit(&s_empty[s]);       // the stage may be refilled once these MMAs have read it
                if (kb + 1 == a.kblocks) a_commit(&s_done);      // the accumulator is final when this arrives
            }
        }
    }
    __syncwarp();

    // ---- epilogue: warp w reads lanes 32 w .. 32 w + 31 of the accumulator, 32 columns at a time ----
    const bool done = ok && warp_wait(&s_done, 0);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int64_t gp = row0 + warp * 32 + lane;      // this thread's pixel, over the whole batch
    const int64_t n = gp / a.P, p = gp - n * a.P;
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
        uint32_t v[32];
        const uint32_t taddr = tmem + ((warp * 32u) << 16) + (uint32_t)c;
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
            "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,"
            "%30,%31}, [%32];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
              "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
              "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
              "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
            : "r"(taddr)
            : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (done && gp < a.rows) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const int64_t o = (int64_t)col0 + c + j;
                if (o < a.O) {
                    const float val = __fsub_rn(__uint_as_float(v[j]), __ldg(a.bias + o));
                    if constexpr (NHWC) a.y[gp * a.O + o] = val;
                    else a.y[(n * a.O + o) * a.P + p] = val;
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)BN) : "memory");
}

// 16 consecutive columns of this warp's 32 lanes of tensor memory (lane = thread), not yet waited for
__device__ __forceinline__ void a_tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}

// ---- the persistent form: one CTA per SM walks over row tiles, its warps split into three roles ----
//   warps 0 .. 15  four groups of 128 threads expand codes into a ring of operand stages, turn and turn about
//                  (loading and converting is a chain of dependent integer instructions and memory latency, so
//                  it is warps, not issue slots, that are short);
//   warp  16       one thread loads both weight halves for all K blocks once (TMA) and issues every MMA
//                  (4 per K block);
//   warps 17 .. 24 two groups of four warps take the finished accumulators in turn (a warp reads the 32 lanes of
//                  its quarter, warp % 4, 16 columns of each half at a time), add the halves, subtract the bias and
//                  store y; while one group stores, the other reads tensor memory.
// Both weight halves sit one after the other in shared memory and are multiplied as ONE operand of 2 BN columns
// (an MMA of 128 x 64 x 16 spends its time fetching the 128 x 16 code operand, not computing: with both halves
// behind one fetch the tensor core is busy half as long); the epilogue adds the two column blocks.
// The CTA owns all 512 columns of its SM's tensor memory: 512 / (2 BN) accumulators in turn, so the MMAs run
// tiles ahead of the epilogue (a hand-over from the tensor core to the epilogue and back costs about a
// microsecond; with two accumulators that latency, not the work, set the pace).  Needs the weight halves of
// all K blocks resident in shared memory.
constexpr int kPStages = 6;               // operand stages of 128 x 64 codes
constexpr int kPTmemCols = 512;           // all of an SM's tensor memory
constexpr int kPGroups = 4;                // groups of 128 threads that expand codes, turn and turn about
constexpr int kPProducers = 128 * kPGroups;
constexpr int kPEpilogue = 256;           // threads that read accumulators out and store y
constexpr int kPThreads = kPProducers + 32 + kPEpilogue;
constexpr size_t kPWeightBytes = 128 * 1024;      // resident weight halves at most (channels-last: 16 KB less,
                                                  // which the epilogue's staging tiles take)

struct PBars {
    uint64_t a_full[kPStages], a_empty[kPStages], acc_full[8], acc_empty[8], b_full;
};

template <int BN, bool NHWC>
__global__ void __launch_bounds__(kPThreads, 1)
accumulate_persistent_kernel(const __grid_constant__ CUtensorMap map_hi, const __grid_constant__ CUtensorMap map_lo,
                             const AArgs a) {
    constexpr uint32_t kABytes = kABm * kABk * 2, kBBytes = BN * kABk * 2;
    constexpr int kAcc = kPTmemCols / (2 * BN);    // accumulators (each: BN columns for the hi half, BN for the lo half)
    static_assert(kAcc <= 8, "barriers for at most 8 accumulators");
    // A parity wait tells "the phase before the current one" from "two phases before" no more than a clock tells
    // noon from midnight: whoever waits for completion k of a barrier must know that completion k - 1 has
    // happened.  With an even number of accumulators and two epilogue groups taking tiles in turn every
    // accumulator is read out by one group only, which has itself seen its previous completion; the producers,
    // who share stages between groups, cannot get a whole turn of the ring ahead of the MMAs they wait for.
    static_assert(kAcc % 2 == 0 && kPEpilogue == 256, "each accumulator belongs to one of the two epilogue groups");
    extern __shared__ __align__(1024) unsigned char a_smem[];
    __shared__ __align__(8) PBars bars;
    __shared__ float s_bias[BN];
    __shared__ uint32_t s_tmem, s_abort;
    __shared__ __align__(16) float4 s_stage[NHWC ? kPEpilogue / 32 : 1][NHWC ? 128 : 1];      // channels-last epilogue
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    unsigned char* ring = a_smem + ((1024u - (a_smem_u32(a_smem) & 1023u)) & 1023u);
    unsigned char* wts = ring + (size_t)kPStages * kABytes;          // per K block: hi half, lo half
    const int col0 = (int)blockIdx.y * BN;
    const int64_t row_tiles = (a.rows + kABm - 1) / kABm;
    const int kblocks = a.kblocks;
    // this CTA's row tiles: blockIdx.x, blockIdx.x + gridDim.x, ...
    const int my_tiles = (int)((row_tiles - (int64_t)blockIdx.x + gridDim.x - 1) / gridDim.x);
    const int my_iters = my_tiles * kblocks;

    if (tid == 0) {
        for (int s = 0; s < kPStages; ++s) {
            a_mbar_init(&bars.a_full[s], 4);                 // one arrival per warp of a producer group
            a_mbar_init(&bars.a_empty[s], 1);
        }
        for (int b = 0; b < kAcc; ++b) {
            a_mbar_init(&bars.acc_full[b], 1);
            a_mbar_init(&bars.acc_empty[b], 4);     // one arrival per warp of the epilogue group that reads it out
        }
        a_mbar_init(&bars.b_full, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = tid; i < BN; i += kPThreads) s_bias[i] = (col0 + i < a.O) ? a.bias[col0 + i] : 0.0f;
    if (warp == kPProducers / 32) {       // kAcc accumulators of BN columns each
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(a_smem_u32(&s_tmem)),
                     "r"((uint32_t)kPTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;

    // bounded wait; false when it ran out or another thread of this CTA has given up
    auto wait = [&](uint64_t* bar, uint32_t parity) -> bool {
        for (uint32_t i = 0; i < a.spin_limit; ++i) {
            if (a_mbar_try_wait(bar, parity)) return true;
            if ((i & 1023u) == 1023u && *(volatile uint32_t*)&s_abort) return false;
        }
        atomicExch(a.status, kATimeout);
        *(volatile uint32_t*)&s_abort = 1;
        return false;
    };
    // the same for a whole warp: one lane polls (hundreds of threads polling one barrier word keep the shared-memory
    // atomic unit busy for a microsecond per hand-over), the shuffle hands the outcome and the ordering to the rest
    auto warp_wait = [&](uint64_t* bar, uint32_t parity) -> bool {
        uint32_t ok = 0;
        if (lane == 0) ok = wait(bar, parity) ? 1u : 0u;
        return __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
    };

    if (warp < kPProducers / 32) {
        // ---- producers: group g takes the iterations (tile, K block) with it % kPGroups == g ----
        const uint32_t group = tid >> 7, pt = tid & 127;
        const int bits = a.bits;
        const bool wide = bits == 8;
        const uint32_t code_mask = (1u << bits) - 1u;
        const uint32_t cg = pt & 7, rq = pt >> 3;          // 8 channels of the stage's 64; row group
        // The eight code strings of this thread for iteration `it`, as loaded words (three per string) and shifts
        // (5 bits each).  NCHW: 8 channels x rows 8 rq .. 8 rq + 7 (code j of string i = channel i, row j);
        // channels-last: rows rq + 16 r x 8 channels (string r = row).
        struct Raw {
            uint32_t w0[8], w1[8], w2[8];
            uint64_t shifts;
            int keep;                 // bits of a string that hold codes
        };
        // (pixel counts are below 2^31: 32-bit index arithmetic; only bit offsets need 64 bits)
        const uint32_t rows32 = (uint32_t)a.rows, P32 = (uint32_t)a.P, C32 = (uint32_t)a.C;
        // 4-bit codes and strings (8 codes) that are whole words of the bit string: planes (NCHW) or pixels'
        // channel vectors (channels-last) of a multiple of 8 elements
        const bool words4 = bits == 4 && ((NHWC ? C32 : P32) & 7u) == 0;
        auto fetch = [&](int it, Raw& r) {
            const int ti = it / kblocks, kb = it - ti * kblocks;
            const uint32_t row0 = (blockIdx.x + (uint32_t)ti * gridDim.x) * (uint32_t)kABm;
            const uint32_t c0 = (uint32_t)kb * kABk + 8u * cg;
            r.shifts = 0;
            if (words4) {
                // 4-bit codes whose strings are whole, aligned words: one load per string, 32-bit arithmetic throughout
                r.keep = 32;
                if constexpr (NHWC) {
                    const uint32_t* src = a.packed + ((size_t)(row0 + rq) * (C32 >> 3) + (c0 >> 3));
                    const uint32_t stepw = 16u * (C32 >> 3);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        r.w0[i] = (row0 + rq + 16u * i < rows32 && c0 < C32) ? __ldg(src + (size_t)i * stepw) : 0u;
                        r.w1[i] = r.w2[i] = 0;
                    }
                } else {
                    const uint32_t gp0 = row0 + 8u * rq;
                    const uint32_t n0 = gp0 / P32, p0 = gp0 - n0 * P32;
                    const uint32_t* src = a.packed + ((((size_t)n0 * C32 + c0) * P32 + p0) >> 3);
                    const uint32_t stepw = P32 >> 3;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        r.w0[i] = (gp0 < rows32 && c0 + i < C32) ? __ldg(src + (size_t)i * stepw) : 0u;
                        r.w1[i] = r.w2[i] = 0;
                    }
                }
                return;
            }
            if constexpr (NHWC) {
                const uint32_t count = c0 < C32 ? min(8u, C32 - c0) : 0u;
                r.keep = (int)count * bits;
                uint64_t bit = ((uint64_t)(row0 + rq) * C32 + c0) * (uint32_t)bits;
                const uint64_t step = (uint64_t)16 * C32 * (uint32_t)bits;           // 16 rows on
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    r.w0[i] = r.w1[i] = r.w2[i] = 0;
                    if (row0 + rq + 16u * i < rows32 && count > 0)
                        r.shifts |= (uint64_t)a_codes8_load(a.packed, bit, (uint32_t)r.keep, a.nwords, r.w0[i], r.w1[i], r.w2[i])
                                    << (5 * i);
                    bit += step;
                }
            } else {
                const uint32_t gp0 = row0 + 8u * rq;
                const uint32_t n0 = gp0 / P32, p0 = gp0 - n0 * P32;
                const bool together = (p0 + 7 < P32) && (gp0 + 7 < rows32);
                r.keep = 8 * bits;
                uint64_t bit = (((uint64_t)n0 * C32 + c0) * P32 + p0) * (uint32_t)bits;
                const uint64_t step = (uint64_t)P32 * (uint32_t)bits;                 // one channel on
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const uint32_t c = c0 + i;
                    r.w0[i] = r.w1[i] = r.w2[i] = 0;
                    if (c < C32 && gp0 < rows32) {
                        if (together) {
                            r.shifts |= (uint64_t)a_codes8_load(a.packed, bit, (uint32_t)r.keep, a.nwords, r.w0[i], r.w1[i],
                                                                r.w2[i])
                                        << (5 * i);
                        } else if (P32 >= 8) {
                            // a sample boundary or the end of the batch inside: the rows up to the boundary are one run of
                            // this channel's codes in sample n0, the rest the first codes of the channel in sample n0 + 1
                            const uint32_t live = min(8u, rows32 - gp0), first = min(live, P32 - p0), rest = live - first;
                            uint32_t x0, x1, x2;
                            uint32_t sh = a_codes8_load(a.packed, bit, first * (uint32_t)bits, a.nwords, x0, x1, x2);
                            uint64_t v = a_codes8_finish(x0, x1, x2, sh, (int)first * bits);
                            if (rest) {
                                const uint64_t bit2 = (((uint64_t)(n0 + 1) * C32 + c) * P32) * (uint32_t)bits;
                                sh = a_codes8_load(a.packed, bit2, rest * (uint32_t)bits, a.nwords, x0, x1, x2);
                                v |= a_codes8_finish(x0, x1, x2, sh, (int)rest * bits) << (first * (uint32_t)bits);
                            }
                            r.w0[i] = (uint32_t)v;
                            r.w1[i] = (uint32_t)(v >> 32);
                        } else {                                 // planes of fewer than 8 pixels: code by code
                            uint64_t v = 0;
                            for (uint32_t j = 0; j < 8; ++j) {
                                const uint32_t gp = gp0 + j;
                                if (gp < rows32) {
                                    const uint32_t n = gp / P32, p = gp - n * P32;
                                    v |= (uint64_t)a_code_at(a.packed, ((int64_t)n * C32 + c) * P32 + p, bits) << (j * bits);
                                }
                            }
                            r.w0[i] = (uint32_t)v;
                            r.w1[i] = (uint32_t)(v >> 32);
                        }
                    }
                    bit += step;
                }
            }
        };
        auto store = [&](unsigned char* tile, const Raw& r) {
            if (bits == 4) {
                // 4-bit codes: a string is the 8 nibbles of one word.  Even and odd nibbles are spread to bytes with two
                // masks, byte permutes put a pair of codes beside the constant 0x43 (0x43cc is the bf16 number 128 + cc),
                // and one packed subtraction of 128 leaves the two codes as bf16: 13 instructions for 8 codes.
                const uint32_t k43 = 0x43434343u, k128 = 0x43004300u;
                auto two = [&](uint32_t x, uint32_t sel) -> uint32_t {
                    const uint32_t biased = __byte_perm(x, k43, sel);
                    const __nv_bfloat162 d = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&biased),
                                                     *reinterpret_cast<const __nv_bfloat162*>(&k128));
                    return *reinterpret_cast<const uint32_t*>(&d);
                };
                uint32_t u[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    u[i] = __funnelshift_r(r.w0[i], r.w1[i], (uint32_t)(r.shifts >> (5 * i)) & 31u);
                    if (r.keep < 32) u[i] &= (1u << r.keep) - 1u;
                }
                if constexpr (NHWC) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {          // string i = row rq + 16 i, its nibbles = 8 channels
                        const uint32_t lo = u[i] & 0x0F0F0F0Fu, hi = (u[i] >> 4) & 0x0F0F0F0Fu;
                        const uint32_t x01 = __byte_perm(lo, hi, 0x5140), x23 = __byte_perm(lo, hi, 0x7362);
                        const uint32_t w[4] = {two(x01, 0x4140), two(x01, 0x4342), two(x23, 0x4140), two(x23, 0x4342)};
                        a_store_chunk(tile, rq + 16u * i, cg, w);
                    }
                } else {
                    uint32_t w[8][4];                      // [row][pair of channels]
#pragma unroll
                    for (int h = 0; h < 4; ++h) {          // strings 2h, 2h + 1 = two channels, nibble j = row 8 rq + j
                        const uint32_t alo = u[2 * h] & 0x0F0F0F0Fu, ahi = (u[2 * h] >> 4) & 0x0F0F0F0Fu;
                        const uint32_t blo = u[2 * h + 1] & 0x0F0F0F0Fu, bhi = (u[2 * h + 1] >> 4) & 0x0F0F0F0Fu;
                        const uint32_t e01 = __byte_perm(alo, blo, 0x5140), e23 = __byte_perm(alo, blo, 0x7362);    // rows 0 2 | 4 6
                        const uint32_t o01 = __byte_perm(ahi, bhi, 0x5140), o23 = __byte_perm(ahi, bhi, 0x7362);    // rows 1 3 | 5 7
                        w[0][h] = two(e01, 0x4140);
                        w[2][h] = two(e01, 0x4342);
                        w[4][h] = two(e23, 0x4140);
                        w[6][h] = two(e23, 0x4342);
                        w[1][h] = two(o01, 0x4140);
                        w[3][h] = two(o01, 0x4342);
                        w[5][h] = two(o23, 0x4140);
                        w[7][h] = two(o23, 0x4342);
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) a_store_chunk(tile, 8u * rq + j, cg, w[j]);
                }
                return;
            }
            uint64_t v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)
                v[i] = a_codes8_finish(r.w0[i], r.w1[i], r.w2[i], (uint32_t)(r.shifts >> (5 * i)) & 31u, r.keep);
            if constexpr (NHWC) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    uint32_t w[4];
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const uint32_t e0 = (uint32_t)v[i] & code_mask;
                        v[i] >>= bits;
                        const uint32_t e1 = (uint32_t)v[i] & code_mask;
                        v[i] >>= bits;
                        w[h] = a_pair_bf16(e0, e1, wide);
                    }
                    a_store_chunk(tile, rq + 16u * i, cg, w);
                }
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint32_t w[4];
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        w[h] = a_pair_bf16((uint32_t)v[2 * h] & code_mask, (uint32_t)v[2 * h + 1] & code_mask, wide);
                        v[2 * h] >>= bits;
                        v[2 * h + 1] >>= bits;
                    }
                    a_store_chunk(tile, 8u * rq + j, cg, w);
                }
            }
        };
        // One iteration: load the words, wait for the stage, convert and store, publish.  The latency of the loads is
        // covered by the other groups' turns, not by loading ahead: a second set of registers for words in flight
        // cost more (register pressure, and the proxy fence below waits for them anyway) than it brought.
        Raw r;
        for (int it = (int)group; it < my_iters; it += kPGroups) {
            fetch(it, r);
            const int s = it % kPStages;
            // the MMAs that read this stage kPStages iterations ago have completed (passes at once the first time round)
            if (!warp_wait(&bars.a_empty[s], (uint32_t)(((it / kPStages) & 1) ^ 1))) break;
            store(ring + (size_t)s * kABytes, r);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the stores above, for the tensor core
            __syncwarp();
            if (lane == 0) a_mbar_arrive(&bars.a_full[s]);
        }
    } else if (warp == kPProducers / 32) {
        if (lane == 0) {
            // ---- weights once, then every MMA: per K block 4 steps of 16, each against the hi and the lo half ----
            a_mbar_expect_tx(&bars.b_full, (uint32_t)(2 * kBBytes) * (uint32_t)kblocks);
            for (int kb = 0; kb < kblocks; ++kb) {
                a_tma_load_2d(wts + (size_t)kb * 2 * kBBytes, &map_hi, kb * kABk, col0, &bars.b_full);
                a_tma_load_2d(wts + (size_t)kb * 2 * kBBytes + kBBytes, &map_lo, kb * kABk, col0, &bars.b_full);
            }
            const uint32_t idesc = a_instr_desc(2 * BN);        // hi and lo halves as one operand
            bool ok = wait(&bars.b_full, 0);
            int it = 0;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const uint32_t buf = (uint32_t)(t % kAcc);
                // the epilogue has read this accumulator out (passes at once the first time round)
                ok = wait(&bars.acc_empty[buf], (uint32_t)(((t / kAcc) & 1) ^ 1));
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % kPStages;
                    ok = wait(&bars.a_full[s], (uint32_t)((it / kPStages) & 1));
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t dq = a_smem_desc(ring + (size_t)s * kABytes);
                    const uint64_t dw = a_smem_desc(wts + (size_t)kb * 2 * kBBytes);      // 2 BN rows: hi, then lo
#pragma unroll
                    for (int k = 0; k < kABk / 16; ++k)      // 16 bf16 = 32 bytes = 2 sixteen-byte units along K
                        a_mma(tmem + buf * (2 * BN), dq + 2 * k, dw + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    a_commit(&bars.a_empty[s]);       // the stage may be refilled once these MMAs have read it
                }
                if (ok) a_commit(&bars.acc_full[buf]);       // the accumulator is final when this arrives
            }
        }
        __syncwarp();
    } else {
        // ---- epilogue: a warp reads lanes 32 q .. 32 q + 31 (q = warp % 4) of every second accumulator ----
        const uint32_t q = warp & 3u;
        const int egroup = (int)((warp - (kPProducers / 32 + 1)) >> 2);      // two groups of four warps, tiles in turn
        for (int t = egroup; t < my_tiles; t += 2) {
            const uint32_t buf = (uint32_t)(t % kAcc);
            if (!warp_wait(&bars.acc_full[buf], (uint32_t)((t / kAcc) & 1))) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t gp = (blockIdx.x + (uint32_t)t * gridDim.x) * (uint32_t)kABm + q * 32u + lane;      // this thread's pixel
            const uint32_t n = gp / (uint32_t)a.P, p = gp - n * (uint32_t)a.P;
            const bool live = gp < (uint32_t)a.rows;
            // this thread's element of output channel col0: the next channel is P (NCHW) or 1 (channels-last) further
            float* const yrow = NHWC ? a.y + (size_t)gp * (size_t)a.O + col0
                                     : a.y + ((size_t)n * (size_t)a.O + col0) * (size_t)a.P + p;
#pragma unroll 1
            for (int c = 0; c < BN; c += 16) {
                uint32_t vh[16], vl[16];
                const uint32_t taddr = tmem + ((q * 32u) << 16) + buf * (2 * BN) + (uint32_t)c;
                a_tmem_ld16(taddr, vh);              // the hi half's sums
                a_tmem_ld16(taddr + BN, vl);         // the lo half's
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (c + 16 >= BN) {          // this warp's part is in registers: hand the accumulator back
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) a_mbar_arrive(&bars.acc_empty[buf]);
                }
                float f[16];
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    f[j] = __fsub_rn(__fadd_rn(__uint_as_float(vh[j]), __uint_as_float(vl[j])), s_bias[c + j]);
                if constexpr (NHWC) {
                    // channels-last: a thread's 16 values are 64 contiguous bytes of its pixel's row, but the rows of
                    // neighbouring lanes lie O floats apart: stored straight from the registers, every instruction
                    // would touch 32 lines.  The warp passes the chunk through a 2 KB staging tile (quads swizzled
                    // by the row so that neither side has bank conflicts worth naming) and stores 8 rows x 64
                    // bytes per instruction instead.
                    const bool vec = (a.O & 3) == 0 && col0 + c + 16 <= a.O && ((uintptr_t)a.y & 15) == 0;      // same for the warp
                    if (vec) {
                        float4* stg = s_stage[warp - (kPProducers / 32 + 1)];
                        __syncwarp();                                   // the previous chunk has been read out
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            stg[lane * 4 + (j ^ (lane & 3))] = make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
                        __syncwarp();
                        const uint32_t gp_first = gp - lane, quad = lane & 3;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint32_t row = 8u * i + (lane >> 2);
                            const float4 v = stg[row * 4 + (quad ^ (row & 3))];
                            if (gp_first + row < (uint32_t)a.rows)
                                *reinterpret_cast<float4*>(a.y + (size_t)(gp_first + row) * (size_t)a.O + col0 + c + 4 * quad) = v;
                        }
                    } else if (live) {
                        float* out = yrow + c;
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (col0 + c + j < a.O) out[j] = f[j];
                    }
                } else if (live) {
                    {
                        float* out = yrow + (size_t)c * (size_t)a.P;
                        const int left = (int)a.O - col0 - c;          // channels of this chunk that exist
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            if (j < left) *out = f[j];
                            out += (uint32_t)a.P;
                        }
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == kPProducers / 32)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kPTmemCols)
                     : "memory");
}

// W' = w * s in fp32, split into hi + lo (bf16 each), rows padded with zeros to Cpad; one CTA per output channel.
// bias[o] = sum_c (hi + lo)[o][c] * z_c in fp64 (the matrix that is really multiplied), rounded once to fp32.
__global__ void accumulate_weights_kernel(const float* __restrict__ w, const float* __restrict__ s,
                                          const float* __restrict__ z, int C, int Cpad, __nv_bfloat16* hi,
                                          __nv_bfloat16* lo, float* bias) {
    const int o = blockIdx.x;
    double acc = 0.0;
    for (int c = threadIdx.x; c < Cpad; c += blockDim.x) {
        float h = 0.0f, l = 0.0f;
        if (c < C) {
            const float wp = __fmul_rn(w[(size_t)o * C + c], s[c]);
            const __nv_bfloat16 hb = __float2bfloat16_rn(wp);
            h = __bfloat162float(hb);
            const __nv_bfloat16 lb = __float2bfloat16_rn(__fsub_rn(wp, h));
            l = __bfloat162float(lb);
            acc += ((double)h + (double)l) * (double)z[c];
            hi[(size_t)o * Cpad + c] = hb;
            lo[(size_t)o * Cpad + c] = lb;
        } else {
            hi[(size_t)o * Cpad + c] = __float2bfloat16_rn(0.0f);
            lo[(size_t)o * Cpad + c] = __float2bfloat16_rn(0.0f);
        }
    }
    __shared__ double red[32];
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, d);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int i = 0; i < (int)(blockDim.x + 31) / 32; ++i) t += red[i];
        bias[o] = (float)t;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 matrix [rows, cols] (cols contiguous) cut into boxes of 64 columns x box_rows rows, 128-byte swizzle;
// columns and rows beyond the matrix read as zero
bool a_make_map(EncodeTiledFn encode, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols,
                uint32_t box_rows) {
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kABk, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct ALayout {
    int64_t N, C, P, Cpad, rows;
    size_t off_hi, off_lo, off_bias, total;
};

bool a_layout(const int64_t dims[4], int channel_axis, int64_t O, ALayout& L) {
    if (!dims || (channel_axis != 1 && channel_axis != 3) || O <= 0 || O >= (1ll << 24)) return false;
    for (int d = 0; d < 4; ++d)
        if (dims[d] <= 0 || dims[d] >= (1ll << 31)) return false;
    L.N = dims[0];
    L.C = channel_axis == 1 ? dims[1] : dims[3];
    L.P = channel_axis == 1 ? dims[2] * dims[3] : dims[1] * dims[2];
    if (L.C >= (1ll << 20) || L.P >= (1ll << 31) || L.N * L.P >= (1ll << 31)) return false;
    L.Cpad = (L.C + 7) & ~7ll;                 // rows of 16-byte multiples for the tile loads
    L.rows = L.N * L.P;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    L.off_hi = 256;
    L.off_lo = L.off_hi + up((size_t)O * L.Cpad * 2);
    L.off_bias = L.off_lo + up((size_t)O * L.Cpad * 2);
    L.total = L.off_bias + up((size_t)O * 4);
    return true;
}

template <int BN, bool NHWC>
cudaError_t a_launch(const CUtensorMap& mh, const CUtensorMap& ml, const AArgs& args, cudaStream_t st) {
    // a short ring leaves room for several CTAs per SM, whose load / multiply / store chains then overlap
    const size_t smem = (size_t)args.stages * (kABm * kABk * 2 + 2 * BN * kABk * 2) + 1024;
    auto kern = accumulate_kernel<BN, NHWC>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)((args.rows + kABm - 1) / kABm), (unsigned)((args.O + BN - 1) / BN));
    kern<<<grid, kAThreads, smem, st>>>(mh, ml, args);
    return cudaGetLastError();
}

// the persistent form, when the weight halves of all K blocks fit beside the ring of stages
template <int BN, bool NHWC>
cudaError_t p_launch(const CUtensorMap& mh, const CUtensorMap& ml, const AArgs& args, cudaStream_t st) {
    const size_t smem = (size_t)kPStages * kABm * kABk * 2 + (size_t)args.kblocks * 2 * BN * kABk * 2 + 1024;
    auto kern = accumulate_persistent_kernel<BN, NHWC>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const int64_t row_tiles = (args.rows + kABm - 1) / kABm;
    const unsigned col_tiles = (unsigned)((args.O + BN - 1) / BN);
    // one CTA per SM, shared out among the column tiles; no CTA without a row tile
    const unsigned per_col = (unsigned)std::max<int64_t>(1, std::min<int64_t>(row_tiles, sms / (int)std::min<unsigned>(col_tiles, (unsigned)sms)));
    const dim3 grid(per_col, col_tiles);
    kern<<<grid, kPThreads, smem, st>>>(mh, ml, args);
    return cudaGetLastError();
}

}  // namespace

}  // namespace granq

using namespace granq;

extern "C" size_t granq_accumulate_workspace_bytes(const int64_t dims[4], int channel_axis, int64_t out_channels) {
    ALayout L;
    if (!a_layout(dims, channel_axis, out_channels, L)) return 0;
    return L.total;
}

extern "C" int granq_accumulate_codes(const uint32_t* packed_codes, const int64_t dims[4], int channel_axis, int bits,
                                      const float* scale, const float* zp, const float* weights, int64_t out_channels,
                                      float* y, void* workspace, size_t workspace_bytes, uint32_t flags,
                                      void* cuda_stream) {
    ALayout L;
    if (!packed_codes || !scale || !zp || !weights || !y || bits < 1 || bits > 8 || ((uintptr_t)packed_codes & 3) ||
        !a_layout(dims, channel_axis, out_channels, L))
        return GRANQ_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < L.total) return GRANQ_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // the tile-load descriptors are made by the driver: look its encoder up (no link-time dependency on the driver)
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
        return GRANQ_ERR_CUDA;
    EncodeTiledFn encode = (EncodeTiledFn)fn;
    char* ws = (char*)workspace;
    __nv_bfloat16* hi = (__nv_bfloat16*)(ws + L.off_hi);
    __nv_bfloat16* lo = (__nv_bfloat16*)(ws + L.off_lo);
    float* bias = (float*)(ws + L.off_bias);
    // Output channels per tile: 128 when there are more than 64 of them, unless only the narrower tile lets the
    // weight halves of all K blocks stay resident in shared memory (the persistent kernel's condition).
    const int kblocks = (int)((L.Cpad + kABk - 1) / kABk);
    const size_t weight_room = kPWeightBytes - (channel_axis == 3 ? 16 * 1024 : 0);
    auto resident = [&](int bn) { return (size_t)kblocks * 2 * bn * kABk * 2 <= weight_room; };
    const bool one_tile_per_cta = (flags & GRANQ_FLAG_FORCE_TWO_PASS) != 0;
    int BN = out_channels <= 64 ? 64 : 128;
    if (!one_tile_per_cta && BN == 128 && !resident(128) && resident(64)) BN = 64;
    CUtensorMap mh, ml;
    if (!a_make_map(encode, &mh, hi, (uint64_t)out_channels, (uint64_t)L.Cpad, (uint32_t)BN) ||
        !a_make_map(encode, &ml, lo, (uint64_t)out_channels, (uint64_t)L.Cpad, (uint32_t)BN))
        return GRANQ_ERR_CUDA;

    cudaError_t e = cudaMemsetAsync(workspace, 0, sizeof(uint32_t), st);       // the status word
    if (e != cudaSuccess) return GRANQ_ERR_CUDA;
    accumulate_weights_kernel<<<(unsigned)out_channels, 128, 0, st>>>(weights, scale, zp, (int)L.C, (int)L.Cpad, hi, lo,
                                                                    bias);
    if (cudaGetLastError() != cudaSuccess) return GRANQ_ERR_CUDA;
    AArgs args{};
    args.y = y;
    args.bias = bias;
    args.status = (uint32_t*)workspace;
    args.packed = packed_codes;
    args.nwords = (L.rows * L.C * bits + 31) / 32;
    args.rows = L.rows;
    args.P = L.P;
    args.C = L.C;
    args.O = out_channels;
    args.bits = bits;
    args.kblocks = kblocks;
    args.spin_limit = kASpin;
    args.stages = std::min(args.kblocks, 2);
    const bool persistent = !one_tile_per_cta && resident(BN);
    if (persistent) {
        if (channel_axis == 3)
            e = BN == 64 ? p_launch<64, true>(mh, ml, args, st) : p_launch<128, true>(mh, ml, args, st);
        else
            e = BN == 64 ? p_launch<64, false>(mh, ml, args, st) : p_launch<128, false>(mh, ml, args, st);
    } else if (channel_axis == 3) {
        e = BN == 64 ? a_launch<64, true>(mh, ml, args, st) : a_launch<128, true>(mh, ml, args, st);
    } else {
        e = BN == 64 ? a_launch<64, false>(mh, ml, args, st) : a_launch<128, false>(mh, ml, args, st);
    }
    return e == cudaSuccess ? GRANQ_OK : GRANQ_ERR_CUDA;
}
