// On-chip staged GranQ kernel: one persistent cooperative launch in which every activation
// is read from HBM exactly once.
//
// The tensor is processed in waves of whole channel groups.  A wave is cut into chunks
// (contiguous runs inside one slab), dealt round-robin to the CTAs, and each CTA pulls its
// chunks into shared memory with bulk asynchronous copies (TMA, no multicast) that complete
// on an mbarrier.  Phase 1 of a wave reduces the staged data to per-group min/max keys
// (Eq. 4): warps combine in shared memory and the last warp of the CTA publishes the
// CTA's keys with global atomics and bumps the wave's arrival counter.  Phase 2 waits for
// that counter to reach the grid size, turns the keys into (s, z) (Eq. 5) and quantizes the
// wave from shared memory (Eq. 1, clamp, Eq. 6) while streaming gy in and y / gx out (STE).
//
// The warps of a CTA are specialised and there is no CTA-wide barrier in the steady state.
// A few reducer warps run phase 1 wave after wave, as far ahead as loaded buffers allow;
// the other (quantizer) warps run phase 2 wave after wave over rows of 128 units (4 per
// lane), fetching the gy packs of their next row before doing the arithmetic of the current
// one.  The last quantizer warp to finish a wave re-fills that wave's buffer with wave
// w + depth.  With depth >= 2 a wave's arrival counter has filled up long before the
// quantizers reach it, so neither the loads nor the grid-wide wait are exposed.
//
// Every wait is bounded: when one runs out the warp records GRANQ_ERR_TIMEOUT in the
// workspace status word and raises the CTA's abort flag; all warps then leave their loops,
// the CTA waits (bounded again) for its own copies in flight and returns.
#include "granq_internal.h"

#include <algorithm>

namespace granq {

namespace {

constexpr int kThreadsPerSm = 512;           // split over the CTAs that share an SM
constexpr uint32_t kDefaultCtasPerSm = 1;
constexpr uint32_t kRowUnits = 128;          // units one warp handles per step: 4 per lane
constexpr uint32_t kReduceWarpsAligned = 2;  // warps of a CTA that run phase 1 (planes of whole packs)
constexpr uint32_t kReduceWarpsRagged = 4;   // ... when packs straddle channels (more work per unit)
constexpr uint32_t kMaxDepth = 3;
constexpr uint32_t kMaxChunks = 64;          // chunks of one wave per CTA
constexpr uint32_t kTabMax = 2048;           // channel groups per wave
constexpr uint32_t kSmemBars = 128;          // mbarriers
constexpr uint32_t kSmemCtl = 128;           // control words
constexpr uint32_t kMbarTries = 1u << 22;    // bounded wait on a bulk-copy barrier
constexpr uint32_t kSpinLimit = 1u << 24;    // bounded wait on a wave counter (x ~64 ns)
constexpr uint32_t kStatusTimeout = 5;       // GRANQ_ERR_TIMEOUT

struct WaveShape {
    uint32_t channels;   // groups in the wave
    uint32_t units;      // 16-byte units of one slab of the wave
    uint32_t cps;        // chunks per slab
    uint32_t nchunks;    // outer * cps
    FastDiv div_cps;
};

// One chunk of a wave as staged by this CTA.
struct ChunkDesc {
    uint32_t gu0;    // global 16-byte unit index of its first unit
    uint32_t su0;    // unit offset inside the wave's slab (gives the channel)
    uint32_t len;    // units
    uint32_t pad;
};

// control words in shared memory
struct Control {
    uint32_t p2_done[kMaxDepth];  // quantizer warps that finished phase 2 on this buffer
    uint32_t issued;              // waves whose loads have been issued
    uint32_t abort;               // a bounded wait ran out somewhere in this CTA
};

struct StagedArgs {
    const void* x;
    const void* gy;
    void* y;
    void* gx;
    uint8_t* codes;
    uint8_t* mask;
    uint32_t* status;
    uint32_t* kmin;
    uint32_t* kmax;
    uint32_t* counters;
    float* lo;
    float* hi;
    float* s_out;
    float* z_out;
    float qmax;
    uint32_t inner;          // elements of one plane
    uint32_t slab_units;     // units of one slab (all channels)
    uint32_t cw;             // channels per regular wave
    uint32_t wave_units;     // units of one slab of a regular wave (= cw * inner / V)
    uint32_t cu;             // units per chunk
    uint32_t rpc;            // rows (of kRowUnits units) per chunk
    uint32_t nwaves, depth, buf_units, tab_entries;
    uint32_t spin_limit, mbar_tries, expected;
    WaveShape shape[2];      // regular wave, last wave
    FastDiv div_rpc;
    FastDiv div_plane;       // units per plane (aligned planes) or elements per plane
};

// ---- mbarrier / bulk copy wrappers -----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// global -> shared bulk copy; src, dst 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst_smem)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_volatile_shared(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}

// ---- chunk bookkeeping ---------------------------------------------------------------------------
struct WaveCtx {
    uint32_t c0;           // first channel
    uint32_t base_units;   // unit offset of the wave's first channel inside a slab
    const WaveShape* sh;
    uint32_t nk;           // chunks of this CTA
};

__device__ __forceinline__ WaveCtx wave_ctx(const StagedArgs& a, uint32_t w) {
    WaveCtx c;
    c.c0 = w * a.cw;
    c.base_units = w * a.wave_units;
    c.sh = &a.shape[(w + 1 == a.nwaves) ? 1 : 0];
    c.nk = (blockIdx.x < c.sh->nchunks) ? (c.sh->nchunks - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u;
    return c;
}

// chunk k of this CTA
__device__ __forceinline__ ChunkDesc chunk_of(const StagedArgs& a, const WaveCtx& c, uint32_t k) {
    uint32_t j = blockIdx.x + k * gridDim.x, slab, ci;
    c.sh->div_cps.divmod(j, slab, ci);
    ChunkDesc d;
    d.su0 = ci * a.cu;
    d.len = min(a.cu, c.sh->units - d.su0);
    d.gu0 = slab * a.slab_units + c.base_units + d.su0;
    d.pad = 0;
    return d;
}

// scale, zero-point and reciprocal of one group from its published keys
__device__ __forceinline__ GroupParam group_param(const StagedArgs& a, uint32_t g, float& lo, float& hi) {
    return group_param_from_keys(a.kmin, a.kmax, g, a.qmax, lo, hi);
}

__device__ __forceinline__ void named_barrier(uint32_t id, uint32_t threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// EXTRAS: the optional per-element codes / mask outputs are compiled in
template <typename T, int MODE, bool ALIGNED, bool EXTRAS, int NT>
__global__ void __launch_bounds__(NT, kThreadsPerSm / NT) staged_kernel(const StagedArgs a) {
    constexpr uint32_t kWarps = NT / 32;
    constexpr uint32_t kRWarps = ALIGNED ? kReduceWarpsAligned : kReduceWarpsRagged;   // reducer warps
    constexpr uint32_t kQWarps = kWarps - kRWarps;                                     // quantizer warps
    constexpr int V = Pack<T>::V;
    constexpr bool kBwd = (MODE & MODE_BWD) != 0;
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);                                        // [depth]
    Control* ctl = reinterpret_cast<Control*>(smem + kSmemBars);
    ChunkDesc* descs = reinterpret_cast<ChunkDesc*>(smem + kSmemBars + kSmemCtl);             // [kMaxDepth][kMaxChunks]
    uint32_t* s_keys = reinterpret_cast<uint32_t*>(descs + kMaxDepth * kMaxChunks);           // [2][2][tab_entries]
    uint4* bufs = reinterpret_cast<uint4*>(s_keys + 4 * a.tab_entries);
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint4* xg = reinterpret_cast<const uint4*>(a.x);
    const uint4* gyg = reinterpret_cast<const uint4*>(a.gy);
    uint4* yg = reinterpret_cast<uint4*>(a.y);
    uint4* gxg = reinterpret_cast<uint4*>(a.gx);
    const uint32_t W = a.nwaves, D = a.depth;

    if (tid == 0) {
        for (uint32_t d = 0; d < D; ++d) mbar_init(&bars[d], 1);
        *ctl = Control{};
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (uint32_t i = tid; i < 4 * a.tab_entries; i += NT) s_keys[i] = 0;
    __syncthreads();

    auto give_up = [&]() {
        if (lane == 0) {
            atomicExch(a.status, kStatusTimeout);
            atomicExch(&ctl->abort, 1u);
        }
    };

    // ---- issue the bulk loads of wave w into its buffer (one warp; one chunk per lane and round) ----
    auto issue = [&](uint32_t w) {
        const WaveCtx c = wave_ctx(a, w);
        const uint32_t b = w % D;
        uint64_t* bar = &bars[b];
        uint4* buf = bufs + (size_t)b * a.buf_units;
        ChunkDesc* dsc = descs + b * kMaxChunks;
        uint32_t total = 0;
        for (uint32_t k = lane; k < c.nk; k += 32) {
            const ChunkDesc d = chunk_of(a, c, k);
            dsc[k] = d;
            total += d.len;
        }
        total = __reduce_add_sync(kFullMask, total);
        __syncwarp();
        if (lane == 0) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_expect_tx(bar, total * 16u);      // release: the descriptors are visible to whoever sees the phase
            atomicAdd(&ctl->issued, 1u);
        }
        __syncwarp();
        for (uint32_t k = lane; k < c.nk; k += 32) {
            const ChunkDesc d = dsc[k];
            bulk_load(buf + (size_t)k * a.cu, xg + d.gu0, d.len * 16u, bar);
        }
    };

    // ---- wait (bounded) until the loads of wave w have landed in its buffer ----
    auto wait_loaded = [&](uint32_t w) -> bool {
        uint64_t* bar = &bars[w % D];
        const uint32_t parity = (w / D) & 1u;
        for (uint32_t i = 0; i < a.mbar_tries; ++i) {
            if (mbar_try_wait(bar, parity)) return true;
            if ((i & 63u) == 63u && ld_volatile_shared(&ctl->abort)) return false;
        }
        return false;
    };

    if (warp == 0)
        for (uint32_t w = 0; w < min(D, W); ++w) issue(w);

    if (warp < kRWarps) {
        // =========================== reducer warps: phase 1 of every wave ===========================
        for (uint32_t w = 0; w < W; ++w) {
            const WaveCtx c = wave_ctx(a, w);
            const uint32_t b = w % D, par = w & 1u;
            const uint4* buf = bufs + (size_t)b * a.buf_units;
            const ChunkDesc* dsc = descs + b * kMaxChunks;
            uint32_t* kmn = s_keys + (2 * par) * a.tab_entries;
            uint32_t* kmx = kmn + a.tab_entries;
            const bool landed = __all_sync(kFullMask, wait_loaded(w));
            if (!landed) give_up();
            WarpRun run{kNoGroup, 0u, 0u}, run2{kNoGroup, 0u, 0u};
            const uint32_t rows = landed ? c.nk * a.rpc : 0u;
            for (uint32_t row = warp; row < rows; row += kRWarps) {
                const uint32_t k = a.div_rpc.div(row), rr = row - k * a.rpc;
                const ChunkDesc d = dsc[k];
                const uint32_t r0 = rr * kRowUnits;
                if (r0 >= d.len) continue;
                const uint4* src = buf + (size_t)k * a.cu;
                Pack<T> p[4];
                bool v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t uo = r0 + j * 32 + lane;
                    v[j] = uo < d.len;
                    if (v[j]) p[j].raw = src[uo];
                }
                if constexpr (ALIGNED) {
                    float mn[4], mx[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        mn[j] = INFINITY;
                        mx[j] = -INFINITY;
                        if (v[j]) pack_minmax(p[j], 0, V, mn[j], mx[j]);
                    }
                    const uint32_t ch_first = a.div_plane.div(d.su0 + r0);
                    const uint32_t ch_last = a.div_plane.div(d.su0 + min(r0 + kRowUnits, d.len) - 1);
                    if (ch_first == ch_last) {       // the whole row lies in one channel
                        const float m0 = fminf(fminf(mn[0], mn[1]), fminf(mn[2], mn[3]));
                        const float m1 = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                        run_add(run, v[0], ch_first, ~enc(m0), enc(m1), kmn, kmx);
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t g = a.div_plane.div(d.su0 + r0 + j * 32 + lane);
                            run_add(run, v[j], g, ~enc(mn[j]), enc(mx[j]), kmn, kmx);
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint32_t pl = 0, rem = 0;
                        a.div_plane.divmod((d.su0 + r0 + j * 32 + lane) * V, pl, rem);
                        const int n1 = (int)min((uint32_t)V, a.inner - rem);      // elements of the first channel
                        float mn1 = INFINITY, mx1 = -INFINITY, mn2 = INFINITY, mx2 = -INFINITY;
                        if (v[j]) {
                            pack_minmax(p[j], 0, n1, mn1, mx1);
                            pack_minmax(p[j], n1, V, mn2, mx2);
                        }
                        run_add(run, v[j], pl, ~enc(mn1), enc(mx1), kmn, kmx);
                        run_add(run2, v[j] && n1 < V, pl + 1, ~enc(mn2), enc(mx2), kmn, kmx);
                    }
                }
            }
            run_flush(run, kmn, kmx);               // shared-memory atomics on the wave-local group index
            if constexpr (!ALIGNED) run_flush(run2, kmn, kmx);
            // all reducer warps meet; warp 0 then publishes the groups this CTA touched and arrives
            named_barrier(1, kRWarps * 32);
            const bool aborting = ld_volatile_shared(&ctl->abort) != 0;
            if (warp == 0 && !aborting) {
                for (uint32_t t = lane; t < c.sh->channels; t += 32) {
                    const uint32_t k1 = atomicExch(kmn + t, 0u), k2 = atomicExch(kmx + t, 0u);
                    if (k1 | k2) {
                        atomicMax(a.kmin + c.c0 + t, k1);
                        atomicMax(a.kmax + c.c0 + t, k2);
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    __threadfence();
                    atomicAdd(a.counters + w, 1u);
                }
            }
            if (aborting) break;     // uniform across the reducer warps: the flag was read after their barrier
        }
    } else {
        // =========================== quantizer warps: phase 2 of every wave ===========================
        const uint32_t qwarp = warp - kRWarps;
        const float qmax = a.qmax;
        for (uint32_t w = 0; w < W; ++w) {
            const WaveCtx c = wave_ctx(a, w);
            const uint32_t b = w % D;
            const uint4* buf = bufs + (size_t)b * a.buf_units;
            const ChunkDesc* dsc = descs + b * kMaxChunks;
            // every CTA must have published wave w
            bool ready = true;
            if (lane == 0) {
                ready = false;
                for (uint32_t i = 0; i < a.spin_limit; ++i) {
                    if (ld_acquire(a.counters + w) >= a.expected) {
                        ready = true;
                        break;
                    }
                    if (ld_volatile_shared(&ctl->abort)) break;
                    __nanosleep(64);
                }
            }
            ready = __all_sync(kFullMask, ready) && __all_sync(kFullMask, wait_loaded(w));
            if (!ready) {
                give_up();
                break;
            }
            if (qwarp == 0 && (w % gridDim.x) == blockIdx.x) {       // one warp in the grid reports the wave's groups
                for (uint32_t t = lane; t < c.sh->channels; t += 32) {
                    float lo, hi;
                    const GroupParam gp = group_param(a, c.c0 + t, lo, hi);
                    a.lo[c.c0 + t] = lo;
                    a.hi[c.c0 + t] = hi;
                    if (a.s_out) a.s_out[c.c0 + t] = gp.s;
                    if (a.z_out) a.z_out[c.c0 + t] = gp.z;
                }
            }
            const uint32_t rows = c.nk * a.rpc;

            // a row: where it is, and its gy packs (fetched one row ahead of the arithmetic)
            struct Row {
                ChunkDesc d;
                uint32_t k, r0;
                bool any;
            };
            auto fetch = [&](uint32_t row, Row& r, Pack<T> (&pg)[4]) {
                r.any = row < rows;
                if (!r.any) return;
                r.k = a.div_rpc.div(row);
                r.d = dsc[r.k];
                r.r0 = (row - r.k * a.rpc) * kRowUnits;
                r.any = r.r0 < r.d.len;
                if constexpr (kBwd) {
                    if (r.any) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t uo = r.r0 + j * 32 + lane;
                            if (uo < r.d.len) pg[j].raw = ld_stream_16(gyg + r.d.gu0 + uo);
                        }
                    }
                }
            };
            auto compute = [&](const Row& r, const Pack<T> (&pg)[4]) {
                if (!r.any) return;
                const ChunkDesc d = r.d;
                const uint32_t r0 = r.r0;
                const uint4* src = buf + (size_t)r.k * a.cu;
                // parameters of the channels this row touches: lane l holds channel ch_first + l
                const uint32_t last_u = d.su0 + min(r0 + kRowUnits, d.len) - 1;
                const uint32_t ch_first = ALIGNED ? a.div_plane.div(d.su0 + r0) : a.div_plane.div((d.su0 + r0) * V);
                const uint32_t ch_last = ALIGNED ? a.div_plane.div(last_u) : a.div_plane.div(last_u * V + (V - 1));
                const uint32_t nch = ch_last - ch_first + 1;
                const bool shared_params = nch <= 32;
                GroupParam mine{1.0f, 0.0f, 0.0f};
                if (shared_params && lane < nch) {
                    float lo, hi;
                    mine = group_param(a, c.c0 + ch_first + lane, lo, hi);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t uo = r0 + j * 32 + lane;
                    const bool valid = uo < d.len;
                    uint32_t ci1 = 0, ci2 = 0;
                    int n1 = V;
                    if constexpr (ALIGNED) {
                        ci1 = a.div_plane.div(d.su0 + (valid ? uo : r0));
                        ci2 = ci1;
                    } else {
                        uint32_t rem;
                        a.div_plane.divmod((d.su0 + (valid ? uo : r0)) * V, ci1, rem);
                        n1 = (int)min((uint32_t)V, a.inner - rem);
                        ci2 = min(ci1 + 1, c.sh->channels - 1);
                    }
                    GroupParam g1, g2;
                    if (shared_params) {
                        const uint32_t i1 = ci1 - ch_first, i2 = min(ci2 - ch_first, nch - 1);
                        g1.s = __shfl_sync(kFullMask, mine.s, i1);
                        g1.z = __shfl_sync(kFullMask, mine.z, i1);
                        g1.r = __shfl_sync(kFullMask, mine.r, i1);
                        if constexpr (ALIGNED) {
                            g2 = g1;
                        } else {
                            g2.s = __shfl_sync(kFullMask, mine.s, i2);
                            g2.z = __shfl_sync(kFullMask, mine.z, i2);
                            g2.r = __shfl_sync(kFullMask, mine.r, i2);
                        }
                    } else {
                        float lo, hi;
                        g1 = group_param(a, c.c0 + ci1, lo, hi);
                        g2 = ALIGNED ? g1 : group_param(a, c.c0 + ci2, lo, hi);
                    }
                    if (!valid) continue;
                    Pack<T> px, py, pgx;
                    px.raw = src[uo];
                    uint32_t cb[V / 4] = {}, mb[V / 4] = {};
                    auto element = [&](int i, float t, float s, float z) {
                        float yv;
                        bool in;
                        const float code = quant_from_quotient(t, s, z, qmax, yv, in);
                        py.set(i, yv);
                        if constexpr (kBwd) pgx.set(i, in ? pg[j].get(i) : 0.0f);
                        if constexpr (EXTRAS) {
                            cb[i / 4] |= (uint32_t)code << (8 * (i % 4));
                            mb[i / 4] |= (in ? 1u : 0u) << (8 * (i % 4));
                        }
                    };
                    if ((g1.r != 0.0f) && (g2.r != 0.0f)) {
#pragma unroll
                        for (int i = 0; i < V; ++i) {
                            const bool first = ALIGNED || i < n1;
                            const float s = first ? g1.s : g2.s, z = first ? g1.z : g2.z, rc = first ? g1.r : g2.r;
                            element(i, div_by_scale(px.get(i), s, rc), s, z);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < V; ++i) {
                            const bool first = ALIGNED || i < n1;
                            const float s = first ? g1.s : g2.s, z = first ? g1.z : g2.z;
                            element(i, __fdiv_rn(px.get(i), s), s, z);
                        }
                    }
                    const uint32_t gu = d.gu0 + uo;
                    st_stream_16(yg + gu, py.raw);
                    if constexpr (kBwd) st_stream_16(gxg + gu, pgx.raw);
                    if constexpr (EXTRAS) {
                        if (a.codes) {
#pragma unroll
                            for (int i = 0; i < V / 4; ++i)
                                reinterpret_cast<uint32_t*>(a.codes)[(size_t)gu * (V / 4) + i] = cb[i];
                        }
                        if (kBwd && a.mask) {
#pragma unroll
                            for (int i = 0; i < V / 4; ++i)
                                reinterpret_cast<uint32_t*>(a.mask)[(size_t)gu * (V / 4) + i] = mb[i];
                        }
                    }
                }
            };

            Row ra, rb;
            Pack<T> pa[4], pb[4];
            fetch(qwarp, ra, pa);
            for (uint32_t row = qwarp; row < rows; row += 2 * kQWarps) {
                fetch(row + kQWarps, rb, pb);
                compute(ra, pa);
                fetch(row + 2 * kQWarps, ra, pa);
                compute(rb, pb);
            }

            // the last quantizer warp to leave the buffer re-fills it with wave w + depth
            __syncwarp();
            uint32_t prev = 0;
            if (lane == 0) {
                __threadfence_block();
                prev = atomicAdd(&ctl->p2_done[b], 1u);
            }
            prev = __shfl_sync(kFullMask, prev, 0);
            if (prev == kQWarps - 1) {
                if (lane == 0) atomicExch(&ctl->p2_done[b], 0u);
                __syncwarp();
                if (w + D < W) issue(w + D);
            }
        }
    }
    __syncthreads();
    if (ld_volatile_shared(&ctl->abort)) {
        // let this CTA's outstanding copies land before its shared memory is given away
        const uint32_t n = ld_volatile_shared(&ctl->issued);
        for (uint32_t w = (n > D ? n - D : 0); w < n; ++w) {
            uint64_t* bar = &bars[w % D];
            for (uint32_t i = 0; i < kMbarTries; ++i)
                if (mbar_try_wait(bar, (w / D) & 1u)) break;
        }
    }
}

inline uint32_t gcd_u32(uint32_t a, uint32_t b) {
    while (b) {
        uint32_t t = a % b;
        a = b;
        b = t;
    }
    return a;
}

bool aligned16(const void* p) { return p == nullptr || ((uintptr_t)p & 15) == 0; }

template <typename T, int MODE, bool ALIGNED, bool EXTRAS, int NT>
cudaError_t launch_nt(const StagedPlan& plan, StagedArgs& args, cudaStream_t st) {
    auto kern = staged_kernel<T, MODE, ALIGNED, EXTRAS, NT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
    if (e != cudaSuccess) return e;
    void* params[] = {(void*)&args};
    return cudaLaunchCooperativeKernel((const void*)kern, dim3(plan.grid), dim3(plan.threads), params,
                                       plan.smem_bytes, st);
}

template <typename T, int MODE, bool ALIGNED, bool EXTRAS>
cudaError_t launch_t(const StagedPlan& plan, StagedArgs& args, cudaStream_t st) {
    if (plan.threads == 512) return launch_nt<T, MODE, ALIGNED, EXTRAS, 512>(plan, args, st);
    return launch_nt<T, MODE, ALIGNED, EXTRAS, 256>(plan, args, st);
}

template <typename T, int MODE>
cudaError_t launch_mode(const StagedPlan& plan, StagedArgs& args, bool aligned, bool extras, cudaStream_t st) {
    if (aligned)
        return extras ? launch_t<T, MODE, true, true>(plan, args, st) : launch_t<T, MODE, true, false>(plan, args, st);
    return extras ? launch_t<T, MODE, false, true>(plan, args, st) : launch_t<T, MODE, false, false>(plan, args, st);
}

template <typename T>
cudaError_t launch_dtype(const StagedPlan& plan, StagedArgs& args, int mode, bool aligned, cudaStream_t st) {
    const bool extras = args.codes != nullptr || args.mask != nullptr;
    if (mode == MODE_FWD) return launch_mode<T, MODE_FWD>(plan, args, aligned, extras, st);
    return launch_mode<T, MODE_BOTH>(plan, args, aligned, extras, st);
}

struct DeviceInfo {
    int sms = 0;
    int smem_optin = 0;
};

DeviceInfo device_info(int device) {
    static DeviceInfo cache[64];
    if (device < 0 || device >= 64) device = 0;
    DeviceInfo& d = cache[device];
    if (d.sms == 0) {
        cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
        cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, device);
    }
    return d;
}

uint32_t table_entries(uint32_t cw) { return ((cw + 15u) / 16u) * 16u; }
uint32_t fixed_smem(uint32_t cw) {
    return kSmemBars + kSmemCtl + kMaxDepth * kMaxChunks * (uint32_t)sizeof(ChunkDesc) + 16u * table_entries(cw);
}

}  // namespace

StagedPlan plan_staged(int dtype, const Geom& g, const QuantIO& io, int device, const StagedTuning& tune) {
    const DeviceInfo di = device_info(device);
    return plan_staged_on(dtype, g, io, di.sms, di.smem_optin, tune);
}

// Chooses the wave / chunk geometry.  Cost model: a wave takes as long as its busiest CTA,
// i.e. (chunks per CTA) x (units per chunk rounded up to whole warp rows + a per-copy overhead), plus a
// fixed per-wave overhead.
StagedPlan plan_staged_on(int dtype, const Geom& g, const QuantIO& io, int sm_count, int smem_optin,
                          const StagedTuning& tune) {
    StagedPlan best{};
    best.ok = false;
    const uint32_t V = dtype == 0 ? 4 : 8;
    if (!aligned16(io.x) || !aligned16(io.gy) || !aligned16(io.y) || !aligned16(io.gx)) return best;
    if (((uintptr_t)io.codes & 3) || ((uintptr_t)io.mask & 3)) return best;
    if (g.inner < (int64_t)V || g.inner >= (1ll << 28) || g.C >= (1ll << 28) || g.outer >= (1ll << 28)) return best;
    if ((g.C * g.inner) % V != 0 || g.E / V >= (1ll << 31)) return best;
    if (sm_count <= 0 || smem_optin < 64 * 1024) return best;

    const uint32_t inner = (uint32_t)g.inner, C = (uint32_t)g.C, O = (uint32_t)g.outer;
    const uint32_t q = V / gcd_u32(inner, V);          // waves hold multiples of q channels (16-byte slabs)
    const uint32_t cps_sm = (tune.ctas_per_sm == 1 || tune.ctas_per_sm == 2) ? (uint32_t)tune.ctas_per_sm
                                                                             : kDefaultCtasPerSm;
    const uint32_t full_grid = (uint32_t)sm_count * cps_sm;
    const uint32_t grid = (tune.grid > 0 && (uint32_t)tune.grid < full_grid) ? (uint32_t)tune.grid : full_grid;
    // an SM holds 1 KB more than one CTA may ask for, and reserves 1 KB per resident CTA
    const uint32_t smem_total = cps_sm == 1 ? (uint32_t)smem_optin
                                            : (((uint32_t)smem_optin + 1024u) / cps_sm - 1024u) & ~127u;
    const uint64_t plane_units_x_q = (uint64_t)q * inner / V;   // units of q channels in one slab
    const uint32_t mult_total = C / q;                           // C is a multiple of q (slabs are whole packs)

    double best_cost = 1e300;
    const double wave_overhead = 512.0;   // units-equivalent of per-wave fixed cost
    const double chunk_overhead = 32.0;   // units-equivalent of issuing one bulk copy
    for (uint32_t depth = 1; depth <= kMaxDepth; ++depth) {
        if (tune.depth > 0 && (int)depth != tune.depth) continue;
        if (depth > 1 && best.ok && best.nwaves == 1 && tune.depth == 0) continue;   // a single wave needs no pipeline
        // candidate wave sizes from the largest downwards, until four of them have produced a
        // feasible chunking (imbalance between CTAs can make the largest ones infeasible)
        uint32_t feasible = 0, tried = 0, prev_cw = 0;
        for (uint32_t nw = 1; nw <= mult_total && feasible < 4 && tried < 256; ++nw) {
            if (depth == 1 && nw != 1) break;                    // depth 1 only for a single wave
            const uint32_t cw = ((mult_total + nw - 1) / nw) * q;
            if (cw > kTabMax || cw == prev_cw) continue;
            prev_cw = cw;
            const uint32_t fixed = fixed_smem(cw);
            if (smem_total <= fixed + 2048) continue;
            uint32_t buf_units = (smem_total - fixed) / 16u / depth;
            if (tune.max_buf_units > 0) buf_units = std::min<uint32_t>(buf_units, (uint32_t)tune.max_buf_units);
            if ((uint64_t)grid * buf_units < (uint64_t)O * (cw / q) * plane_units_x_q) continue;   // cannot fit
            ++tried;
            bool any = false;
            const uint32_t nwaves = (C + cw - 1) / cw;
            const uint32_t c_last = C - (nwaves - 1) * cw;
            const uint64_t wu64 = (uint64_t)cw * inner / V, lu64 = (uint64_t)c_last * inner / V;
            if (wu64 >= (1ull << 30)) continue;
            const uint32_t wave_units = (uint32_t)wu64, last_units = (uint32_t)lu64;
            for (uint32_t nk = 1; nk <= kMaxChunks; ++nk) {
                uint64_t cps = ((uint64_t)grid * nk) / O;
                if (cps == 0) continue;
                cps = std::min<uint64_t>(cps, wave_units);
                uint32_t cu = (uint32_t)((wave_units + cps - 1) / cps);
                if ((uint64_t)nk * cu > buf_units) continue;
                const uint32_t cps_r = (wave_units + cu - 1) / cu;
                const uint64_t nk_r = ((uint64_t)O * cps_r + grid - 1) / grid;
                const uint32_t cps_l = (last_units + cu - 1) / cu;
                const uint64_t nk_l = ((uint64_t)O * cps_l + grid - 1) / grid;
                if (nk_r * cu > buf_units || nk_l * cu > buf_units) continue;
                if (nk_r > kMaxChunks || nk_l > kMaxChunks) continue;
                if ((uint64_t)O * cps_r >= (1ull << 30)) continue;
                // a warp works through a chunk in rows of kRowUnits units
                const double row_units = (double)((cu + kRowUnits - 1) / kRowUnits) * kRowUnits;
                double cost = (double)(nwaves - 1) * (double)nk_r * (row_units + chunk_overhead) +
                              (double)nk_l * (row_units + chunk_overhead) +
                              wave_overhead * nwaves * (depth == 2 ? 2.0 : 1.0);
                any = true;
                if (cost < best_cost) {
                    best_cost = cost;
                    best.ok = true;
                    best.grid = (int)grid;
                    best.threads = kThreadsPerSm / (int)cps_sm;
                    best.depth = (int)std::min(depth, nwaves);
                    best.buf_units = buf_units;
                    best.smem_bytes = fixed + depth * buf_units * 16u;
                    best.cw = cw;
                    best.cu = cu;
                    best.nwaves = nwaves;
                }
            }
            if (any) ++feasible;
        }
    }
    return best;
}

cudaError_t launch_staged(const StagedPlan& plan, const QuantIO& io, int mode, int dtype, const Geom& g, int bits,
                          const Workspace& ws, float* lo, float* hi, float* s_opt, float* z_opt,
                          const StagedTuning& tune, cudaStream_t st) {
    const uint32_t V = dtype == 0 ? 4 : 8;
    StagedArgs a{};
    a.x = io.x;
    a.gy = io.gy;
    a.y = io.y;
    a.gx = io.gx;
    a.codes = io.codes;
    a.mask = io.mask;
    a.status = ws.status;
    a.kmin = ws.kmin;
    a.kmax = ws.kmax;
    a.counters = ws.counters;
    a.lo = lo;
    a.hi = hi;
    a.s_out = s_opt;
    a.z_out = z_opt;
    a.qmax = (float)((1 << bits) - 1);
    const uint32_t inner = (uint32_t)g.inner, C = (uint32_t)g.C, O = (uint32_t)g.outer;
    a.inner = inner;
    a.slab_units = (uint32_t)((uint64_t)C * inner / V);
    a.cw = plan.cw;
    a.wave_units = (uint32_t)((uint64_t)plan.cw * inner / V);
    a.cu = plan.cu;
    a.rpc = (plan.cu + kRowUnits - 1) / kRowUnits;
    a.div_rpc = make_fastdiv(a.rpc);
    a.nwaves = plan.nwaves;
    a.depth = (uint32_t)plan.depth;
    a.buf_units = plan.buf_units;
    a.spin_limit = tune.spin_limit > 0 ? (uint32_t)tune.spin_limit : kSpinLimit;
    a.mbar_tries = kMbarTries;
    a.expected = (uint32_t)plan.grid + (uint32_t)(tune.extra_arrivals > 0 ? tune.extra_arrivals : 0);
    a.tab_entries = table_entries(plan.cw);
    const uint32_t c_last = C - (plan.nwaves - 1) * plan.cw;
    const uint32_t ch[2] = {plan.nwaves > 1 ? plan.cw : c_last, c_last};
    for (int i = 0; i < 2; ++i) {
        WaveShape& s = a.shape[i];
        s.channels = ch[i];
        s.units = (uint32_t)((uint64_t)ch[i] * inner / V);
        s.cps = (s.units + plan.cu - 1) / plan.cu;
        s.nchunks = O * s.cps;
        s.div_cps = make_fastdiv(s.cps);
    }
    const bool aligned = (inner % V) == 0;
    a.div_plane = make_fastdiv(aligned ? inner / V : inner);
    if (dtype == 0) return launch_dtype<float>(plan, a, mode, aligned, st);
    return launch_dtype<__nv_bfloat16>(plan, a, mode, aligned, st);
}

}  // namespace granq
