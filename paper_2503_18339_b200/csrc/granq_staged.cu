// On-chip staged GranQ kernel: one persistent cooperative launch in which every activation
// is read from HBM exactly once.
//
// The tensor is processed in waves of whole channel groups.  A wave is cut into chunks
// (contiguous runs inside one slab), dealt round-robin to the CTAs, and each CTA pulls its
// chunks into shared memory with bulk asynchronous copies (TMA, no multicast) that complete
// on an mbarrier.  Phase 1 of a wave reduces the staged data to per-group min/max keys
// (Eq. 4) and publishes them with atomics; a per-wave arrival counter tells when every CTA
// has done so.  Phase 2 turns the keys into (s, z) (Eq. 5) and quantizes the wave from
// shared memory (Eq. 1, clamp, Eq. 6) while streaming gy in and y / gx out (STE).  With
// `depth` buffers per CTA the loads of wave w + depth are in flight, and phase 1 of wave
// w + depth - 1 has already been published, while wave w is quantized, so neither the load
// latency nor the grid-wide wait is exposed.
//
// Every wait is bounded: when one runs out the CTA records GRANQ_ERR_TIMEOUT in the
// workspace status word, waits (bounded again) for its own copies in flight and returns.
#include "granq_internal.h"

#include <algorithm>

namespace granq {

namespace {

constexpr int kStagedThreads = 512;
constexpr int kStagedUnroll = 4;
constexpr uint32_t kMaxDepth = 3;
constexpr uint32_t kTabMax = 2048;           // channel groups per wave (size of the (s, z) table)
constexpr uint32_t kSmemHeader = 128;        // mbarriers
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
    uint32_t nwaves, depth, buf_units, tab_entries;
    uint32_t spin_limit, mbar_tries, expected;
    WaveShape shape[2];      // regular wave, last wave
    FastDiv div_cu;
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
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t tries) {
    for (uint32_t i = 0; i < tries; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
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

// ---- chunk bookkeeping ---------------------------------------------------------------------------
struct WaveCtx {
    uint32_t c0;           // first channel
    uint64_t base_units;   // unit offset of the wave's first channel inside a slab
    const WaveShape* sh;
    uint32_t nk;           // chunks of this CTA
};

__device__ __forceinline__ WaveCtx wave_ctx(const StagedArgs& a, uint32_t w) {
    WaveCtx c;
    c.c0 = w * a.cw;
    c.base_units = (uint64_t)w * a.wave_units;
    c.sh = &a.shape[(w + 1 == a.nwaves) ? 1 : 0];
    c.nk = (blockIdx.x < c.sh->nchunks) ? (c.sh->nchunks - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u;
    return c;
}

// chunk k of this CTA -> (slab, first unit inside the wave's slab, length in units)
__device__ __forceinline__ void chunk_of(const StagedArgs& a, const WaveCtx& c, uint32_t k, uint32_t& slab,
                                         uint32_t& su0, uint32_t& len) {
    uint32_t j = blockIdx.x + k * gridDim.x, ci;
    c.sh->div_cps.divmod(j, slab, ci);
    su0 = ci * a.cu;
    len = min(a.cu, c.sh->units - su0);
}

template <typename T, int MODE, bool ALIGNED>
__global__ void __launch_bounds__(kStagedThreads, 1) staged_kernel(const StagedArgs a) {
    constexpr int V = Pack<T>::V;
    constexpr bool kFwd = (MODE & MODE_FWD) != 0, kBwd = (MODE & MODE_BWD) != 0;
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem);                       // [depth]
    QParam* tab = reinterpret_cast<QParam*>(smem + kSmemHeader);              // [tab_entries]
    uint4* bufs = reinterpret_cast<uint4*>(smem + kSmemHeader + a.tab_entries * sizeof(QParam));
    const uint32_t tid = threadIdx.x;
    const uint4* xg = reinterpret_cast<const uint4*>(a.x);

    if (tid == 0) {
        for (uint32_t d = 0; d < a.depth; ++d) mbar_init(&bars[d], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    uint32_t issued = 0;   // waves whose loads have been issued
    uint32_t reduced = 0;  // waves whose phase 1 is done
    bool ok = true;

    // ---- issue the bulk loads of wave w into its buffer (warp 0, one chunk per lane and round) ----
    auto issue = [&](uint32_t w) {
        if (tid < 32) {
            const WaveCtx c = wave_ctx(a, w);
            uint64_t* bar = &bars[w % a.depth];
            uint4* buf = bufs + (size_t)(w % a.depth) * a.buf_units;
            uint32_t total = 0;
            for (uint32_t k = tid; k < c.nk; k += 32) {
                uint32_t slab, su0, len;
                chunk_of(a, c, k, slab, su0, len);
                total += len;
            }
            total = __reduce_add_sync(kFullMask, total);
            if (tid == 0) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_expect_tx(bar, total * 16u);
            }
            __syncwarp();
            for (uint32_t k = tid; k < c.nk; k += 32) {
                uint32_t slab, su0, len;
                chunk_of(a, c, k, slab, su0, len);
                const uint4* src = xg + ((uint64_t)slab * a.slab_units + c.base_units + su0);
                bulk_load(buf + (size_t)k * a.cu, src, len * 16u, bar);
            }
        }
    };

    // ---- phase 1: staged data -> min/max keys of the wave's groups; then arrive ----
    auto reduce_wave = [&](uint32_t w) -> bool {
        const WaveCtx c = wave_ctx(a, w);
        const uint4* buf = bufs + (size_t)(w % a.depth) * a.buf_units;
        bool landed = mbar_wait_bounded(&bars[w % a.depth], (w / a.depth) & 1u, a.mbar_tries);
        if (!__syncthreads_and(landed)) return false;
        WarpRun run{kNoGroup, 0u, 0u}, run2{kNoGroup, 0u, 0u};
        const uint32_t total = c.nk * a.cu;
        for (uint32_t f0 = 0; f0 < total; f0 += kStagedThreads) {
            const uint32_t f = f0 + tid;
            uint32_t k, uo, slab, su0 = 0, len = 0;
            a.div_cu.divmod(f, k, uo);
            bool valid = f < total;
            if (valid) {
                chunk_of(a, c, k, slab, su0, len);
                valid = uo < len;
            }
            uint32_t g1 = kNoGroup, mn1 = 0, mx1 = 0, g2 = kNoGroup, mn2 = 0, mx2 = 0;
            bool valid2 = false;
            if (valid) {
                Pack<T> p;
                p.raw = buf[f];
                const uint32_t su = su0 + uo;
                if constexpr (ALIGNED) {
                    g1 = c.c0 + a.div_plane.div(su);
#pragma unroll
                    for (int i = 0; i < V; ++i) {
                        uint32_t e = enc(p.get(i));
                        mn1 = max(mn1, ~e);
                        mx1 = max(mx1, e);
                    }
                } else {
                    uint32_t pl, rem;
                    a.div_plane.divmod(su * V, pl, rem);
                    g1 = c.c0 + pl;
                    const uint32_t n1 = min((uint32_t)V, a.inner - rem);   // elements that belong to g1
                    valid2 = n1 < (uint32_t)V;
                    g2 = valid2 ? g1 + 1 : kNoGroup;
#pragma unroll
                    for (int i = 0; i < V; ++i) {
                        uint32_t e = enc(p.get(i));
                        if ((uint32_t)i < n1) {
                            mn1 = max(mn1, ~e);
                            mx1 = max(mx1, e);
                        } else {
                            mn2 = max(mn2, ~e);
                            mx2 = max(mx2, e);
                        }
                    }
                }
            }
            run_add(run, valid, g1, mn1, mx1, a.kmin, a.kmax);
            if constexpr (!ALIGNED) run_add(run2, valid2, g2, mn2, mx2, a.kmin, a.kmax);
        }
        run_flush(run, a.kmin, a.kmax);
        if constexpr (!ALIGNED) run_flush(run2, a.kmin, a.kmax);
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            atomicAdd(a.counters + w, 1u);
        }
        return true;
    };

    // ---- wait until every CTA has published wave w, then build the (s, z) table ----
    auto params_of_wave = [&](uint32_t w) -> bool {
        bool done = true;
        if (tid == 0) {
            done = false;
            for (uint32_t i = 0; i < a.spin_limit; ++i) {
                if (ld_acquire(a.counters + w) >= a.expected) {
                    done = true;
                    break;
                }
                __nanosleep(64);
            }
        }
        if (!__syncthreads_and(done)) return false;
        const WaveCtx c = wave_ctx(a, w);
        const bool writer = (w % gridDim.x) == blockIdx.x;
        for (uint32_t t = tid; t < c.sh->channels; t += kStagedThreads) {
            const uint32_t g = c.c0 + t;
            float lo, hi;
            keys_to_range(__ldcg(a.kmin + g), __ldcg(a.kmax + g), lo, hi);
            const QParam p = make_qparam(lo, hi, a.qmax);
            tab[t] = p;
            if (writer) {
                a.lo[g] = lo;
                a.hi[g] = hi;
                if (a.s_out) a.s_out[g] = p.s;
                if (a.z_out) a.z_out[g] = p.z;
            }
        }
        __syncthreads();
        return true;
    };

    // ---- phase 2: quantize the wave from shared memory ----
    auto quantize_wave = [&](uint32_t w) {
        const WaveCtx c = wave_ctx(a, w);
        const uint4* buf = bufs + (size_t)(w % a.depth) * a.buf_units;
        const uint32_t total = c.nk * a.cu;
        for (uint32_t f0 = 0; f0 < total; f0 += kStagedThreads * kStagedUnroll) {
            uint32_t f[kStagedUnroll], su[kStagedUnroll];
            uint64_t gu[kStagedUnroll];   // global unit index
            bool valid[kStagedUnroll];
            Pack<T> pg[kStagedUnroll];
#pragma unroll
            for (int j = 0; j < kStagedUnroll; ++j) {
                f[j] = f0 + j * kStagedThreads + tid;
                uint32_t k, uo, slab, su0, len;
                a.div_cu.divmod(f[j], k, uo);
                valid[j] = f[j] < total;
                su[j] = 0;
                gu[j] = 0;
                if (valid[j]) {
                    chunk_of(a, c, k, slab, su0, len);
                    valid[j] = uo < len;
                    su[j] = su0 + uo;
                    gu[j] = (uint64_t)slab * a.slab_units + c.base_units + su[j];
                    if constexpr (kBwd) {
                        if (valid[j]) pg[j].raw = ld_stream_16(reinterpret_cast<const uint4*>(a.gy) + gu[j]);
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < kStagedUnroll; ++j) {
                if (!valid[j]) continue;
                Pack<T> px, py, pgx;
                px.raw = buf[f[j]];
                QParam p1, p2;
                uint32_t n1 = V;
                if constexpr (ALIGNED) {
                    p1 = tab[a.div_plane.div(su[j])];
                    p2 = p1;
                } else {
                    uint32_t pl, rem;
                    a.div_plane.divmod(su[j] * V, pl, rem);
                    n1 = min((uint32_t)V, a.inner - rem);
                    p1 = tab[pl];
                    p2 = tab[min(pl + 1, c.sh->channels - 1)];
                }
                uint32_t cb[V / 4] = {}, mb[V / 4] = {};
#pragma unroll
                for (int i = 0; i < V; ++i) {
                    const QParam p = (ALIGNED || (uint32_t)i < n1) ? p1 : p2;
                    float yv;
                    bool in;
                    float code = quant_one(px.get(i), p, a.qmax, yv, in);
                    py.set(i, yv);
                    cb[i / 4] |= (uint32_t)code << (8 * (i % 4));
                    mb[i / 4] |= (in ? 1u : 0u) << (8 * (i % 4));
                    if constexpr (kBwd) pgx.set(i, in ? pg[j].get(i) : 0.0f);
                }
                if constexpr (kFwd) {
                    st_stream_16(reinterpret_cast<uint4*>(a.y) + gu[j], py.raw);
                    if (a.codes) {
#pragma unroll
                        for (int i = 0; i < V / 4; ++i)
                            reinterpret_cast<uint32_t*>(a.codes)[gu[j] * (V / 4) + i] = cb[i];
                    }
                }
                if constexpr (kBwd) {
                    st_stream_16(reinterpret_cast<uint4*>(a.gx) + gu[j], pgx.raw);
                    if (a.mask) {
#pragma unroll
                        for (int i = 0; i < V / 4; ++i)
                            reinterpret_cast<uint32_t*>(a.mask)[gu[j] * (V / 4) + i] = mb[i];
                    }
                }
            }
        }
    };

    // ---- the pipeline ----
    const uint32_t W = a.nwaves, D = a.depth;
    for (; issued < min(D, W); ++issued) issue(issued);
    if (D > 1) {
        const uint32_t npre = min(D - 1, W);
        while (ok && reduced < npre) {
            ok = reduce_wave(reduced);
            if (ok) ++reduced;
        }
    }
    for (uint32_t w = 0; ok && w < W; ++w) {
        if (D == 1) {
            ok = reduce_wave(w);
            if (!ok) break;
            reduced = w + 1;
        }
        ok = params_of_wave(w);
        if (!ok) break;
        quantize_wave(w);
        if (issued < W) {
            __syncthreads();          // every thread is done reading the buffer that is refilled
            issue(issued);
            ++issued;
        }
        if (D > 1 && reduced < W) {
            ok = reduce_wave(reduced);
            if (ok) ++reduced;
        }
    }
    if (!ok) {
        // a bounded wait ran out: flag it, then let this CTA's outstanding copies land before leaving
        if (tid == 0) atomicExch(a.status, kStatusTimeout);
        for (uint32_t w = reduced; w < issued; ++w) mbar_wait_bounded(&bars[w % D], (w / D) & 1u, kMbarTries);
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

template <typename T, int MODE, bool ALIGNED>
cudaError_t launch_t(const StagedPlan& plan, StagedArgs& args, cudaStream_t st) {
    auto kern = staged_kernel<T, MODE, ALIGNED>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
    if (e != cudaSuccess) return e;
    void* params[] = {(void*)&args};
    return cudaLaunchCooperativeKernel((const void*)kern, dim3(plan.grid), dim3(plan.threads), params,
                                       plan.smem_bytes, st);
}

template <typename T>
cudaError_t launch_dtype(const StagedPlan& plan, StagedArgs& args, int mode, bool aligned, cudaStream_t st) {
    if (mode == MODE_FWD)
        return aligned ? launch_t<T, MODE_FWD, true>(plan, args, st) : launch_t<T, MODE_FWD, false>(plan, args, st);
    return aligned ? launch_t<T, MODE_BOTH, true>(plan, args, st) : launch_t<T, MODE_BOTH, false>(plan, args, st);
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

}  // namespace

StagedPlan plan_staged(int dtype, const Geom& g, const QuantIO& io, int device, const StagedTuning& tune) {
    const DeviceInfo di = device_info(device);
    return plan_staged_on(dtype, g, io, di.sms, di.smem_optin, tune);
}

// Chooses the wave / chunk geometry.  Cost model: a wave takes as long as its busiest CTA,
// i.e. (chunks per CTA) x (units per chunk + a per-copy overhead), plus a fixed per-wave overhead.
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
    const uint32_t grid = (uint32_t)((tune.grid > 0 && tune.grid < sm_count) ? tune.grid : sm_count);
    const uint32_t tab_entries = ((std::min(C, kTabMax) + 15u) / 16u) * 16u;
    const uint32_t smem_total = (uint32_t)smem_optin;
    const uint32_t fixed = kSmemHeader + tab_entries * (uint32_t)sizeof(QParam);
    if (smem_total <= fixed + 4096) return best;
    const uint32_t units_total = (smem_total - fixed) / 16u;
    const uint64_t plane_units_x_q = (uint64_t)q * inner / V;   // units of q channels in one slab
    const uint32_t mult_total = C / q;                           // C is a multiple of q (slabs are whole packs)

    double best_cost = 1e300;
    const double wave_overhead = 512.0;   // units-equivalent of per-wave fixed cost
    const double chunk_overhead = 32.0;   // units-equivalent of issuing one bulk copy
    for (uint32_t depth = 1; depth <= kMaxDepth; ++depth) {
        if (tune.depth > 0 && (int)depth != tune.depth) continue;
        uint32_t buf_units = units_total / depth;
        if (tune.max_buf_units > 0) buf_units = std::min<uint32_t>(buf_units, (uint32_t)tune.max_buf_units);
        // largest wave (in multiples of q channels) whose data fits the grid's buffers
        uint64_t cap_units = (uint64_t)grid * buf_units;
        uint64_t max_mult = cap_units / ((uint64_t)O * plane_units_x_q);
        max_mult = std::min<uint64_t>(max_mult, kTabMax / q);
        if (max_mult == 0) continue;
        if (depth == 1 && max_mult < mult_total) continue;        // depth 1 only for a single wave
        if (depth > 1 && max_mult >= mult_total && best.ok && tune.depth == 0) continue;
        const uint32_t waves_min = (uint32_t)((mult_total + max_mult - 1) / max_mult);
        // candidate wave sizes: from the largest that fits downwards, until four of them
        // have produced a feasible chunking (imbalance can make the largest ones infeasible)
        uint32_t feasible = 0, tried = 0, prev_cw = 0;
        for (uint32_t nw = waves_min; nw <= mult_total && feasible < 4 && tried < 256; ++nw) {
            if (depth == 1 && nw != 1) break;
            const uint32_t cw = ((mult_total + nw - 1) / nw) * q;
            if (cw > kTabMax || cw == prev_cw) continue;
            prev_cw = cw;
            ++tried;
            bool any = false;
            const uint32_t nwaves = (C + cw - 1) / cw;
            const uint32_t c_last = C - (nwaves - 1) * cw;
            const uint64_t wu64 = (uint64_t)cw * inner / V, lu64 = (uint64_t)c_last * inner / V;
            if (wu64 >= (1ull << 30)) continue;
            const uint32_t wave_units = (uint32_t)wu64, last_units = (uint32_t)lu64;
            for (uint32_t nk = 1; nk <= 64; ++nk) {
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
                if ((uint64_t)O * cps_r >= (1ull << 30)) continue;
                double cost = (double)(nwaves - 1) * (double)nk_r * (cu + chunk_overhead) +
                              (double)nk_l * (cu + chunk_overhead) +
                              wave_overhead * nwaves * (depth == 2 ? 2.0 : 1.0);
                any = true;
                if (cost < best_cost) {
                    best_cost = cost;
                    best.ok = true;
                    best.grid = (int)grid;
                    best.threads = kStagedThreads;
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
    a.nwaves = plan.nwaves;
    a.depth = (uint32_t)plan.depth;
    a.buf_units = plan.buf_units;
    a.spin_limit = tune.spin_limit > 0 ? (uint32_t)tune.spin_limit : kSpinLimit;
    a.mbar_tries = kMbarTries;
    a.expected = (uint32_t)plan.grid + (uint32_t)(tune.extra_arrivals > 0 ? tune.extra_arrivals : 0);
    a.tab_entries = ((std::min(C, kTabMax) + 15u) / 16u) * 16u;
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
    a.div_cu = make_fastdiv(plan.cu);
    const bool aligned = (inner % V) == 0;
    a.div_plane = make_fastdiv(aligned ? inner / V : inner);
    if (dtype == 0) return launch_dtype<float>(plan, a, mode, aligned, st);
    return launch_dtype<__nv_bfloat16>(plan, a, mode, aligned, st);
}

}  // namespace granq
