// L2-resident-wave GranQ kernel: one persistent cooperative launch with many resident warps
// and no shared-memory staging.
//
// The tensor is processed in waves of whole channel groups, sized (64 MB of x by default)
// so that a wave's x stays in the L2 cache between its two phases.  A wave is cut into tiles (contiguous runs inside one
// slab) dealt round-robin to the CTAs; the same CTA handles a tile in both phases.
//   phase 1 (Eq. 4): read the tile's x with an evict-last L2 policy, reduce to per-group
//                    min/max keys (warp runs -> shared memory -> one global atomic per group
//                    and CTA), then bump the wave's arrival counter;
//   phase 2 (Eq. 5, 1, 6, STE): once the counter shows every CTA has arrived, turn the wave's keys
//                    into a shared-memory table of (s, z, 1/s), read x again (an L2 hit),
//                    stream gy in and y / gx out with evict-first policies.
// Each CTA runs  P1(0);  then for every wave w:  P1(w+1), wait(w), P2(w)  - so a wave's
// counter has had a whole phase to fill up before anybody waits on it.
//
// The wait is bounded: when it runs out the CTA records GRANQ_ERR_TIMEOUT in the workspace
// status word and returns (nothing asynchronous is in flight in this kernel).
#include "granq_internal.h"

#include <algorithm>

namespace granq {

namespace {

constexpr int kLThreads = 256;
constexpr int kLWarps = kLThreads / 32;
constexpr uint32_t kLTabMax = 2048;          // channel groups per wave
constexpr uint32_t kLSpinLimit = 1u << 24;   // bounded wait on a wave counter (x ~64 ns)
constexpr uint32_t kLStatusTimeout = 5;      // GRANQ_ERR_TIMEOUT

struct LShape {
    uint32_t channels;   // groups in the wave
    uint32_t units;      // 16-byte units of one slab of the wave
    uint32_t tps;        // tiles per slab
    uint32_t ntiles;     // outer * tps
    FastDiv div_tps;
};

struct LArgs {
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
    uint32_t inner;        // elements of one plane
    uint32_t slab_units;   // units of one slab (all channels)
    uint32_t cw;           // channels per regular wave
    uint32_t wave_units;   // units of one slab of a regular wave
    uint32_t nwaves;
    uint32_t spin_limit, expected;
    LShape shape[2];       // regular wave, last wave
    FastDiv div_plane;     // units per plane (aligned planes) or elements per plane
};

__device__ __forceinline__ uint32_t l_ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// UPL = 16-byte units per lane and step; a warp handles rows of 32 * UPL consecutive units
template <typename T, int MODE, bool ALIGNED, bool EXTRAS, int UPL>
__global__ void __launch_bounds__(kLThreads, UPL == 2 ? 4 : 3) l2wave_kernel(const LArgs a) {
    constexpr int V = Pack<T>::V;
    constexpr bool kBwd = (MODE & MODE_BWD) != 0;
    constexpr uint32_t kRow = 32 * UPL, kTile = kLWarps * kRow;
    extern __shared__ uint32_t s_keys[];                       // [2][tab] min / max keys, then the wave's parameters
    const uint32_t tab = ((a.cw + 15u) / 16u) * 16u;
    uint32_t* s_kmn = s_keys;
    uint32_t* s_kmx = s_keys + tab;
    float2* s_sz = reinterpret_cast<float2*>(s_keys + 2 * tab);   // [tab] (scale, zero-point)
    float* s_rcp = reinterpret_cast<float*>(s_sz + tab);          // [tab] RN(1 / scale), or 0 = use IEEE division
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint4* xg = reinterpret_cast<const uint4*>(a.x);
    const uint4* gyg = reinterpret_cast<const uint4*>(a.gy);
    uint4* yg = reinterpret_cast<uint4*>(a.y);
    uint4* gxg = reinterpret_cast<uint4*>(a.gx);
    const uint64_t keep = l2_policy_evict_last(), drop = l2_policy_evict_first();
    const uint32_t W = a.nwaves;

    for (uint32_t i = tid; i < 2 * tab; i += kLThreads) s_keys[i] = 0;
    __syncthreads();

    // Tiles are dealt round-robin over the CTAs and the deal carries on from wave to wave, so the
    // CTAs that get one tile more differ from wave to wave; both phases of a wave use the same deal.
    auto first_tile = [&](uint32_t w) -> uint32_t {
        const uint32_t dealt = (uint32_t)(((uint64_t)w * a.shape[0].ntiles) % gridDim.x);
        return (blockIdx.x + gridDim.x - dealt) % gridDim.x;
    };

    // ---- phase 1: this CTA's tiles of wave w -> min / max keys, then arrive ----
    auto phase1 = [&](uint32_t w) {
        const LShape& sh = a.shape[(w + 1 == W) ? 1 : 0];
        const uint32_t c0 = w * a.cw, base = w * a.wave_units;
        WarpRun run{kNoGroup, 0u, 0u}, run2{kNoGroup, 0u, 0u};
        for (uint32_t tile = first_tile(w); tile < sh.ntiles; tile += gridDim.x) {
            uint32_t slab, ti;
            sh.div_tps.divmod(tile, slab, ti);
            const uint32_t r0 = ti * kTile + warp * kRow;
            if (r0 >= sh.units) continue;
            const uint4* src = xg + (slab * a.slab_units + base);
            Pack<T> p[UPL];
            bool v[UPL];
#pragma unroll
            for (int j = 0; j < UPL; ++j) {
                const uint32_t uo = r0 + j * 32 + lane;
                v[j] = uo < sh.units;
                if (v[j]) p[j].raw = ld_hint_16(src + uo, keep);
            }
            if constexpr (ALIGNED) {
                float mn[UPL], mx[UPL];
                float m0 = INFINITY, m1 = -INFINITY;
#pragma unroll
                for (int j = 0; j < UPL; ++j) {
                    mn[j] = INFINITY;
                    mx[j] = -INFINITY;
                    if (v[j]) pack_minmax(p[j], 0, V, mn[j], mx[j]);
                    m0 = fminf(m0, mn[j]);
                    m1 = fmaxf(m1, mx[j]);
                }
                const uint32_t ch_first = a.div_plane.div(r0);
                const uint32_t ch_last = a.div_plane.div(min(r0 + kRow, sh.units) - 1);
                if (ch_first == ch_last) {       // the whole row lies in one channel
                    run_add(run, v[0], ch_first, ~enc(m0), enc(m1), s_kmn, s_kmx);
                } else {
#pragma unroll
                    for (int j = 0; j < UPL; ++j)
                        run_add(run, v[j], a.div_plane.div(r0 + j * 32 + lane), ~enc(mn[j]), enc(mx[j]), s_kmn, s_kmx);
                }
            } else {
#pragma unroll
                for (int j = 0; j < UPL; ++j) {
                    uint32_t pl = 0, rem = 0;
                    a.div_plane.divmod((r0 + j * 32 + lane) * V, pl, rem);
                    const int n1 = (int)min((uint32_t)V, a.inner - rem);      // elements of the first channel
                    float mn1 = INFINITY, mx1 = -INFINITY, mn2 = INFINITY, mx2 = -INFINITY;
                    if (v[j]) {
                        pack_minmax(p[j], 0, n1, mn1, mx1);
                        pack_minmax(p[j], n1, V, mn2, mx2);
                    }
                    run_add(run, v[j], pl, ~enc(mn1), enc(mx1), s_kmn, s_kmx);
                    run_add(run2, v[j] && n1 < V, pl + 1, ~enc(mn2), enc(mx2), s_kmn, s_kmx);
                }
            }
        }
        run_flush(run, s_kmn, s_kmx);
        if constexpr (!ALIGNED) run_flush(run2, s_kmn, s_kmx);
        __syncthreads();
        for (uint32_t t = tid; t < sh.channels; t += kLThreads) {     // publish what this CTA touched
            const uint32_t k1 = atomicExch(s_kmn + t, 0u), k2 = atomicExch(s_kmx + t, 0u);
            if (k1 | k2) {
                atomicMax(a.kmin + c0 + t, k1);
                atomicMax(a.kmax + c0 + t, k2);
            }
        }
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            atomicAdd(a.counters + w, 1u);
        }
    };

    // ---- wait (bounded) until every CTA has published wave w ----
    __shared__ uint32_t s_ready;
    auto wait_wave = [&](uint32_t w) -> bool {
        if (tid == 0) {
            uint32_t ready = 0;
            for (uint32_t i = 0; i < a.spin_limit; ++i) {
                if (l_ld_acquire(a.counters + w) >= a.expected) {
                    ready = 1;
                    break;
                }
                __nanosleep(64);
            }
            s_ready = ready;
            if (!ready) atomicExch(a.status, kLStatusTimeout);
        }
        __syncthreads();
        const bool ok = s_ready != 0;
        __syncthreads();
        return ok;
    };

    // ---- phase 2: this CTA's tiles of wave w, quantized ----
    auto phase2 = [&](uint32_t w) {
        const LShape& sh = a.shape[(w + 1 == W) ? 1 : 0];
        const uint32_t c0 = w * a.cw, base = w * a.wave_units;
        const float qmax = a.qmax;
        // the wave's parameters (Eq. 5), once per CTA; one CTA in the grid also reports them
        const bool writer = (w % gridDim.x) == blockIdx.x;
        for (uint32_t t = tid; t < sh.channels; t += kLThreads) {
            float lo, hi;
            const GroupParam gp = group_param_from_keys(a.kmin, a.kmax, c0 + t, qmax, lo, hi);
            s_sz[t] = make_float2(gp.s, gp.z);
            s_rcp[t] = gp.r;
            if (writer) {
                a.lo[c0 + t] = lo;
                a.hi[c0 + t] = hi;
                if (a.s_out) a.s_out[c0 + t] = gp.s;
                if (a.z_out) a.z_out[c0 + t] = gp.z;
            }
        }
        __syncthreads();
        for (uint32_t tile = first_tile(w); tile < sh.ntiles; tile += gridDim.x) {
            uint32_t slab, ti;
            sh.div_tps.divmod(tile, slab, ti);
            const uint32_t r0 = ti * kTile + warp * kRow;
            if (r0 >= sh.units) continue;
            const uint32_t gbase = slab * a.slab_units + base;
            Pack<T> px[UPL], pg[UPL];
#pragma unroll
            for (int j = 0; j < UPL; ++j) {
                const uint32_t uo = r0 + j * 32 + lane;
                if (uo < sh.units) {
                    px[j].raw = ld_hint_16(xg + gbase + uo, drop);
                    if constexpr (kBwd) pg[j].raw = ld_hint_16(gyg + gbase + uo, drop);
                }
            }
            // a row that lies in one channel looks its parameters up once
            const uint32_t last_u = min(r0 + kRow, sh.units) - 1;
            const uint32_t ch_first = ALIGNED ? a.div_plane.div(r0) : a.div_plane.div(r0 * V);
            const uint32_t ch_last = ALIGNED ? a.div_plane.div(last_u) : a.div_plane.div(last_u * V + (V - 1));
            const bool one_channel = ch_first == ch_last;
            GroupParam row_g;
            {
                const float2 sz = s_sz[ch_first];
                row_g.s = sz.x;
                row_g.z = sz.y;
                row_g.r = s_rcp[ch_first];
            }
#pragma unroll
            for (int j = 0; j < UPL; ++j) {
                const uint32_t uo = r0 + j * 32 + lane;
                const bool valid = uo < sh.units;
                int n1 = V;
                GroupParam g1 = row_g, g2 = row_g;
                if (!one_channel && valid) {
                    uint32_t ci1, ci2;
                    if constexpr (ALIGNED) {
                        ci1 = a.div_plane.div(uo);
                        ci2 = ci1;
                    } else {
                        uint32_t rem;
                        a.div_plane.divmod(uo * V, ci1, rem);
                        n1 = (int)min((uint32_t)V, a.inner - rem);
                        ci2 = min(ci1 + 1, sh.channels - 1);
                    }
                    const float2 sz1 = s_sz[ci1];
                    g1.s = sz1.x;
                    g1.z = sz1.y;
                    g1.r = s_rcp[ci1];
                    if constexpr (ALIGNED) {
                        g2 = g1;
                    } else {
                        const float2 sz2 = s_sz[ci2];
                        g2.s = sz2.x;
                        g2.z = sz2.y;
                        g2.r = s_rcp[ci2];
                    }
                }
                if (!valid) continue;
                Pack<T> py, pgx;
                uint32_t cb[V / 4], mb[V / 4];
                quantize_pack<T, kBwd, !ALIGNED, EXTRAS, true>(px[j], pg[j], g1, g2, n1, qmax, py, pgx, cb, mb);
                const uint32_t gu = gbase + uo;
                st_hint_16(yg + gu, py.raw, drop);
                if constexpr (kBwd) st_hint_16(gxg + gu, pgx.raw, drop);
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
        }
    };

    // ---- the program of a CTA ----
    phase1(0);
    for (uint32_t w = 0; w < W; ++w) {
        if (w + 1 < W) phase1(w + 1);
        if (!wait_wave(w)) return;
        phase2(w);
    }
}



inline uint32_t l_gcd(uint32_t a, uint32_t b) {
    while (b) {
        uint32_t t = a % b;
        a = b;
        b = t;
    }
    return a;
}

bool l_aligned16(const void* p) { return p == nullptr || ((uintptr_t)p & 15) == 0; }

// CTAs of one instantiation that fit on an SM (queried once per kernel and shared-memory size class)
template <typename K>
int resident_ctas(K kern, uint32_t smem) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, kLThreads, smem) != cudaSuccess) return 0;
    return n;
}

template <typename T, int MODE, bool ALIGNED, bool EXTRAS, int UPL>
cudaError_t l_launch_upl(const L2Plan& plan, LArgs& args, int sm_count, int cta_cap, cudaStream_t st) {
    auto kern = l2wave_kernel<T, MODE, ALIGNED, EXTRAS, UPL>;
    if (plan.smem_bytes > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
        if (e != cudaSuccess) return e;
    }
    int per_sm = resident_ctas(kern, plan.smem_bytes);
    if (per_sm <= 0) return cudaErrorLaunchOutOfResources;
    if (cta_cap > 0 && per_sm > cta_cap) per_sm = cta_cap;
    const int grid = sm_count * per_sm;
    args.expected += (uint32_t)grid;
    void* params[] = {(void*)&args};
    return cudaLaunchCooperativeKernel((const void*)kern, dim3(grid), dim3(kLThreads), params, plan.smem_bytes, st);
}

template <typename T, int MODE, bool ALIGNED, bool EXTRAS>
cudaError_t l_launch_t(const L2Plan& plan, LArgs& args, int sm_count, int cta_cap, cudaStream_t st) {
    if (plan.upl == 4) return l_launch_upl<T, MODE, ALIGNED, EXTRAS, 4>(plan, args, sm_count, cta_cap, st);
    return l_launch_upl<T, MODE, ALIGNED, EXTRAS, 2>(plan, args, sm_count, cta_cap, st);
}

template <typename T, int MODE>
cudaError_t l_launch_mode(const L2Plan& plan, LArgs& a, bool aligned, bool extras, int sms, int cap, cudaStream_t st) {
    if (aligned)
        return extras ? l_launch_t<T, MODE, true, true>(plan, a, sms, cap, st)
                      : l_launch_t<T, MODE, true, false>(plan, a, sms, cap, st);
    return extras ? l_launch_t<T, MODE, false, true>(plan, a, sms, cap, st)
                  : l_launch_t<T, MODE, false, false>(plan, a, sms, cap, st);
}

}  // namespace

// Wave size: the largest whole number of channel groups (in multiples that keep every slab of
// the wave on 16-byte boundaries) whose x bytes stay under the target, then evened out over
// the waves.
L2Plan plan_l2wave(int dtype, const Geom& g, const QuantIO& io, const StagedTuning& tune) {
    L2Plan p{};
    p.ok = false;
    const uint32_t V = dtype == 0 ? 4 : 8;
    if (!l_aligned16(io.x) || !l_aligned16(io.gy) || !l_aligned16(io.y) || !l_aligned16(io.gx)) return p;
    if (((uintptr_t)io.codes & 3) || ((uintptr_t)io.mask & 3)) return p;
    if (g.inner < (int64_t)V || g.inner >= (1ll << 28) || g.C >= (1ll << 28) || g.outer >= (1ll << 28)) return p;
    if ((g.C * g.inner) % V != 0 || g.E / V >= (1ll << 31)) return p;
    const uint32_t inner = (uint32_t)g.inner, C = (uint32_t)g.C;
    const uint32_t q = V / l_gcd(inner, V);
    const uint64_t target = (tune.l2_wave_kb > 0 ? (uint64_t)tune.l2_wave_kb : 64ull * 1024) * 1024;
    const uint64_t group_bytes = (uint64_t)g.outer * inner * (16 / V);           // x bytes of one channel group
    const uint32_t mult_total = C / q;
    uint64_t max_mult = target / (group_bytes * q);
    max_mult = std::max<uint64_t>(1, std::min<uint64_t>(max_mult, kLTabMax / q ? kLTabMax / q : 1));
    if (q > kLTabMax) return p;
    const uint32_t nw = (uint32_t)((mult_total + max_mult - 1) / max_mult);
    p.cw = ((mult_total + nw - 1) / nw) * q;
    p.nwaves = (C + p.cw - 1) / p.cw;
    if ((uint64_t)p.cw * inner / V >= (1ull << 30)) return p;
    // long planes: rows of 128 units lie in one channel and amortise the row set-up; short planes: 64
    p.upl = tune.l2_upl == 4 ? 4 : (tune.l2_upl == 2 ? 2 : ((inner / V) >= 512 ? 4 : 2));
    p.smem_bytes = 20u * (((p.cw + 15u) / 16u) * 16u);     // keys (8 B) and parameters (12 B) per group
    p.ok = true;
    return p;
}

cudaError_t launch_l2wave(const L2Plan& plan, const QuantIO& io, int mode, int dtype, const Geom& g, int bits,
                          const Workspace& ws, float* lo, float* hi, float* s_opt, float* z_opt,
                          const StagedTuning& tune, cudaStream_t st) {
    const uint32_t V = dtype == 0 ? 4 : 8;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    LArgs a{};
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
    a.nwaves = plan.nwaves;
    a.spin_limit = tune.spin_limit > 0 ? (uint32_t)tune.spin_limit : kLSpinLimit;
    a.expected = (uint32_t)(tune.extra_arrivals > 0 ? tune.extra_arrivals : 0);   // + grid, added at launch
    const uint32_t tile_units = (uint32_t)kLWarps * 32u * (uint32_t)plan.upl;
    const uint32_t c_last = C - (plan.nwaves - 1) * plan.cw;
    const uint32_t ch[2] = {plan.nwaves > 1 ? plan.cw : c_last, c_last};
    for (int i = 0; i < 2; ++i) {
        LShape& s = a.shape[i];
        s.channels = ch[i];
        s.units = (uint32_t)((uint64_t)ch[i] * inner / V);
        s.tps = (s.units + tile_units - 1) / tile_units;
        s.ntiles = O * s.tps;
        s.div_tps = make_fastdiv(s.tps);
    }
    const bool aligned = (inner % V) == 0;
    a.div_plane = make_fastdiv(aligned ? inner / V : inner);
    const bool extras = io.codes != nullptr || io.mask != nullptr;
    const int cap = tune.l2_ctas_per_sm;
    if (dtype == 0) {
        if (mode == MODE_FWD) return l_launch_mode<float, MODE_FWD>(plan, a, aligned, extras, sms, cap, st);
        return l_launch_mode<float, MODE_BOTH>(plan, a, aligned, extras, sms, cap, st);
    }
    if (mode == MODE_FWD) return l_launch_mode<__nv_bfloat16, MODE_FWD>(plan, a, aligned, extras, sms, cap, st);
    return l_launch_mode<__nv_bfloat16, MODE_BOTH>(plan, a, aligned, extras, sms, cap, st);
}


}  // namespace granq
