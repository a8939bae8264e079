// Column-walk GranQ kernel: the L2-resident-wave scheme with a thread-to-channel mapping
// that never changes while a thread works.
//
// In a contiguous [outer, C, inner] tensor the 16-byte unit at offset u of a slab belongs to
// the same channel (or pair of channels, when a unit straddles a plane boundary) in EVERY
// slab.  So a thread is given one unit column u and walks it down a run of slabs:
//   phase 1 (Eq. 4): per-element running min / max stay in registers for the whole walk and
//                    are combined once at its end (warp reduction when the warp lies in one
//                    channel, shared-memory atomics otherwise, then one global atomic per
//                    channel and CTA);
//   phase 2 (Eq. 5, 1, 6, STE): scale, zero-point and reciprocal are worked out once per
//                    walk from the published keys and stay in registers.
// Neither phase divides an index or looks anything up inside the walk.
//
// As in the L2-wave kernel the tensor is cut into waves of whole channel groups that stay in
// L2 between the phases; a wave's work items (column tile x slab chunk) are dealt round-robin
// to the CTAs of one persistent cooperative launch, the same item to the same CTA in both
// phases; each CTA runs  P1(0..lag-1);  for w:  P1(w+lag), wait(w), P2(w).
// The wait is bounded: when it runs out the CTA records GRANQ_ERR_TIMEOUT in the workspace
// status word and returns (nothing asynchronous is in flight in this kernel).
// The kernel expects zeroed keys and counters and, when no wait ran out, leaves them zeroed
// (slot `nwaves` of the counters counts the CTAs that have finished; the last one clears).
#include "granq_internal.h"

#include <algorithm>
#include <atomic>
#include <mutex>

namespace granq {

namespace {

constexpr int kCThreads = 256;
constexpr uint32_t kCSpinLimit = 1u << 24;   // bounded wait on a wave counter (x ~64 ns)
constexpr uint32_t kCStatusTimeout = 5;      // GRANQ_ERR_TIMEOUT
constexpr uint32_t kCTab = 264;              // channels one column tile can touch (inner >= V): 256 + 2, padded

struct CShape {
    uint32_t channels;   // groups in the wave
    uint32_t units;      // 16-byte units of one slab of the wave
    uint32_t ncol;       // column tiles of kCThreads units
    uint32_t chunks;     // slab chunks
    uint32_t nitems;     // ncol * chunks
    FastDiv div_ncol;
};

struct CArgs {
    const void* x;
    const void* gy;
    void* y;
    void* gx;
    uint8_t* codes;
    uint8_t* mask;
    uint32_t* pmask;       // mask at one bit per element, or null
    uint32_t* pcodes;      // the codes as a bit string of code_bits each, or null (forward calls; y is then not written)
    int code_bits;
    double* dist;          // four running sums of Table 2's statistics, or null
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
    uint32_t outer;        // slabs
    uint32_t slab_units;   // units of one slab (all channels)
    uint32_t cw;           // channels per regular wave
    uint32_t wave_units;   // units of one slab of a regular wave
    uint32_t nwaves;
    uint32_t groups;       // channel groups of the tensor
    uint32_t lag;          // waves of phase 1 that run ahead of phase 2
    uint32_t spin_limit, expected;
    CShape shape[2];       // regular wave, last wave
    FastDiv div_plane;     // units per plane (aligned planes) or elements per plane
};

__device__ __forceinline__ uint32_t c_ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// per-element running min / max of one unit column
template <typename T>
struct ColRange {
    float mn[Pack<T>::V], mx[Pack<T>::V];
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int i = 0; i < Pack<T>::V; ++i) {
            mn[i] = INFINITY;
            mx[i] = -INFINITY;
        }
    }
    __device__ __forceinline__ void add(const Pack<T>& p) {
#pragma unroll
        for (int i = 0; i < Pack<T>::V; ++i) {
            const float v = p.get(i);
            mn[i] = fminf(mn[i], v);
            mx[i] = fmaxf(mx[i], v);
        }
    }
    // keys of elements [first, last)
    __device__ __forceinline__ void keys(int first, int last, uint32_t& kmn, uint32_t& kmx) const {
        float a = INFINITY, b = -INFINITY;
#pragma unroll
        for (int i = 0; i < Pack<T>::V; ++i) {
            if (i >= first && i < last) {
                a = fminf(a, mn[i]);
                b = fmaxf(b, mx[i]);
            }
        }
        kmn = (a <= b) ? ~enc(a) : 0u;
        kmx = (a <= b) ? enc(b) : 0u;
    }
};

// U1 / U2 = slabs a thread has in flight in phase 1 / phase 2
template <typename T, int MODE, bool ALIGNED, int EXTRAS, int U1, int U2>
__global__ void __launch_bounds__(kCThreads, 4) colwalk_kernel(const CArgs a) {
    constexpr int V = Pack<T>::V;
    constexpr bool kBwd = (MODE & MODE_BWD) != 0;
    __shared__ uint32_t s_kmn[2][kCTab], s_kmx[2][kCTab];     // double-buffered per-tile keys
    __shared__ uint32_t s_ready;
    const uint32_t tid = threadIdx.x, lane = tid & 31;
    const uint4* xg = reinterpret_cast<const uint4*>(a.x);
    const uint4* gyg = reinterpret_cast<const uint4*>(a.gy);
    uint4* yg = reinterpret_cast<uint4*>(a.y);
    uint4* gxg = reinterpret_cast<uint4*>(a.gx);
    const uint64_t keep = l2_policy_evict_last(), drop = l2_policy_evict_first();
    const uint32_t W = a.nwaves;
    const size_t slab = a.slab_units;

    for (uint32_t i = tid; i < 2 * kCTab; i += kCThreads) {
        (&s_kmn[0][0])[i] = 0;
        (&s_kmx[0][0])[i] = 0;
    }
    __syncthreads();

    // Items are dealt round-robin over the CTAs and the deal carries on from wave to wave, so the
    // CTAs that get one item more differ from wave to wave; both phases of a wave use the same deal.
    auto first_item = [&](uint32_t w) -> uint32_t {
        const uint32_t dealt = (uint32_t)(((uint64_t)w * a.shape[0].nitems) % gridDim.x);
        return (blockIdx.x + gridDim.x - dealt) % gridDim.x;
    };

    // one work item: column tile `col`, slabs [n0, n1); this thread's unit column, its channel
    // (relative to the wave) and how many of the unit's elements lie in that channel
    struct Item {
        uint32_t u, n0, n1, ci, ch_base;
        int ne;
        bool valid;
    };
    auto make_item = [&](const CShape& sh, uint32_t item) -> Item {
        Item it;
        uint32_t chunk, col;
        sh.div_ncol.divmod(item, chunk, col);
        it.n0 = (uint32_t)(((uint64_t)chunk * a.outer) / sh.chunks);
        it.n1 = (uint32_t)(((uint64_t)(chunk + 1) * a.outer) / sh.chunks);
        it.u = col * kCThreads + tid;
        it.valid = it.u < sh.units;
        const uint32_t uu = it.valid ? it.u : sh.units - 1;
        if constexpr (ALIGNED) {
            it.ci = a.div_plane.div(uu);
            it.ne = V;
            it.ch_base = a.div_plane.div(col * kCThreads);
        } else {
            uint32_t rem;
            a.div_plane.divmod(uu * V, it.ci, rem);
            it.ne = (int)min((uint32_t)V, a.inner - rem);
            it.ch_base = a.div_plane.div(col * kCThreads * V);
        }
        return it;
    };

    uint32_t p1_items = 0;      // items this CTA has reduced so far (selects the shared-memory buffer)
    DistAcc dacc;               // Table 2's sums over everything this thread quantizes (EXTRAS only)
    dacc.reset();

    // ---- phase 1: this CTA's items of wave w -> min / max keys, then arrive ----
    auto phase1 = [&](uint32_t w) {
        const CShape& sh = a.shape[(w + 1 == W) ? 1 : 0];
        const uint32_t c0 = w * a.cw, base = w * a.wave_units;
        for (uint32_t item = first_item(w); item < sh.nitems; item += gridDim.x) {
            const Item it = make_item(sh, item);
            ColRange<T> acc;
            acc.reset();
            if (it.valid) {
                const uint4* p = xg + ((size_t)it.n0 * slab + base + it.u);
                uint32_t n = it.n0;
                for (; n + U1 <= it.n1; n += U1) {
                    Pack<T> r[U1];
#pragma unroll
                    for (int j = 0; j < U1; ++j) r[j].raw = ld_hint_16(p + (size_t)j * slab, keep);
#pragma unroll
                    for (int j = 0; j < U1; ++j) acc.add(r[j]);
                    p += (size_t)U1 * slab;
                }
                if (n < it.n1) {                                     // a short last batch, still loaded together
                    Pack<T> r[U1 - 1];
#pragma unroll
                    for (int j = 0; j < U1 - 1; ++j)
                        if (n + j < it.n1) r[j].raw = ld_hint_16(p + (size_t)j * slab, keep);
#pragma unroll
                    for (int j = 0; j < U1 - 1; ++j)
                        if (n + j < it.n1) acc.add(r[j]);
                }
            }
            // combine into this item's shared-memory buffer
            uint32_t* tmn = s_kmn[p1_items & 1];
            uint32_t* tmx = s_kmx[p1_items & 1];
            uint32_t ka, kb;
            acc.keys(0, it.ne, ka, kb);
            if (!it.valid) {
                ka = 0;
                kb = 0;
            }
            const uint32_t rel = it.ci - it.ch_base;
            const uint32_t rel0 = __shfl_sync(kFullMask, rel, 0);
            const bool whole = ALIGNED || it.ne == V;
            if (__all_sync(kFullMask, rel == rel0 && whole)) {      // the warp lies in one channel
                ka = __reduce_max_sync(kFullMask, ka);
                kb = __reduce_max_sync(kFullMask, kb);
                if (lane == 0 && (ka | kb)) {
                    atomicMax(tmn + rel0, ka);
                    atomicMax(tmx + rel0, kb);
                }
            } else if (it.valid) {
                atomicMax(tmn + rel, ka);
                atomicMax(tmx + rel, kb);
                if constexpr (!ALIGNED) {
                    if (it.ne < V) {
                        uint32_t kc, kd;
                        acc.keys(it.ne, V, kc, kd);
                        atomicMax(tmn + rel + 1, kc);
                        atomicMax(tmx + rel + 1, kd);
                    }
                }
            }
            __syncthreads();
            // publish what the tile touched and clear the buffer (it is used again two items on,
            // with the next item's barrier in between)
            for (uint32_t t = tid; t < kCTab; t += kCThreads) {
                const uint32_t k1 = tmn[t], k2 = tmx[t];
                if (k1 | k2) {
                    tmn[t] = 0;
                    tmx[t] = 0;
                    atomicMax(a.kmin + c0 + it.ch_base + t, k1);
                    atomicMax(a.kmax + c0 + it.ch_base + t, k2);
                }
            }
            ++p1_items;
        }
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            atomicAdd(a.counters + w, 1u);
        }
    };

    // ---- wait (bounded) until every CTA has published wave w ----
    auto wait_wave = [&](uint32_t w) -> bool {
        if (tid == 0) {
            uint32_t ready = 0;
            for (uint32_t i = 0; i < a.spin_limit; ++i) {
                if (c_ld_acquire(a.counters + w) >= a.expected) {
                    ready = 1;
                    break;
                }
                __nanosleep(64);
            }
            s_ready = ready;
            if (!ready) atomicExch(a.status, kCStatusTimeout);
        }
        __syncthreads();
        const bool ok = s_ready != 0;
        __syncthreads();
        return ok;
    };

    // ---- phase 2: this CTA's items of wave w, quantized ----
    auto phase2 = [&](uint32_t w) {
        const CShape& sh = a.shape[(w + 1 == W) ? 1 : 0];
        const uint32_t c0 = w * a.cw, base = w * a.wave_units;
        const float qmax = a.qmax;
        if ((w % gridDim.x) == blockIdx.x) {        // one CTA in the grid reports the wave's parameters (Eq. 5)
            for (uint32_t t = tid; t < sh.channels; t += kCThreads) {
                float lo, hi;
                const GroupParam gp = group_param_from_keys(a.kmin, a.kmax, c0 + t, qmax, lo, hi);
                a.lo[c0 + t] = lo;
                a.hi[c0 + t] = hi;
                if (a.s_out) a.s_out[c0 + t] = gp.s;
                if (a.z_out) a.z_out[c0 + t] = gp.z;
            }
        }
        for (uint32_t item = first_item(w); item < sh.nitems; item += gridDim.x) {
            const Item it = make_item(sh, item);
            if (!it.valid) continue;
            size_t gu = (size_t)it.n0 * slab + base + it.u;
            // the channel's parameters (Eq. 5), once per walk
            float lo, hi;
            const GroupParam g1 = group_param_from_keys(a.kmin, a.kmax, c0 + it.ci, qmax, lo, hi);
            GroupParam g2 = g1;
            if constexpr (!ALIGNED) {
                if (it.ne < V) g2 = group_param_from_keys(a.kmin, a.kmax, c0 + it.ci + 1, qmax, lo, hi);
            }
            auto emit = [&](const Pack<T>& px, const Pack<T>& pg, size_t at) {
                Pack<T> py, pgx;
                uint32_t cb[V / 4], mb[V / 4];
                quantize_pack<T, kBwd, !ALIGNED, EXTRAS, true>(px, pg, g1, g2, it.ne, qmax, py, pgx, cb, mb, EXTRAS == 3 ? a.code_bits : 8);
                if constexpr (EXTRAS == 3) {
                    // the packed codes are the only output: 8 codes = b bytes per pair of fp32 lanes (per bf16 lane);
                    // the planner has made every slab and wave whole groups of 8 elements
                    store_code_bytes<V>(a.pcodes, at * V, code_string_of<V>(cb, a.code_bits), a.code_bits, lane);
                    return;
                }
                st_hint_16(yg + at, py.raw, drop);
                if constexpr (kBwd) st_hint_16(gxg + at, pgx.raw, drop);
                if constexpr (EXTRAS != 0) {
                    if constexpr (EXTRAS == 1) {
                        if (a.codes) {
#pragma unroll
                            for (int i = 0; i < V / 4; ++i) reinterpret_cast<uint32_t*>(a.codes)[at * (V / 4) + i] = cb[i];
                        }
                        if (kBwd && a.mask) {
#pragma unroll
                            for (int i = 0; i < V / 4; ++i) reinterpret_cast<uint32_t*>(a.mask)[at * (V / 4) + i] = mb[i];
                        }
                        if (a.dist) dacc.add(px, py);
                    }
                    if (a.pmask) {
                        // the mask is written byte by byte (8 elements: two fp32 packs of neighbouring lanes, one
                        // bf16 pack); the planner has made every slab and wave whole mask words, so both lanes of a
                        // byte are here together
                        store_mask_byte<V>(a.pmask, at * V, mask_bits_of<V, EXTRAS>(mb), lane);
                    }
                }
            };
            uint32_t n = it.n0;
            for (; n + U2 <= it.n1; n += U2) {
                Pack<T> px[U2], pg[U2];
#pragma unroll
                for (int j = 0; j < U2; ++j) {
                    px[j].raw = ld_hint_16(xg + gu + (size_t)j * slab, drop);
                    if constexpr (kBwd) pg[j].raw = ld_hint_16(gyg + gu + (size_t)j * slab, drop);
                }
#pragma unroll
                for (int j = 0; j < U2; ++j) emit(px[j], pg[j], gu + (size_t)j * slab);
                gu += (size_t)U2 * slab;
            }
            if (n < it.n1) {                                         // a short last batch, still loaded together
                Pack<T> px[U2 - 1], pg[U2 - 1];
#pragma unroll
                for (int j = 0; j < U2 - 1; ++j) {
                    if (n + j < it.n1) {
                        px[j].raw = ld_hint_16(xg + gu + (size_t)j * slab, drop);
                        if constexpr (kBwd) pg[j].raw = ld_hint_16(gyg + gu + (size_t)j * slab, drop);
                    }
                }
#pragma unroll
                for (int j = 0; j < U2 - 1; ++j)
                    if (n + j < it.n1) emit(px[j], pg[j], gu + (size_t)j * slab);
            }
        }
    };

    // ---- the program of a CTA ----
    const uint32_t lag = a.lag;
    for (uint32_t w = 0; w < lag && w < W; ++w) phase1(w);
    for (uint32_t w = 0; w < W; ++w) {
        if (w + lag < W) phase1(w + lag);
        if (!wait_wave(w)) return;
        phase2(w);
    }

    if constexpr (EXTRAS == 1) {
        if (a.dist) dacc.flush(a.dist);
    }

    // ---- leave the workspace as it was found: the last CTA to finish clears keys and counters ----
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        s_ready = (atomicAdd(a.counters + W, 1u) == gridDim.x - 1) ? 1u : 0u;
    }
    __syncthreads();
    if (s_ready) {
        for (uint32_t i = tid; i < a.groups; i += kCThreads) {
            a.kmin[i] = 0;
            a.kmax[i] = 0;
        }
        for (uint32_t i = tid; i <= W; i += kCThreads) a.counters[i] = 0;
    }
}

inline uint32_t c_gcd(uint32_t a, uint32_t b) {
    while (b) {
        uint32_t t = a % b;
        a = b;
        b = t;
    }
    return a;
}

bool c_aligned16(const void* p) { return p == nullptr || ((uintptr_t)p & 15) == 0; }

// Slab chunks for a wave of `ncol` column tiles over `outer` slabs on `grid` CTAs: the count that
// minimises the walk of the busiest CTA, a fixed cost per item included.
uint32_t c_pick_chunks(uint32_t ncol, uint32_t outer, uint32_t grid, uint64_t* cost_out = nullptr) {
    const uint64_t kItemCost = 3;      // set-up and combine of one item, in slabs walked
    uint64_t best = ~0ull;
    uint32_t best_k = 1;
    // more than a few items per CTA and wave only adds per-item cost
    const uint32_t kmax = std::min<uint32_t>(std::min<uint32_t>(outer, 4096), 4 * (grid / ncol + 1));
    for (uint32_t k = 1; k <= kmax; ++k) {
        const uint64_t items = (uint64_t)ncol * k;
        const uint64_t per_cta = (items + grid - 1) / grid;
        const uint64_t len = (outer + k - 1) / k;
        const uint64_t cost = per_cta * (len + kItemCost);
        if (cost < best) {
            best = cost;
            best_k = k;
        }
    }
    if (cost_out) *cost_out = best;
    return best_k;
}

// CTAs the planner assumes when it sizes waves (the launch recomputes the chunks for the real grid)
uint32_t c_assumed_grid(int cta_cap) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    const int per_sm = (cta_cap > 0 && cta_cap < 4) ? cta_cap : 4;
    return (uint32_t)(sms * per_sm);
}

template <typename T, int MODE, bool ALIGNED, int EXTRAS>
cudaError_t c_launch_t(CArgs& args, int sm_count, int cta_cap, cudaStream_t st) {
    auto kern = colwalk_kernel<T, MODE, ALIGNED, EXTRAS, 4, 2>;
    // resident CTAs per SM of this instantiation, remembered per device (a pure function of both)
    static std::atomic<int> per_sm_cached[64] = {};
    int dev = 0;
    cudaError_t de = cudaGetDevice(&dev);
    if (de != cudaSuccess) return de;
    int per_sm = (dev >= 0 && dev < 64) ? per_sm_cached[dev].load(std::memory_order_relaxed) : 0;
    if (per_sm == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, kCThreads, 0) != cudaSuccess || n <= 0)
            return cudaErrorLaunchOutOfResources;
        per_sm = n;
        if (dev >= 0 && dev < 64) per_sm_cached[dev].store(n, std::memory_order_relaxed);
    }
    if (cta_cap > 0 && per_sm > cta_cap) per_sm = cta_cap;
    const uint32_t grid = (uint32_t)(sm_count * per_sm);
    for (int i = 0; i < 2; ++i) {
        CShape& s = args.shape[i];
        s.chunks = c_pick_chunks(s.ncol, args.outer, grid);
        s.nitems = s.ncol * s.chunks;
    }
    args.expected += grid;
    void* params[] = {(void*)&args};
    return cudaLaunchCooperativeKernel((const void*)kern, dim3(grid), dim3(kCThreads), params, 0, st);
}

template <typename T, int MODE>
cudaError_t c_launch_mode(CArgs& a, bool aligned, int extras, int sms, int cap, cudaStream_t st) {
    if constexpr (MODE == MODE_FWD) {
        if (extras == 2)       // the packed mask alone: a leaner instantiation of the forward kernel
            return aligned ? c_launch_t<T, MODE, true, 2>(a, sms, cap, st) : c_launch_t<T, MODE, false, 2>(a, sms, cap, st);
        if (extras == 3)       // the packed codes alone
            return aligned ? c_launch_t<T, MODE, true, 3>(a, sms, cap, st) : c_launch_t<T, MODE, false, 3>(a, sms, cap, st);
    }
    if (aligned)
        return extras ? c_launch_t<T, MODE, true, 1>(a, sms, cap, st) : c_launch_t<T, MODE, true, 0>(a, sms, cap, st);
    return extras ? c_launch_t<T, MODE, false, 1>(a, sms, cap, st) : c_launch_t<T, MODE, false, 0>(a, sms, cap, st);
}

}  // namespace

// Wave size: the largest whole number of channel groups (in multiples that keep every slab of
// the wave on 16-byte boundaries) whose x bytes stay under the target, then evened out over
// the waves.  The plan needs slabs to walk: tensors with fewer than kMinOuter slabs are left to
// the other plans.
ColPlan plan_colwalk(int dtype, const Geom& g, const QuantIO& io, const StagedTuning& tune) {
    constexpr int64_t kMinOuter = 8;
    ColPlan p{};
    p.ok = false;
    const uint32_t V = dtype == 0 ? 4 : 8;
    if (!c_aligned16(io.x) || !c_aligned16(io.gy) || !c_aligned16(io.y) || !c_aligned16(io.gx)) return p;
    if (((uintptr_t)io.codes & 3) || ((uintptr_t)io.mask & 3)) return p;
    if (g.outer < kMinOuter || g.outer >= (1ll << 28)) return p;
    if (g.inner < (int64_t)V || g.inner >= (1ll << 28) || g.C >= (1ll << 28)) return p;
    if ((g.C * g.inner) % V != 0 || g.E / V >= (1ll << 31)) return p;
    const uint32_t inner = (uint32_t)g.inner, C = (uint32_t)g.C;
    // waves are whole 16-byte units; with a packed mask also whole 32-element mask words
    if (io.pmask && (((uintptr_t)io.pmask & 3) || (g.C * g.inner) % 32 != 0)) return p;
    // packed codes: nothing else beside them, slabs and waves of whole groups of 8 elements, whole words of codes
    if (io.pcodes && (io.gy || io.codes || io.mask || io.pmask || io.dist || ((uintptr_t)io.pcodes & 3) ||
                      io.code_bits < 1 || io.code_bits > 8 || (g.C * g.inner) % 8 != 0 || g.E % 32 != 0))
        return p;
    const uint32_t q = io.pmask ? 32 / c_gcd(inner, 32) : io.pcodes ? std::max(8 / c_gcd(inner, 8), V / c_gcd(inner, V))
                                                                    : V / c_gcd(inner, V);
    // x bytes of a wave: 32 MB with a gradient (gy and gx stream through the L2 beside the wave), 64 MB without
    // (measured: 3-6 % faster forward-only; larger waves lose to eviction either way)
    const uint64_t target = (tune.l2_wave_kb > 0 ? (uint64_t)tune.l2_wave_kb : (io.gy ? 32ull : 64ull) * 1024) * 1024;
    const uint64_t group_bytes = (uint64_t)g.outer * inner * (16 / V);           // x bytes of one channel group
    const uint32_t mult_total = C / q;
    const uint64_t cap = std::max<uint64_t>(1, ((1ull << 30) / inner) / q);       // keeps cw * inner below 2^30
    const uint64_t max_mult = std::max<uint64_t>(1, std::min<uint64_t>(target / (group_bytes * q), cap));
    if ((uint64_t)q * inner >= (1ull << 30)) return p;
    const uint32_t nw = (uint32_t)((mult_total + max_mult - 1) / max_mult);
    p.cw = ((mult_total + nw - 1) / nw) * q;
    if (tune.l2_wave_kb <= 0 && nw > 1) {
        // Several waves: among the wave sizes from half the target up to the target take the one whose
        // work items load the CTAs most evenly (the busiest CTA's walk, summed over the waves).
        const uint32_t grid = c_assumed_grid(tune.l2_ctas_per_sm);
        // the search is host work on every call: remember the last few answers
        struct Memo {
            uint32_t V, inner, C, grid, q;
            int64_t outer;
            uint64_t target;
            uint32_t cw;
        };
        static Memo memo[8] = {};
        static unsigned memo_next = 0;
        static std::mutex memo_lock;
        bool found = false;
        {
            std::lock_guard<std::mutex> hold(memo_lock);
            for (const Memo& e : memo)
                if (e.cw && e.V == V && e.inner == inner && e.C == C && e.grid == grid && e.q == q && e.outer == g.outer &&
                    e.target == target) {
                    p.cw = e.cw;
                    found = true;
                    break;
                }
        }
        uint64_t best = ~0ull;
        const uint64_t m_lo = std::max<uint64_t>(1, max_mult / 2);
        const uint64_t m_step = std::max<uint64_t>(1, (max_mult - m_lo) / 24);       // at most ~25 candidates
        for (uint64_t m = max_mult; !found && m >= m_lo; m -= std::min(m_step, m - m_lo + 1)) {
            const uint32_t waves = (uint32_t)((mult_total + m - 1) / m);
            const uint32_t m_last = mult_total - (waves - 1) * (uint32_t)m;
            uint64_t c_reg = 0, c_last = 0;
            const uint64_t u_reg = m * q * (uint64_t)inner / V, u_last = (uint64_t)m_last * q * inner / V;
            c_pick_chunks((uint32_t)((u_reg + kCThreads - 1) / kCThreads), (uint32_t)g.outer, grid, &c_reg);
            c_pick_chunks((uint32_t)((u_last + kCThreads - 1) / kCThreads), (uint32_t)g.outer, grid, &c_last);
            const uint64_t total = (waves - 1) * c_reg + c_last;
            if (total < best) {
                best = total;
                p.cw = (uint32_t)m * q;
            }
        }
        if (!found) {
            std::lock_guard<std::mutex> hold(memo_lock);
            memo[memo_next++ % 8] = Memo{V, inner, C, grid, q, g.outer, target, p.cw};
        }
    }
    p.nwaves = (C + p.cw - 1) / p.cw;
    p.lag = tune.l2_lag > 0 ? (uint32_t)tune.l2_lag : 1u;
    p.ok = true;
    return p;
}

cudaError_t launch_colwalk(const ColPlan& plan, const QuantIO& io, int mode, int dtype, const Geom& g, int bits,
                           const Workspace& ws, float* lo, float* hi, float* s_opt, float* z_opt,
                           const StagedTuning& tune, cudaStream_t st) {
    const uint32_t V = dtype == 0 ? 4 : 8;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    CArgs a{};
    a.x = io.x;
    a.gy = io.gy;
    a.y = io.y;
    a.gx = io.gx;
    a.codes = io.codes;
    a.mask = io.mask;
    a.pmask = io.pmask;
    a.pcodes = io.pcodes;
    a.code_bits = io.code_bits;
    a.dist = io.dist;
    a.status = ws.status;
    a.kmin = ws.kmin;
    a.kmax = ws.kmax;
    a.counters = ws.counters;
    a.lo = lo;
    a.hi = hi;
    a.s_out = s_opt;
    a.z_out = z_opt;
    a.qmax = (float)((1 << bits) - 1);
    const uint32_t inner = (uint32_t)g.inner, C = (uint32_t)g.C;
    a.inner = inner;
    a.outer = (uint32_t)g.outer;
    a.slab_units = (uint32_t)((uint64_t)C * inner / V);
    a.cw = plan.cw;
    a.wave_units = (uint32_t)((uint64_t)plan.cw * inner / V);
    a.nwaves = plan.nwaves;
    a.groups = C;
    a.lag = plan.lag;
    a.spin_limit = tune.spin_limit > 0 ? (uint32_t)tune.spin_limit : kCSpinLimit;
    a.expected = (uint32_t)(tune.extra_arrivals > 0 ? tune.extra_arrivals : 0);   // + grid, added at launch
    const uint32_t c_last = C - (plan.nwaves - 1) * plan.cw;
    const uint32_t ch[2] = {plan.nwaves > 1 ? plan.cw : c_last, c_last};
    // The packed mask is assembled by groups of lanes that must be present together: every slab and
    // every wave has to be a whole number of 32-element mask words (the planner sees to it; a plan
    // that is not is refused here rather than launched).
    if (io.pmask && (((uint64_t)C * inner) % 32 != 0 || ((uint64_t)plan.cw * inner) % 32 != 0 ||
                     ((uint64_t)c_last * inner) % 32 != 0))
        return cudaErrorInvalidValue;
    const bool aligned = (inner % V) == 0;
    for (int i = 0; i < 2; ++i) {
        CShape& s = a.shape[i];
        s.channels = ch[i];
        s.units = (uint32_t)((uint64_t)ch[i] * inner / V);
        s.ncol = (s.units + kCThreads - 1) / kCThreads;
        s.div_ncol = make_fastdiv(s.ncol);
    }
    a.div_plane = make_fastdiv(aligned ? inner / V : inner);
    // 1: codes / mask bytes / sums compiled in; 2: the packed mask alone
    const int extras = (io.codes != nullptr || io.mask != nullptr || io.dist != nullptr) ? 1 : (io.pmask != nullptr ? 2 : (io.pcodes != nullptr ? 3 : 0));
    const int cap = tune.l2_ctas_per_sm;
    if (dtype == 0) {
        if (mode == MODE_FWD) return c_launch_mode<float, MODE_FWD>(a, aligned, extras, sms, cap, st);
        return c_launch_mode<float, MODE_BOTH>(a, aligned, extras, sms, cap, st);
    }
    if (mode == MODE_FWD) return c_launch_mode<__nv_bfloat16, MODE_FWD>(a, aligned, extras, sms, cap, st);
    return c_launch_mode<__nv_bfloat16, MODE_BOTH>(a, aligned, extras, sms, cap, st);
}

}  // namespace granq
