// Cluster-local GranQ kernel: every activation is read from HBM exactly once and no CTA ever
// waits for the rest of the grid.
//
// Channels are independent (Section 4.2.1: per-channel vectors; Section 4.2.2: channels as
// independent lanes), and a channel group of a thin-plane tensor is small: 25 KB for 7x7
// planes at batch 128, 100 KB for 14x14, 401 KB for 28x28.  A "run" of k adjacent channels is
// k * inner contiguous elements in every slab (sample); k is chosen so that a run is a whole
// number of 16-byte units.  One thread-block cluster of R CTAs owns one run: each CTA takes a
// share of the slabs and stages its part of x ONCE in shared memory,
//   - with bulk asynchronous copies (one per slab, completing on mbarriers; no multicast), or
//   - with plain 128-bit loads that reduce on the way (the range is then ready when the
//     last load lands),
// reduces it to per-channel min / max keys (Eq. 4), exchanges the keys with the other CTAs of
// the cluster through distributed shared memory (one cluster barrier), works out scale,
// zero-point and reciprocal per channel (Eq. 5), and quantizes from shared memory (Eq. 1,
// clamp, Eq. 6) while gy streams in and y / gx stream out (STE).  There are no global
// atomics, no arrival counters and no workspace; the only waits are on the CTA's own copies
// (bounded: GRANQ_ERR_TIMEOUT in the status word) and on the cluster's hardware barrier.
//
// Thread mapping: with ncol units per slab of the run, thread t owns unit column t % P
// (P = min(ncol, threads)) and walks it down the CTA's slabs, so its channel - and with it
// its parameters - never change during a walk; the first access of the CTA is one contiguous
// sweep of the tile.
#include "granq_internal.h"

#include <algorithm>

namespace granq {

namespace {

constexpr int kKMaxThreads = 512;
constexpr int kKBars = 8;                    // mbarriers per tile: the range walk starts on the first eighth
constexpr uint32_t kKSpinLimit = 1u << 22;   // bounded wait on a bulk-copy barrier
constexpr uint32_t kKStatusTimeout = 5;      // GRANQ_ERR_TIMEOUT
constexpr uint32_t kKMaxRunChannels = 2048;  // channels of one run (keys and parameters live in shared memory)

struct KArgs {
    const void* x;
    const void* gy;
    void* y;
    void* gx;
    uint8_t* codes;
    uint8_t* mask;
    uint32_t* pmask;       // the STE mask at one bit per element, or null (forward plans with whole mask bytes per run)
    uint32_t* pcodes;      // the codes as a bit string of code_bits each, or null (forward plans; y is then not written)
    int code_bits;
    double* dist;          // four running sums of Table 2's statistics, or null
    uint32_t* status;
    float* lo;
    float* hi;
    float* s_out;
    float* z_out;
    float qmax;
    uint32_t inner;        // elements of one plane
    uint32_t outer;        // slabs
    uint32_t C;            // channel groups
    uint32_t slab_units;   // 16-byte units of one slab
    uint32_t k;            // channels of a regular run
    uint32_t R;            // CTAs of a cluster
    uint32_t tile_bytes;   // shared-memory bytes of the staged tile (keys and parameters follow)
    uint32_t spin_limit;
    uint32_t prefetch_gy;  // ask the L2 for gy while x is on its way
    uint32_t test_stall;   // test hook: after a tile has landed, wait (bounded) for a phase that never completes
    FastDiv div_inner;     // elements per plane
};

__device__ __forceinline__ uint32_t k_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void k_mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(k_smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void k_mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(k_smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool k_mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(k_smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// global -> shared bulk copy of this GPU's own memory into this CTA's shared memory; src and dst
// 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void k_bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::
            "r"(k_smem_u32(dst_smem)),
        "l"(src), "r"(bytes), "r"(k_smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void k_bulk_prefetch_l2(const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t k_cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void k_cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void k_cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// unsigned max into the same shared-memory word of CTA `rank` of this cluster
__device__ __forceinline__ void k_red_max_peer(const uint32_t* local, uint32_t rank, uint32_t v) {
    uint32_t addr;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(addr) : "r"(k_smem_u32(local)), "r"(rank));
    asm volatile("red.relaxed.cluster.shared::cluster.max.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
// per-thread asynchronous 16-byte copy global -> shared (both 16-byte aligned), L2 eviction hint
__device__ __forceinline__ void k_cp_async_16(void* dst_smem, const void* src, uint64_t policy) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(k_smem_u32(dst_smem)), "l"(src),
                 "l"(policy)
                 : "memory");
}
__device__ __forceinline__ void k_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void k_cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// per-element running min / max of one unit column
template <typename T>
struct KRange {
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
    // ordered keys of elements [first, last); (0, 0) when that range is empty or nothing was added
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

// All 32 lanes: fold the lanes' (channel, keys) into the keys in shared memory - of this CTA and of
// every other CTA of its cluster - with one pair of atomics per distinct channel of the warp and CTA.
__device__ __forceinline__ void k_warp_fold(bool valid, uint32_t ch, uint32_t ka, uint32_t kb, uint32_t* s_kmn,
                                            uint32_t* s_kmx, uint32_t R) {
    uint32_t pending = __ballot_sync(kFullMask, valid);
    const uint32_t lane = threadIdx.x & 31;
    while (pending) {
        const int src = __ffs(pending) - 1;
        const uint32_t cur = __shfl_sync(kFullMask, ch, src);
        const bool mine = valid && ch == cur;
        const uint32_t a = __reduce_max_sync(kFullMask, mine ? ka : 0u);
        const uint32_t b = __reduce_max_sync(kFullMask, mine ? kb : 0u);
        if (R == 1) {
            if (lane == (uint32_t)src) {
                atomicMax(s_kmn + cur, a);
                atomicMax(s_kmx + cur, b);
            }
        } else if (lane < R) {                 // lane r tells CTA r of the cluster (its own CTA included)
            k_red_max_peer(s_kmn + cur, lane, a);
            k_red_max_peer(s_kmx + cur, lane, b);
        }
        pending &= ~__ballot_sync(kFullMask, mine);
    }
}

// How the tile gets into shared memory.
enum : int {
    K_LOAD_PLAIN = 0,      // 128-bit loads that reduce on the way and store to the tile; gy read in the quantize walk
    K_LOAD_BULK_X = 1,     // bulk copies (one per slab) of x; gy read in the quantize walk
    K_LOAD_BULK_XG = 2,    // bulk copies of x and gy
    K_LOAD_ASYNC_X = 3,    // per-thread 16-byte asynchronous copies of x; gy read in the quantize walk
    K_LOAD_ASYNC_XG = 4    // per-thread asynchronous copies of x and gy: the quantize walk reads nothing from global memory
};

// U1 / U2 = slabs a thread has in flight in the range walk (plain-load variant) / the quantize walk
template <typename T, int MODE, bool ALIGNED, int EXTRAS, int LOAD, int U1, int U2>
__global__ void __launch_bounds__(kKMaxThreads, 2) cluster_kernel(const KArgs a) {
    constexpr int V = Pack<T>::V;
    constexpr bool kBwd = (MODE & MODE_BWD) != 0;
    constexpr bool BULK = LOAD == K_LOAD_BULK_X || LOAD == K_LOAD_BULK_XG;
    constexpr bool ASYNC = LOAD == K_LOAD_ASYNC_X || LOAD == K_LOAD_ASYNC_XG;
    constexpr bool GY = kBwd && (LOAD == K_LOAD_BULK_XG || LOAD == K_LOAD_ASYNC_XG);      // gy staged as well
    extern __shared__ __align__(128) unsigned char k_smem[];
    __shared__ __align__(8) uint64_t s_bar[2 * kKBars];      // x tile, then gy tile (bulk copies only)

    const uint32_t tid = threadIdx.x, NT = blockDim.x;
    const uint32_t R = a.R;
    const uint32_t rank = R > 1 ? k_cluster_rank() : 0u;
    const uint32_t run = blockIdx.x / R;
    const uint32_t c0 = run * a.k;
    const uint32_t kc = min(a.k, a.C - c0);                               // channels of this run
    const uint32_t ncol = (uint32_t)(((uint64_t)kc * a.inner) / V);       // units of one slab of the run
    const uint32_t n0 = (uint32_t)(((uint64_t)rank * a.outer) / R);
    const uint32_t nl = (uint32_t)(((uint64_t)(rank + 1) * a.outer) / R) - n0;   // this CTA's slabs
    const size_t slab = a.slab_units;
    const size_t gbase = (size_t)n0 * slab + (size_t)(((uint64_t)c0 * a.inner) / V);

    uint4* tile = reinterpret_cast<uint4*>(k_smem);
    uint4* tileg = reinterpret_cast<uint4*>(k_smem + a.tile_bytes);           // staged gy (GY only)
    uint32_t* s_kmn = reinterpret_cast<uint32_t*>(k_smem + (GY ? 2u : 1u) * a.tile_bytes);
    uint32_t* s_kmx = s_kmn + a.k;
    GroupParam* s_par = reinterpret_cast<GroupParam*>(s_kmx + a.k);

    const uint4* xg = reinterpret_cast<const uint4*>(a.x) + gbase;
    const uint4* gyg = reinterpret_cast<const uint4*>(a.gy) + gbase;
    uint4* yg = reinterpret_cast<uint4*>(a.y) + gbase;
    uint4* gxg = reinterpret_cast<uint4*>(a.gx) + gbase;
    const uint64_t drop = l2_policy_evict_first();

    // the walk of thread t: unit column tile0 + t % P, slabs t / P, t / P + nrows, ...
    const uint32_t P = min(ncol, NT), nrows = NT / P;
    const uint32_t r0 = tid / P, cin = tid - r0 * P;
    const bool rowed = r0 < nrows;
    const size_t gstep = (size_t)nrows * slab;
    const uint32_t sstep = nrows * ncol;

    // ---- keys to zero; with a cluster, tell the peers (they fold their keys into this CTA's copy too) ----
    for (uint32_t t = tid; t < kc; t += NT) {
        s_kmn[t] = 0;
        s_kmx[t] = 0;
    }
    const uint32_t CS = (nl + kKBars - 1) / kKBars;                       // slabs per barrier (bulk copies)
    if constexpr (BULK) {
        if (tid < 2u * kKBars) {
            const uint32_t b = tid % kKBars;
            const uint32_t first = min(nl, b * CS), last = min(nl, (b + 1) * CS);
            k_mbar_init(&s_bar[tid], 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            k_mbar_expect_tx(&s_bar[tid], (tid < (uint32_t)kKBars || GY) ? (last - first) * ncol * 16u : 0u);
        }
    }
    if (R > 1) k_cluster_arrive();
    else __syncthreads();

    // Everything above touched only this CTA's own state.  When the launch allows this grid to start before
    // the kernel ahead of it in the stream has finished (programmatic dependent launch), this is where it
    // waits for that kernel's memory; dependents of this grid may start their own preamble from here on.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- stage x (and gy) ----
    if constexpr (BULK) {
        if (R > 1) __syncthreads();          // the barriers are initialised before anyone copies onto them
        for (uint32_t s = tid; s < nl; s += NT)
            k_bulk_load(tile + (size_t)s * ncol, xg + (size_t)s * slab, ncol * 16u, &s_bar[s / CS], drop);
        if constexpr (GY) {
            for (uint32_t s = tid; s < nl; s += NT)
                k_bulk_load(tileg + (size_t)s * ncol, gyg + (size_t)s * slab, ncol * 16u, &s_bar[kKBars + s / CS], drop);
        } else if constexpr (kBwd) {
            if (a.prefetch_gy)
                for (uint32_t s = tid; s < nl; s += NT) k_bulk_prefetch_l2(gyg + (size_t)s * slab, ncol * 16u);
        }
    }
    if constexpr (ASYNC) {
        // every thread copies exactly the units it will read: no barrier between the copy and the walks
        if (rowed) {
            for (uint32_t col = cin; col < ncol; col += P) {
                const uint4* p = xg + (size_t)r0 * slab + col;
                uint4* q = tile + (size_t)r0 * ncol + col;
                for (uint32_t s = r0; s < nl; s += nrows, p += gstep, q += sstep) k_cp_async_16(q, p, drop);
            }
        }
        k_cp_async_commit();
        if constexpr (GY) {
            if (rowed) {
                for (uint32_t col = cin; col < ncol; col += P) {
                    const uint4* p = gyg + (size_t)r0 * slab + col;
                    uint4* q = tileg + (size_t)r0 * ncol + col;
                    for (uint32_t s = r0; s < nl; s += nrows, p += gstep, q += sstep) k_cp_async_16(q, p, drop);
                }
            }
            k_cp_async_commit();
        }
    }

    // bounded wait for barrier b of a tile; false when it ran out (status recorded)
    auto wait_bar = [&](uint32_t b, uint32_t parity) -> bool {
        for (uint32_t i = 0; i < a.spin_limit; ++i)
            if (k_mbar_try_wait(&s_bar[b], parity)) return true;
        atomicExch(a.status, kKStatusTimeout);
        return false;
    };
    bool ok = true;          // false once one of this thread's waits ran out: it then only keeps the barriers company
    uint32_t nb_done = 0;    // barriers of the x tile this thread has seen complete
    uint32_t ng_done = 0;    // ... of the gy tile

    auto column = [&](uint32_t col, uint32_t& ch, int& ne) {
        if constexpr (ALIGNED) {
            ch = a.div_inner.div(col * V);
            ne = V;
        } else {
            uint32_t rem;
            a.div_inner.divmod(col * V, ch, rem);
            ne = (int)min((uint32_t)V, a.inner - rem);
        }
    };

    // ---- range (Eq. 4): per-element running min / max down the walk, folded per channel ----
    if constexpr (ASYNC) {
        if constexpr (GY) k_cp_async_wait<1>();
        else k_cp_async_wait<0>();
    }
    bool peers_ready = R == 1;      // the peers' key tables are known to be zeroed
    for (uint32_t tile0 = 0; tile0 < ncol; tile0 += P) {
        const uint32_t col = tile0 + cin;
        const bool valid = rowed && col < ncol;
        KRange<T> acc;
        acc.reset();
        if (valid) {
            if constexpr (LOAD != K_LOAD_PLAIN) {
                const uint4* p = tile + col;
                for (uint32_t s = r0; s < nl && ok; s += nrows) {
                    if constexpr (BULK) {
                        while (ok && s >= nb_done * CS) {
                            ok = wait_bar(nb_done, 0);
                            if (ok && a.test_stall) ok = wait_bar(nb_done, 1);
                            if (!ok) wait_bar(nb_done, 0);      // its own copies, once more, before it moves on
                            ++nb_done;
                        }
                        if (!ok) break;
                    }
                    Pack<T> v;
                    v.raw = p[(size_t)s * ncol];
                    acc.add(v);
                }
            } else {
                const uint4* p = xg + (size_t)r0 * slab + col;
                uint4* q = tile + (size_t)r0 * ncol + col;
                uint32_t s = r0;
                for (; s + (U1 - 1) * nrows < nl; s += U1 * nrows) {
                    Pack<T> v[U1];
#pragma unroll
                    for (int j = 0; j < U1; ++j) v[j].raw = ld_hint_16(p + (size_t)j * gstep, drop);
#pragma unroll
                    for (int j = 0; j < U1; ++j) {
                        acc.add(v[j]);
                        q[(size_t)j * sstep] = v[j].raw;
                    }
                    p += (size_t)U1 * gstep;
                    q += (size_t)U1 * sstep;
                }
                if (s < nl) {                                    // a short last batch, still loaded together
                    Pack<T> v[U1 - 1];
#pragma unroll
                    for (int j = 0; j < U1 - 1; ++j)
                        if (s + j * nrows < nl) v[j].raw = ld_hint_16(p + (size_t)j * gstep, drop);
#pragma unroll
                    for (int j = 0; j < U1 - 1; ++j)
                        if (s + j * nrows < nl) {
                            acc.add(v[j]);
                            q[(size_t)j * sstep] = v[j].raw;
                        }
                }
            }
        }
        if (!peers_ready) {          // first fold: by now every CTA of the cluster has long zeroed its keys
            k_cluster_wait();
            peers_ready = true;
        }
        uint32_t ch = 0;
        int ne = V;
        if (valid) column(col, ch, ne);
        uint32_t ka, kb;
        acc.keys(0, ne, ka, kb);
        k_warp_fold(valid, ch, ka, kb, s_kmn, s_kmx, R);
        if constexpr (!ALIGNED) {
            uint32_t kc2, kd2;
            acc.keys(ne, V, kc2, kd2);
            k_warp_fold(valid && ne < V, ch + 1, kc2, kd2, s_kmn, s_kmx, R);
        }
    }
    // every CTA of the cluster has folded its keys into every copy once all have arrived here
    if (R > 1) {
        if (!peers_ready) k_cluster_wait();
        k_cluster_arrive();
        k_cluster_wait();
    } else {
        __syncthreads();
    }

    // ---- keys -> lo, hi, scale, zero-point, reciprocal per channel (Eq. 5) ----
    for (uint32_t t = tid; t < kc; t += NT) {
        float lo, hi;
        keys_to_range(s_kmn[t], s_kmx[t], lo, hi);
        const QParam qp = make_qparam(lo, hi, a.qmax);
        GroupParam gp;
        gp.s = qp.s;
        gp.z = qp.z;
        gp.r = div_is_safe(qp.s, lo, hi) ? __frcp_rn(qp.s) : 0.0f;
        s_par[t] = gp;
        if (rank == 0) {
            a.lo[c0 + t] = lo;
            a.hi[c0 + t] = hi;
            if (a.s_out) a.s_out[c0 + t] = gp.s;
            if (a.z_out) a.z_out[c0 + t] = gp.z;
        }
    }
    __syncthreads();

    // ---- quantize, clamp, dequantize from shared memory; STE backward (Eq. 1, 6, Section 2.1) ----
    const float qmax = a.qmax;
    DistAcc dacc;               // Table 2's sums over everything this thread quantizes (EXTRAS only)
    dacc.reset();
    if constexpr (ASYNC && GY) k_cp_async_wait<0>();
    for (uint32_t tile0 = 0; tile0 < ncol; tile0 += P) {
        const uint32_t col = tile0 + cin;
        if (!(rowed && col < ncol) || !ok) continue;
        uint32_t ch;
        int ne;
        column(col, ch, ne);
        const GroupParam g1 = s_par[ch];
        GroupParam g2 = g1;
        if constexpr (!ALIGNED) {
            if (ne < V) g2 = s_par[ch + 1];
        }
        auto emit = [&](const Pack<T>& px, const Pack<T>& pg, size_t at) {
            Pack<T> py, pgx;
            uint32_t cb[V / 4], mb[V / 4];
            quantize_pack<T, kBwd, !ALIGNED, EXTRAS, true>(px, pg, g1, g2, ne, qmax, py, pgx, cb, mb, EXTRAS == 3 ? a.code_bits : 8);
            if constexpr (EXTRAS == 3) {
                // the packed codes are the only output: 8 codes = b bytes per pair of fp32 lanes (per bf16 lane); the
                // planner has made every run and slab whole groups of 8 elements, so both lanes of a pair are here
                store_code_bytes<V>(a.pcodes, (gbase + at) * V, code_string_of<V>(cb, a.code_bits), a.code_bits, tid & 31);
                return;
            }
            st_hint_16(yg + at, py.raw, drop);
            if constexpr (kBwd) st_hint_16(gxg + at, pgx.raw, drop);
            if constexpr (EXTRAS != 0) {
                if constexpr (EXTRAS == 1) {
                    const size_t w = (gbase + at) * (V / 4);
                    if (a.codes) {
#pragma unroll
                        for (int i = 0; i < V / 4; ++i) reinterpret_cast<uint32_t*>(a.codes)[w + i] = cb[i];
                    }
                    if (kBwd && a.mask) {
#pragma unroll
                        for (int i = 0; i < V / 4; ++i) reinterpret_cast<uint32_t*>(a.mask)[w + i] = mb[i];
                    }
                    if (a.dist) dacc.add(px, py);
                }
                if (a.pmask) {
                    // the mask is written byte by byte (8 elements: two fp32 packs of neighbouring lanes, one bf16
                    // pack): the planner has made every run and slab whole bytes of mask and the rows of columns
                    // whole pairs of lanes, so both lanes of a byte are here together, in the same slab
                    store_mask_byte<V>(a.pmask, (gbase + at) * V, mask_bits_of<V, EXTRAS>(mb), tid & 31);
                }
            }
        };
        size_t gu = (size_t)r0 * slab + col;
        const uint4* q = tile + (size_t)r0 * ncol + col;
        const uint4* qg = tileg + (size_t)r0 * ncol + col;
        uint32_t s = r0;
        // the staged gy of slabs up to `last` has landed (bounded wait; false when it ran out)
        auto gy_ready = [&](uint32_t last) -> bool {
            if constexpr (BULK) {
                while (ok && last >= ng_done * CS) {
                    ok = wait_bar(kKBars + ng_done, 0);
                    if (!ok) wait_bar(kKBars + ng_done, 0);
                    ++ng_done;
                }
            }
            return ok;
        };
        for (; s + (U2 - 1) * nrows < nl; s += U2 * nrows) {
            Pack<T> px[U2], pg[U2];
            if constexpr (GY) {
                if (!gy_ready(s + (U2 - 1) * nrows)) break;
            }
#pragma unroll
            for (int j = 0; j < U2; ++j) {
                if constexpr (GY) pg[j].raw = qg[(size_t)j * sstep];
                else if constexpr (kBwd) pg[j].raw = ld_hint_16(gyg + gu + (size_t)j * gstep, drop);
            }
#pragma unroll
            for (int j = 0; j < U2; ++j) px[j].raw = q[(size_t)j * sstep];
#pragma unroll
            for (int j = 0; j < U2; ++j) emit(px[j], pg[j], gu + (size_t)j * gstep);
            gu += (size_t)U2 * gstep;
            q += (size_t)U2 * sstep;
            qg += (size_t)U2 * sstep;
        }
        for (; s < nl && ok; s += nrows) {
            Pack<T> px, pg;
            if constexpr (GY) {
                if (!gy_ready(s)) break;
                pg.raw = *qg;
            } else if constexpr (kBwd) {
                pg.raw = ld_hint_16(gyg + gu, drop);
            }
            px.raw = *q;
            emit(px, pg, gu);
            gu += gstep;
            q += sstep;
            qg += sstep;
        }
    }
    if constexpr (EXTRAS == 1) {
        if (a.dist) dacc.flush(a.dist);       // all lanes of every warp are here
    }
    if constexpr (BULK) {
        // Nothing of this CTA may still be in flight when it leaves: every barrier once more (a no-op unless a
        // wait above gave up early), with the built-in limit.
        __syncthreads();
        if (tid < 2u * kKBars) {
            for (uint32_t i = 0; i < kKSpinLimit; ++i)
                if (k_mbar_try_wait(&s_bar[tid], 0)) break;
        }
        __syncthreads();
    }
}

bool k_aligned16(const void* p) { return p == nullptr || ((uintptr_t)p & 15) == 0; }

uint32_t k_gcd(uint32_t a, uint32_t b) {
    while (b) {
        uint32_t t = a % b;
        a = b;
        b = t;
    }
    return a;
}

template <typename T, int MODE, bool ALIGNED, int EXTRAS>
cudaError_t k_launch_t(const KArgs& args, const ClusterPlan& plan, uint32_t grid, cudaStream_t st) {
    auto launch = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
        if (e != cudaSuccess) return e;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(plan.threads);
        cfg.dynamicSmemBytes = plan.smem_bytes;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = plan.R;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        // the grid may be set up while the kernel ahead of it in the stream drains (it waits for that
        // kernel's memory itself, before its first global access)
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = plan.early_launch ? 2 : 1;
        return cudaLaunchKernelEx(&cfg, kern, args);
    };
    if constexpr (EXTRAS == 2 || EXTRAS == 3) {      // packed mask or packed codes alone: forward plans with per-thread copies or plain loads
        if (plan.load == K_LOAD_ASYNC_X) return launch(cluster_kernel<T, MODE, ALIGNED, EXTRAS, K_LOAD_ASYNC_X, 4, 2>);
        return launch(cluster_kernel<T, MODE, ALIGNED, EXTRAS, K_LOAD_PLAIN, 4, 2>);
    } else {
        switch (plan.load) {
            case K_LOAD_BULK_X: return launch(cluster_kernel<T, MODE, ALIGNED, EXTRAS, K_LOAD_BULK_X, 4, 2>);
            case K_LOAD_BULK_XG: return launch(cluster_kernel<T, MODE, ALIGNED, EXTRAS, K_LOAD_BULK_XG, 4, 2>);
            case K_LOAD_ASYNC_X: return launch(cluster_kernel<T, MODE, ALIGNED, EXTRAS, K_LOAD_ASYNC_X, 4, 2>);
            case K_LOAD_ASYNC_XG: return launch(cluster_kernel<T, MODE, ALIGNED, EXTRAS, K_LOAD_ASYNC_XG, 4, 2>);
            default: return launch(cluster_kernel<T, MODE, ALIGNED, EXTRAS, K_LOAD_PLAIN, 4, 2>);
        }
    }
}

template <typename T, int MODE>
cudaError_t k_launch_mode(const KArgs& a, const ClusterPlan& p, bool aligned, int extras, uint32_t grid,
                          cudaStream_t st) {
    if constexpr (MODE == MODE_FWD) {
        if (extras == 2)
            return aligned ? k_launch_t<T, MODE, true, 2>(a, p, grid, st) : k_launch_t<T, MODE, false, 2>(a, p, grid, st);
        if (extras == 3)
            return aligned ? k_launch_t<T, MODE, true, 3>(a, p, grid, st) : k_launch_t<T, MODE, false, 3>(a, p, grid, st);
    }
    if (aligned)
        return extras ? k_launch_t<T, MODE, true, 1>(a, p, grid, st) : k_launch_t<T, MODE, true, 0>(a, p, grid, st);
    return extras ? k_launch_t<T, MODE, false, 1>(a, p, grid, st) : k_launch_t<T, MODE, false, 0>(a, p, grid, st);
}

}  // namespace

// The cut: k channels per run (the smallest count that makes a run whole 16-byte units, times a
// multiplier when a whole group is far below the tile target), R CTAs per run so that a CTA's
// share of the slabs fits the tile limit, and a thread count whose rows of columns waste the
// fewest lanes.
ClusterPlan plan_cluster(int dtype, const Geom& g, const QuantIO& io, bool backward, const StagedTuning& tune) {
    ClusterPlan p{};
    p.ok = false;
    const uint32_t V = dtype == 0 ? 4 : 8, esize = 16 / V;
    // packed codes: forward only, nothing else beside them, whole words of codes (no padding to clear)
    if (io.pcodes && (backward || io.codes || io.mask || io.pmask || io.dist || ((uintptr_t)io.pcodes & 3) ||
                      io.code_bits < 1 || io.code_bits > 8 || g.E % 32 != 0))
        return p;
    if ((io.pmask || io.pcodes) && (g.C * g.inner) % 8 != 0) return p;
    if (!k_aligned16(io.x) || !k_aligned16(io.gy) || !k_aligned16(io.y) || !k_aligned16(io.gx)) return p;
    if (((uintptr_t)io.codes & 3) || ((uintptr_t)io.mask & 3)) return p;
    if (g.inner < (int64_t)V || g.inner >= (1ll << 24) || g.C >= (1ll << 28) || g.outer >= (1ll << 24)) return p;
    if ((g.C * g.inner) % V != 0 || g.E / V >= (1ll << 31)) return p;
    const uint32_t inner = (uint32_t)g.inner, C = (uint32_t)g.C, outer = (uint32_t)g.outer;
    // How the tile is staged.  Knob: 1 = bulk copies for x, 2 = plain loads, 3 = bulk copies for x and gy,
    // 4 = per-thread asynchronous copies for x, 5 = for x and gy.  Default: asynchronous copies; gy is staged
    // too for fp32 tensors with a gradient when that still fits a portable cluster (measured faster there;
    // bf16 halves the bytes per element, and reading gy in the quantize walk measured faster).
    const uint64_t limit = tune.cl_tile_kb > 0 ? (uint64_t)tune.cl_tile_kb * 1024 : 112ull * 1024;   // two CTAs per SM
    // a run is whole 16-byte units; with a packed mask also whole bytes of mask (8 elements)
    const uint32_t unit = (io.pmask || io.pcodes) ? 8u : V;
    const uint64_t group_bytes = (uint64_t)g.outer * (unit / k_gcd((uint32_t)g.inner, unit)) * g.inner * esize;
    switch (tune.cl_load) {
        case 1: p.load = K_LOAD_BULK_X; break;
        case 2: p.load = K_LOAD_PLAIN; break;
        case 3: p.load = backward ? K_LOAD_BULK_XG : K_LOAD_BULK_X; break;
        case 4: p.load = K_LOAD_ASYNC_X; break;
        case 5: p.load = backward ? K_LOAD_ASYNC_XG : K_LOAD_ASYNC_X; break;
        default:
            p.load = (backward && dtype == 0 && 2 * group_bytes <= 8 * limit) ? K_LOAD_ASYNC_XG : K_LOAD_ASYNC_X;
            break;
    }
    // the two lanes that assemble a byte of mask must both be there: only the variants without a give-up path qualify
    if ((io.pmask || io.pcodes) && p.load != K_LOAD_ASYNC_X && p.load != K_LOAD_ASYNC_XG && p.load != K_LOAD_PLAIN) return p;
    const uint64_t tiles = (p.load == K_LOAD_BULK_XG || p.load == K_LOAD_ASYNC_XG) ? 2 : 1;   // staged tiles per CTA
    const uint32_t k0 = unit / k_gcd(inner, unit);
    const uint64_t target = std::min<uint64_t>(limit, 64ull * 1024);
    const uint64_t run0 = (uint64_t)k0 * inner * esize;                  // bytes of a minimal run in one slab
    // CTAs per run: the smallest power of two (at most 8, the portable cluster size) that fits the limit
    uint32_t R = 1;
    auto share = [&](uint32_t r) { return tiles * (uint64_t)((outer + r - 1) / r) * run0; };
    if (tune.cl_r > 0) {
        R = (uint32_t)tune.cl_r;
        if (R > 8 || (R & (R - 1)) || R > outer) return p;
    } else {
        while (R < 8 && R * 2 <= outer && share(R) > limit) R *= 2;
        // small tensors: more, smaller CTAs keep more SMs busy
        while (R < 8 && R * 2 <= outer && share(R) > target && (uint64_t)(C / k0) * R < 2 * 148) R *= 2;
    }
    if (share(R) > limit) return p;
    // channels per run: widen a run while the tile stays under the target (groups far smaller than a tile)
    uint32_t m = 1;
    if (tune.cl_kmul > 0) {
        m = (uint32_t)tune.cl_kmul;
    } else if (R == 1) {
        const uint64_t fit = target / std::max<uint64_t>(1, share(1));
        m = (uint32_t)std::max<uint64_t>(1, std::min<uint64_t>(fit, (C + k0 - 1) / k0));
    }
    m = std::min<uint32_t>(m, std::max<uint32_t>(1, kKMaxRunChannels / k0));
    m = std::min<uint32_t>(m, (C + k0 - 1) / k0);
    p.k = k0 * m;
    if (p.k > kKMaxRunChannels) return p;
    p.R = R;
    const uint32_t nl = (outer + R - 1) / R;
    const uint64_t run_units = (uint64_t)p.k * inner / V;
    if (run_units >= (1ull << 24) || (uint64_t)nl * run_units * 16 * tiles > limit) return p;
    p.tile_bytes = (uint32_t)((uint64_t)nl * run_units * 16);
    p.smem_bytes = (uint32_t)tiles * p.tile_bytes + p.k * (2 * sizeof(uint32_t) + sizeof(GroupParam));
    p.smem_bytes = (p.smem_bytes + 15) & ~15u;
    if (p.smem_bytes > 227u * 1024) return p;
    // threads: rows of P = min(columns, threads) lanes; take the count that wastes the fewest lanes
    if (tune.cl_threads > 0 && (tune.cl_threads % 32 != 0 || tune.cl_threads > kKMaxThreads)) return p;
    const uint32_t top = tune.cl_threads > 0 ? (uint32_t)tune.cl_threads
                                             : (p.smem_bytes > 56u * 1024 ? 512u : 256u);
    double best = -1.0;
    p.threads = top;
    for (uint32_t nt = top; nt >= 128 && nt + 160 > top; nt -= 32) {
        const uint64_t P = std::min<uint64_t>(run_units, nt), rows = nt / P;
        const uint64_t walks = ((nl + rows - 1) / rows) * ((run_units + P - 1) / P);
        const double eff = (double)nl * (double)run_units / ((double)nt * (double)walks);
        if (eff > best + 1e-9) {
            best = eff;
            p.threads = nt;
        }
        if (tune.cl_threads > 0) break;
    }
    p.prefetch_gy = tune.cl_prefetch != 2;
    p.early_launch = tune.cl_pdl != 2;
    p.ok = true;
    return p;
}

cudaError_t launch_cluster(const ClusterPlan& plan, const QuantIO& io, int mode, int dtype, const Geom& g, int bits,
                           const Workspace& ws, float* lo, float* hi, float* s_opt, float* z_opt,
                           const StagedTuning& tune, cudaStream_t st) {
    const uint32_t V = dtype == 0 ? 4 : 8;
    KArgs a{};
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
    a.lo = lo;
    a.hi = hi;
    a.s_out = s_opt;
    a.z_out = z_opt;
    a.qmax = (float)((1 << bits) - 1);
    a.inner = (uint32_t)g.inner;
    a.outer = (uint32_t)g.outer;
    a.C = (uint32_t)g.C;
    a.slab_units = (uint32_t)((uint64_t)g.C * g.inner / V);
    a.k = plan.k;
    a.R = plan.R;
    a.tile_bytes = plan.tile_bytes;
    a.spin_limit = tune.spin_limit > 0 ? (uint32_t)tune.spin_limit : kKSpinLimit;
    a.prefetch_gy = plan.prefetch_gy ? 1u : 0u;
    a.test_stall = tune.extra_arrivals > 0 ? 1u : 0u;
    a.div_inner = make_fastdiv(a.inner);
    const uint32_t nruns = (a.C + plan.k - 1) / plan.k;
    const uint32_t grid = nruns * plan.R;
    const bool aligned = (a.inner % V) == 0;
    // 1: codes / mask bytes / sums compiled in; 2: the packed mask alone (a leaner instantiation of the forward kernel)
    const int extras = (io.codes != nullptr || io.mask != nullptr || io.dist != nullptr) ? 1 : (io.pmask != nullptr ? 2 : (io.pcodes != nullptr ? 3 : 0));
    if (dtype == 0) {
        if (mode == MODE_FWD) return k_launch_mode<float, MODE_FWD>(a, plan, aligned, extras, grid, st);
        return k_launch_mode<float, MODE_BOTH>(a, plan, aligned, extras, grid, st);
    }
    if (mode == MODE_FWD) return k_launch_mode<__nv_bfloat16, MODE_FWD>(a, plan, aligned, extras, grid, st);
    return k_launch_mode<__nv_bfloat16, MODE_BOTH>(a, plan, aligned, extras, grid, st);
}

}  // namespace granq
