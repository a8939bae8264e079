// Channels-last GranQ kernels: geometries whose channel is the innermost axis ([N, H, W, C] with the
// channel axis last, or [N, C, 1, 1]), i.e. a row-major matrix [rows, C] with one group per column.
//
// Every channel is spread over the whole tensor, so nothing can be quantized before all of it has been
// read: x is read twice (20 instead of 16 bytes per element with a gradient; the second read comes from
// the L2 when the tensor fits), and two plain launches are the right shape - there is nothing for a
// grid-wide hand-over to save.  What makes them fast is the mapping: a 16-byte unit holds V consecutive
// channels of one row, so a thread keeps ONE unit column and walks it down the rows;
//   range pass (Eq. 4):    per-element running min / max stay in registers for the whole walk, are folded
//                          per channel in shared memory and reach global memory as one pair of atomics per
//                          channel and CTA;
//   quantize pass (Eq. 5, 1, 6, STE): the CTA turns the keys into a table of (s, z, 1/s) once; a thread
//                          loads the V parameter sets of its column once and then streams.
// Neither pass divides an index or looks anything up inside the walk.
#include "granq_internal.h"

#include <algorithm>

namespace granq {

namespace {

constexpr int kRThreads = 256;
constexpr uint32_t kRMaxChannels = 4096;      // keys / parameter table in shared memory

struct RArgs {
    const void* x;
    const void* gy;
    void* y;
    void* gx;
    uint8_t* codes;
    uint8_t* mask;
    uint32_t* kmin;
    uint32_t* kmax;
    float* lo;
    float* hi;
    float* s_out;
    float* z_out;
    float qmax;
    uint32_t C;          // channels
    uint32_t ncol;       // 16-byte units per row
    uint64_t rows;
};

// the walk of thread t of CTA b: unit column tile0 + t % P, rows (b * nrows + t / P), + gridDim * nrows, ...
struct RWalk {
    uint32_t P, nrows, r0, cin;
    bool rowed;
    __device__ __forceinline__ RWalk(uint32_t ncol) {
        P = min(ncol, (uint32_t)kRThreads);
        nrows = kRThreads / P;
        r0 = threadIdx.x / P;
        cin = threadIdx.x - r0 * P;
        rowed = r0 < nrows;
    }
};

template <typename T, int U>
__global__ void __launch_bounds__(kRThreads, 4) rows_range_kernel(const RArgs a) {
    constexpr int V = Pack<T>::V;
    extern __shared__ uint32_t r_keys[];          // C min keys, C max keys
    uint32_t* s_kmn = r_keys;
    uint32_t* s_kmx = r_keys + a.C;
    for (uint32_t t = threadIdx.x; t < 2 * a.C; t += kRThreads) r_keys[t] = 0;
    __syncthreads();
    const RWalk w(a.ncol);
    const uint4* xg = reinterpret_cast<const uint4*>(a.x);
    const uint64_t first = (uint64_t)blockIdx.x * w.nrows + w.r0, step = (uint64_t)gridDim.x * w.nrows;
    for (uint32_t tile0 = 0; tile0 < a.ncol; tile0 += w.P) {
        const uint32_t col = tile0 + w.cin;
        if (!w.rowed || col >= a.ncol) continue;
        float mn[V], mx[V];
#pragma unroll
        for (int i = 0; i < V; ++i) {
            mn[i] = INFINITY;
            mx[i] = -INFINITY;
        }
        auto add = [&](const Pack<T>& p) {
#pragma unroll
            for (int i = 0; i < V; ++i) {
                const float v = p.get(i);
                mn[i] = fminf(mn[i], v);
                mx[i] = fmaxf(mx[i], v);
            }
        };
        uint64_t r = first;
        for (; r + (uint64_t)(U - 1) * step < a.rows; r += (uint64_t)U * step) {
            Pack<T> v[U];
#pragma unroll
            for (int j = 0; j < U; ++j) v[j].raw = ld_stream_16(xg + (r + (uint64_t)j * step) * a.ncol + col);
#pragma unroll
            for (int j = 0; j < U; ++j) add(v[j]);
        }
        for (; r < a.rows; r += step) {
            Pack<T> v;
            v.raw = ld_stream_16(xg + r * a.ncol + col);
            add(v);
        }
        if (first < a.rows) {
#pragma unroll
            for (int i = 0; i < V; ++i) {
                atomicMax(s_kmn + col * V + i, ~enc(mn[i]));
                atomicMax(s_kmx + col * V + i, enc(mx[i]));
            }
        }
    }
    __syncthreads();
    for (uint32_t t = threadIdx.x; t < a.C; t += kRThreads) {
        const uint32_t k1 = s_kmn[t], k2 = s_kmx[t];
        if (k1 | k2) {
            atomicMax(a.kmin + t, k1);
            atomicMax(a.kmax + t, k2);
        }
    }
}

template <typename T, int MODE, bool EXTRAS, int U>
__global__ void __launch_bounds__(kRThreads, 3) rows_quant_kernel(const RArgs a) {
    constexpr int V = Pack<T>::V;
    constexpr bool kBwd = (MODE & MODE_BWD) != 0;
    extern __shared__ GroupParam r_par[];         // one (s, z, 1/s) per channel
    for (uint32_t t = threadIdx.x; t < a.C; t += kRThreads) {
        float lo, hi;
        const GroupParam gp = group_param_from_keys(a.kmin, a.kmax, t, a.qmax, lo, hi);
        r_par[t] = gp;
        if (blockIdx.x == 0) {
            a.lo[t] = lo;
            a.hi[t] = hi;
            if (a.s_out) a.s_out[t] = gp.s;
            if (a.z_out) a.z_out[t] = gp.z;
        }
    }
    __syncthreads();
    const RWalk w(a.ncol);
    const uint4* xg = reinterpret_cast<const uint4*>(a.x);
    const uint4* gyg = reinterpret_cast<const uint4*>(a.gy);
    uint4* yg = reinterpret_cast<uint4*>(a.y);
    uint4* gxg = reinterpret_cast<uint4*>(a.gx);
    const uint64_t first = (uint64_t)blockIdx.x * w.nrows + w.r0, step = (uint64_t)gridDim.x * w.nrows;
    const float qmax = a.qmax;
    for (uint32_t tile0 = 0; tile0 < a.ncol; tile0 += w.P) {
        const uint32_t col = tile0 + w.cin;
        if (!w.rowed || col >= a.ncol) continue;
        GroupParam g[V];
#pragma unroll
        for (int i = 0; i < V; ++i) g[i] = r_par[col * V + i];
        auto emit = [&](const Pack<T>& px, const Pack<T>& pg, uint64_t at) {
            Pack<T> py, pgx;
            uint32_t cb[V / 4], mb[V / 4];
            quantize_pack_each<T, kBwd, EXTRAS>(px, pg, g, qmax, py, pgx, cb, mb);
            st_stream_16(yg + at, py.raw);
            if constexpr (kBwd) st_stream_16(gxg + at, pgx.raw);
            if constexpr (EXTRAS) {
                if (a.codes) {
#pragma unroll
                    for (int i = 0; i < V / 4; ++i) reinterpret_cast<uint32_t*>(a.codes)[at * (V / 4) + i] = cb[i];
                }
                if (kBwd && a.mask) {
#pragma unroll
                    for (int i = 0; i < V / 4; ++i) reinterpret_cast<uint32_t*>(a.mask)[at * (V / 4) + i] = mb[i];
                }
            }
        };
        uint64_t r = first;
        for (; r + (uint64_t)(U - 1) * step < a.rows; r += (uint64_t)U * step) {
            Pack<T> px[U], pg[U];
#pragma unroll
            for (int j = 0; j < U; ++j) {
                const uint64_t at = (r + (uint64_t)j * step) * a.ncol + col;
                px[j].raw = ld_stream_16(xg + at);
                if constexpr (kBwd) pg[j].raw = ld_stream_16(gyg + at);
            }
#pragma unroll
            for (int j = 0; j < U; ++j) emit(px[j], pg[j], (r + (uint64_t)j * step) * a.ncol + col);
        }
        for (; r < a.rows; r += step) {
            const uint64_t at = r * a.ncol + col;
            Pack<T> px, pg;
            px.raw = ld_stream_16(xg + at);
            if constexpr (kBwd) pg.raw = ld_stream_16(gyg + at);
            emit(px, pg, at);
        }
    }
}

bool r_aligned16(const void* p) { return p == nullptr || ((uintptr_t)p & 15) == 0; }

template <typename T, int MODE>
cudaError_t r_launch_quant(const RArgs& a, bool extras, int grid, cudaStream_t st) {
    const size_t smem = (size_t)a.C * sizeof(GroupParam);
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<grid, kRThreads, smem, st>>>(a);
        return cudaGetLastError();
    };
    return extras ? go(rows_quant_kernel<T, MODE, true, 2>) : go(rows_quant_kernel<T, MODE, false, 2>);
}

}  // namespace

// inner == 1 (the channel is the innermost axis), rows of whole 16-byte units, everything 16-byte aligned
bool plan_rows(int dtype, const Geom& g, const QuantIO& io) {
    const int64_t V = dtype == 0 ? 4 : 8;
    if (io.pmask || io.dist || io.pcodes) return false;
    if (g.inner != 1 || g.C < V || g.C % V != 0 || g.C > (int64_t)kRMaxChannels || g.outer < 1) return false;
    if (!r_aligned16(io.x) || !r_aligned16(io.gy) || !r_aligned16(io.y) || !r_aligned16(io.gx)) return false;
    if (((uintptr_t)io.codes & 3) || ((uintptr_t)io.mask & 3)) return false;
    return true;
}

cudaError_t launch_rows(const QuantIO& io, int mode, int dtype, const Geom& g, int bits, const Workspace& ws,
                        float* lo, float* hi, float* s_opt, float* z_opt, cudaStream_t st) {
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const uint32_t V = dtype == 0 ? 4 : 8;
    RArgs a{};
    a.x = io.x;
    a.gy = io.gy;
    a.y = io.y;
    a.gx = io.gx;
    a.codes = io.codes;
    a.mask = io.mask;
    a.kmin = ws.kmin;
    a.kmax = ws.kmax;
    a.lo = lo;
    a.hi = hi;
    a.s_out = s_opt;
    a.z_out = z_opt;
    a.qmax = (float)((1 << bits) - 1);
    a.C = (uint32_t)g.C;
    a.ncol = (uint32_t)(g.C / V);
    a.rows = (uint64_t)g.outer;
    // row lanes in the grid: no more CTAs than there are rows to give each row lane at least one
    const uint32_t P = std::min<uint32_t>(a.ncol, kRThreads), nrows = kRThreads / P;
    const uint64_t want = (a.rows + nrows - 1) / nrows;
    const int grid_r = (int)std::min<uint64_t>(want, (uint64_t)sms * 4);
    const int grid_q = (int)std::min<uint64_t>(want, (uint64_t)sms * 3);
    const size_t smem_r = (size_t)a.C * 2 * sizeof(uint32_t);
    if (dtype == 0) {
        auto kr = rows_range_kernel<float, 4>;
        e = cudaFuncSetAttribute(kr, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_r);
        if (e != cudaSuccess) return e;
        kr<<<grid_r, kRThreads, smem_r, st>>>(a);
    } else {
        auto kr = rows_range_kernel<__nv_bfloat16, 4>;
        e = cudaFuncSetAttribute(kr, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_r);
        if (e != cudaSuccess) return e;
        kr<<<grid_r, kRThreads, smem_r, st>>>(a);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const bool extras = io.codes != nullptr || io.mask != nullptr;
    if (dtype == 0) {
        if (mode == MODE_FWD) return r_launch_quant<float, MODE_FWD>(a, extras, grid_q, st);
        return r_launch_quant<float, MODE_BOTH>(a, extras, grid_q, st);
    }
    if (mode == MODE_FWD) return r_launch_quant<__nv_bfloat16, MODE_FWD>(a, extras, grid_q, st);
    return r_launch_quant<__nv_bfloat16, MODE_BOTH>(a, extras, grid_q, st);
}

}  // namespace granq
