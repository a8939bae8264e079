// Channel-wise fake-quantization of many small tensors in one launch (Section 5.1: every weight
// tensor is quantized per output channel).  A weight tensor [channels, group_elems] has one group
// per leading index and each group is a short contiguous run (27 .. a few thousand values), so a
// whole group fits in one warp's reach: a warp reads its group once for the range (Eq. 4), works
// out scale and zero-point (Eq. 5), reads it again (an L1 / L2 hit) to quantize, clamp, dequantize
// (Eq. 1, 6) and, when an upstream gradient is given, to mask it (STE).  No shared memory, no
// block-wide or grid-wide synchronisation; warps take groups grid-stride over ALL tensors of the
// batch, found by a binary search in a table of first-group indices.
#include "../../include/granq.h"

#include "granq_internal.h"

#include <vector>

namespace granq {

namespace {

constexpr int kWThreads = 256;

struct WDesc {
    const void* x;
    const void* gy;
    void* y;
    void* gx;
    float* lo;
    float* hi;
    float* s;
    float* z;
    uint32_t group_elems;
    uint32_t first_group;   // index of this tensor's first group in the batch
    float qmax;
    uint32_t vec;           // groups start on 16-byte boundaries and are whole packs
};

template <typename T>
__global__ void __launch_bounds__(kWThreads) weights_kernel(const WDesc* __restrict__ descs, uint32_t n,
                                                            uint32_t total_groups) {
    constexpr int V = Pack<T>::V;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warps = gridDim.x * (kWThreads / 32);
    for (uint32_t g = blockIdx.x * (kWThreads / 32) + (threadIdx.x >> 5); g < total_groups; g += warps) {
        // the tensor that holds group g: last descriptor with first_group <= g
        uint32_t a = 0, b = n - 1;
        while (a < b) {
            const uint32_t m = (a + b + 1) >> 1;
            if (descs[m].first_group <= g) a = m;
            else b = m - 1;
        }
        const WDesc d = descs[a];
        const uint32_t c = g - d.first_group, ge = d.group_elems;
        const T* x = reinterpret_cast<const T*>(d.x) + (size_t)c * ge;
        const T* gy = d.gy ? reinterpret_cast<const T*>(d.gy) + (size_t)c * ge : nullptr;
        T* y = reinterpret_cast<T*>(d.y) + (size_t)c * ge;
        T* gx = d.gx ? reinterpret_cast<T*>(d.gx) + (size_t)c * ge : nullptr;

        // ---- Eq. 4: the group's range ----
        float mn = INFINITY, mx = -INFINITY;
        if (d.vec) {
            for (uint32_t u = lane; u < ge / V; u += 32) {
                Pack<T> p;
                p.raw = *reinterpret_cast<const uint4*>(x + (size_t)u * V);
                pack_minmax(p, 0, V, mn, mx);
            }
        } else {
            for (uint32_t e = lane; e < ge; e += 32) {
                const float v = load_scalar(x + e);
                mn = fminf(mn, v);
                mx = fmaxf(mx, v);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mn = fminf(mn, __shfl_xor_sync(kFullMask, mn, o));
            mx = fmaxf(mx, __shfl_xor_sync(kFullMask, mx, o));
        }
        const float lo = __fadd_rn(mn, 0.0f), hi = __fadd_rn(mx, 0.0f);      // -0 -> +0
        const QParam qp = make_qparam(lo, hi, d.qmax);                        // Eq. 5
        if (lane == 0) {
            d.lo[c] = lo;
            d.hi[c] = hi;
            if (d.s) d.s[c] = qp.s;
            if (d.z) d.z[c] = qp.z;
        }

        // ---- Eq. 1, clamp, Eq. 6, STE ----
        if (d.vec) {
            for (uint32_t u = lane; u < ge / V; u += 32) {
                Pack<T> p, pg, py, pgx;
                p.raw = *reinterpret_cast<const uint4*>(x + (size_t)u * V);
                if (gy) pg.raw = *reinterpret_cast<const uint4*>(gy + (size_t)u * V);
#pragma unroll
                for (int i = 0; i < V; ++i) {
                    float yv;
                    bool in;
                    quant_one(p.get(i), qp, d.qmax, yv, in);
                    py.set(i, yv);
                    if (gy) pgx.set(i, in ? pg.get(i) : 0.0f);
                }
                *reinterpret_cast<uint4*>(y + (size_t)u * V) = py.raw;
                if (gy) *reinterpret_cast<uint4*>(gx + (size_t)u * V) = pgx.raw;
            }
        } else {
            for (uint32_t e = lane; e < ge; e += 32) {
                float yv;
                bool in;
                quant_one(load_scalar(x + e), qp, d.qmax, yv, in);
                store_scalar(y + e, yv);
                if (gy) store_scalar(gx + e, in ? load_scalar(gy + e) : 0.0f);
            }
        }
    }
}

size_t table_bytes(int n) { return (((size_t)n * sizeof(WDesc)) + 255) & ~(size_t)255; }

}  // namespace

}  // namespace granq

using namespace granq;

extern "C" {

size_t granq_weights_workspace_bytes(int n_tensors) { return n_tensors > 0 ? table_bytes(n_tensors) : 0; }

int granq_fakequant_weights(const granq_weight_desc* descs, int n_tensors, int dtype, void* workspace,
                            size_t workspace_bytes, uint32_t flags, void* cuda_stream) {
    (void)flags;
    if (!descs || n_tensors <= 0 || (dtype != GRANQ_F32 && dtype != GRANQ_BF16)) return GRANQ_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < table_bytes(n_tensors)) return GRANQ_ERR_WORKSPACE;
    const size_t esz = dtype == GRANQ_F32 ? 4 : 2;
    const uint32_t V = dtype == GRANQ_F32 ? 4 : 8;
    std::vector<WDesc> table((size_t)n_tensors);
    uint64_t total = 0;
    for (int i = 0; i < n_tensors; ++i) {
        const granq_weight_desc& s = descs[i];
        if (!s.x || !s.y || !s.min_out || !s.max_out || s.bits < 1 || s.bits > 8 || s.channels <= 0 ||
            s.group_elems <= 0 || (s.gy_opt == nullptr) != (s.gx_opt == nullptr))
            return GRANQ_ERR_INVALID_ARG;
        if (s.channels >= (1ll << 31) || s.group_elems >= (1ll << 31)) return GRANQ_ERR_UNSUPPORTED;
        const size_t nb = (size_t)s.channels * (size_t)s.group_elems * esz;
        const char *px = (const char*)s.x, *py = (const char*)s.y, *pgy = (const char*)s.gy_opt,
                   *pgx = (const char*)s.gx_opt;
        auto hit = [nb](const char* a, const char* b) { return a && b && a < b + nb && b < a + nb; };
        if (hit(px, py) || hit(px, pgx) || hit(pgy, py) || hit(pgy, pgx) || hit(py, pgx)) return GRANQ_ERR_INVALID_ARG;
        WDesc& d = table[(size_t)i];
        d.x = s.x;
        d.gy = s.gy_opt;
        d.y = s.y;
        d.gx = s.gx_opt;
        d.lo = s.min_out;
        d.hi = s.max_out;
        d.s = s.scale_opt;
        d.z = s.zp_opt;
        d.group_elems = (uint32_t)s.group_elems;
        d.first_group = (uint32_t)total;
        d.qmax = (float)((1 << s.bits) - 1);
        const uintptr_t all = (uintptr_t)s.x | (uintptr_t)s.y | (uintptr_t)s.gy_opt | (uintptr_t)s.gx_opt;
        d.vec = ((all & 15) == 0 && s.group_elems % V == 0) ? 1u : 0u;
        total += (uint64_t)s.channels;
        if (total >= (1ull << 31)) return GRANQ_ERR_UNSUPPORTED;
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // The table below is pageable host memory that lives until this call returns: fine for an eager copy (the
    // runtime has read it by then), wrong for a captured one (a replay would read freed memory) - so a
    // capturing stream is refused.
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &capturing) != cudaSuccess) return GRANQ_ERR_CUDA;
    if (capturing != cudaStreamCaptureStatusNone) return GRANQ_ERR_UNSUPPORTED;
    // the table is pageable host memory: the copy has read it by the time the call returns
    cudaError_t e = cudaMemcpyAsync(workspace, table.data(), table.size() * sizeof(WDesc), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return GRANQ_ERR_CUDA;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const uint64_t ctas = (total + kWThreads / 32 - 1) / (kWThreads / 32), cap = (uint64_t)sms * 8;
    const int grid = (int)(ctas < cap ? ctas : cap);
    if (dtype == GRANQ_F32)
        weights_kernel<float><<<grid, kWThreads, 0, st>>>((const WDesc*)workspace, (uint32_t)n_tensors, (uint32_t)total);
    else
        weights_kernel<__nv_bfloat16><<<grid, kWThreads, 0, st>>>((const WDesc*)workspace, (uint32_t)n_tensors,
                                                                  (uint32_t)total);
    return cudaGetLastError() == cudaSuccess ? GRANQ_OK : GRANQ_ERR_CUDA;
}

}  // extern "C"
