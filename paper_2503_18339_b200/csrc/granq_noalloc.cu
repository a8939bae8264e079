// granq_range_noalloc(): the per-group range (Eq. 4) for callers that cannot hand over a
// workspace because they cannot allocate device memory at the point of the call - code running
// inside a framework's allocator callback or out-of-memory handler, a plugin that only receives
// its input and output buffers, a real-time loop that must not touch the driver's allocator.
//
// The min/max keys that granq_range() keeps in the caller's workspace live here in one array
// that is part of the library image: every GPU that loads the library holds these 256 KB until
// the process exits.  All calls share the array, so two calls that overlap on the GPU (different
// streams, or different host threads) race; calls on one stream are safe.
#include "../../include/granq.h"

#include "granq_internal.h"

#include <atomic>

namespace {

constexpr int64_t kNoAllocMaxGroups = GRANQ_NOALLOC_MAX_GROUPS;

// [0, max): min keys, [max, 2 max): max keys
static __device__ __align__(256) uint32_t g_noalloc_keys[2 * kNoAllocMaxGroups];

// Device address of the array, looked up once per device with that device current.  In host
// code `g_noalloc_keys` itself is only a handle for the runtime, not something a kernel can
// dereference.  Two host threads that make the first call on a device together both look the
// address up and store the same value (the entries are atomic, the lookup is idempotent).
uint32_t* noalloc_keys_on_current_device(cudaError_t* err) {
    static std::atomic<uint32_t*> cached[64] = {};
    int dev = 0;
    *err = cudaGetDevice(&dev);
    if (*err != cudaSuccess) return nullptr;
    if (dev < 0 || dev >= 64) {
        *err = cudaErrorInvalidDevice;
        return nullptr;
    }
    uint32_t* keys = cached[dev].load(std::memory_order_acquire);
    if (!keys) {
        void* p = nullptr;
        *err = cudaGetSymbolAddress(&p, g_noalloc_keys);
        if (*err != cudaSuccess) return nullptr;
        keys = static_cast<uint32_t*>(p);
        cached[dev].store(keys, std::memory_order_release);
    }
    return keys;
}

}  // namespace

extern "C" int granq_range_noalloc(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group,
                                   float* min_out, float* max_out, void* cuda_stream) {
    using namespace granq;
    if (!x || !min_out || !max_out || !dims || (dtype != GRANQ_F32 && dtype != GRANQ_BF16))
        return GRANQ_ERR_INVALID_ARG;
    Geom g;
    int64_t G = 0;
    if (!make_geom(dims, channel_axis, group, g, G)) return GRANQ_ERR_INVALID_ARG;
    if (G > kNoAllocMaxGroups) return GRANQ_ERR_UNSUPPORTED;      // more groups than the built-in scratch holds
    cudaError_t e = cudaSuccess;
    uint32_t* keys = noalloc_keys_on_current_device(&e);
    if (!keys) return GRANQ_ERR_CUDA;
    uint32_t* kmin = keys;
    uint32_t* kmax = keys + kNoAllocMaxGroups;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // the array keeps the previous call's keys: both halves must start at the identity (0)
    e = cudaMemsetAsync(kmin, 0, (size_t)G * sizeof(uint32_t), st);
    if (e == cudaSuccess) e = cudaMemsetAsync(kmax, 0, (size_t)G * sizeof(uint32_t), st);
    if (e == cudaSuccess) e = launch_range_flat(x, dtype, g, kmin, kmax, st);
    if (e == cudaSuccess) e = launch_finalize_range(kmin, kmax, G, min_out, max_out, 0, nullptr, nullptr, st);
    return e == cudaSuccess ? GRANQ_OK : GRANQ_ERR_CUDA;
}
