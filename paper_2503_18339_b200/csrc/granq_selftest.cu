// Device self-test of the reciprocal-based division used by the staged kernel: it must give
// the same bits as IEEE division (__fdiv_rn) for every divisor and dividend in the range
// div_is_safe() admits.  Pairs come from a counter-based generator and include the shapes
// that are hard for such schemes: divisors whose significand is all ones or a power of two,
// quotients next to a rounding boundary (k + 1/2 for small integers k), tiny and huge ratios.
#include "../../include/granq.h"

#include "granq_internal.h"

namespace granq {
namespace {

__device__ __forceinline__ uint64_t mix64(uint64_t v) {   // splitmix64 finaliser
    v += 0x9E3779B97F4A7C15ull;
    v = (v ^ (v >> 30)) * 0xBF58476D1CE4E5B9ull;
    v = (v ^ (v >> 27)) * 0x94D049BB133111EBull;
    return v ^ (v >> 31);
}

__device__ __forceinline__ float make_float(uint32_t mant, int exp2) {   // 1.mant * 2^exp2
    return __uint_as_float(((uint32_t)(exp2 + 127) << 23) | (mant & 0x7FFFFFu));
}

__global__ void division_selftest_kernel(uint64_t pairs, uint64_t seed, unsigned long long* mismatches) {
    unsigned long long bad = 0;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < pairs;
         i += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t h1 = mix64(seed * 0x100000001B3ull + i), h2 = mix64(h1);
        // divisor: exponent in [-60, 60]; significand random, all ones, a power of two, or nearly so
        uint32_t ms = (uint32_t)h1 & 0x7FFFFFu;
        const uint32_t kind = (uint32_t)(h1 >> 23) & 7u;
        if (kind == 0) ms = 0x7FFFFFu;
        if (kind == 1) ms = 0;
        if (kind == 2) ms = 0x7FFFFFu - ((uint32_t)(h1 >> 40) & 7u);
        if (kind == 3) ms = (uint32_t)(h1 >> 40) & 7u;
        const int es = (int)((h1 >> 48) % 121u) - 60;
        const float s = make_float(ms, es);
        // dividend: random, or s * (k + 1/2) nudged by a few ulps (a quotient next to a rounding boundary)
        float x;
        const uint32_t xkind = (uint32_t)(h2 >> 60);
        if (xkind < 8) {
            int ex = es + (int)((h2 >> 32) % 61u) - 30;
            ex = max(-60, min(60, ex));
            x = make_float((uint32_t)h2 & 0x7FFFFFu, ex);
        } else {
            const float k = (float)((h2 >> 8) & 511u) + 0.5f;
            x = __fmul_rn(s, k);
            int nudge = (int)((h2 >> 20) & 7u) - 3;
            x = __uint_as_float(__float_as_uint(x) + nudge);
            if (!(fabsf(x) <= 1152921504606846976.0f)) x = s;
        }
        if (h2 & 1u) x = -x;
        const float want = __fdiv_rn(x, s);
        const float got = div_by_scale(x, s, __frcp_rn(s));
        if (__float_as_uint(want) != __float_as_uint(got)) ++bad;
    }
    bad = __reduce_add_sync(0xFFFFFFFFu, (unsigned)bad);
    if ((threadIdx.x & 31) == 0 && bad) atomicAdd(mismatches, bad);
}

}  // namespace
}  // namespace granq

extern "C" int granq_selftest_division(uint64_t pairs, uint64_t seed, unsigned long long* device_mismatches,
                                       void* cuda_stream) {
    if (!device_mismatches || pairs == 0) return GRANQ_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(device_mismatches, 0, sizeof(unsigned long long), st) != cudaSuccess) return GRANQ_ERR_CUDA;
    granq::division_selftest_kernel<<<148 * 8, 256, 0, st>>>(pairs, seed, device_mismatches);
    return cudaGetLastError() == cudaSuccess ? GRANQ_OK : GRANQ_ERR_CUDA;
}
