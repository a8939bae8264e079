// Host-side declarations shared by the translation units of the GranQ library.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "granq_device.cuh"

namespace granq {

// A tensor reduced to channel-group form: element e lies in plane p = e / inner and in
// group p % C.  Sample-channel grouping is (outer = 1, C = outer * C); tensor grouping is
// (outer = 1, C = 1, inner = E).
struct Geom {
    int64_t E;      // elements
    int64_t outer;  // slabs
    int64_t C;      // groups (< 2^31)
    int64_t inner;  // contiguous elements of one (slab, group) plane
};

// (dims, channel axis, group mode) -> channel-group form and the number of groups; false when the
// arguments are invalid (null dims, axis or mode out of range, a non-positive dim, more than 2^40 elements).
constexpr int64_t kMaxElements = 1ll << 40;
inline bool make_geom(const int64_t dims[4], int axis, int group, Geom& g, int64_t& G) {
    if (!dims || axis < 0 || axis > 3 || group < 0 || group > 2) return false;
    int64_t E = 1;
    for (int d = 0; d < 4; ++d) {
        if (dims[d] <= 0 || dims[d] > kMaxElements) return false;
        if (E > kMaxElements / dims[d]) return false;
        E *= dims[d];
    }
    if (E > kMaxElements) return false;
    int64_t outer = 1, inner = 1;
    for (int d = 0; d < axis; ++d) outer *= dims[d];
    for (int d = axis + 1; d < 4; ++d) inner *= dims[d];
    const int64_t C = dims[axis];
    g.E = E;
    if (group == 0) {            // GRANQ_GROUP_CHANNEL
        g.outer = outer; g.C = C; g.inner = inner;
    } else if (group == 1) {     // GRANQ_GROUP_SAMPLE_CHANNEL
        g.outer = 1; g.C = outer * C; g.inner = inner;
    } else {                     // GRANQ_GROUP_TENSOR
        g.outer = 1; g.C = 1; g.inner = E;
    }
    G = g.C;
    return true;
}

// Workspace layout (all plans): a 256-byte header whose first word is the device status,
// then G min-keys, G max-keys, then G + 1 wave arrival counters.
constexpr size_t kWsHeaderBytes = 256;
struct Workspace {
    uint32_t* status;
    uint32_t* kmin;
    uint32_t* kmax;
    uint32_t* counters;
    size_t clear_bytes;  // bytes from the start that must be zero before a launch
};
inline size_t workspace_bytes_for(int64_t G) {
    size_t b = kWsHeaderBytes + (size_t)G * 8 + ((size_t)G + 1) * 4;
    return (b + 255) & ~(size_t)255;
}
inline Workspace carve_workspace(void* ws, int64_t G) {
    Workspace w;
    char* p = (char*)ws;
    w.status = (uint32_t*)p;
    w.kmin = (uint32_t*)(p + kWsHeaderBytes);
    w.kmax = w.kmin + G;
    w.counters = w.kmax + G;
    w.clear_bytes = kWsHeaderBytes + (size_t)G * 8 + ((size_t)G + 1) * 4;
    return w;
}

enum { MODE_FWD = 1, MODE_BWD = 2, MODE_BOTH = 3 };

struct QuantIO {
    const void* x;
    const void* gy;   // MODE_BWD / MODE_BOTH
    void* y;          // MODE_FWD / MODE_BOTH
    void* gx;         // MODE_BWD / MODE_BOTH
    uint8_t* codes;   // optional
    uint8_t* mask;    // optional
    uint32_t* pmask;  // optional: the mask at one bit per element (forward plans that support it)
    double* dist;     // optional: 4 running sums of Table 2's statistics, zero on entry (same plans)
    uint32_t* pcodes; // optional: the integer codes as a bit string, code_bits each (flat forward kernel; y may then be null)
    int code_bits;
};

// ---- generic ("flat") kernels: any geometry, any alignment --------------------------------
// keys must be zero on entry; accumulates ordered min/max keys per group
cudaError_t launch_range_flat(const void* x, int dtype, const Geom& g, uint32_t* kmin, uint32_t* kmax,
                              cudaStream_t st);
// keys -> lo / hi (and s / z when bits > 0 and the pointers are given)
cudaError_t launch_finalize_range(const uint32_t* kmin, const uint32_t* kmax, int64_t G, float* lo, float* hi,
                                  int bits, float* s_opt, float* z_opt, cudaStream_t st);
// lo / hi -> s / z
cudaError_t launch_params(const float* lo, const float* hi, int64_t G, int bits, float* s_opt, float* z_opt,
                          cudaStream_t st);
// elementwise quantize / backward with a per-group range in lo / hi
cudaError_t launch_quant_flat(const QuantIO& io, int mode, int dtype, const Geom& g, int bits, const float* lo,
                              const float* hi, cudaStream_t st);
// STE backward from the mask at one bit per element (bit e % 32 of word e / 32)
cudaError_t launch_bwd_packmask(const void* gy, const uint32_t* pmask, void* gx, int dtype, int64_t E,
                                cudaStream_t st);
// sums[0..3] += sum x^2, sum q^2, sum x*q, sum (x-q)^2 over E elements (Table 2's raw material)
cudaError_t launch_distortion(const void* x, const void* q, int dtype, int64_t E, double* sums, cudaStream_t st);
// Eq. 6 from the packed integer codes (element e in bits [e*b, (e+1)*b) of the bit string)
cudaError_t launch_dequant_packed(const uint32_t* pcodes, void* y, int dtype, const Geom& g, int bits, const float* s,
                                  const float* z, cudaStream_t st);
// the "conventional" scheme: a host loop over groups with three launches each
cudaError_t launch_naive(const QuantIO& io, int mode, int dtype, const Geom& g, int bits, uint32_t* kmin,
                         uint32_t* kmax, float* lo, float* hi, cudaStream_t st, int* launches);

// ---- on-chip staged persistent kernel ------------------------------------------------------
struct StagedPlan {
    bool ok;
    int grid, threads, depth;      // CTAs, threads per CTA, buffers per CTA
    uint32_t smem_bytes;           // dynamic shared memory per CTA
    uint32_t buf_units;            // 16-byte units per buffer
    uint32_t cw;                   // channels per wave
    uint32_t cu;                   // units per chunk
    uint32_t nwaves;
};
// Test / tuning overrides of the planner (0 = automatic).
struct StagedTuning {
    int depth;            // force the number of buffers per CTA (1..3)
    int max_buf_units;    // cap on 16-byte units per buffer (forces many small waves)
    int grid;             // cap on the number of CTAs
    int spin_limit;       // iteration limit of the wait on a wave's arrival count
    int extra_arrivals;   // test hook: arrivals a wave waits for beyond the grid size (never come)
    int ctas_per_sm;      // CTAs sharing one SM (1 or 2); they split its threads and shared memory
    int l2_wave_kb;       // L2-wave plan: target x bytes of one wave, in KiB
    int l2_upl;           // L2-wave plan: 16-byte units per lane and step (2 or 4)
    int l2_ctas_per_sm;   // L2-wave and column-walk plans: cap on resident CTAs per SM
    int l2_lag;           // column-walk plan: waves of phase 1 running ahead of phase 2 (1..3)
    int cl_tile_kb;       // cluster plan: limit on the staged tile of one CTA, in KiB
    int cl_r;             // cluster plan: CTAs per cluster (1, 2, 4, 8)
    int cl_threads;       // cluster plan: threads per CTA
    int cl_load;          // cluster plan: 1 = bulk copies for x, 2 = plain loads that reduce on the way, 3 = bulk copies for x and gy
    int cl_prefetch;      // cluster plan: 1 = ask the L2 for gy while x is loading, 2 = do not
    int cl_kmul;          // cluster plan: multiplier of the minimal channel count of a run
    int cl_pdl;           // cluster plan: 2 = no programmatic dependent launch
};
StagedPlan plan_staged(int dtype, const Geom& g, const QuantIO& io, int device, const StagedTuning& tune);
StagedPlan plan_staged_on(int dtype, const Geom& g, const QuantIO& io, int sm_count, int smem_optin,
                          const StagedTuning& tune);
cudaError_t launch_staged(const StagedPlan& plan, const QuantIO& io, int mode, int dtype, const Geom& g, int bits,
                          const Workspace& ws, float* lo, float* hi, float* s_opt, float* z_opt,
                          const StagedTuning& tune, cudaStream_t st);

// ---- L2-resident-wave persistent kernel ---------------------------------------------------
struct L2Plan {
    bool ok;
    int upl;                 // 16-byte units per lane and step
    uint32_t smem_bytes;     // dynamic shared memory per CTA
    uint32_t cw;             // channels per wave
    uint32_t nwaves;
};
L2Plan plan_l2wave(int dtype, const Geom& g, const QuantIO& io, const StagedTuning& tune);
cudaError_t launch_l2wave(const L2Plan& plan, const QuantIO& io, int mode, int dtype, const Geom& g, int bits,
                          const Workspace& ws, float* lo, float* hi, float* s_opt, float* z_opt,
                          const StagedTuning& tune, cudaStream_t st);

// ---- column-walk persistent kernel (L2-resident waves, one unit column per thread) ----------
struct ColPlan {
    bool ok;
    uint32_t cw;             // channels per wave
    uint32_t nwaves;
    uint32_t lag;            // waves of phase 1 running ahead of phase 2
};
ColPlan plan_colwalk(int dtype, const Geom& g, const QuantIO& io, const StagedTuning& tune);
cudaError_t launch_colwalk(const ColPlan& plan, const QuantIO& io, int mode, int dtype, const Geom& g, int bits,
                           const Workspace& ws, float* lo, float* hi, float* s_opt, float* z_opt,
                           const StagedTuning& tune, cudaStream_t st);

// ---- channels-last kernels (the channel is the innermost axis: one 16-byte unit holds V channels of a row) ----
bool plan_rows(int dtype, const Geom& g, const QuantIO& io);
cudaError_t launch_rows(const QuantIO& io, int mode, int dtype, const Geom& g, int bits, const Workspace& ws,
                        float* lo, float* hi, float* s_opt, float* z_opt, cudaStream_t st);

// ---- cluster-local kernel (a run of channels staged once in the shared memory of one cluster) ----
struct ClusterPlan {
    bool ok;
    uint32_t k;              // channels per run
    uint32_t R;              // CTAs per cluster
    uint32_t threads;        // threads per CTA
    uint32_t tile_bytes;     // staged tile of one CTA
    uint32_t smem_bytes;     // dynamic shared memory per CTA (tile + keys + parameters)
    int load;                // 0 = plain loads, 1 = x staged by bulk copies, 2 = x and gy staged by bulk copies
    bool prefetch_gy;
    bool early_launch;       // programmatic dependent launch: set the grid up while the kernel ahead drains
};
ClusterPlan plan_cluster(int dtype, const Geom& g, const QuantIO& io, bool backward, const StagedTuning& tune);
cudaError_t launch_cluster(const ClusterPlan& plan, const QuantIO& io, int mode, int dtype, const Geom& g, int bits,
                           const Workspace& ws, float* lo, float* hi, float* s_opt, float* z_opt,
                           const StagedTuning& tune, cudaStream_t st);

}  // namespace granq
