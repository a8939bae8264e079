// C ABI of the GranQ library: argument validation, reduction of (dims, channel axis, group
// mode) to channel-group geometry, plan selection and launches.  See include/granq.h.
#include "../../include/granq.h"

#include "granq_internal.h"

#include <math.h>

using namespace granq;

namespace {

StagedTuning g_tune = {};

bool dtype_ok(int dtype) { return dtype == GRANQ_F32 || dtype == GRANQ_BF16; }
size_t elt_size(int dtype) { return dtype == GRANQ_F32 ? 4 : 2; }

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    if (!a || !b) return false;
    const char* pa = (const char*)a;
    const char* pb = (const char*)b;
    return pa < pb + nb && pb < pa + na;
}

int check_workspace(const void* ws, size_t bytes, int64_t G) {
    if (!ws || ((uintptr_t)ws & 255) != 0) return GRANQ_ERR_WORKSPACE;
    if (bytes < workspace_bytes_for(G)) return GRANQ_ERR_WORKSPACE;
    return GRANQ_OK;
}

int cuda_status(cudaError_t e) { return e == cudaSuccess ? GRANQ_OK : GRANQ_ERR_CUDA; }

enum { PLAN_TWO_PASS = 0, PLAN_NAIVE = 1, PLAN_STAGED = 2, PLAN_L2WAVE = 3, PLAN_COLWALK = 4, PLAN_CLUSTER = 5, PLAN_ROWS = 6 };

// plan of the fused entry point; `plan_out` is filled when the staged plan is taken
int choose_plan(int dtype, const Geom& g, const QuantIO& io, bool backward, uint32_t flags, StagedPlan* plan_out,
                L2Plan* l2_out, ColPlan* col_out, ClusterPlan* cl_out) {
    if (flags & GRANQ_FLAG_FORCE_NAIVE) return PLAN_NAIVE;
    if (flags & GRANQ_FLAG_FORCE_TWO_PASS) return PLAN_TWO_PASS;
    if (flags & GRANQ_FLAG_FORCE_CLUSTER) {
        ClusterPlan kp = plan_cluster(dtype, g, io, backward, g_tune);
        if (!kp.ok) return -GRANQ_ERR_UNSUPPORTED;
        if (cl_out) *cl_out = kp;
        return PLAN_CLUSTER;
    }
    if (flags & GRANQ_FLAG_FORCE_COLWALK) {
        ColPlan cp = plan_colwalk(dtype, g, io, g_tune);
        if (!cp.ok) return -GRANQ_ERR_UNSUPPORTED;
        if (col_out) *col_out = cp;
        return PLAN_COLWALK;
    }
    if (flags & GRANQ_FLAG_FORCE_L2WAVE) {
        L2Plan lp = plan_l2wave(dtype, g, io, g_tune);
        if (!lp.ok) return -GRANQ_ERR_UNSUPPORTED;
        if (l2_out) *l2_out = lp;
        return PLAN_L2WAVE;
    }
    if (flags & GRANQ_FLAG_FORCE_STAGED) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return -GRANQ_ERR_CUDA;
        StagedPlan p = plan_staged(dtype, g, io, dev, g_tune);
        if (!p.ok) return -GRANQ_ERR_UNSUPPORTED;
        if (plan_out) *plan_out = p;
        return PLAN_STAGED;
    }
    // channels-last geometries (the channel is the innermost axis) have plans of their own: the cluster-local
    // kernel cannot stage them (a run of channels is a few bytes per row) and there are no planes to walk
    if (g.inner == 1 && plan_rows(dtype, g, io)) return PLAN_ROWS;
    // default: the cluster-local kernel where a run of channels fits the shared memory of one cluster
    // (x is then read once and nothing waits on the grid), else the column-walk kernel where there are
    // slabs to walk, else the L2-resident-wave kernel
    ClusterPlan kp = plan_cluster(dtype, g, io, backward, g_tune);
    ColPlan cp{};
    cp.ok = false;
    // Measured exception: forward-only bf16 tensors of 48 MB and more (a 100 KB tile then holds 51 200 elements
    // and a CTA's chain of copy, fold and quantize is twice as long as for fp32) run 6-15 % faster on the
    // column walk; with a gradient, and for fp32, the cluster-local kernel wins wherever it fits.
    const bool long_chain = dtype == 1 && !backward && !(io.codes || io.mask || io.pmask || io.dist) &&
                            (uint64_t)g.E * 2 >= (48ull << 20);
    if (kp.ok && long_chain) {
        cp = plan_colwalk(dtype, g, io, g_tune);
        if (cp.ok) {
            if (col_out) *col_out = cp;
            return PLAN_COLWALK;
        }
    }
    if (kp.ok) {
        if (cl_out) *cl_out = kp;
        return PLAN_CLUSTER;
    }
    cp = plan_colwalk(dtype, g, io, g_tune);
    if (cp.ok) {
        if (col_out) *col_out = cp;
        return PLAN_COLWALK;
    }
    L2Plan lp = plan_l2wave(dtype, g, io, g_tune);
    if (lp.ok) {
        if (l2_out) *l2_out = lp;
        return PLAN_L2WAVE;
    }
    return PLAN_TWO_PASS;
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace

extern "C" {

const char* granq_status_string(int status) {
    switch (status) {
        case GRANQ_OK: return "ok";
        case GRANQ_ERR_INVALID_ARG: return "invalid argument";
        case GRANQ_ERR_UNSUPPORTED: return "unsupported geometry or plan";
        case GRANQ_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case GRANQ_ERR_CUDA: return "CUDA error";
        case GRANQ_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        default: return "unknown status";
    }
}

int64_t granq_num_groups(const int64_t dims[4], int channel_axis, int group) {
    Geom g;
    int64_t G;
    if (!make_geom(dims, channel_axis, group, g, G)) return -1;
    return G;
}

size_t granq_workspace_bytes(int dtype, const int64_t dims[4], int channel_axis, int group) {
    Geom g;
    int64_t G;
    if (!dtype_ok(dtype) || !make_geom(dims, channel_axis, group, g, G)) return 0;
    return workspace_bytes_for(G);
}

int granq_range(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group, float* min_out,
                float* max_out, void* workspace, size_t workspace_bytes, uint32_t flags, void* cuda_stream) {
    (void)flags;
    Geom g;
    int64_t G;
    if (!x || !min_out || !max_out || !dtype_ok(dtype) || !make_geom(dims, channel_axis, group, g, G))
        return GRANQ_ERR_INVALID_ARG;
    if (G >= (1ll << 31)) return GRANQ_ERR_UNSUPPORTED;
    if (int rc = check_workspace(workspace, workspace_bytes, G)) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    Workspace ws = carve_workspace(workspace, G);
    cudaError_t e = cudaMemsetAsync(workspace, 0, ws.clear_bytes, st);
    if (e == cudaSuccess) e = launch_range_flat(x, dtype, g, ws.kmin, ws.kmax, st);
    if (e == cudaSuccess) e = launch_finalize_range(ws.kmin, ws.kmax, G, min_out, max_out, 0, nullptr, nullptr, st);
    return cuda_status(e);
}

int granq_fakequant_fwd(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group, int bits,
                        const float* min_in, const float* max_in, void* y, uint8_t* codes_opt, float* scale_opt,
                        float* zp_opt, uint32_t flags, void* cuda_stream) {
    (void)flags;
    Geom g;
    int64_t G;
    if (!x || !y || !min_in || !max_in || bits < 1 || bits > 8 || !dtype_ok(dtype) ||
        !make_geom(dims, channel_axis, group, g, G))
        return GRANQ_ERR_INVALID_ARG;
    if (G >= (1ll << 31)) return GRANQ_ERR_UNSUPPORTED;
    const size_t nb = (size_t)g.E * elt_size(dtype);
    if (overlaps(x, nb, y, nb)) return GRANQ_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    QuantIO io{x, nullptr, y, nullptr, codes_opt, nullptr};
    cudaError_t e = launch_quant_flat(io, MODE_FWD, dtype, g, bits, min_in, max_in, st);
    if (e == cudaSuccess && (scale_opt || zp_opt)) e = launch_params(min_in, max_in, G, bits, scale_opt, zp_opt, st);
    return cuda_status(e);
}

int granq_fakequant_bwd(const void* gy, const void* x, int dtype, const int64_t dims[4], int channel_axis, int group,
                        int bits, const float* min_in, const float* max_in, void* gx, uint8_t* mask_opt,
                        uint32_t flags, void* cuda_stream) {
    (void)flags;
    Geom g;
    int64_t G;
    if (!gy || !x || !gx || !min_in || !max_in || bits < 1 || bits > 8 || !dtype_ok(dtype) ||
        !make_geom(dims, channel_axis, group, g, G))
        return GRANQ_ERR_INVALID_ARG;
    if (G >= (1ll << 31)) return GRANQ_ERR_UNSUPPORTED;
    const size_t nb = (size_t)g.E * elt_size(dtype);
    if (overlaps(x, nb, gx, nb) || overlaps(gy, nb, gx, nb)) return GRANQ_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    QuantIO io{x, gy, nullptr, gx, nullptr, mask_opt};
    return cuda_status(launch_quant_flat(io, MODE_BWD, dtype, g, bits, min_in, max_in, st));
}

int granq_fakequant_fused(const void* x, const void* gy_opt, int dtype, const int64_t dims[4], int channel_axis,
                          int group, int bits, void* y, void* gx_opt, float* min_out, float* max_out,
                          uint8_t* codes_opt, uint8_t* mask_opt, float* scale_opt, float* zp_opt, void* workspace,
                          size_t workspace_bytes, uint32_t flags, void* cuda_stream) {
    Geom g;
    int64_t G;
    if (!x || !y || !min_out || !max_out || bits < 1 || bits > 8 || !dtype_ok(dtype) ||
        !make_geom(dims, channel_axis, group, g, G))
        return GRANQ_ERR_INVALID_ARG;
    if ((gy_opt == nullptr) != (gx_opt == nullptr)) return GRANQ_ERR_INVALID_ARG;
    if (mask_opt && !gy_opt) return GRANQ_ERR_INVALID_ARG;
    if (G >= (1ll << 31)) return GRANQ_ERR_UNSUPPORTED;
    const size_t nb = (size_t)g.E * elt_size(dtype);
    if (overlaps(x, nb, y, nb) || overlaps(x, nb, gx_opt, nb) || overlaps(gy_opt, nb, y, nb) ||
        overlaps(gy_opt, nb, gx_opt, nb) || overlaps(y, nb, gx_opt, nb))
        return GRANQ_ERR_INVALID_ARG;
    if (int rc = check_workspace(workspace, workspace_bytes, G)) return rc;

    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int mode = gy_opt ? MODE_BOTH : MODE_FWD;
    QuantIO io{x, gy_opt, y, gx_opt, codes_opt, mask_opt};
    StagedPlan sp{};
    L2Plan lp{};
    ColPlan cp{};
    ClusterPlan kp{};
    const int plan = choose_plan(dtype, g, io, gy_opt != nullptr, flags, &sp, &lp, &cp, &kp);
    if (plan < 0) return -plan;

    Workspace ws = carve_workspace(workspace, G);
    // The column-walk kernel leaves a zeroed workspace zeroed and the cluster-local kernel writes
    // nothing but the status word (and that only when a wait ran out); with the caller's word that
    // the workspace is zero on entry nothing has to be cleared.  The other plans clear before and, to
    // keep that word true for the next call, after.
    const bool zeroed = (flags & GRANQ_FLAG_WORKSPACE_ZEROED) != 0;
    const bool keeps_zero = plan == PLAN_COLWALK || plan == PLAN_CLUSTER;
    cudaError_t e = cudaSuccess;
    if (plan == PLAN_CLUSTER) {
        if (!zeroed) e = cudaMemsetAsync(workspace, 0, sizeof(uint32_t), st);      // the status word
    } else if (!(zeroed && keeps_zero)) {
        e = cudaMemsetAsync(workspace, 0, ws.clear_bytes, st);
    }
    if (e != cudaSuccess) return GRANQ_ERR_CUDA;
    if (plan == PLAN_CLUSTER) {
        e = launch_cluster(kp, io, mode, dtype, g, bits, ws, min_out, max_out, scale_opt, zp_opt, g_tune, st);
    } else if (plan == PLAN_ROWS) {
        e = launch_rows(io, mode, dtype, g, bits, ws, min_out, max_out, scale_opt, zp_opt, st);
    } else if (plan == PLAN_STAGED) {
        e = launch_staged(sp, io, mode, dtype, g, bits, ws, min_out, max_out, scale_opt, zp_opt, g_tune, st);
    } else if (plan == PLAN_L2WAVE) {
        e = launch_l2wave(lp, io, mode, dtype, g, bits, ws, min_out, max_out, scale_opt, zp_opt, g_tune, st);
    } else if (plan == PLAN_COLWALK) {
        e = launch_colwalk(cp, io, mode, dtype, g, bits, ws, min_out, max_out, scale_opt, zp_opt, g_tune, st);
    } else if (plan == PLAN_NAIVE) {
        e = launch_naive(io, mode, dtype, g, bits, ws.kmin, ws.kmax, min_out, max_out, st, nullptr);
        if (e == cudaSuccess && (scale_opt || zp_opt))
            e = launch_params(min_out, max_out, G, bits, scale_opt, zp_opt, st);
    } else {
        e = launch_range_flat(x, dtype, g, ws.kmin, ws.kmax, st);
        if (e == cudaSuccess)
            e = launch_finalize_range(ws.kmin, ws.kmax, G, min_out, max_out, bits, scale_opt, zp_opt, st);
        if (e == cudaSuccess) e = launch_quant_flat(io, mode, dtype, g, bits, min_out, max_out, st);
    }
    if (e == cudaSuccess && zeroed && !keeps_zero)
        e = cudaMemsetAsync((char*)workspace + sizeof(uint32_t), 0, ws.clear_bytes - sizeof(uint32_t), st);
    return cuda_status(e);
}

size_t granq_packmask_bytes(const int64_t dims[4]) {
    Geom g;
    int64_t G;
    if (!make_geom(dims, 1, GRANQ_GROUP_TENSOR, g, G)) return 0;
    return (size_t)((g.E + 31) / 32) * 4;
}

int granq_fakequant_fwd_packmask(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group,
                                 int bits, const float* min_in, const float* max_in, void* y,
                                 uint32_t* packed_mask, float* scale_opt, float* zp_opt, uint32_t flags,
                                 void* cuda_stream) {
    (void)flags;
    Geom g;
    int64_t G;
    if (!x || !y || !packed_mask || !min_in || !max_in || bits < 1 || bits > 8 || !dtype_ok(dtype) ||
        !make_geom(dims, channel_axis, group, g, G) || ((uintptr_t)packed_mask & 3))
        return GRANQ_ERR_INVALID_ARG;
    if (G >= (1ll << 31)) return GRANQ_ERR_UNSUPPORTED;
    const size_t nb = (size_t)g.E * elt_size(dtype), mb = (size_t)((g.E + 31) / 32) * 4;
    if (overlaps(x, nb, y, nb) || overlaps(x, nb, packed_mask, mb) || overlaps(y, nb, packed_mask, mb))
        return GRANQ_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    QuantIO io{x, nullptr, y, nullptr, nullptr, nullptr, packed_mask};
    cudaError_t e = launch_quant_flat(io, MODE_FWD, dtype, g, bits, min_in, max_in, st);
    if (e == cudaSuccess && (scale_opt || zp_opt)) e = launch_params(min_in, max_in, G, bits, scale_opt, zp_opt, st);
    return cuda_status(e);
}

int granq_fakequant_bwd_packmask(const void* gy, const uint32_t* packed_mask, int dtype, const int64_t dims[4],
                                 void* gx, uint32_t flags, void* cuda_stream) {
    (void)flags;
    Geom g;
    int64_t G;
    if (!gy || !gx || !packed_mask || !dtype_ok(dtype) || !make_geom(dims, 1, GRANQ_GROUP_TENSOR, g, G) ||
        ((uintptr_t)packed_mask & 3))
        return GRANQ_ERR_INVALID_ARG;
    const size_t nb = (size_t)g.E * elt_size(dtype), mb = (size_t)((g.E + 31) / 32) * 4;
    if (overlaps(gy, nb, gx, nb) || overlaps(packed_mask, mb, gx, nb)) return GRANQ_ERR_INVALID_ARG;
    return cuda_status(launch_bwd_packmask(gy, packed_mask, gx, dtype, g.E, (cudaStream_t)cuda_stream));
}

int granq_fakequant_fused_fwd_packmask(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group,
                                       int bits, void* y, uint32_t* packed_mask, float* min_out, float* max_out,
                                       float* scale_opt, float* zp_opt, void* workspace, size_t workspace_bytes,
                                       uint32_t flags, void* cuda_stream) {
    Geom g;
    int64_t G;
    if (!x || !y || !packed_mask || !min_out || !max_out || bits < 1 || bits > 8 || !dtype_ok(dtype) ||
        !make_geom(dims, channel_axis, group, g, G) || ((uintptr_t)packed_mask & 3))
        return GRANQ_ERR_INVALID_ARG;
    if (G >= (1ll << 31)) return GRANQ_ERR_UNSUPPORTED;
    const size_t nb = (size_t)g.E * elt_size(dtype), mb = (size_t)((g.E + 31) / 32) * 4;
    if (overlaps(x, nb, y, nb) || overlaps(x, nb, packed_mask, mb) || overlaps(y, nb, packed_mask, mb))
        return GRANQ_ERR_INVALID_ARG;
    if (int rc = check_workspace(workspace, workspace_bytes, G)) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    QuantIO io{x, nullptr, y, nullptr, nullptr, nullptr, packed_mask};
    // the cluster-local kernel where a run of whole mask words fits one cluster, else the column-walk kernel
    // where the geometry allows whole mask words per wave, else range pass + flat pass
    ColPlan cp{};
    ClusterPlan kp{};
    const bool two_pass = (flags & GRANQ_FLAG_FORCE_TWO_PASS) != 0;
    if (!two_pass && !(flags & GRANQ_FLAG_FORCE_COLWALK)) kp = plan_cluster(dtype, g, io, false, g_tune);
    if ((flags & GRANQ_FLAG_FORCE_CLUSTER) && !kp.ok) return GRANQ_ERR_UNSUPPORTED;
    if (!two_pass && !kp.ok) cp = plan_colwalk(dtype, g, io, g_tune);
    if ((flags & GRANQ_FLAG_FORCE_COLWALK) && !cp.ok) return GRANQ_ERR_UNSUPPORTED;
    Workspace ws = carve_workspace(workspace, G);
    const bool zeroed = (flags & GRANQ_FLAG_WORKSPACE_ZEROED) != 0;
    cudaError_t e = cudaSuccess;
    if (kp.ok) {
        if (!zeroed) e = cudaMemsetAsync(workspace, 0, sizeof(uint32_t), st);      // the status word
        // the kernel writes the mask byte by byte: the padding bits of a last, partial word are cleared here
        if (e == cudaSuccess && g.E % 32 != 0) e = cudaMemsetAsync(packed_mask + g.E / 32, 0, sizeof(uint32_t), st);
        if (e != cudaSuccess) return GRANQ_ERR_CUDA;
        return cuda_status(launch_cluster(kp, io, MODE_FWD, dtype, g, bits, ws, min_out, max_out, scale_opt, zp_opt,
                                          g_tune, st));
    }
    if (!(zeroed && cp.ok)) e = cudaMemsetAsync(workspace, 0, ws.clear_bytes, st);
    if (e != cudaSuccess) return GRANQ_ERR_CUDA;
    if (cp.ok) {
        e = launch_colwalk(cp, io, MODE_FWD, dtype, g, bits, ws, min_out, max_out, scale_opt, zp_opt, g_tune, st);
    } else {
        e = launch_range_flat(x, dtype, g, ws.kmin, ws.kmax, st);
        if (e == cudaSuccess)
            e = launch_finalize_range(ws.kmin, ws.kmax, G, min_out, max_out, bits, scale_opt, zp_opt, st);
        if (e == cudaSuccess) e = launch_quant_flat(io, MODE_FWD, dtype, g, bits, min_out, max_out, st);
        if (e == cudaSuccess && zeroed)
            e = cudaMemsetAsync((char*)workspace + sizeof(uint32_t), 0, ws.clear_bytes - sizeof(uint32_t), st);
    }
    return cuda_status(e);
}

int granq_fakequant_fused_batch(const granq_fused_desc* descs, int n_tensors, int dtype, int channel_axis, int group,
                                uint32_t flags, void* cuda_stream, int* failed_opt) {
    if (failed_opt) *failed_opt = -1;
    if (!descs || n_tensors < 0) return GRANQ_ERR_INVALID_ARG;
    for (int i = 0; i < n_tensors; ++i) {
        const granq_fused_desc& d = descs[i];
        const int rc = granq_fakequant_fused(d.x, d.gy_opt, dtype, d.dims, channel_axis, group, d.bits, d.y, d.gx_opt,
                                             d.min_out, d.max_out, nullptr, nullptr, d.scale_opt, d.zp_opt, d.workspace,
                                             d.workspace_bytes, flags, cuda_stream);
        if (rc != GRANQ_OK) {
            if (failed_opt) *failed_opt = i;
            return rc;
        }
    }
    return GRANQ_OK;
}

int granq_distortion(const void* x, const void* q, int dtype, const int64_t dims[4], double* sums_out,
                     uint32_t flags, void* cuda_stream) {
    (void)flags;
    Geom g;
    int64_t G;
    if (!x || !q || !sums_out || !dtype_ok(dtype) || !make_geom(dims, 1, GRANQ_GROUP_TENSOR, g, G) ||
        ((uintptr_t)sums_out & 7))
        return GRANQ_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemsetAsync(sums_out, 0, 4 * sizeof(double), st);
    if (e == cudaSuccess) e = launch_distortion(x, q, dtype, g.E, sums_out, st);
    return cuda_status(e);
}

int granq_distortion_stats(const double sums[4], double* cosine_out, double* rel_error_out) {
    if (!sums) return GRANQ_ERR_INVALID_ARG;
    const double sxx = sums[0], sqq = sums[1], sxq = sums[2], sdd = sums[3];
    const double den = sqrt(sxx) * sqrt(sqq);
    if (cosine_out) *cosine_out = den > 0.0 ? sxq / den : 0.0;
    if (rel_error_out) *rel_error_out = sxx > 0.0 ? sqrt(sdd) / sqrt(sxx) : 0.0;
    return GRANQ_OK;
}

int granq_fakequant_fused_stats(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group,
                                int bits, void* y, float* min_out, float* max_out, float* scale_opt, float* zp_opt,
                                double* sums_out, void* workspace, size_t workspace_bytes, uint32_t flags,
                                void* cuda_stream) {
    Geom g;
    int64_t G;
    if (!x || !y || !sums_out || !min_out || !max_out || bits < 1 || bits > 8 || !dtype_ok(dtype) ||
        !make_geom(dims, channel_axis, group, g, G) || ((uintptr_t)sums_out & 7))
        return GRANQ_ERR_INVALID_ARG;
    if (G >= (1ll << 31)) return GRANQ_ERR_UNSUPPORTED;
    const size_t nb = (size_t)g.E * elt_size(dtype);
    if (overlaps(x, nb, y, nb) || overlaps(x, nb, sums_out, 32) || overlaps(y, nb, sums_out, 32))
        return GRANQ_ERR_INVALID_ARG;
    if (int rc = check_workspace(workspace, workspace_bytes, G)) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    QuantIO io{x, nullptr, y, nullptr, nullptr, nullptr, nullptr, sums_out};
    // the column-walk kernel where there are slabs to walk, else range pass + flat pass (layer-wise and
    // per-sample groups): the statistics are gathered in the pass that writes y either way
    ColPlan cp{};
    ClusterPlan kp{};
    const bool two_pass = (flags & GRANQ_FLAG_FORCE_TWO_PASS) != 0;
    if (!two_pass && !(flags & GRANQ_FLAG_FORCE_COLWALK)) kp = plan_cluster(dtype, g, io, false, g_tune);
    if ((flags & GRANQ_FLAG_FORCE_CLUSTER) && !kp.ok) return GRANQ_ERR_UNSUPPORTED;
    if (!two_pass && !kp.ok) cp = plan_colwalk(dtype, g, io, g_tune);
    if ((flags & GRANQ_FLAG_FORCE_COLWALK) && !cp.ok) return GRANQ_ERR_UNSUPPORTED;
    Workspace ws = carve_workspace(workspace, G);
    const bool zeroed = (flags & GRANQ_FLAG_WORKSPACE_ZEROED) != 0;
    cudaError_t e = cudaMemsetAsync(sums_out, 0, 4 * sizeof(double), st);
    if (e == cudaSuccess && kp.ok) {
        if (!zeroed) e = cudaMemsetAsync(workspace, 0, sizeof(uint32_t), st);      // the status word
        if (e != cudaSuccess) return GRANQ_ERR_CUDA;
        return cuda_status(launch_cluster(kp, io, MODE_FWD, dtype, g, bits, ws, min_out, max_out, scale_opt, zp_opt,
                                          g_tune, st));
    }
    if (e == cudaSuccess && !(zeroed && cp.ok)) e = cudaMemsetAsync(workspace, 0, ws.clear_bytes, st);
    if (e != cudaSuccess) return GRANQ_ERR_CUDA;
    if (cp.ok) {
        e = launch_colwalk(cp, io, MODE_FWD, dtype, g, bits, ws, min_out, max_out, scale_opt, zp_opt, g_tune, st);
    } else {
        e = launch_range_flat(x, dtype, g, ws.kmin, ws.kmax, st);
        if (e == cudaSuccess)
            e = launch_finalize_range(ws.kmin, ws.kmax, G, min_out, max_out, bits, scale_opt, zp_opt, st);
        if (e == cudaSuccess) e = launch_quant_flat(io, MODE_FWD, dtype, g, bits, min_out, max_out, st);
        if (e == cudaSuccess && zeroed)
            e = cudaMemsetAsync((char*)workspace + sizeof(uint32_t), 0, ws.clear_bytes - sizeof(uint32_t), st);
    }
    return cuda_status(e);
}

size_t granq_packed_codes_bytes(const int64_t dims[4], int bits) {
    Geom g;
    int64_t G;
    if (bits < 1 || bits > 8 || !make_geom(dims, 1, GRANQ_GROUP_TENSOR, g, G)) return 0;
    return (size_t)((g.E * bits + 31) / 32) * 4;
}

int granq_quantize_packed(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group, int bits,
                          const float* min_in, const float* max_in, uint32_t* packed_codes, void* y_opt,
                          float* scale_out, float* zp_out, uint32_t flags, void* cuda_stream) {
    (void)flags;
    Geom g;
    int64_t G;
    if (!x || !packed_codes || !min_in || !max_in || !scale_out || !zp_out || bits < 1 || bits > 8 ||
        !dtype_ok(dtype) || !make_geom(dims, channel_axis, group, g, G) || ((uintptr_t)packed_codes & 3))
        return GRANQ_ERR_INVALID_ARG;
    if (G >= (1ll << 31)) return GRANQ_ERR_UNSUPPORTED;
    const size_t nb = (size_t)g.E * elt_size(dtype), cbytes = (size_t)((g.E * bits + 31) / 32) * 4;
    if (overlaps(x, nb, y_opt, nb) || overlaps(x, nb, packed_codes, cbytes) || overlaps(y_opt, nb, packed_codes, cbytes))
        return GRANQ_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    QuantIO io{x, nullptr, y_opt, nullptr, nullptr, nullptr, nullptr, nullptr, packed_codes, bits};
    cudaError_t e = launch_quant_flat(io, MODE_FWD, dtype, g, bits, min_in, max_in, st);
    if (e == cudaSuccess) e = launch_params(min_in, max_in, G, bits, scale_out, zp_out, st);
    return cuda_status(e);
}

int granq_quantize_packed_fused(const void* x, int dtype, const int64_t dims[4], int channel_axis, int group, int bits,
                                uint32_t* packed_codes, float* min_out, float* max_out, float* scale_out, float* zp_out,
                                void* workspace, size_t workspace_bytes, uint32_t flags, void* cuda_stream) {
    Geom g;
    int64_t G;
    if (!x || !packed_codes || !min_out || !max_out || !scale_out || !zp_out || bits < 1 || bits > 8 ||
        !dtype_ok(dtype) || !make_geom(dims, channel_axis, group, g, G) || ((uintptr_t)packed_codes & 3))
        return GRANQ_ERR_INVALID_ARG;
    if (G >= (1ll << 31)) return GRANQ_ERR_UNSUPPORTED;
    const size_t nb = (size_t)g.E * elt_size(dtype), cbytes = (size_t)((g.E * bits + 31) / 32) * 4;
    if (overlaps(x, nb, packed_codes, cbytes)) return GRANQ_ERR_INVALID_ARG;
    if (int rc = check_workspace(workspace, workspace_bytes, G)) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    QuantIO io{x, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, packed_codes, bits};
    // the cluster-local kernel where a run of whole groups of 8 codes fits one cluster, the column walk where
    // slabs and waves are such groups, else range pass, parameters, elementwise pass
    ColPlan cp{};
    ClusterPlan kp{};
    const bool two_pass = (flags & GRANQ_FLAG_FORCE_TWO_PASS) != 0;
    if (!two_pass && !(flags & GRANQ_FLAG_FORCE_COLWALK)) kp = plan_cluster(dtype, g, io, false, g_tune);
    if ((flags & GRANQ_FLAG_FORCE_CLUSTER) && !kp.ok) return GRANQ_ERR_UNSUPPORTED;
    if (!two_pass && !kp.ok) cp = plan_colwalk(dtype, g, io, g_tune);
    if ((flags & GRANQ_FLAG_FORCE_COLWALK) && !cp.ok) return GRANQ_ERR_UNSUPPORTED;
    Workspace ws = carve_workspace(workspace, G);
    const bool zeroed = (flags & GRANQ_FLAG_WORKSPACE_ZEROED) != 0;
    cudaError_t e = cudaSuccess;
    if (kp.ok) {
        if (!zeroed) e = cudaMemsetAsync(workspace, 0, sizeof(uint32_t), st);      // the status word
        if (e != cudaSuccess) return GRANQ_ERR_CUDA;
        return cuda_status(launch_cluster(kp, io, MODE_FWD, dtype, g, bits, ws, min_out, max_out, scale_out, zp_out,
                                          g_tune, st));
    }
    if (!(zeroed && cp.ok)) e = cudaMemsetAsync(workspace, 0, ws.clear_bytes, st);
    if (e != cudaSuccess) return GRANQ_ERR_CUDA;
    if (cp.ok) {
        e = launch_colwalk(cp, io, MODE_FWD, dtype, g, bits, ws, min_out, max_out, scale_out, zp_out, g_tune, st);
    } else {
        e = launch_range_flat(x, dtype, g, ws.kmin, ws.kmax, st);
        if (e == cudaSuccess)
            e = launch_finalize_range(ws.kmin, ws.kmax, G, min_out, max_out, bits, scale_out, zp_out, st);
        if (e == cudaSuccess) e = launch_quant_flat(io, MODE_FWD, dtype, g, bits, min_out, max_out, st);
        if (e == cudaSuccess && zeroed)
            e = cudaMemsetAsync((char*)workspace + sizeof(uint32_t), 0, ws.clear_bytes - sizeof(uint32_t), st);
    }
    return cuda_status(e);
}

int granq_dequantize_packed(const uint32_t* packed_codes, int dtype, const int64_t dims[4], int channel_axis,
                            int group, int bits, const float* scale_in, const float* zp_in, void* y, uint32_t flags,
                            void* cuda_stream) {
    (void)flags;
    Geom g;
    int64_t G;
    if (!packed_codes || !scale_in || !zp_in || !y || bits < 1 || bits > 8 || !dtype_ok(dtype) ||
        !make_geom(dims, channel_axis, group, g, G) || ((uintptr_t)packed_codes & 3))
        return GRANQ_ERR_INVALID_ARG;
    const size_t nb = (size_t)g.E * elt_size(dtype), cbytes = (size_t)((g.E * bits + 31) / 32) * 4;
    if (overlaps(y, nb, packed_codes, cbytes)) return GRANQ_ERR_INVALID_ARG;
    return cuda_status(launch_dequant_packed(packed_codes, y, dtype, g, bits, scale_in, zp_in, (cudaStream_t)cuda_stream));
}

int granq_workspace_status(const void* workspace, void* cuda_stream) {
    if (!workspace) return GRANQ_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return GRANQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return GRANQ_ERR_CUDA;
    return word == 0 ? GRANQ_OK : (word == GRANQ_ERR_TIMEOUT ? GRANQ_ERR_TIMEOUT : GRANQ_ERR_CUDA);
}

// arena layout: x | gy | y | gx | lo | hi | s | z | workspace, each piece 256-byte aligned
size_t granq_host_arena_bytes(int dtype, const int64_t dims[4], int channel_axis, int group, int with_backward) {
    Geom g;
    int64_t G;
    if (!dtype_ok(dtype) || !make_geom(dims, channel_axis, group, g, G)) return 0;
    const size_t nb = align256((size_t)g.E * elt_size(dtype));
    return nb * (with_backward ? 4 : 2) + 4 * align256((size_t)G * 4) + workspace_bytes_for(G);
}

int granq_fakequant_fused_host(const void* x_host, const void* gy_host_opt, int dtype, const int64_t dims[4],
                               int channel_axis, int group, int bits, void* y_host, void* gx_host_opt,
                               float* min_host, float* max_host, float* scale_host_opt, float* zp_host_opt,
                               void* device_arena, size_t arena_bytes, uint32_t flags, void* cuda_stream) {
    Geom g;
    int64_t G;
    if (!x_host || !y_host || !min_host || !max_host || bits < 1 || bits > 8 || !dtype_ok(dtype) ||
        !make_geom(dims, channel_axis, group, g, G))
        return GRANQ_ERR_INVALID_ARG;
    if ((gy_host_opt == nullptr) != (gx_host_opt == nullptr)) return GRANQ_ERR_INVALID_ARG;
    if (G >= (1ll << 31)) return GRANQ_ERR_UNSUPPORTED;
    const int bwd = gy_host_opt ? 1 : 0;
    if (!device_arena || ((uintptr_t)device_arena & 255) ||
        arena_bytes < granq_host_arena_bytes(dtype, dims, channel_axis, group, bwd))
        return GRANQ_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t raw = (size_t)g.E * elt_size(dtype), nb = align256(raw), gb = align256((size_t)G * 4);
    char* p = (char*)device_arena;
    char* dx = p; p += nb;
    char* dgy = nullptr; if (bwd) { dgy = p; p += nb; }
    char* dy = p; p += nb;
    char* dgx = nullptr; if (bwd) { dgx = p; p += nb; }
    float* dlo = (float*)p; p += gb;
    float* dhi = (float*)p; p += gb;
    float* ds = (float*)p; p += gb;
    float* dz = (float*)p; p += gb;
    void* ws = p;
    if (cudaMemcpyAsync(dx, x_host, raw, cudaMemcpyHostToDevice, st) != cudaSuccess) return GRANQ_ERR_CUDA;
    if (bwd && cudaMemcpyAsync(dgy, gy_host_opt, raw, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return GRANQ_ERR_CUDA;
    int rc = granq_fakequant_fused(dx, dgy, dtype, dims, channel_axis, group, bits, dy, dgx, dlo, dhi, nullptr,
                                   nullptr, scale_host_opt ? ds : nullptr, zp_host_opt ? dz : nullptr, ws,
                                   workspace_bytes_for(G), flags, cuda_stream);
    if (rc != GRANQ_OK) return rc;
    cudaError_t e = cudaMemcpyAsync(y_host, dy, raw, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && bwd) e = cudaMemcpyAsync(gx_host_opt, dgx, raw, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(min_host, dlo, (size_t)G * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(max_host, dhi, (size_t)G * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && scale_host_opt)
        e = cudaMemcpyAsync(scale_host_opt, ds, (size_t)G * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && zp_host_opt) e = cudaMemcpyAsync(zp_host_opt, dz, (size_t)G * 4, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return GRANQ_ERR_CUDA;
    if (flags & GRANQ_FLAG_HOST_ASYNC) return GRANQ_OK;
    return granq_workspace_status(ws, cuda_stream);
}

int granq_host_arena_status(int dtype, const int64_t dims[4], int channel_axis, int group, int with_backward,
                            const void* device_arena, void* cuda_stream) {
    Geom g;
    int64_t G;
    if (!device_arena || !dtype_ok(dtype) || !make_geom(dims, channel_axis, group, g, G)) return GRANQ_ERR_INVALID_ARG;
    const size_t nb = align256((size_t)g.E * elt_size(dtype)), gb = align256((size_t)G * 4);
    const char* ws = (const char*)device_arena + nb * (with_backward ? 4 : 2) + 4 * gb;
    return granq_workspace_status(ws, cuda_stream);
}

int granq_fused_plan(int dtype, const int64_t dims[4], int channel_axis, int group, int with_backward,
                     uint32_t flags, int* launches_out) {
    Geom g;
    int64_t G;
    if (!dtype_ok(dtype) || !make_geom(dims, channel_axis, group, g, G)) return -GRANQ_ERR_INVALID_ARG;
    QuantIO io{};   // null pointers: alignment is assumed
    const int plan = choose_plan(dtype, g, io, with_backward != 0, flags, nullptr, nullptr, nullptr, nullptr);
    if (launches_out) {
        if (plan == PLAN_STAGED || plan == PLAN_L2WAVE || plan == PLAN_COLWALK || plan == PLAN_CLUSTER) *launches_out = 1;
        else if (plan == PLAN_ROWS) *launches_out = 2;
        else if (plan == PLAN_NAIVE) *launches_out = (int)(3 * g.C);
        else if (plan == PLAN_TWO_PASS) *launches_out = 3;
    }
    return plan;
}

int granq_staged_geometry(int dtype, const int64_t dims[4], int channel_axis, int group, int sm_count,
                          int smem_bytes, int64_t out[8]) {
    Geom g;
    int64_t G;
    if (!out || !dtype_ok(dtype) || !make_geom(dims, channel_axis, group, g, G)) return GRANQ_ERR_INVALID_ARG;
    QuantIO io{};
    StagedPlan p = plan_staged_on(dtype, g, io, sm_count, smem_bytes, g_tune);
    if (!p.ok) return GRANQ_ERR_UNSUPPORTED;
    out[0] = p.grid; out[1] = p.threads; out[2] = p.depth; out[3] = p.smem_bytes;
    out[4] = p.buf_units; out[5] = p.cw; out[6] = p.cu; out[7] = p.nwaves;
    return GRANQ_OK;
}

int granq_cluster_geometry(int dtype, const int64_t dims[4], int channel_axis, int group, int with_backward,
                           int64_t out[8]) {
    Geom g;
    int64_t G;
    if (!out || !dtype_ok(dtype) || !make_geom(dims, channel_axis, group, g, G)) return GRANQ_ERR_INVALID_ARG;
    QuantIO io{};
    ClusterPlan p = plan_cluster(dtype, g, io, with_backward != 0, g_tune);
    if (!p.ok) return GRANQ_ERR_UNSUPPORTED;
    out[0] = (int64_t)((g.C + p.k - 1) / p.k) * p.R; out[1] = p.threads; out[2] = p.R; out[3] = p.smem_bytes;
    out[4] = p.tile_bytes; out[5] = p.k; out[6] = p.load; out[7] = p.prefetch_gy ? 1 : 0;
    return GRANQ_OK;
}

int granq_tune(int knob, int value) {
    switch (knob) {
        case GRANQ_KNOB_STAGED_DEPTH: g_tune.depth = value; return GRANQ_OK;
        case GRANQ_KNOB_STAGED_MAX_BUF_UNITS: g_tune.max_buf_units = value; return GRANQ_OK;
        case GRANQ_KNOB_STAGED_GRID: g_tune.grid = value; return GRANQ_OK;
        case GRANQ_KNOB_SPIN_LIMIT: g_tune.spin_limit = value; return GRANQ_OK;
        case GRANQ_KNOB_TEST_EXTRA_ARRIVALS: g_tune.extra_arrivals = value; return GRANQ_OK;
        case GRANQ_KNOB_STAGED_CTAS_PER_SM: g_tune.ctas_per_sm = value; return GRANQ_OK;
        case GRANQ_KNOB_L2_WAVE_KB: g_tune.l2_wave_kb = value; return GRANQ_OK;
        case GRANQ_KNOB_L2_UPL: g_tune.l2_upl = value; return GRANQ_OK;
        case GRANQ_KNOB_L2_CTAS_PER_SM: g_tune.l2_ctas_per_sm = value; return GRANQ_OK;
        case GRANQ_KNOB_L2_LAG: g_tune.l2_lag = value; return GRANQ_OK;
        case GRANQ_KNOB_CLUSTER_TILE_KB: g_tune.cl_tile_kb = value; return GRANQ_OK;
        case GRANQ_KNOB_CLUSTER_CTAS: g_tune.cl_r = value; return GRANQ_OK;
        case GRANQ_KNOB_CLUSTER_THREADS: g_tune.cl_threads = value; return GRANQ_OK;
        case GRANQ_KNOB_CLUSTER_LOAD: g_tune.cl_load = value; return GRANQ_OK;
        case GRANQ_KNOB_CLUSTER_PREFETCH: g_tune.cl_prefetch = value; return GRANQ_OK;
        case GRANQ_KNOB_CLUSTER_KMUL: g_tune.cl_kmul = value; return GRANQ_OK;
        case GRANQ_KNOB_CLUSTER_EARLY_LAUNCH: g_tune.cl_pdl = value; return GRANQ_OK;
        default: return GRANQ_ERR_INVALID_ARG;
    }
}

}  // extern "C"
