// Generic GranQ kernels: they accept any geometry and any pointer alignment and make no
// assumption about what fits on chip.  The fused two-pass plan is
//   range_flat_kernel (Eq. 4)  ->  finalize_range_kernel (Eq. 5)  ->  quant_flat_kernel (Eq. 1, 6, STE)
// and the stand-alone entry points (range / forward / backward) use the same kernels.
// Also here: the "conventional" per-channel loop the paper measures against (Section 5.3.2).
#include "granq_internal.h"

namespace granq {

namespace {

constexpr int kThreads = 256;
constexpr uint32_t kTile = 8192;          // elements per CTA tile
constexpr int kUnroll = 4;                // 16-byte loads in flight per thread
constexpr uint32_t kTableMax = 1026;      // planes of one tile whose (s, z) are tabled in shared memory

struct FlatGeom {
    int64_t E, inner, C, ntiles;
    FastDiv div_inner, div_C;   // valid when the divisor is < 2^30
    int inner_big, C_big;       // divisor >= 2^30: at most one wrap inside a tile
};

FlatGeom make_flat(const Geom& g) {
    FlatGeom f;
    f.E = g.E;
    f.inner = g.inner;
    f.C = g.C;
    f.ntiles = (g.E + kTile - 1) / kTile;
    f.inner_big = g.inner >= (1ll << 30);
    f.C_big = g.C >= (1ll << 30);
    f.div_inner = make_fastdiv(f.inner_big ? 1u : (uint32_t)g.inner);
    f.div_C = make_fastdiv(f.C_big ? 1u : (uint32_t)g.C);
    return f;
}

// Position of a tile's first element: plane remainder and group of its first plane.
struct TileBase {
    int64_t rem;      // e0 % inner
    uint32_t c;       // (e0 / inner) % C
};

__device__ __forceinline__ TileBase tile_base(const FlatGeom& g, int64_t e0) {
    TileBase b;
    int64_t p = e0 / g.inner;
    b.rem = e0 - p * g.inner;
    b.c = (uint32_t)(p % g.C);
    return b;
}

// plane offset (relative to the tile's first plane) of the element k elements into the tile
__device__ __forceinline__ uint32_t plane_offset(const FlatGeom& g, const TileBase& b, uint32_t k) {
    if (g.inner_big) return (b.rem + (int64_t)k >= g.inner) ? 1u : 0u;
    return g.div_inner.div((uint32_t)b.rem + k);
}
// group of the plane `q` planes after the tile's first plane
__device__ __forceinline__ uint32_t group_at(const FlatGeom& g, const TileBase& b, uint32_t q) {
    if (g.C_big) {
        int64_t v = (int64_t)b.c + q;
        return (uint32_t)(v >= g.C ? v - g.C : v);
    }
    uint32_t v = b.c + q, quo, r;
    g.div_C.divmod(v, quo, r);
    return r;
}

// ---- Eq. 4: range ------------------------------------------------------------------------------
// V = elements per load: a 16-byte pack when planes and pointers allow it, else 1.
template <typename T, int V>
__global__ void __launch_bounds__(kThreads) range_flat_kernel(const T* __restrict__ x, FlatGeom g,
                                                              uint32_t* __restrict__ kmin,
                                                              uint32_t* __restrict__ kmax) {
    __shared__ TileBase s_base;
    WarpRun run{kNoGroup, 0u, 0u};
    for (int64_t tile = blockIdx.x; tile < g.ntiles; tile += gridDim.x) {
        const int64_t e0 = tile * (int64_t)kTile;
        const uint32_t ne = (uint32_t)min((int64_t)kTile, g.E - e0);
        __syncthreads();
        if (threadIdx.x == 0) s_base = tile_base(g, e0);
        __syncthreads();
        const TileBase base = s_base;
        for (uint32_t k0 = 0; k0 < ne; k0 += kThreads * V * kUnroll) {
            uint32_t mn[kUnroll], mx[kUnroll], k[kUnroll];
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                k[j] = k0 + (j * kThreads + threadIdx.x) * V;
                mn[j] = 0;
                mx[j] = 0;
                if (k[j] < ne) {
                    if constexpr (V == 1) {
                        uint32_t e = enc(load_scalar(x + e0 + k[j]));
                        mn[j] = ~e;
                        mx[j] = e;
                    } else {
                        Pack<T> p;
                        p.raw = *reinterpret_cast<const uint4*>(x + e0 + k[j]);
                        float lo = INFINITY, hi = -INFINITY;
                        pack_minmax(p, 0, V, lo, hi);
                        mn[j] = ~enc(lo);
                        mx[j] = enc(hi);
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                bool valid = k[j] < ne;
                uint32_t grp = valid ? group_at(g, base, plane_offset(g, base, k[j])) : kNoGroup;
                run_add(run, valid, grp, mn[j], mx[j], kmin, kmax);
            }
        }
    }
    run_flush(run, kmin, kmax);
}

// ---- Eq. 4: range, vector path -----------------------------------------------------------------
// Planes made of whole 16-byte packs, fewer than 2^31 packs: a warp takes rows of 128 consecutive
// packs (two rows in flight), a row that lies in one plane costs one run update, and the CTA
// combines its warps' keys in shared memory before touching the global keys.
constexpr uint32_t kRangeSmemGroups = 1024;

// ALIGNED: planes are whole packs (div_plane divides pack indices); otherwise a pack may straddle two
// planes (div_plane divides element indices, `inner` >= V elements per plane).
template <typename T, bool ALIGNED>
__global__ void __launch_bounds__(kThreads) range_rows_kernel(const uint4* __restrict__ x, uint32_t n_units,
                                                              uint32_t inner, FastDiv div_plane, FastDiv div_C,
                                                              uint32_t groups, uint32_t* __restrict__ kmin,
                                                              uint32_t* __restrict__ kmax) {
    constexpr int V = Pack<T>::V;
    __shared__ uint32_t s_kmn[kRangeSmemGroups], s_kmx[kRangeSmemGroups];
    const bool combine = groups <= kRangeSmemGroups;       // else: straight to the global keys
    if (combine) {
        for (uint32_t i = threadIdx.x; i < groups; i += kThreads) {
            s_kmn[i] = 0;
            s_kmx[i] = 0;
        }
        __syncthreads();
    }
    uint32_t* dmn = combine ? s_kmn : kmin;
    uint32_t* dmx = combine ? s_kmx : kmax;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t nwarps = gridDim.x * (kThreads / 32), gw = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    const uint32_t nrows = (n_units + 127u) / 128u;
    WarpRun run{kNoGroup, 0u, 0u}, run2{kNoGroup, 0u, 0u};
    auto fetch = [&](uint32_t row, Pack<T> (&p)[4]) {
        if (row >= nrows) return;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t u = row * 128u + j * 32 + lane;
            if (u < n_units) p[j].raw = ld_stream_16(x + u);
        }
    };
    auto reduce = [&](uint32_t row, const Pack<T> (&p)[4]) {
        if (row >= nrows) return;
        const uint32_t r0 = row * 128u;
        bool v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = r0 + j * 32 + lane < n_units;
        if constexpr (ALIGNED) {
            float mn[4], mx[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                mn[j] = INFINITY;
                mx[j] = -INFINITY;
                if (v[j]) pack_minmax(p[j], 0, V, mn[j], mx[j]);
            }
            const uint32_t pl_first = div_plane.div(r0), pl_last = div_plane.div(min(r0 + 128u, n_units) - 1);
            if (pl_first == pl_last) {
                uint32_t q, g;
                div_C.divmod(pl_first, q, g);
                const float m0 = fminf(fminf(mn[0], mn[1]), fminf(mn[2], mn[3]));
                const float m1 = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                run_add(run, v[0], g, ~enc(m0), enc(m1), dmn, dmx);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t q, g;
                    div_C.divmod(div_plane.div(v[j] ? r0 + j * 32 + lane : r0), q, g);
                    run_add(run, v[j], g, ~enc(mn[j]), enc(mx[j]), dmn, dmx);
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint32_t pl, rem, q, g1, g2;
                div_plane.divmod((v[j] ? r0 + j * 32 + lane : r0) * V, pl, rem);
                const int n1 = (int)min((uint32_t)V, inner - rem);          // elements of the first plane
                div_C.divmod(pl, q, g1);
                div_C.divmod(pl + 1, q, g2);
                float mn1 = INFINITY, mx1 = -INFINITY, mn2 = INFINITY, mx2 = -INFINITY;
                if (v[j]) {
                    pack_minmax(p[j], 0, n1, mn1, mx1);
                    pack_minmax(p[j], n1, V, mn2, mx2);
                }
                run_add(run, v[j], g1, ~enc(mn1), enc(mx1), dmn, dmx);
                run_add(run2, v[j] && n1 < V, g2, ~enc(mn2), enc(mx2), dmn, dmx);
            }
        }
    };
    for (uint32_t row = gw; row < nrows; row += 2 * nwarps) {
        Pack<T> pa[4], pb[4];
        fetch(row, pa);
        fetch(row + nwarps, pb);
        reduce(row, pa);
        reduce(row + nwarps, pb);
    }
    run_flush(run, dmn, dmx);
    if constexpr (!ALIGNED) run_flush(run2, dmn, dmx);
    if (combine) {
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < groups; i += kThreads) {
            const uint32_t k1 = s_kmn[i], k2 = s_kmx[i];
            if (k1 | k2) {
                atomicMax(kmin + i, k1);
                atomicMax(kmax + i, k2);
            }
        }
    }
}

__global__ void finalize_range_kernel(const uint32_t* __restrict__ kmin, const uint32_t* __restrict__ kmax,
                                      int64_t G, float* __restrict__ lo, float* __restrict__ hi, int bits,
                                      float* __restrict__ s_opt, float* __restrict__ z_opt) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= G) return;
    float l, h;
    keys_to_range(kmin[i], kmax[i], l, h);
    lo[i] = l;
    hi[i] = h;
    if (bits > 0) {
        QParam p = make_qparam(l, h, (float)((1 << bits) - 1));
        if (s_opt) s_opt[i] = p.s;
        if (z_opt) z_opt[i] = p.z;
    }
}

__global__ void params_kernel(const float* __restrict__ lo, const float* __restrict__ hi, int64_t G, int bits,
                              float* __restrict__ s_opt, float* __restrict__ z_opt) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= G) return;
    QParam p = make_qparam(__fadd_rn(lo[i], 0.0f), __fadd_rn(hi[i], 0.0f), (float)((1 << bits) - 1));
    if (s_opt) s_opt[i] = p.s;
    if (z_opt) z_opt[i] = p.z;
}

// Packing a warp's row of integer codes into a bit string.  Every lane holds `nb` bits (its V codes
// of b bits, nb = V * b <= 64): lane i owns bits [i * nb, (i + 1) * nb) of a row of nb 32-bit words.
// Lane k returns word k of the row in out[0] and word k + 32 in out[1] (0 where the row has no such
// word); all 32 lanes must call.
__device__ __forceinline__ void warp_pack_row(uint64_t mine, uint32_t nb, uint32_t lane, uint32_t first0,
                                              uint32_t first1, uint32_t (&out)[2]) {
    // first0 / first1 = (32 * lane) / nb and (32 * (lane + 32)) / nb: the first lane that reaches into the
    // word(s) this lane assembles (lane constants, worked out once per kernel)
    out[0] = 0;
    out[1] = 0;
    if ((nb & (nb - 1)) == 0 && nb <= 32) {              // 32 / nb lanes make up one word exactly
        const uint32_t lpw = 32 / nb;
        uint32_t w = (uint32_t)mine << (nb * (lane & (lpw - 1)));
        for (uint32_t d = 1; d < lpw; d <<= 1) w |= __shfl_xor_sync(kFullMask, w, d);
        out[0] = __shfl_sync(kFullMask, w, (lane * lpw) & 31);      // word k sits in lanes k * lpw ...
        return;
    }
    const uint32_t nsrc = 32 / nb + 2;                   // lanes whose bits can fall into one word
    if (nb <= 32) {                                      // one word per lane at most, 32-bit shuffles
        const uint32_t lo = (uint32_t)mine;
        uint32_t acc = 0;
        for (uint32_t j = 0; j < nsrc; ++j) {
            const uint32_t src = first0 + j;
            const uint32_t v = __shfl_sync(kFullMask, lo, src & 31);
            const int off = (int)(src * nb) - (int)(32 * lane);     // where src's bits start, relative to the word
            if (src < 32 && off < 32 && lane < nb) acc |= off >= 0 ? (v << off) : (v >> (-off));
        }
        out[0] = acc;
        return;
    }
    for (int h = 0; h < 2; ++h) {
        const uint32_t wk = lane + 32 * h;               // word of the row this lane assembles
        const uint32_t first = h ? first1 : first0;
        uint32_t acc = 0;
        for (uint32_t j = 0; j < nsrc; ++j) {
            const uint32_t src = first + j;
            const uint64_t v = __shfl_sync(kFullMask, mine, src & 31);
            const int off = (int)(src * nb) - (int)(32 * wk);
            if (src < 32 && off < 32 && wk < nb) acc |= (uint32_t)(off >= 0 ? (v << off) : (v >> (-off)));
        }
        out[h] = acc;
    }
}

// ---- Eq. 1, clamp, Eq. 6, STE: elementwise pass with a given per-group range ----------------------
// EXTRAS = 1: the optional codes / mask / packed-mask outputs are compiled in; 2: the packed mask alone.  The packed mask holds
// one bit per element (bit e % 32 of word e / 32): a warp's lanes own consecutive elements or packs
// starting at a multiple of 32 elements, so whole words are assembled with warp shuffles.
// PACKONLY: the packed integer codes are the only output (everything else is compiled out).  With EXTRAS = 3
// (tensors of a multiple of 32 elements) the bit string is written 8 codes = b bytes at a time by every second
// fp32 lane (every bf16 lane) with plain stores: no word assembly across the warp.
// RAGGED: planes are not whole 16-byte packs (7x7 planes), so a pack may straddle two planes and takes the
// parameters of both (planes of at least one pack: never more than two).
template <typename T, int V, int MODE, int EXTRAS, bool PACKONLY = false, bool RAGGED = false>
__global__ void __launch_bounds__(kThreads) quant_flat_kernel(const T* __restrict__ x, const T* __restrict__ gy,
                                                              T* __restrict__ y, T* __restrict__ gx,
                                                              uint8_t* __restrict__ codes,
                                                              uint8_t* __restrict__ mask,
                                                              uint32_t* __restrict__ pmask,
                                                              double* __restrict__ dist,
                                                              uint32_t* __restrict__ pcodes, int code_bits,
                                                              FlatGeom g, float qmax,
                                                              const float* __restrict__ lo,
                                                              const float* __restrict__ hi) {
    __shared__ TileBase s_base;
    __shared__ float s_tab_s[kTableMax], s_tab_z[kTableMax], s_tab_r[kTableMax];
    constexpr bool kFwd = (MODE & MODE_FWD) != 0, kBwd = (MODE & MODE_BWD) != 0;
    DistAcc dacc;
    dacc.reset();
    const uint32_t pk_nb = (uint32_t)(V * (code_bits > 0 ? code_bits : 1));
    const uint32_t pk_first0 = (32 * (threadIdx.x & 31)) / pk_nb, pk_first1 = (32 * ((threadIdx.x & 31) + 32)) / pk_nb;
    for (int64_t tile = blockIdx.x; tile < g.ntiles; tile += gridDim.x) {
        const int64_t e0 = tile * (int64_t)kTile;
        const uint32_t ne = (uint32_t)min((int64_t)kTile, g.E - e0);
        __syncthreads();
        if (threadIdx.x == 0) s_base = tile_base(g, e0);
        __syncthreads();
        const TileBase base = s_base;
        const uint32_t nplanes = plane_offset(g, base, ne - 1) + 1;
        const bool tabled = nplanes <= kTableMax;
        if (tabled) {
            for (uint32_t q = threadIdx.x; q < nplanes; q += kThreads) {
                uint32_t grp = group_at(g, base, q);
                const QParam qp = make_qparam(__fadd_rn(lo[grp], 0.0f), __fadd_rn(hi[grp], 0.0f), qmax);
                s_tab_s[q] = qp.s;
                s_tab_z[q] = qp.z;
                s_tab_r[q] = div_is_safe(qp.s, 0.0f, 0.0f) ? __frcp_rn(qp.s) : 0.0f;
            }
            __syncthreads();
        }
        for (uint32_t k0 = 0; k0 < ne; k0 += kThreads * V * kUnroll) {
            uint32_t k[kUnroll];
            Pack<T> px[kUnroll], pg[kUnroll];
            float sx[kUnroll], sg[kUnroll];
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                k[j] = k0 + (j * kThreads + threadIdx.x) * V;
                if (k[j] < ne) {
                    if constexpr (V == 1) {
                        sx[j] = load_scalar(x + e0 + k[j]);
                        if constexpr (kBwd) sg[j] = load_scalar(gy + e0 + k[j]);
                    } else {
                        px[j].raw = ld_stream_16(x + e0 + k[j]);
                        if constexpr (kBwd) pg[j].raw = ld_stream_16(gy + e0 + k[j]);
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                const bool valid = k[j] < ne;
                uint32_t inside_bits = 0;            // bit i: the clamp was inactive for this thread's element i
                uint64_t code_string = 0;            // this thread's V codes, b bits each, first element lowest
                if (valid) {
                const uint32_t q = plane_offset(g, base, k[j]);
                QParam p;
                float rcp = 0.0f;            // reciprocal of the scale when the short division applies
                if (tabled) {
                    p.s = s_tab_s[q];
                    p.z = s_tab_z[q];
                    rcp = s_tab_r[q];
                } else {
                    uint32_t grp = group_at(g, base, q);
                    p = make_qparam(__fadd_rn(lo[grp], 0.0f), __fadd_rn(hi[grp], 0.0f), qmax);
                }
                const int64_t e = e0 + k[j];
                if constexpr (V == 1) {
                    float yv;
                    bool in;
                    float code = quant_one(sx[j], p, qmax, yv, in);
                    inside_bits = in ? 1u : 0u;
                    code_string = (uint64_t)code;
                    if constexpr (kFwd) {
                        if (dist) dacc.add_one(sx[j], as_stored(yv, y));
                        if (y) store_scalar(y + e, yv);
                        if (codes) codes[e] = (uint8_t)code;
                    }
                    if constexpr (kBwd) {
                        store_scalar(gx + e, in ? sg[j] : 0.0f);
                        if (mask) mask[e] = in ? 1 : 0;
                    }
                } else {
                    Pack<T> py, pgx;
                    uint32_t cb[V / 4 > 0 ? V / 4 : 1], mb[V / 4 > 0 ? V / 4 : 1];
                    // x may lie outside the given range: the short division needs |x| <= 2^60
                    float amax = 0.0f;
#pragma unroll
                    for (int i = 0; i < V; ++i) amax = fmaxf(amax, fabsf(px[j].get(i)));
                    GroupParam gp{p.s, p.z, (amax <= 1152921504606846976.0f) ? rcp : 0.0f};
                    GroupParam gp2 = gp;
                    int n1 = V;
                    if constexpr (RAGGED) {
                        const uint32_t rem = (uint32_t)base.rem + k[j] - q * (uint32_t)g.inner;      // position inside plane q
                        n1 = (int)min((uint32_t)V, (uint32_t)g.inner - rem);
                        if (n1 < V) {                                                           // the rest lies in plane q + 1
                            if (tabled) {
                                gp2.s = s_tab_s[q + 1];
                                gp2.z = s_tab_z[q + 1];
                                gp2.r = (amax <= 1152921504606846976.0f) ? s_tab_r[q + 1] : 0.0f;
                            } else {
                                const uint32_t grp2 = group_at(g, base, q + 1);
                                const QParam p2 = make_qparam(__fadd_rn(lo[grp2], 0.0f), __fadd_rn(hi[grp2], 0.0f), qmax);
                                gp2.s = p2.s;
                                gp2.z = p2.z;
                                gp2.r = 0.0f;
                            }
                        }
                    }
                    quantize_pack<T, kBwd, RAGGED, EXTRAS>(px[j], pg[j], gp, gp2, n1, qmax, py, pgx, cb, mb, EXTRAS == 3 ? code_bits : 8);
                    if constexpr (EXTRAS == 3) {
                        code_string = code_string_of<V>(cb, code_bits);
                    } else if constexpr (EXTRAS != 0) {
                        if constexpr (!PACKONLY) inside_bits = mask_bits_of<V, EXTRAS>(mb);
                        if constexpr (kFwd && EXTRAS == 1) {
                            if constexpr (!PACKONLY) {
                                if (dist) dacc.add(px[j], py);
                            }
                            if (PACKONLY || pcodes) {
#pragma unroll
                                for (int i = 0; i < V; ++i)
                                    code_string |= (uint64_t)((cb[i / 4] >> (8 * (i % 4))) & 0xFFu) << (i * code_bits);
                            }
                        }
                    }
                    if constexpr (kFwd && !PACKONLY) {
                        if (EXTRAS != 1 || y) st_stream_16(y + e, py.raw);
                        if constexpr (EXTRAS == 1) {
                            if (codes) {
#pragma unroll
                                for (int i = 0; i < V / 4; ++i) reinterpret_cast<uint32_t*>(codes + e)[i] = cb[i];
                            }
                        }
                    }
                    if constexpr (kBwd) {
                        st_stream_16(gx + e, pgx.raw);
                        if constexpr (EXTRAS == 1) {
                            if (mask) {
#pragma unroll
                                for (int i = 0; i < V / 4; ++i) reinterpret_cast<uint32_t*>(mask + e)[i] = mb[i];
                            }
                        }
                    }
                }
                }
                if constexpr (EXTRAS != 0 && kFwd) {
                    if (!PACKONLY && pmask) {          // every lane of the warp is here: assemble whole 32-bit words
                        const uint32_t lane = threadIdx.x & 31;
                        const int64_t word = (e0 + k[j]) >> 5;
                        if constexpr (V == 1) {
                            const uint32_t w = __ballot_sync(kFullMask, inside_bits != 0);
                            if (lane == 0 && valid) pmask[word] = w;
                        } else {
                            constexpr uint32_t kLanes = 32 / V;             // lanes that share one word
                            uint32_t w = inside_bits << (V * (lane & (kLanes - 1)));
#pragma unroll
                            for (uint32_t d = 1; d < kLanes; d <<= 1) w |= __shfl_xor_sync(kFullMask, w, d);
                            if ((lane & (kLanes - 1)) == 0 && valid) pmask[word] = w;
                        }
                    }
                    if constexpr (EXTRAS == 3) {
                        // 8 consecutive codes are b whole bytes of the bit string (the tensor is a multiple of 32
                        // elements, so the lanes of a pair are valid or not together, and a lane without a pack has
                        // nothing to say)
                        if constexpr (V > 1) {
                            if (valid) store_code_bytes<V>(pcodes, (size_t)(e0 + k[j]), code_string, code_bits, threadIdx.x & 31);
                        }
                    } else if (EXTRAS == 1 && (PACKONLY || pcodes)) {      // the warp's 32 * V codes are V * b whole words of the bit string
                        const uint32_t lane = threadIdx.x & 31;
                        const uint32_t nb = (uint32_t)(V * code_bits);
                        const int64_t row_e = e0 + k0 + (int64_t)(j * kThreads + (threadIdx.x & ~31u)) * V;
                        const int64_t word0 = (row_e >> 5) * code_bits, nwords = (g.E * code_bits + 31) >> 5;
                        uint32_t out[2];
                        warp_pack_row(code_string, nb, lane, pk_first0, pk_first1, out);
                        if (lane < nb && word0 + lane < nwords) pcodes[word0 + lane] = out[0];
                        if (lane + 32 < nb && word0 + lane + 32 < nwords) pcodes[word0 + lane + 32] = out[1];
                    }
                }
            }
        }
    }
    if constexpr (EXTRAS == 1 && kFwd && !PACKONLY) {
        if (dist) dacc.flush(dist);
    }
}

// ---- the "conventional" per-channel scheme (Section 5.3.2): one group per launch ------------------
template <typename T, bool IS_MAX>
__global__ void __launch_bounds__(kThreads) naive_extreme_kernel(const T* __restrict__ x, Geom g, int64_t c,
                                                                 uint32_t* __restrict__ key) {
    uint32_t acc = 0;
    for (int64_t o = blockIdx.x; o < g.outer; o += gridDim.x) {
        const T* plane = x + (o * g.C + c) * g.inner;
        for (int64_t i = threadIdx.x; i < g.inner; i += kThreads) {
            uint32_t e = enc(load_scalar(plane + i));
            acc = max(acc, IS_MAX ? e : ~e);
        }
    }
    acc = __reduce_max_sync(kFullMask, acc);
    if ((threadIdx.x & 31) == 0) atomicMax(key, acc);
}

template <typename T, int MODE>
__global__ void __launch_bounds__(kThreads) naive_quant_kernel(const T* __restrict__ x, const T* __restrict__ gy,
                                                               T* __restrict__ y, T* __restrict__ gx,
                                                               uint8_t* __restrict__ codes,
                                                               uint8_t* __restrict__ mask, Geom g, int64_t c,
                                                               float qmax, const uint32_t* __restrict__ kmin,
                                                               const uint32_t* __restrict__ kmax,
                                                               float* __restrict__ lo_out,
                                                               float* __restrict__ hi_out) {
    constexpr bool kFwd = (MODE & MODE_FWD) != 0, kBwd = (MODE & MODE_BWD) != 0;
    float lo, hi;
    keys_to_range(kmin[c], kmax[c], lo, hi);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        lo_out[c] = lo;
        hi_out[c] = hi;
    }
    const QParam p = make_qparam(lo, hi, qmax);
    for (int64_t o = blockIdx.x; o < g.outer; o += gridDim.x) {
        const int64_t b = (o * g.C + c) * g.inner;
        for (int64_t i = threadIdx.x; i < g.inner; i += kThreads) {
            float yv;
            bool in;
            float code = quant_one(load_scalar(x + b + i), p, qmax, yv, in);
            if constexpr (kFwd) {
                store_scalar(y + b + i, yv);
                if (codes) codes[b + i] = (uint8_t)code;
            }
            if constexpr (kBwd) {
                store_scalar(gx + b + i, in ? load_scalar(gy + b + i) : 0.0f);
                if (mask) mask[b + i] = in ? 1 : 0;
            }
        }
    }
}

// ---- STE backward from the packed mask alone (Section 2.1): gx = gy where the element's bit is set ----
// V = elements per thread and step: a 16-byte pack when E and the pointers allow it, else 1.
template <typename T, int V>
__global__ void __launch_bounds__(kThreads) bwd_packmask_kernel(const T* __restrict__ gy,
                                                                const uint32_t* __restrict__ pmask,
                                                                T* __restrict__ gx, int64_t E) {
    const int64_t nunits = E / V;
    const int64_t stride = (int64_t)gridDim.x * kThreads * kUnroll;
    for (int64_t u0 = (int64_t)blockIdx.x * kThreads * kUnroll; u0 < nunits; u0 += stride) {
        int64_t e[kUnroll];
        Pack<T> pg[kUnroll];
        float sg[kUnroll];
        uint32_t w[kUnroll];
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) {
            e[j] = (u0 + j * kThreads + threadIdx.x) * V;
            if (e[j] < E) {
                if constexpr (V == 1) sg[j] = load_scalar(gy + e[j]);
                else pg[j].raw = ld_stream_16(gy + e[j]);
                w[j] = __ldg(pmask + (e[j] >> 5));
            }
        }
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) {
            if (e[j] >= E) continue;
            const uint32_t bits = w[j] >> (uint32_t)(e[j] & 31);
            if constexpr (V == 1) {
                store_scalar(gx + e[j], (bits & 1u) ? sg[j] : 0.0f);
            } else {
                Pack<T> out;
                out.select(pg[j], bits);
                st_stream_16(gx + e[j], out.raw);
            }
        }
    }
}

// ---- Table 2's raw material for an existing pair (x, q): four fp64 sums -----------------------------
template <typename T, int V>
__global__ void __launch_bounds__(kThreads) distortion_kernel(const T* __restrict__ x, const T* __restrict__ q,
                                                              int64_t E, double* __restrict__ sums) {
    DistAcc acc;
    acc.reset();
    const int64_t nunits = E / V;
    const int64_t stride = (int64_t)gridDim.x * kThreads * 2;
    for (int64_t u0 = (int64_t)blockIdx.x * kThreads * 2; u0 < nunits; u0 += stride) {
        int64_t e[2];
        Pack<T> px[2], pq[2];
        float sx[2], sq[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            e[j] = (u0 + j * kThreads + threadIdx.x) * V;
            if (e[j] < E) {
                if constexpr (V == 1) {
                    sx[j] = load_scalar(x + e[j]);
                    sq[j] = load_scalar(q + e[j]);
                } else {
                    px[j].raw = ld_stream_16(x + e[j]);
                    pq[j].raw = ld_stream_16(q + e[j]);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            if (e[j] >= E) continue;
            if constexpr (V == 1) acc.add_one(sx[j], sq[j]);
            else acc.add(px[j], pq[j]);
        }
    }
    acc.flush(sums);
}

// ---- Eq. 6 from the packed integer codes: y = s * (code - z) --------------------------------------
// V = elements per thread and step (a 16-byte pack of y when E and the pointer allow it, else 1).
template <typename T, int V>
__global__ void __launch_bounds__(kThreads) dequant_packed_kernel(const uint32_t* __restrict__ pcodes,
                                                                  T* __restrict__ y, int64_t E, int64_t inner,
                                                                  int64_t C, int bits,
                                                                  const float* __restrict__ s,
                                                                  const float* __restrict__ z) {
    const int64_t nunits = E / V;
    const uint32_t field = (1u << bits) - 1u;
    for (int64_t u = (int64_t)blockIdx.x * kThreads + threadIdx.x; u < nunits; u += (int64_t)gridDim.x * kThreads) {
        const int64_t e = u * V;
        int64_t rem, grp;
        if (E < (1ll << 31)) {                       // 32-bit divisions are several times cheaper
            const uint32_t plane = (uint32_t)e / (uint32_t)inner;
            rem = (uint32_t)e - plane * (uint32_t)inner;
            grp = plane % (uint32_t)C;
        } else {
            const int64_t plane = e / inner;
            rem = e - plane * inner;
            grp = plane % C;
        }
        float sg = __ldg(s + grp), zg = __ldg(z + grp);
        Pack<T> out;
        // the thread's V * b <= 64 bits lie in at most three consecutive words
        const int64_t first_bit = e * bits, last_word = (E * bits - 1) >> 5;
        const uint32_t bit0 = (uint32_t)(first_bit & 31);
        const int64_t w0 = first_bit >> 5;
        const uint32_t q0 = __ldg(pcodes + w0);
        const uint32_t q1 = w0 + 1 <= last_word ? __ldg(pcodes + w0 + 1) : 0u;
        const uint32_t q2 = (V * 8 > 32 && w0 + 2 <= last_word) ? __ldg(pcodes + w0 + 2) : 0u;
        const uint64_t lo64 = ((uint64_t)q1 << 32) | q0, hi64 = ((uint64_t)q2 << 32) | q1;
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const uint32_t pos = bit0 + (uint32_t)(i * bits);               // < 96
            const uint32_t v = pos < 32u ? (uint32_t)(lo64 >> pos) : (uint32_t)(hi64 >> (pos - 32u));
            const float yv = __fmul_rn(sg, __fsub_rn((float)(v & field), zg));
            if constexpr (V == 1) store_scalar(y + e, yv);
            else out.set(i, yv);
            if (V > 1 && ++rem == inner) {          // the next element starts the next plane
                rem = 0;
                grp = (grp + 1 == C) ? 0 : grp + 1;
                sg = __ldg(s + grp);
                zg = __ldg(z + grp);
            }
        }
        if constexpr (V > 1) st_stream_16(y + e, out.raw);
    }
}

bool aligned16(const void* p) { return p == nullptr || ((uintptr_t)p & 15) == 0; }

int flat_grid(const FlatGeom& f) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int64_t cap = (int64_t)sms * 8;
    return (int)(f.ntiles < cap ? f.ntiles : cap);
}

int range_rows_ctas() {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms * 4;
}

template <typename T>
cudaError_t range_flat_t(const void* x, const Geom& g, uint32_t* kmin, uint32_t* kmax, cudaStream_t st) {
    FlatGeom f = make_flat(g);
    constexpr int VF = Pack<T>::V;
    bool vec = aligned16(x) && (g.inner % VF == 0);
    int grid = flat_grid(f);
    const bool rows_ok = aligned16(x) && g.E % VF == 0 && g.inner >= VF && g.E < (1ll << 31) &&
                         g.C < (1ll << 30) && g.inner < (1ll << 30);
    if (rows_ok) {
        const uint32_t n_units = (uint32_t)(g.E / VF);
        int64_t rows = ((int64_t)n_units + 127) / 128, ctas = (rows + 2 * (kThreads / 32) - 1) / (2 * (kThreads / 32));
        const int64_t cap = (int64_t)range_rows_ctas();                 // 4 resident CTAs per SM at 64 registers
        int rgrid = (int)(ctas < cap ? ctas : cap);
        if (vec)
            range_rows_kernel<T, true><<<rgrid, kThreads, 0, st>>>((const uint4*)x, n_units, (uint32_t)g.inner,
                                                                   make_fastdiv((uint32_t)(g.inner / VF)),
                                                                   make_fastdiv((uint32_t)g.C), (uint32_t)g.C, kmin, kmax);
        else
            range_rows_kernel<T, false><<<rgrid, kThreads, 0, st>>>((const uint4*)x, n_units, (uint32_t)g.inner,
                                                                    make_fastdiv((uint32_t)g.inner),
                                                                    make_fastdiv((uint32_t)g.C), (uint32_t)g.C, kmin, kmax);
    } else if (vec)
        range_flat_kernel<T, VF><<<grid, kThreads, 0, st>>>((const T*)x, f, kmin, kmax);
    else
        range_flat_kernel<T, 1><<<grid, kThreads, 0, st>>>((const T*)x, f, kmin, kmax);
    return cudaGetLastError();
}

template <typename T, int MODE>
cudaError_t quant_flat_t(const QuantIO& io, const Geom& g, int bits, const float* lo, const float* hi,
                         cudaStream_t st) {
    FlatGeom f = make_flat(g);
    constexpr int VF = Pack<T>::V;
    bool vec = (g.inner % VF == 0) && aligned16(io.x) && aligned16(io.gy) && aligned16(io.y) && aligned16(io.gx) &&
               ((uintptr_t)io.codes % 4 == 0) && ((uintptr_t)io.mask % 4 == 0);
    int grid = flat_grid(f);
    float qmax = (float)((1 << bits) - 1);
    const bool extras = io.codes != nullptr || io.mask != nullptr || io.pmask != nullptr || io.dist != nullptr ||
                        io.pcodes != nullptr;
    // forward with y and the packed mask as the only outputs: a leaner instantiation
    const bool pmask_only = io.pmask != nullptr && io.y != nullptr && io.codes == nullptr && io.mask == nullptr &&
                            io.dist == nullptr && io.pcodes == nullptr;
    const bool pack_only = io.pcodes != nullptr && io.y == nullptr && io.codes == nullptr && io.mask == nullptr &&
                           io.pmask == nullptr && io.dist == nullptr;
    // planes that are not whole packs, everything else in place for 16-byte accesses: the vector kernel with
    // packs that may straddle two planes
    const bool ragged = !vec && g.inner >= VF && g.inner % VF != 0 && g.E % VF == 0 && !f.inner_big && aligned16(io.x) &&
                        aligned16(io.gy) && aligned16(io.y) && aligned16(io.gx) && ((uintptr_t)io.codes % 4 == 0) &&
                        ((uintptr_t)io.mask % 4 == 0);
    if constexpr (MODE == MODE_FWD) {
        if ((vec || ragged) && pack_only && g.E % 32 == 0) {       // whole words of codes: the byte-wise writer
            if (vec)
                quant_flat_kernel<T, VF, MODE, 3, true><<<grid, kThreads, 0, st>>>(
                    (const T*)io.x, (const T*)io.gy, (T*)io.y, (T*)io.gx, io.codes, io.mask, io.pmask, io.dist, io.pcodes,
                    io.code_bits, f, qmax, lo, hi);
            else
                quant_flat_kernel<T, VF, MODE, 3, true, true><<<grid, kThreads, 0, st>>>(
                    (const T*)io.x, (const T*)io.gy, (T*)io.y, (T*)io.gx, io.codes, io.mask, io.pmask, io.dist, io.pcodes,
                    io.code_bits, f, qmax, lo, hi);
            return cudaGetLastError();
        }
        if ((vec || ragged) && pack_only) {
            if (vec)
                quant_flat_kernel<T, VF, MODE, 1, true><<<grid, kThreads, 0, st>>>(
                    (const T*)io.x, (const T*)io.gy, (T*)io.y, (T*)io.gx, io.codes, io.mask, io.pmask, io.dist, io.pcodes,
                    io.code_bits, f, qmax, lo, hi);
            else
                quant_flat_kernel<T, VF, MODE, 1, true, true><<<grid, kThreads, 0, st>>>(
                    (const T*)io.x, (const T*)io.gy, (T*)io.y, (T*)io.gx, io.codes, io.mask, io.pmask, io.dist, io.pcodes,
                    io.code_bits, f, qmax, lo, hi);
            return cudaGetLastError();
        }
        if ((vec || ragged) && pmask_only) {
            if (vec)
                quant_flat_kernel<T, VF, MODE, 2><<<grid, kThreads, 0, st>>>(
                    (const T*)io.x, (const T*)io.gy, (T*)io.y, (T*)io.gx, io.codes, io.mask, io.pmask, io.dist, io.pcodes,
                    io.code_bits, f, qmax, lo, hi);
            else
                quant_flat_kernel<T, VF, MODE, 2, false, true><<<grid, kThreads, 0, st>>>(
                    (const T*)io.x, (const T*)io.gy, (T*)io.y, (T*)io.gx, io.codes, io.mask, io.pmask, io.dist, io.pcodes,
                    io.code_bits, f, qmax, lo, hi);
            return cudaGetLastError();
        }
    }
    if (ragged) {
        if (extras)
            quant_flat_kernel<T, VF, MODE, 1, false, true><<<grid, kThreads, 0, st>>>(
                (const T*)io.x, (const T*)io.gy, (T*)io.y, (T*)io.gx, io.codes, io.mask, io.pmask, io.dist, io.pcodes,
                io.code_bits, f, qmax, lo, hi);
        else
            quant_flat_kernel<T, VF, MODE, 0, false, true><<<grid, kThreads, 0, st>>>(
                (const T*)io.x, (const T*)io.gy, (T*)io.y, (T*)io.gx, io.codes, io.mask, io.pmask, io.dist, io.pcodes,
                io.code_bits, f, qmax, lo, hi);
        return cudaGetLastError();
    }
    if (vec && extras)
        quant_flat_kernel<T, VF, MODE, 1><<<grid, kThreads, 0, st>>>((const T*)io.x, (const T*)io.gy, (T*)io.y,
                                                                        (T*)io.gx, io.codes, io.mask, io.pmask, io.dist, io.pcodes, io.code_bits, f, qmax, lo, hi);
    else if (vec)
        quant_flat_kernel<T, VF, MODE, 0><<<grid, kThreads, 0, st>>>((const T*)io.x, (const T*)io.gy, (T*)io.y,
                                                                         (T*)io.gx, io.codes, io.mask, io.pmask, io.dist, io.pcodes, io.code_bits, f, qmax, lo, hi);
    else
        quant_flat_kernel<T, 1, MODE, 1><<<grid, kThreads, 0, st>>>((const T*)io.x, (const T*)io.gy, (T*)io.y,
                                                                       (T*)io.gx, io.codes, io.mask, io.pmask, io.dist, io.pcodes, io.code_bits, f, qmax, lo, hi);
    return cudaGetLastError();
}

template <typename T, int MODE>
cudaError_t naive_t(const QuantIO& io, const Geom& g, int bits, uint32_t* kmin, uint32_t* kmax, float* lo,
                    float* hi, cudaStream_t st, int* launches) {
    int grid = (int)(g.outer < 1024 ? g.outer : 1024);
    float qmax = (float)((1 << bits) - 1);
    int n = 0;
    for (int64_t c = 0; c < g.C; ++c) {
        naive_extreme_kernel<T, false><<<grid, kThreads, 0, st>>>((const T*)io.x, g, c, kmin + c);
        naive_extreme_kernel<T, true><<<grid, kThreads, 0, st>>>((const T*)io.x, g, c, kmax + c);
        naive_quant_kernel<T, MODE><<<grid, kThreads, 0, st>>>((const T*)io.x, (const T*)io.gy, (T*)io.y,
                                                               (T*)io.gx, io.codes, io.mask, g, c, qmax, kmin,
                                                               kmax, lo, hi);
        n += 3;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (launches) *launches = n;
    return cudaSuccess;
}

}  // namespace

cudaError_t launch_range_flat(const void* x, int dtype, const Geom& g, uint32_t* kmin, uint32_t* kmax,
                              cudaStream_t st) {
    return dtype == 0 ? range_flat_t<float>(x, g, kmin, kmax, st) : range_flat_t<__nv_bfloat16>(x, g, kmin, kmax, st);
}

cudaError_t launch_finalize_range(const uint32_t* kmin, const uint32_t* kmax, int64_t G, float* lo, float* hi,
                                  int bits, float* s_opt, float* z_opt, cudaStream_t st) {
    int grid = (int)((G + 255) / 256);
    finalize_range_kernel<<<grid, 256, 0, st>>>(kmin, kmax, G, lo, hi, bits, s_opt, z_opt);
    return cudaGetLastError();
}

cudaError_t launch_params(const float* lo, const float* hi, int64_t G, int bits, float* s_opt, float* z_opt,
                          cudaStream_t st) {
    int grid = (int)((G + 255) / 256);
    params_kernel<<<grid, 256, 0, st>>>(lo, hi, G, bits, s_opt, z_opt);
    return cudaGetLastError();
}

cudaError_t launch_quant_flat(const QuantIO& io, int mode, int dtype, const Geom& g, int bits, const float* lo,
                              const float* hi, cudaStream_t st) {
    if (dtype == 0) {
        if (mode == MODE_FWD) return quant_flat_t<float, MODE_FWD>(io, g, bits, lo, hi, st);
        if (mode == MODE_BWD) return quant_flat_t<float, MODE_BWD>(io, g, bits, lo, hi, st);
        return quant_flat_t<float, MODE_BOTH>(io, g, bits, lo, hi, st);
    }
    if (mode == MODE_FWD) return quant_flat_t<__nv_bfloat16, MODE_FWD>(io, g, bits, lo, hi, st);
    if (mode == MODE_BWD) return quant_flat_t<__nv_bfloat16, MODE_BWD>(io, g, bits, lo, hi, st);
    return quant_flat_t<__nv_bfloat16, MODE_BOTH>(io, g, bits, lo, hi, st);
}

cudaError_t launch_naive(const QuantIO& io, int mode, int dtype, const Geom& g, int bits, uint32_t* kmin,
                         uint32_t* kmax, float* lo, float* hi, cudaStream_t st, int* launches) {
    if (dtype == 0) {
        if (mode == MODE_FWD) return naive_t<float, MODE_FWD>(io, g, bits, kmin, kmax, lo, hi, st, launches);
        return naive_t<float, MODE_BOTH>(io, g, bits, kmin, kmax, lo, hi, st, launches);
    }
    if (mode == MODE_FWD) return naive_t<__nv_bfloat16, MODE_FWD>(io, g, bits, kmin, kmax, lo, hi, st, launches);
    return naive_t<__nv_bfloat16, MODE_BOTH>(io, g, bits, kmin, kmax, lo, hi, st, launches);
}

cudaError_t launch_bwd_packmask(const void* gy, const uint32_t* pmask, void* gx, int dtype, int64_t E,
                                cudaStream_t st) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int VF = dtype == 0 ? 4 : 8;
    const bool vec = aligned16(gy) && aligned16(gx) && (E % VF == 0);
    const int64_t units = vec ? E / VF : E;
    const int64_t per_cta = (int64_t)kThreads * kUnroll;
    int64_t ctas = (units + per_cta - 1) / per_cta;
    const int64_t cap = (int64_t)sms * 16;
    const int grid = (int)(ctas < 1 ? 1 : (ctas < cap ? ctas : cap));
    if (dtype == 0) {
        if (vec) bwd_packmask_kernel<float, 4><<<grid, kThreads, 0, st>>>((const float*)gy, pmask, (float*)gx, E);
        else bwd_packmask_kernel<float, 1><<<grid, kThreads, 0, st>>>((const float*)gy, pmask, (float*)gx, E);
    } else {
        if (vec)
            bwd_packmask_kernel<__nv_bfloat16, 8><<<grid, kThreads, 0, st>>>((const __nv_bfloat16*)gy, pmask,
                                                                             (__nv_bfloat16*)gx, E);
        else
            bwd_packmask_kernel<__nv_bfloat16, 1><<<grid, kThreads, 0, st>>>((const __nv_bfloat16*)gy, pmask,
                                                                             (__nv_bfloat16*)gx, E);
    }
    return cudaGetLastError();
}

cudaError_t launch_distortion(const void* x, const void* q, int dtype, int64_t E, double* sums, cudaStream_t st) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int VF = dtype == 0 ? 4 : 8;
    const bool vec = aligned16(x) && aligned16(q) && (E % VF == 0);
    const int64_t units = vec ? E / VF : E;
    const int64_t per_cta = (int64_t)kThreads * 2;
    const int64_t ctas = (units + per_cta - 1) / per_cta, cap = (int64_t)sms * 8;
    const int grid = (int)(ctas < 1 ? 1 : (ctas < cap ? ctas : cap));
    if (dtype == 0) {
        if (vec) distortion_kernel<float, 4><<<grid, kThreads, 0, st>>>((const float*)x, (const float*)q, E, sums);
        else distortion_kernel<float, 1><<<grid, kThreads, 0, st>>>((const float*)x, (const float*)q, E, sums);
    } else {
        if (vec)
            distortion_kernel<__nv_bfloat16, 8><<<grid, kThreads, 0, st>>>((const __nv_bfloat16*)x,
                                                                           (const __nv_bfloat16*)q, E, sums);
        else
            distortion_kernel<__nv_bfloat16, 1><<<grid, kThreads, 0, st>>>((const __nv_bfloat16*)x,
                                                                           (const __nv_bfloat16*)q, E, sums);
    }
    return cudaGetLastError();
}

cudaError_t launch_dequant_packed(const uint32_t* pcodes, void* y, int dtype, const Geom& g, int bits,
                                  const float* s, const float* z, cudaStream_t st) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int VF = dtype == 0 ? 4 : 8;
    const bool vec = aligned16(y) && (g.E % VF == 0);
    const int64_t units = vec ? g.E / VF : g.E;
    const int64_t ctas = (units + kThreads - 1) / kThreads, cap = (int64_t)sms * 16;
    const int grid = (int)(ctas < 1 ? 1 : (ctas < cap ? ctas : cap));
    if (dtype == 0) {
        if (vec) dequant_packed_kernel<float, 4><<<grid, kThreads, 0, st>>>(pcodes, (float*)y, g.E, g.inner, g.C, bits, s, z);
        else dequant_packed_kernel<float, 1><<<grid, kThreads, 0, st>>>(pcodes, (float*)y, g.E, g.inner, g.C, bits, s, z);
    } else {
        if (vec)
            dequant_packed_kernel<__nv_bfloat16, 8><<<grid, kThreads, 0, st>>>(pcodes, (__nv_bfloat16*)y, g.E, g.inner,
                                                                               g.C, bits, s, z);
        else
            dequant_packed_kernel<__nv_bfloat16, 1><<<grid, kThreads, 0, st>>>(pcodes, (__nv_bfloat16*)y, g.E, g.inner,
                                                                               g.C, bits, s, z);
    }
    return cudaGetLastError();
}

}  // namespace granq
