"""Thin ctypes binding of libgranq.so (include/granq.h): argument marshalling only.

PyTorch supplies device memory and the CUDA stream; every step of the path runs in the
library's kernels.  There is no fallback: if the shared library is missing, or a tensor is
not a contiguous CUDA tensor, the call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgranq.so")

F32, BF16 = 0, 1
GROUP_CHANNEL, GROUP_SAMPLE_CHANNEL, GROUP_TENSOR = 0, 1, 2
FLAG_FORCE_TWO_PASS, FLAG_FORCE_NAIVE, FLAG_FORCE_STAGED, FLAG_FORCE_L2WAVE, FLAG_FORCE_COLWALK = 1, 2, 4, 8, 16
FLAG_WORKSPACE_ZEROED = 32
FLAG_HOST_ASYNC = 64
FLAG_FORCE_CLUSTER = 128
PLAN_TWO_PASS, PLAN_NAIVE, PLAN_STAGED, PLAN_L2WAVE, PLAN_COLWALK, PLAN_CLUSTER, PLAN_ROWS = 0, 1, 2, 3, 4, 5, 6
(KNOB_STAGED_DEPTH, KNOB_STAGED_MAX_BUF_UNITS, KNOB_STAGED_GRID, KNOB_SPIN_LIMIT, KNOB_TEST_EXTRA_ARRIVALS,
 KNOB_STAGED_CTAS_PER_SM, KNOB_L2_WAVE_KB, KNOB_L2_UPL, KNOB_L2_CTAS_PER_SM, KNOB_L2_LAG,
 KNOB_CLUSTER_TILE_KB, KNOB_CLUSTER_CTAS, KNOB_CLUSTER_THREADS, KNOB_CLUSTER_LOAD, KNOB_CLUSTER_PREFETCH,
 KNOB_CLUSTER_KMUL, KNOB_CLUSTER_EARLY_LAUNCH) = range(17)
N_KNOBS = 17
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)

EXPORTS = [
    "granq_status_string", "granq_num_groups", "granq_workspace_bytes", "granq_range",
    "granq_fakequant_fwd", "granq_fakequant_bwd", "granq_fakequant_fused", "granq_workspace_status",
    "granq_host_arena_bytes", "granq_fakequant_fused_host", "granq_fused_plan", "granq_staged_geometry",
    "granq_tune", "granq_selftest_division", "granq_range_noalloc", "granq_packmask_bytes",
    "granq_fakequant_fwd_packmask", "granq_fakequant_bwd_packmask", "granq_fakequant_fused_fwd_packmask",
    "granq_host_arena_status", "granq_distortion", "granq_fakequant_fused_stats",
    "granq_weights_workspace_bytes", "granq_fakequant_weights", "granq_packed_codes_bytes",
    "granq_quantize_packed", "granq_dequantize_packed", "granq_cluster_geometry", "granq_distortion_stats",
    "granq_accumulate_workspace_bytes", "granq_accumulate_codes", "granq_fakequant_fused_batch",
    "granq_quantize_packed_fused",
]
NOALLOC_MAX_GROUPS = 32768


class GranqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (status {status})")


_lib = None


class WeightDesc(ctypes.Structure):
    """granq_weight_desc of include/granq.h."""
    _fields_ = [("x", ctypes.c_void_p), ("gy_opt", ctypes.c_void_p), ("y", ctypes.c_void_p),
                ("gx_opt", ctypes.c_void_p), ("min_out", ctypes.c_void_p), ("max_out", ctypes.c_void_p),
                ("scale_opt", ctypes.c_void_p), ("zp_opt", ctypes.c_void_p), ("channels", ctypes.c_int64),
                ("group_elems", ctypes.c_int64), ("bits", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class FusedDesc(ctypes.Structure):
    """granq_fused_desc of include/granq.h."""
    _fields_ = [("x", ctypes.c_void_p), ("gy_opt", ctypes.c_void_p), ("y", ctypes.c_void_p),
                ("gx_opt", ctypes.c_void_p), ("min_out", ctypes.c_void_p), ("max_out", ctypes.c_void_p),
                ("scale_opt", ctypes.c_void_p), ("zp_opt", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
                ("workspace_bytes", ctypes.c_size_t), ("dims", ctypes.c_int64 * 4), ("bits", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2503_18339_b200.build` "
                "(needs nvcc); there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64p, ci, u32, sz = (ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64), ctypes.c_int, ctypes.c_uint32,
                                 ctypes.c_size_t)
        L.granq_status_string.restype = ctypes.c_char_p
        L.granq_status_string.argtypes = [ci]
        L.granq_num_groups.restype = ctypes.c_int64
        L.granq_num_groups.argtypes = [i64p, ci, ci]
        L.granq_workspace_bytes.restype = sz
        L.granq_workspace_bytes.argtypes = [ci, i64p, ci, ci]
        L.granq_range.restype = ci
        L.granq_range.argtypes = [vp, ci, i64p, ci, ci, vp, vp, vp, sz, u32, vp]
        L.granq_fakequant_fwd.restype = ci
        L.granq_fakequant_fwd.argtypes = [vp, ci, i64p, ci, ci, ci, vp, vp, vp, vp, vp, vp, u32, vp]
        L.granq_fakequant_bwd.restype = ci
        L.granq_fakequant_bwd.argtypes = [vp, vp, ci, i64p, ci, ci, ci, vp, vp, vp, vp, u32, vp]
        L.granq_fakequant_fused.restype = ci
        L.granq_fakequant_fused.argtypes = [vp, vp, ci, i64p, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz,
                                            u32, vp]
        L.granq_workspace_status.restype = ci
        L.granq_workspace_status.argtypes = [vp, vp]
        L.granq_host_arena_bytes.restype = sz
        L.granq_host_arena_bytes.argtypes = [ci, i64p, ci, ci, ci]
        L.granq_fakequant_fused_host.restype = ci
        L.granq_fakequant_fused_host.argtypes = [vp, vp, ci, i64p, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, sz, u32,
                                                 vp]
        L.granq_fused_plan.restype = ci
        L.granq_fused_plan.argtypes = [ci, i64p, ci, ci, ci, u32, ctypes.POINTER(ci)]
        L.granq_staged_geometry.restype = ci
        L.granq_staged_geometry.argtypes = [ci, i64p, ci, ci, ci, ci, i64p]
        L.granq_distortion_stats.restype = ci
        L.granq_distortion_stats.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
                                             ctypes.POINTER(ctypes.c_double)]
        L.granq_fakequant_fused_batch.restype = ci
        L.granq_fakequant_fused_batch.argtypes = [ctypes.POINTER(FusedDesc), ci, ci, ci, ci, u32, vp,
                                                  ctypes.POINTER(ci)]
        L.granq_accumulate_workspace_bytes.restype = sz
        L.granq_accumulate_workspace_bytes.argtypes = [i64p, ci, ctypes.c_int64]
        L.granq_accumulate_codes.restype = ci
        L.granq_accumulate_codes.argtypes = [vp, i64p, ci, ci, vp, vp, vp, ctypes.c_int64, vp, vp, sz, u32, vp]
        L.granq_cluster_geometry.restype = ci
        L.granq_cluster_geometry.argtypes = [ci, i64p, ci, ci, ci, i64p]
        L.granq_selftest_division.restype = ci
        L.granq_selftest_division.argtypes = [ctypes.c_uint64, ctypes.c_uint64, vp, vp]
        L.granq_range_noalloc.restype = ci
        L.granq_range_noalloc.argtypes = [vp, ci, i64p, ci, ci, vp, vp, vp]
        L.granq_tune.restype = ci
        L.granq_tune.argtypes = [ci, ci]
        L.granq_host_arena_status.restype = ci
        L.granq_host_arena_status.argtypes = [ci, i64p, ci, ci, ci, vp, vp]
        L.granq_distortion.restype = ci
        L.granq_distortion.argtypes = [vp, vp, ci, i64p, vp, u32, vp]
        L.granq_fakequant_fused_stats.restype = ci
        L.granq_fakequant_fused_stats.argtypes = [vp, ci, i64p, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, sz, u32, vp]
        L.granq_weights_workspace_bytes.restype = sz
        L.granq_weights_workspace_bytes.argtypes = [ci]
        L.granq_fakequant_weights.restype = ci
        L.granq_fakequant_weights.argtypes = [ctypes.POINTER(WeightDesc), ci, ci, vp, sz, u32, vp]
        L.granq_packed_codes_bytes.restype = sz
        L.granq_packed_codes_bytes.argtypes = [i64p, ci]
        L.granq_quantize_packed.restype = ci
        L.granq_quantize_packed.argtypes = [vp, ci, i64p, ci, ci, ci, vp, vp, vp, vp, vp, vp, u32, vp]
        L.granq_quantize_packed_fused.restype = ci
        L.granq_quantize_packed_fused.argtypes = [vp, ci, i64p, ci, ci, ci, vp, vp, vp, vp, vp, vp, sz, u32, vp]
        L.granq_dequantize_packed.restype = ci
        L.granq_dequantize_packed.argtypes = [vp, ci, i64p, ci, ci, ci, vp, vp, vp, u32, vp]
        L.granq_packmask_bytes.restype = sz
        L.granq_packmask_bytes.argtypes = [i64p]
        L.granq_fakequant_fwd_packmask.restype = ci
        L.granq_fakequant_fwd_packmask.argtypes = [vp, ci, i64p, ci, ci, ci, vp, vp, vp, vp, vp, vp, u32, vp]
        L.granq_fakequant_bwd_packmask.restype = ci
        L.granq_fakequant_bwd_packmask.argtypes = [vp, vp, ci, i64p, vp, u32, vp]
        L.granq_fakequant_fused_fwd_packmask.restype = ci
        L.granq_fakequant_fused_fwd_packmask.argtypes = [vp, ci, i64p, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, sz,
                                                         u32, vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().granq_status_string(int(status)).decode()


def _check(rc: int, what: str) -> None:
    if rc != OK:
        raise GranqError(rc, what)


def _new(shape, dtype, device) -> torch.Tensor:
    """Every output tensor the binding allocates itself comes from here (tests swap it for an allocator
    that surrounds each tensor with guard bands)."""
    return torch.empty(shape, dtype=dtype, device=device)


def _new_like(t: torch.Tensor) -> torch.Tensor:
    return _new(tuple(t.shape), t.dtype, t.device)


def _dims(shape):
    if len(shape) != 4:
        raise ValueError("granq tensors are 4-d (NCHW)")
    return (ctypes.c_int64 * 4)(*[int(d) for d in shape])


def _dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"granq supports float32 and bfloat16 tensors, got {t.dtype}")


def _dev(t: Optional[torch.Tensor], name: str) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (there is no CPU path)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t.data_ptr()


def _host(t: Optional[torch.Tensor], name: str) -> Optional[int]:
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous host tensor")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def num_groups(shape, channel_axis: int = 1, group: int = GROUP_CHANNEL) -> int:
    g = lib().granq_num_groups(_dims(shape), channel_axis, group)
    if g < 0:
        raise ValueError("invalid geometry")
    return int(g)


def workspace_bytes(dtype: int, shape, channel_axis: int = 1, group: int = GROUP_CHANNEL) -> int:
    return int(lib().granq_workspace_bytes(dtype, _dims(shape), channel_axis, group))


def make_workspace(x: torch.Tensor, channel_axis: int = 1, group: int = GROUP_CHANNEL,
                   zeroed: bool = False) -> torch.Tensor:
    """Scratch for the entry points that take a workspace; `zeroed` clears it, as calls made with
    FLAG_WORKSPACE_ZEROED expect of a workspace they see for the first time."""
    n = workspace_bytes(_dtype(x), x.shape, channel_axis, group)
    return (torch.zeros if zeroed else torch.empty)(n, dtype=torch.uint8, device=x.device)


def tune(knob: int, value: int) -> None:
    _check(lib().granq_tune(knob, value), "granq_tune")


def fused_plan(dtype: int, shape, channel_axis: int = 1, group: int = GROUP_CHANNEL, with_backward: bool = True,
               flags: int = 0):
    """(plan, launches) the fused entry point would take for this geometry on the current device."""
    n = ctypes.c_int(0)
    p = lib().granq_fused_plan(dtype, _dims(shape), channel_axis, group, int(with_backward), flags, ctypes.byref(n))
    if p < 0:
        raise GranqError(-p, "granq_fused_plan")
    return p, n.value


def staged_geometry(dtype: int, shape, channel_axis: int = 1, group: int = GROUP_CHANNEL, sm_count: int = 148,
                    smem_bytes: int = 232448):
    """Host-only: wave / chunk geometry of the staged plan, or None if the geometry does not qualify."""
    out = (ctypes.c_int64 * 8)()
    rc = lib().granq_staged_geometry(dtype, _dims(shape), channel_axis, group, sm_count, smem_bytes, out)
    if rc == ERR_UNSUPPORTED:
        return None
    _check(rc, "granq_staged_geometry")
    keys = ["grid", "threads", "depth", "smem_bytes", "buf_units", "cw", "cu", "nwaves"]
    return dict(zip(keys, [int(v) for v in out]))


def cluster_geometry(dtype: int, shape, channel_axis: int = 1, group: int = GROUP_CHANNEL,
                     with_backward: bool = True):
    """Host-only: the cut of the cluster-local plan, or None if the geometry does not qualify."""
    out = (ctypes.c_int64 * 8)()
    rc = lib().granq_cluster_geometry(dtype, _dims(shape), channel_axis, group, int(with_backward), out)
    if rc == ERR_UNSUPPORTED:
        return None
    _check(rc, "granq_cluster_geometry")
    keys = ["grid", "threads", "cluster", "smem_bytes", "tile_bytes", "channels_per_run", "staging", "prefetch_gy"]
    return dict(zip(keys, [int(v) for v in out]))


@dataclass
class FakeQuantOut:
    y: Optional[torch.Tensor] = None
    gx: Optional[torch.Tensor] = None
    lo: Optional[torch.Tensor] = None
    hi: Optional[torch.Tensor] = None
    s: Optional[torch.Tensor] = None
    z: Optional[torch.Tensor] = None
    codes: Optional[torch.Tensor] = None
    mask: Optional[torch.Tensor] = None
    workspace: Optional[torch.Tensor] = None
    packed_mask: Optional[torch.Tensor] = None      # int32 words, one bit per element
    sums: Optional[torch.Tensor] = None             # 4 doubles: sum x^2, sum q^2, sum x*q, sum (x-q)^2
    packed_codes: Optional[torch.Tensor] = None     # int32 words: the codes as a bit string, b bits each


def granq_range(x: torch.Tensor, channel_axis: int = 1, group: int = GROUP_CHANNEL, lo: torch.Tensor = None,
                hi: torch.Tensor = None, workspace: torch.Tensor = None, flags: int = 0, stream=None):
    """Per-group (lo, hi) of x: Eq. 4."""
    G = num_groups(x.shape, channel_axis, group)
    lo = _new(G, torch.float32, x.device) if lo is None else lo
    hi = _new(G, torch.float32, x.device) if hi is None else hi
    ws = make_workspace(x, channel_axis, group) if workspace is None else workspace
    _check(lib().granq_range(_dev(x, "x"), _dtype(x), _dims(x.shape), channel_axis, group, _dev(lo, "lo"),
                             _dev(hi, "hi"), _dev(ws, "workspace"), ws.numel(), flags, _stream(stream)),
           "granq_range")
    return lo, hi


def granq_range_noalloc(x: torch.Tensor, lo: torch.Tensor, hi: torch.Tensor, channel_axis: int = 1,
                        group: int = GROUP_CHANNEL, stream=None) -> None:
    """Per-group (lo, hi) of x into caller-provided tensors, using the library's built-in scratch:
    for callers that cannot allocate device memory at this point (nothing is allocated here either)."""
    _check(lib().granq_range_noalloc(_dev(x, "x"), _dtype(x), _dims(x.shape), channel_axis, group, _dev(lo, "lo"),
                                     _dev(hi, "hi"), _stream(stream)), "granq_range_noalloc")


def granq_fakequant_fwd(x: torch.Tensor, bits: int, lo: torch.Tensor, hi: torch.Tensor, channel_axis: int = 1,
                        group: int = GROUP_CHANNEL, y: torch.Tensor = None, want_codes: bool = False,
                        want_params: bool = False, flags: int = 0, stream=None) -> FakeQuantOut:
    """Quantize -> clamp -> dequantize with a given per-group range: Eq. 1, 2, 6."""
    G = num_groups(x.shape, channel_axis, group)
    o = FakeQuantOut(lo=lo, hi=hi)
    o.y = _new_like(x) if y is None else y
    if want_codes:
        o.codes = _new(x.shape, torch.uint8, x.device)
    if want_params:
        o.s = _new(G, torch.float32, x.device)
        o.z = _new(G, torch.float32, x.device)
    _check(lib().granq_fakequant_fwd(_dev(x, "x"), _dtype(x), _dims(x.shape), channel_axis, group, bits,
                                     _dev(lo, "lo"), _dev(hi, "hi"), _dev(o.y, "y"), _dev(o.codes, "codes"),
                                     _dev(o.s, "s"), _dev(o.z, "z"), flags, _stream(stream)),
           "granq_fakequant_fwd")
    return o


def granq_fakequant_bwd(gy: torch.Tensor, x: torch.Tensor, bits: int, lo: torch.Tensor, hi: torch.Tensor,
                        channel_axis: int = 1, group: int = GROUP_CHANNEL, gx: torch.Tensor = None,
                        want_mask: bool = False, flags: int = 0, stream=None) -> FakeQuantOut:
    """Straight-through-estimator backward with a given per-group range."""
    if gy.shape != x.shape or gy.dtype != x.dtype:
        raise ValueError("gy must match x")
    o = FakeQuantOut(lo=lo, hi=hi)
    o.gx = _new_like(x) if gx is None else gx
    if want_mask:
        o.mask = _new(x.shape, torch.uint8, x.device)
    _check(lib().granq_fakequant_bwd(_dev(gy, "gy"), _dev(x, "x"), _dtype(x), _dims(x.shape), channel_axis, group,
                                     bits, _dev(lo, "lo"), _dev(hi, "hi"), _dev(o.gx, "gx"), _dev(o.mask, "mask"),
                                     flags, _stream(stream)),
           "granq_fakequant_bwd")
    return o


def granq_fakequant_fused(x: torch.Tensor, bits: int, gy: torch.Tensor = None, channel_axis: int = 1,
                          group: int = GROUP_CHANNEL, out: FakeQuantOut = None, want_codes: bool = False,
                          want_mask: bool = False, want_params: bool = False, flags: int = 0,
                          stream=None) -> FakeQuantOut:
    """Range of x itself -> scale / zero-point -> y (and gx when gy is given), in one call.

    `out` may carry preallocated tensors (y, gx, lo, hi, s, z, codes, mask, workspace);
    whatever is missing is allocated here.
    """
    if gy is not None and (gy.shape != x.shape or gy.dtype != x.dtype):
        raise ValueError("gy must match x")
    G = num_groups(x.shape, channel_axis, group)
    o = out if out is not None else FakeQuantOut()
    dev = x.device
    if o.y is None:
        o.y = _new_like(x)
    if gy is not None and o.gx is None:
        o.gx = _new_like(x)
    if o.lo is None:
        o.lo = _new(G, torch.float32, dev)
    if o.hi is None:
        o.hi = _new(G, torch.float32, dev)
    if want_params and o.s is None:
        o.s = _new(G, torch.float32, dev)
        o.z = _new(G, torch.float32, dev)
    if want_codes and o.codes is None:
        o.codes = _new(x.shape, torch.uint8, dev)
    if want_mask and gy is not None and o.mask is None:
        o.mask = _new(x.shape, torch.uint8, dev)
    if o.workspace is None:
        o.workspace = make_workspace(x, channel_axis, group)
    _check(lib().granq_fakequant_fused(
        _dev(x, "x"), _dev(gy, "gy"), _dtype(x), _dims(x.shape), channel_axis, group, bits,
        _dev(o.y, "y"), _dev(o.gx if gy is not None else None, "gx"), _dev(o.lo, "lo"), _dev(o.hi, "hi"),
        _dev(o.codes, "codes"), _dev(o.mask if gy is not None else None, "mask"), _dev(o.s, "s"), _dev(o.z, "z"),
        _dev(o.workspace, "workspace"), o.workspace.numel(), flags, _stream(stream)), "granq_fakequant_fused")
    return o


def packmask_bytes(shape) -> int:
    return int(lib().granq_packmask_bytes(_dims(shape)))


def make_packed_mask(x: torch.Tensor) -> torch.Tensor:
    """Buffer for the STE mask of x at one bit per element (int32 words)."""
    return _new(packmask_bytes(x.shape) // 4, torch.int32, x.device)


def granq_fakequant_fwd_packmask(x: torch.Tensor, bits: int, lo: torch.Tensor, hi: torch.Tensor,
                                 channel_axis: int = 1, group: int = GROUP_CHANNEL, y: torch.Tensor = None,
                                 packed_mask: torch.Tensor = None, want_params: bool = False, flags: int = 0,
                                 stream=None) -> FakeQuantOut:
    """Forward with a given range that also stores the STE mask at one bit per element (Section 2.1)."""
    G = num_groups(x.shape, channel_axis, group)
    o = FakeQuantOut(lo=lo, hi=hi)
    o.y = _new_like(x) if y is None else y
    o.packed_mask = make_packed_mask(x) if packed_mask is None else packed_mask
    if want_params:
        o.s = _new(G, torch.float32, x.device)
        o.z = _new(G, torch.float32, x.device)
    _check(lib().granq_fakequant_fwd_packmask(_dev(x, "x"), _dtype(x), _dims(x.shape), channel_axis, group, bits,
                                              _dev(lo, "lo"), _dev(hi, "hi"), _dev(o.y, "y"),
                                              _dev(o.packed_mask, "packed_mask"), _dev(o.s, "s"), _dev(o.z, "z"),
                                              flags, _stream(stream)), "granq_fakequant_fwd_packmask")
    return o


def granq_fakequant_bwd_packmask(gy: torch.Tensor, packed_mask: torch.Tensor, gx: torch.Tensor = None,
                                 flags: int = 0, stream=None) -> torch.Tensor:
    """STE backward from the packed mask alone: gx = gy where the bit is set, else 0."""
    if packed_mask.numel() * packed_mask.element_size() < packmask_bytes(gy.shape):
        raise ValueError("packed mask too small for gy")
    gx = _new_like(gy) if gx is None else gx
    _check(lib().granq_fakequant_bwd_packmask(_dev(gy, "gy"), _dev(packed_mask, "packed_mask"), _dtype(gy),
                                              _dims(gy.shape), _dev(gx, "gx"), flags, _stream(stream)),
           "granq_fakequant_bwd_packmask")
    return gx


class FusedBatch:
    """A list of tensors for granq_fakequant_fused_batch(): descriptors are marshalled once, run() is one C call.
    items: (x, bits, gy or None) triples of one dtype; outputs are allocated here (or taken from `outs`)."""

    def __init__(self, items, channel_axis: int = 1, group: int = GROUP_CHANNEL, outs=None, want_params: bool = False,
                 zeroed: bool = False):
        if not items:
            raise ValueError("no tensors")
        self.channel_axis, self.group = channel_axis, group
        self.dtype = _dtype(items[0][0])
        self.items = list(items)
        self.outs = []
        self.flags = FLAG_WORKSPACE_ZEROED if zeroed else 0
        self._descs = (FusedDesc * len(self.items))()
        for i, (x, bits, gy) in enumerate(self.items):
            if _dtype(x) != self.dtype:
                raise ValueError("all tensors of a batch have one dtype")
            o = outs[i] if outs is not None else FakeQuantOut()
            G = num_groups(x.shape, channel_axis, group)
            if o.y is None:
                o.y = _new_like(x)
            if gy is not None and o.gx is None:
                o.gx = _new_like(x)
            if o.lo is None:
                o.lo = _new(G, torch.float32, x.device)
            if o.hi is None:
                o.hi = _new(G, torch.float32, x.device)
            if want_params and o.s is None:
                o.s = _new(G, torch.float32, x.device)
                o.z = _new(G, torch.float32, x.device)
            if o.workspace is None:
                o.workspace = make_workspace(x, channel_axis, group, zeroed=zeroed)
            d = self._descs[i]
            d.x, d.gy_opt, d.y, d.gx_opt = _dev(x, "x"), _dev(gy, "gy"), _dev(o.y, "y"), _dev(o.gx, "gx")
            d.min_out, d.max_out, d.scale_opt, d.zp_opt = _dev(o.lo, "lo"), _dev(o.hi, "hi"), _dev(o.s, "s"), _dev(o.z, "z")
            d.workspace, d.workspace_bytes = _dev(o.workspace, "workspace"), o.workspace.numel()
            for k in range(4):
                d.dims[k] = int(x.shape[k])
            d.bits = int(bits)
            self.outs.append(o)

    def run(self, stream=None, flags: int = 0):
        failed = ctypes.c_int(-1)
        rc = lib().granq_fakequant_fused_batch(self._descs, len(self.items), self.dtype, self.channel_axis, self.group,
                                               self.flags | flags, _stream(stream), ctypes.byref(failed))
        if rc != OK:
            raise GranqError(rc, f"granq_fakequant_fused_batch (tensor {failed.value})")
        return self.outs


def granq_fakequant_fused_fwd_packmask(x: torch.Tensor, bits: int, channel_axis: int = 1,
                                       group: int = GROUP_CHANNEL, out: FakeQuantOut = None,
                                       want_params: bool = False, flags: int = 0, stream=None) -> FakeQuantOut:
    """Range of x itself -> scale / zero-point -> y and the packed STE mask, in one call."""
    G = num_groups(x.shape, channel_axis, group)
    o = out if out is not None else FakeQuantOut()
    dev = x.device
    if o.y is None:
        o.y = _new_like(x)
    if o.packed_mask is None:
        o.packed_mask = make_packed_mask(x)
    if o.lo is None:
        o.lo = _new(G, torch.float32, dev)
    if o.hi is None:
        o.hi = _new(G, torch.float32, dev)
    if want_params and o.s is None:
        o.s = _new(G, torch.float32, dev)
        o.z = _new(G, torch.float32, dev)
    if o.workspace is None:
        o.workspace = make_workspace(x, channel_axis, group)
    _check(lib().granq_fakequant_fused_fwd_packmask(
        _dev(x, "x"), _dtype(x), _dims(x.shape), channel_axis, group, bits, _dev(o.y, "y"),
        _dev(o.packed_mask, "packed_mask"), _dev(o.lo, "lo"), _dev(o.hi, "hi"), _dev(o.s, "s"), _dev(o.z, "z"),
        _dev(o.workspace, "workspace"), o.workspace.numel(), flags, _stream(stream)),
        "granq_fakequant_fused_fwd_packmask")
    return o


def granq_distortion(x: torch.Tensor, q: torch.Tensor, sums: torch.Tensor = None, stream=None) -> torch.Tensor:
    """[sum x^2, sum q^2, sum x*q, sum (x-q)^2] as 4 doubles on the device (Table 2's raw material)."""
    if q.shape != x.shape or q.dtype != x.dtype:
        raise ValueError("q must match x")
    sums = _new(4, torch.float64, x.device) if sums is None else sums
    _check(lib().granq_distortion(_dev(x, "x"), _dev(q, "q"), _dtype(x), _dims(x.shape), _dev(sums, "sums"), 0,
                                  _stream(stream)), "granq_distortion")
    return sums


def distortion_from_sums(sums):
    """(cosine similarity, relative error) of Table 2 from the four sums (granq_distortion_stats)."""
    arr = (ctypes.c_double * 4)(*[float(v) for v in sums])
    cos, rel = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(lib().granq_distortion_stats(arr, ctypes.byref(cos), ctypes.byref(rel)), "granq_distortion_stats")
    return cos.value, rel.value


def granq_fakequant_fused_stats(x: torch.Tensor, bits: int, channel_axis: int = 1, group: int = GROUP_CHANNEL,
                                out: FakeQuantOut = None, want_params: bool = False, flags: int = 0,
                                stream=None) -> FakeQuantOut:
    """Range of x itself -> scale / zero-point -> y, gathering Table 2's sums in the same pass."""
    G = num_groups(x.shape, channel_axis, group)
    o = out if out is not None else FakeQuantOut()
    dev = x.device
    if o.y is None:
        o.y = _new_like(x)
    if o.sums is None:
        o.sums = _new(4, torch.float64, dev)
    if o.lo is None:
        o.lo = _new(G, torch.float32, dev)
    if o.hi is None:
        o.hi = _new(G, torch.float32, dev)
    if want_params and o.s is None:
        o.s = _new(G, torch.float32, dev)
        o.z = _new(G, torch.float32, dev)
    if o.workspace is None:
        o.workspace = make_workspace(x, channel_axis, group)
    _check(lib().granq_fakequant_fused_stats(
        _dev(x, "x"), _dtype(x), _dims(x.shape), channel_axis, group, bits, _dev(o.y, "y"), _dev(o.lo, "lo"),
        _dev(o.hi, "hi"), _dev(o.s, "s"), _dev(o.z, "z"), _dev(o.sums, "sums"), _dev(o.workspace, "workspace"),
        o.workspace.numel(), flags, _stream(stream)), "granq_fakequant_fused_stats")
    return o


class WeightBatch:
    """All weight tensors of a model prepared for channel-wise (leading axis) fake-quantization in one
    launch: descriptors and outputs are built once, `run()` is a single library call.

    `weights`: contiguous CUDA tensors of one dtype, any rank >= 1 (axis 0 = output channels);
    `bits`: one int or one per tensor; `grads`: upstream gradients (all or none)."""

    def __init__(self, weights, bits, grads=None, want_params: bool = False):
        n = len(weights)
        self.n = n
        self.dtype = _dtype(weights[0])
        bits = [bits] * n if isinstance(bits, int) else list(bits)
        self.descs = (WeightDesc * n)()
        self.outs = []
        self._keep = (list(weights), None if grads is None else list(grads))
        for i, w in enumerate(weights):
            if w.dtype != weights[0].dtype:
                raise ValueError("all tensors of a batch must have one dtype")
            c = w.shape[0]
            o = FakeQuantOut(y=_new_like(w), lo=_new(c, torch.float32, w.device),
                             hi=_new(c, torch.float32, w.device))
            g = None if grads is None else grads[i]
            if g is not None:
                if g.shape != w.shape or g.dtype != w.dtype:
                    raise ValueError("gradient must match its weight")
                o.gx = _new_like(w)
            if want_params:
                o.s = _new(c, torch.float32, w.device)
                o.z = _new(c, torch.float32, w.device)
            self.descs[i] = WeightDesc(_dev(w, "w"), _dev(g, "g"), _dev(o.y, "y"), _dev(o.gx, "gx"),
                                       _dev(o.lo, "lo"), _dev(o.hi, "hi"), _dev(o.s, "s"), _dev(o.z, "z"), c,
                                       w.numel() // max(c, 1), bits[i], 0)
            self.outs.append(o)
        self.workspace = torch.empty(int(lib().granq_weights_workspace_bytes(n)), dtype=torch.uint8,
                                     device=weights[0].device)

    def run(self, workspace: torch.Tensor = None, stream=None):
        ws = self.workspace if workspace is None else workspace
        _check(lib().granq_fakequant_weights(self.descs, self.n, self.dtype, _dev(ws, "workspace"), ws.numel(), 0,
                                             _stream(stream)), "granq_fakequant_weights")
        return self.outs


def granq_fakequant_weights(weights, bits, grads=None, want_params: bool = False, workspace: torch.Tensor = None,
                            stream=None):
    """One-shot form of WeightBatch: returns a list of FakeQuantOut (y, gx, lo, hi, and s / z with want_params)."""
    return WeightBatch(weights, bits, grads, want_params).run(workspace, stream)


def packed_codes_bytes(shape, bits: int) -> int:
    return int(lib().granq_packed_codes_bytes(_dims(shape), bits))


def granq_quantize_packed(x: torch.Tensor, bits: int, lo: torch.Tensor, hi: torch.Tensor, channel_axis: int = 1,
                          group: int = GROUP_CHANNEL, want_y: bool = False, packed_codes: torch.Tensor = None,
                          stream=None) -> FakeQuantOut:
    """Eq. 1 + clamp with a given range -> integer codes as a bit string (b bits each), scale, zero-point."""
    G = num_groups(x.shape, channel_axis, group)
    o = FakeQuantOut(lo=lo, hi=hi)
    o.packed_codes = (_new(packed_codes_bytes(x.shape, bits) // 4, torch.int32, x.device)
                      if packed_codes is None else packed_codes)
    o.s = _new(G, torch.float32, x.device)
    o.z = _new(G, torch.float32, x.device)
    if want_y:
        o.y = _new_like(x)
    _check(lib().granq_quantize_packed(_dev(x, "x"), _dtype(x), _dims(x.shape), channel_axis, group, bits,
                                       _dev(lo, "lo"), _dev(hi, "hi"), _dev(o.packed_codes, "packed_codes"),
                                       _dev(o.y, "y"), _dev(o.s, "s"), _dev(o.z, "z"), 0, _stream(stream)),
           "granq_quantize_packed")
    return o


def granq_dequantize_packed(packed_codes: torch.Tensor, shape, dtype: torch.dtype, bits: int, s: torch.Tensor,
                            z: torch.Tensor, channel_axis: int = 1, group: int = GROUP_CHANNEL,
                            y: torch.Tensor = None, stream=None) -> torch.Tensor:
    """Eq. 6 from the packed codes: y = s * (code - z)."""
    y = _new(tuple(shape), dtype, packed_codes.device) if y is None else y
    _check(lib().granq_dequantize_packed(_dev(packed_codes, "packed_codes"), _dtype(y), _dims(shape), channel_axis,
                                         group, bits, _dev(s, "s"), _dev(z, "z"), _dev(y, "y"), 0, _stream(stream)),
           "granq_dequantize_packed")
    return y


def accumulate_workspace_bytes(shape, channel_axis: int, out_channels: int) -> int:
    return int(lib().granq_accumulate_workspace_bytes(_dims(shape), channel_axis, out_channels))


def granq_quantize_packed_fused(x: torch.Tensor, bits: int, channel_axis: int = 1, group: int = GROUP_CHANNEL,
                                packed_codes: torch.Tensor = None, out: FakeQuantOut = None, flags: int = 0,
                                stream=None) -> FakeQuantOut:
    """Range of x itself -> scale / zero-point -> integer codes as a bit string, in one call (lo, hi, s, z and
    packed_codes of the returned record are filled)."""
    G = num_groups(x.shape, channel_axis, group)
    o = out if out is not None else FakeQuantOut()
    dev = x.device
    for name in ("lo", "hi", "s", "z"):
        if getattr(o, name) is None:
            setattr(o, name, _new(G, torch.float32, dev))
    if packed_codes is not None:
        o.packed_codes = packed_codes
    if o.packed_codes is None:
        o.packed_codes = _new(packed_codes_bytes(x.shape, bits) // 4, torch.int32, dev)
    if o.workspace is None:
        o.workspace = make_workspace(x, channel_axis, group)
    _check(lib().granq_quantize_packed_fused(
        _dev(x, "x"), _dtype(x), _dims(x.shape), channel_axis, group, bits, _dev(o.packed_codes, "packed_codes"),
        _dev(o.lo, "lo"), _dev(o.hi, "hi"), _dev(o.s, "s"), _dev(o.z, "z"), _dev(o.workspace, "workspace"),
        o.workspace.numel(), flags, _stream(stream)), "granq_quantize_packed_fused")
    return o


def granq_accumulate_codes(packed_codes: torch.Tensor, shape, bits: int, s: torch.Tensor, z: torch.Tensor,
                           weights: torch.Tensor, channel_axis: int = 1, y: torch.Tensor = None,
                           workspace: torch.Tensor = None, flags: int = 0, stream=None):
    """Eq. 6 left-hand side / Algorithm 1 output step, pointwise case, from the packed integer codes of a
    tensor of `shape` (NCHW for channel_axis 1, N H W C for 3): y = sum_c w[o, c] * s_c * (code - z_c), fp32.
    Returns (y, workspace); the workspace's status word tells whether a bounded wait ran out.
    flags: FLAG_FORCE_TWO_PASS takes the kernel with one tile per CTA instead of the persistent one."""
    shape = tuple(int(d) for d in shape)
    if weights.dtype != torch.float32 or weights.dim() != 2 or weights.shape[1] != shape[channel_axis]:
        raise ValueError("weights must be float32 [out_channels, C]")
    o = int(weights.shape[0])
    if y is None:
        out_shape = (shape[0], o, shape[2], shape[3]) if channel_axis == 1 else (shape[0], shape[1], shape[2], o)
        y = _new(out_shape, torch.float32, packed_codes.device)
    if workspace is None:
        workspace = torch.empty(accumulate_workspace_bytes(shape, channel_axis, o), dtype=torch.uint8,
                                device=packed_codes.device)
    _check(lib().granq_accumulate_codes(_dev(packed_codes, "packed_codes"), _dims(shape), channel_axis, bits,
                                        _dev(s, "s"), _dev(z, "z"), _dev(weights, "weights"), o, _dev(y, "y"),
                                        _dev(workspace, "workspace"), workspace.numel(), flags, _stream(stream)),
           "granq_accumulate_codes")
    return y, workspace


def selftest_division(pairs: int, seed: int = 0, stream=None) -> int:
    """Pairs (out of `pairs` generated ones) on which the kernel's division differs from IEEE division."""
    counter = torch.zeros(1, dtype=torch.int64, device="cuda")
    _check(lib().granq_selftest_division(pairs, seed, _dev(counter, "counter"), _stream(stream)),
           "granq_selftest_division")
    return int(counter.item())


def workspace_status(workspace: torch.Tensor, stream=None) -> int:
    """Synchronises the stream and returns the device status word of the last staged call."""
    return int(lib().granq_workspace_status(_dev(workspace, "workspace"), _stream(stream)))


def host_arena_bytes(dtype: int, shape, channel_axis: int = 1, group: int = GROUP_CHANNEL,
                     with_backward: bool = True) -> int:
    return int(lib().granq_host_arena_bytes(dtype, _dims(shape), channel_axis, group, int(with_backward)))


def granq_fakequant_fused_host(x: torch.Tensor, bits: int, gy: torch.Tensor, y: torch.Tensor, gx: torch.Tensor,
                               lo: torch.Tensor, hi: torch.Tensor, arena: torch.Tensor, channel_axis: int = 1,
                               group: int = GROUP_CHANNEL, s: torch.Tensor = None, z: torch.Tensor = None,
                               flags: int = 0, stream=None) -> None:
    """Fused path on HOST tensors (pinned memory recommended); `arena` is device scratch of
    host_arena_bytes() bytes.  Returns when the host outputs are valid, or right after enqueuing
    with FLAG_HOST_ASYNC (then host_arena_status() waits and reports)."""
    _check(lib().granq_fakequant_fused_host(
        _host(x, "x"), _host(gy, "gy"), _dtype(x), _dims(x.shape), channel_axis, group, bits,
        _host(y, "y"), _host(gx, "gx"), _host(lo, "lo"), _host(hi, "hi"), _host(s, "s"), _host(z, "z"),
        _dev(arena, "arena"), arena.numel(), flags, _stream(stream)), "granq_fakequant_fused_host")


def host_arena_status(dtype: int, shape, arena: torch.Tensor, channel_axis: int = 1, group: int = GROUP_CHANNEL,
                      with_backward: bool = True, stream=None) -> int:
    """Waits for `stream`, then the status of the last FLAG_HOST_ASYNC call that used `arena`."""
    return lib().granq_host_arena_status(dtype, _dims(shape), channel_axis, group, int(with_backward),
                                         _dev(arena, "arena"), _stream(stream))

