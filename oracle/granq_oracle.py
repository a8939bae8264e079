"""ctypes front end of the GranQ CPU oracle (TEST INFRASTRUCTURE).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module; the product path never does.  It compiles ``granq_oracle.c`` with gcc into
``libgranq_oracle.so`` beside the source when the library is missing or older than
its sources, and marshals numpy arrays to the C functions.  No arithmetic of the
method lives here.

fp32 tensors are ``float32`` arrays; bf16 tensors are ``uint16`` arrays holding the
bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = [os.path.join(_HERE, "granq_oracle.c"), os.path.join(_HERE, "granq_oracle.h")]
_LIB = os.path.join(_HERE, "libgranq_oracle.so")

F32, BF16 = 0, 1
GROUP_CHANNEL, GROUP_SAMPLE_CHANNEL, GROUP_TENSOR = 0, 1, 2

CFLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (a second or so); returns the library path."""
    stale = force or not os.path.exists(_LIB) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB) for s in _SRC)
    if stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, _SRC[0], "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        # GRANQ_ORACLE_LIB_OVERRIDE: a deliberately broken build, used by the test that checks that the
        # pins notice planted mistakes
        L = ctypes.CDLL(os.environ.get("GRANQ_ORACLE_LIB_OVERRIDE") or build())
        vp, i64p, fp, u8p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64), ctypes.c_void_p, ctypes.c_void_p
        ci = ctypes.c_int
        L.granq_oracle_num_groups.restype = ctypes.c_int64
        L.granq_oracle_num_groups.argtypes = [i64p, ci, ci]
        L.granq_oracle_range.restype = ci
        L.granq_oracle_range.argtypes = [vp, ci, i64p, ci, ci, fp, fp]
        L.granq_oracle_params.restype = ci
        L.granq_oracle_params.argtypes = [fp, fp, ctypes.c_int64, ci, fp, fp]
        L.granq_oracle_fakequant.restype = ci
        L.granq_oracle_fakequant.argtypes = [vp, vp, ci, i64p, ci, ci, ci, fp, fp, vp, vp, u8p, u8p, fp, fp]
        L.granq_oracle_fused.restype = ci
        L.granq_oracle_fused.argtypes = [vp, vp, ci, i64p, ci, ci, ci, vp, vp, fp, fp, u8p, u8p, fp, fp]
        L.granq_oracle_pack_mask.restype = ci
        L.granq_oracle_pack_mask.argtypes = [u8p, ctypes.c_int64, u8p]
        L.granq_oracle_bwd_packed.restype = ci
        L.granq_oracle_bwd_packed.argtypes = [vp, u8p, ci, ctypes.c_int64, vp]
        L.granq_oracle_distortion_sums.restype = ci
        L.granq_oracle_distortion_sums.argtypes = [vp, vp, ci, ctypes.c_int64, vp]
        L.granq_oracle_distortion.restype = ci
        L.granq_oracle_distortion.argtypes = [vp, vp, vp]
        L.granq_oracle_pack_codes.restype = ci
        L.granq_oracle_pack_codes.argtypes = [u8p, ctypes.c_int64, ci, u8p]
        L.granq_oracle_dequant_packed.restype = ci
        L.granq_oracle_dequant_packed.argtypes = [u8p, ci, i64p, ci, ci, ci, fp, fp, vp]
        _lib = L
    return _lib


def _dims(shape):
    if len(shape) != 4:
        raise ValueError("oracle tensors are 4-d")
    return (ctypes.c_int64 * 4)(*[int(d) for d in shape])


def _dtype_of(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"oracle takes float32 or uint16(bf16 bits), got {a.dtype}")


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"{what} failed with code {rc}")


@dataclass
class FakeQuantResult:
    y: np.ndarray
    gx: Optional[np.ndarray]
    lo: np.ndarray
    hi: np.ndarray
    s: np.ndarray
    z: np.ndarray
    codes: np.ndarray
    mask: np.ndarray


def num_groups(shape, channel_axis: int = 1, group_mode: int = GROUP_CHANNEL) -> int:
    g = lib().granq_oracle_num_groups(_dims(shape), channel_axis, group_mode)
    if g < 0:
        raise ValueError("invalid geometry")
    return int(g)


def range_(x: np.ndarray, channel_axis: int = 1, group_mode: int = GROUP_CHANNEL):
    """Per-group (lo, hi): Eq. 4."""
    x = np.ascontiguousarray(x)
    G = num_groups(x.shape, channel_axis, group_mode)
    lo = np.empty(G, np.float32)
    hi = np.empty(G, np.float32)
    _check(lib().granq_oracle_range(_p(x), _dtype_of(x), _dims(x.shape), channel_axis, group_mode,
                                    _p(lo), _p(hi)), "granq_oracle_range")
    return lo, hi


def params(lo: np.ndarray, hi: np.ndarray, bits: int):
    """Per-group (s, z): Eq. 2 / Eq. 5."""
    lo = np.ascontiguousarray(lo, np.float32)
    hi = np.ascontiguousarray(hi, np.float32)
    s = np.empty_like(lo)
    z = np.empty_like(lo)
    _check(lib().granq_oracle_params(_p(lo), _p(hi), lo.size, bits, _p(s), _p(z)), "granq_oracle_params")
    return s, z


def fakequant(x: np.ndarray, bits: int, lo: np.ndarray, hi: np.ndarray, gy: Optional[np.ndarray] = None,
              channel_axis: int = 1, group_mode: int = GROUP_CHANNEL) -> FakeQuantResult:
    """Quantize -> clamp -> dequantize (+ STE backward when gy is given) with a given range."""
    x = np.ascontiguousarray(x)
    G = num_groups(x.shape, channel_axis, group_mode)
    lo = np.ascontiguousarray(lo, np.float32)
    hi = np.ascontiguousarray(hi, np.float32)
    if lo.size != G or hi.size != G:
        raise ValueError("range vectors must have one entry per group")
    if gy is not None:
        gy = np.ascontiguousarray(gy)
        if gy.shape != x.shape or gy.dtype != x.dtype:
            raise ValueError("gy must match x")
    y = np.empty_like(x)
    gx = None if gy is None else np.empty_like(x)
    codes = np.empty(x.shape, np.uint8)
    mask = np.empty(x.shape, np.uint8)
    s = np.empty(G, np.float32)
    z = np.empty(G, np.float32)
    _check(lib().granq_oracle_fakequant(_p(x), _p(gy), _dtype_of(x), _dims(x.shape), channel_axis, group_mode,
                                        bits, _p(lo), _p(hi), _p(y), _p(gx), _p(codes), _p(mask), _p(s), _p(z)),
           "granq_oracle_fakequant")
    return FakeQuantResult(y, gx, lo, hi, s, z, codes, mask)


def fused(x: np.ndarray, bits: int, gy: Optional[np.ndarray] = None, channel_axis: int = 1,
          group_mode: int = GROUP_CHANNEL, want_codes: bool = True) -> FakeQuantResult:
    """The whole hot path: range from x itself, then fakequant (+ backward when gy is given)."""
    x = np.ascontiguousarray(x)
    G = num_groups(x.shape, channel_axis, group_mode)
    if gy is not None:
        gy = np.ascontiguousarray(gy)
        if gy.shape != x.shape or gy.dtype != x.dtype:
            raise ValueError("gy must match x")
    y = np.empty_like(x)
    gx = None if gy is None else np.empty_like(x)
    codes = np.empty(x.shape, np.uint8) if want_codes else None
    mask = np.empty(x.shape, np.uint8) if want_codes else None
    lo = np.empty(G, np.float32)
    hi = np.empty(G, np.float32)
    s = np.empty(G, np.float32)
    z = np.empty(G, np.float32)
    _check(lib().granq_oracle_fused(_p(x), _p(gy), _dtype_of(x), _dims(x.shape), channel_axis, group_mode, bits,
                                    _p(y), _p(gx), _p(lo), _p(hi), _p(codes), _p(mask), _p(s), _p(z)),
           "granq_oracle_fused")
    return FakeQuantResult(y, gx, lo, hi, s, z, codes, mask)


def pack_mask(mask: np.ndarray) -> np.ndarray:
    """One bit per element, least significant bit first, ceil(E / 8) bytes (Section 2.1: all the
    backward pass needs of the forward pass)."""
    mask = np.ascontiguousarray(mask, np.uint8)
    packed = np.empty((mask.size + 7) // 8, np.uint8)
    _check(lib().granq_oracle_pack_mask(_p(mask), mask.size, _p(packed)), "granq_oracle_pack_mask")
    return packed


def bwd_packed(gy: np.ndarray, packed: np.ndarray) -> np.ndarray:
    """STE backward from the packed mask alone: gx = gy where the bit is set, else +0."""
    gy = np.ascontiguousarray(gy)
    packed = np.ascontiguousarray(packed, np.uint8)
    if packed.size != (gy.size + 7) // 8:
        raise ValueError("packed mask must hold ceil(E / 8) bytes")
    gx = np.empty_like(gy)
    _check(lib().granq_oracle_bwd_packed(_p(gy), _p(packed), _dtype_of(gy), gy.size, _p(gx)),
           "granq_oracle_bwd_packed")
    return gx


def distortion_sums(x: np.ndarray, q: np.ndarray) -> np.ndarray:
    """[sum x^2, sum q^2, sum x*q, sum (x-q)^2] in fp64 (the raw material of Table 2)."""
    x = np.ascontiguousarray(x)
    q = np.ascontiguousarray(q)
    if x.shape != q.shape or x.dtype != q.dtype:
        raise ValueError("q must match x")
    sums = np.empty(4, np.float64)
    _check(lib().granq_oracle_distortion_sums(_p(x), _p(q), _dtype_of(x), x.size, _p(sums)),
           "granq_oracle_distortion_sums")
    return sums


def distortion(sums: np.ndarray):
    """(cosine similarity, relative error) of Table 2 from distortion_sums()."""
    sums = np.ascontiguousarray(sums, np.float64)
    c = ctypes.c_double(0.0)
    r = ctypes.c_double(0.0)
    _check(lib().granq_oracle_distortion(_p(sums), ctypes.byref(c), ctypes.byref(r)), "granq_oracle_distortion")
    return c.value, r.value


def pack_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """b-bit codes as a little-endian bit string: element e in bits [e*b, (e+1)*b); ceil(E*b / 8) bytes."""
    codes = np.ascontiguousarray(codes, np.uint8)
    packed = np.empty((codes.size * bits + 7) // 8, np.uint8)
    _check(lib().granq_oracle_pack_codes(_p(codes), codes.size, bits, _p(packed)), "granq_oracle_pack_codes")
    return packed


def dequant_packed(packed: np.ndarray, shape, bits: int, s: np.ndarray, z: np.ndarray, dtype=np.float32,
                   channel_axis: int = 1, group_mode: int = GROUP_CHANNEL) -> np.ndarray:
    """Eq. 6 from the packed codes: y = s * (code - z); dtype np.float32 or np.uint16 (bf16 bits)."""
    packed = np.ascontiguousarray(packed, np.uint8)
    s = np.ascontiguousarray(s, np.float32)
    z = np.ascontiguousarray(z, np.float32)
    y = np.empty(shape, dtype)
    _check(lib().granq_oracle_dequant_packed(_p(packed), _dtype_of(y), _dims(shape), channel_axis, group_mode, bits,
                                             _p(s), _p(z), _p(y)), "granq_oracle_dequant_packed")
    return y



def accumulate(codes: np.ndarray, s: np.ndarray, z: np.ndarray, w: np.ndarray, channels_last: bool = False,
               inloop: bool = False) -> np.ndarray:
    """Eq. 6 left-hand side / Algorithm 1 output step, pointwise case: y = sum_c w[o, c] * s_c * (code - z_c).
    codes: uint8 [N, C, H, W] (or [N, H, W, C] with channels_last); w: float32 [O, C]; returns float64
    [N, O, H, W] (or [N, H, W, O]).  inloop=True evaluates Eq. 3's order instead (scale inside the loop)."""
    codes = np.ascontiguousarray(codes, np.uint8)
    w = np.ascontiguousarray(w, np.float32)
    s = np.ascontiguousarray(s, np.float32)
    z = np.ascontiguousarray(z, np.float32)
    if codes.ndim != 4 or w.ndim != 2:
        raise ValueError("codes must be 4-d and w 2-d")
    if channels_last:
        n, h, wd, c = codes.shape
    else:
        n, c, h, wd = codes.shape
    o = w.shape[0]
    if w.shape[1] != c or s.size != c or z.size != c:
        raise ValueError("w, s, z must have one entry per channel")
    y = np.empty((n, h, wd, o) if channels_last else (n, o, h, wd), np.float64)
    dims = (ctypes.c_int64 * 3)(n, c, h * wd)
    L = lib()
    fn = L.granq_oracle_accumulate_inloop if inloop else L.granq_oracle_accumulate
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64), ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                   ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
    _check(fn(_p(codes), dims, int(channels_last), _p(s), _p(z), _p(w), o, _p(y)), "granq_oracle_accumulate")
    return y
