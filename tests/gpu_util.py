"""Helpers shared by the GPU parity tests: marshalling, bit comparison, the parity assertion and
output buffers with guard bands (every output lives inside a larger poisoned allocation whose
margins must come back untouched: a store past either end of an output fails the test even
when it lands in memory nobody compares)."""
import numpy as np
import torch

from oracle import granq_oracle as orc
from paper_2503_18339_b200 import workloads as wl

GUARD_BYTES = 4096
POISON = 0xA5


def to_dev(a: np.ndarray) -> torch.Tensor:
    """float32 array -> cuda float32; uint16 (bf16 bits) -> cuda bfloat16."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def to_np(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def widen(a: np.ndarray) -> np.ndarray:
    return wl.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a


def same_bits(a: np.ndarray, c: np.ndarray) -> bool:
    v = {1: np.uint8, 2: np.uint16, 4: np.uint32, 8: np.uint64}[a.dtype.itemsize]
    return np.array_equal(np.ascontiguousarray(a).view(v), np.ascontiguousarray(c).view(v))


def group_index(shape, axis, mode):
    """per-element group id, shaped like the tensor"""
    outer = int(np.prod(shape[:axis], dtype=np.int64))
    C = shape[axis]
    inner = int(np.prod(shape[axis + 1:], dtype=np.int64))
    o = np.arange(outer).reshape(outer, 1, 1)
    c = np.arange(C).reshape(1, C, 1)
    if mode == orc.GROUP_CHANNEL:
        g = np.broadcast_to(c, (outer, C, 1))
    elif mode == orc.GROUP_SAMPLE_CHANNEL:
        g = o * C + c
    else:
        g = np.zeros((outer, C, 1), np.int64)
    return np.broadcast_to(g, (outer, C, inner)).reshape(shape)


def assert_parity(got, ref, shape, axis, mode, backward, exact=True):
    """got: binding.FakeQuantOut on the device; ref: oracle FakeQuantResult.
    lo / hi / s / z / codes / mask / gx bit-exact; y within 1e-6 * s of the oracle (and bit-exact)."""
    if got.lo is not None:
        assert same_bits(to_np(got.lo), ref.lo), "per-group min differs"
        assert same_bits(to_np(got.hi), ref.hi), "per-group max differs"
    if got.s is not None:
        assert same_bits(to_np(got.s), ref.s) and same_bits(to_np(got.z), ref.z), "scale / zero-point differ"
    if got.codes is not None:
        assert np.array_equal(to_np(got.codes), ref.codes), "integer codes differ"
    if got.y is not None:
        y = to_np(got.y)
        tol = 1e-6 * ref.s.astype(np.float64)[group_index(shape, axis, mode)]
        assert np.all(np.abs(widen(y).astype(np.float64) - widen(ref.y).astype(np.float64)) <= tol), "y out of tolerance"
        if exact:
            assert same_bits(y, ref.y), "y not bit-exact"
    if backward:
        if got.mask is not None:
            assert np.array_equal(to_np(got.mask), ref.mask), "STE mask differs"
        assert same_bits(to_np(got.gx), ref.gx), "gx differs"


class Guarded:
    """Device tensors carved out of poisoned allocations; check() asserts that every margin is intact."""

    def __init__(self):
        self._bufs = []

    def empty(self, shape, dtype, align: int = 256, offset: int = 0) -> torch.Tensor:
        """A contiguous tensor of `shape` whose first byte sits `offset` bytes past an `align`-byte
        boundary, with GUARD_BYTES of poison before and after it (the tensor itself is poisoned too)."""
        shape = tuple(int(d) for d in shape)
        esize = torch.empty(0, dtype=dtype).element_size()
        nbytes = int(np.prod(shape, dtype=np.int64)) * esize
        raw = torch.full((GUARD_BYTES + align + offset + nbytes + GUARD_BYTES,), POISON, dtype=torch.uint8,
                         device="cuda")
        start = GUARD_BYTES + (-(raw.data_ptr() + GUARD_BYTES)) % align + offset
        t = raw[start:start + nbytes].view(dtype).view(shape)
        assert t.data_ptr() % align == offset % align
        self._bufs.append((raw, start, nbytes))
        return t

    def check(self):
        for raw, start, nbytes in self._bufs:
            assert bool((raw[:start] == POISON).all()), "an output was written before its first byte"
            assert bool((raw[start + nbytes:] == POISON).all()), "an output was written past its last byte"

    def held_bytes(self) -> int:
        return sum(raw.numel() for raw, _, _ in self._bufs)

    def check_and_release(self):
        """Check every margin, then let go of the allocations (the tensors handed out stay valid: they hold a
        reference to their storage)."""
        torch.cuda.synchronize()
        self.check()
        self._bufs.clear()


def guarded_out(b, g: Guarded, x: torch.Tensor, G: int, backward: bool, codes: bool = True, params: bool = True,
                offset: int = 0):
    """A FakeQuantOut whose every output tensor has guard bands (offset: bytes past a 256-byte boundary for y / gx)."""
    o = b.FakeQuantOut()
    o.y = g.empty(x.shape, x.dtype, offset=offset)
    o.lo = g.empty((G,), torch.float32)
    o.hi = g.empty((G,), torch.float32)
    if backward:
        o.gx = g.empty(x.shape, x.dtype, offset=offset)
    if params:
        o.s = g.empty((G,), torch.float32)
        o.z = g.empty((G,), torch.float32)
    if codes:
        o.codes = g.empty(x.shape, torch.uint8)
        if backward:
            o.mask = g.empty(x.shape, torch.uint8)
    return o


def make_case(shape, seed, dtype="f32", relu=False, spread=1.0):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal(shape) * np.exp(spread * rng.standard_normal((1, shape[1], 1, 1)))
    x = x.astype(np.float32)
    if relu:
        x = np.maximum(x, 0)
    x = x + np.float32(0)
    gy = rng.standard_normal(shape).astype(np.float32)
    if dtype == "bf16":
        return wl.to_bf16_bits(x), wl.to_bf16_bits(gy)
    return x, gy
