"""The accumulation over the integer codes on the tensor cores (Eq. 6 left-hand side, Algorithm 1 output
step, pointwise case) against the CPU oracle, through the C ABI.

Tolerance, derived from the arithmetic (not tuned): the kernel multiplies the exact codes by the scaled
weights w * s_c split into two bf16 halves (what the split leaves out is below 2^-17 of each weight),
accumulates the 2 C exact products in fp32 in an order of the hardware's choosing (at most one unit in the
last place, 2^-23, of the running sum per addition, and the running sum never exceeds sum_c |w s_c| code),
rounds the bias once and subtracts it in fp32; the split also touches the bias terms w s_c z_c, and the oracle
itself rounds every pre-scaled activation s_c (code - z_c) to fp32 once.  With S = sum_c |w s_c| (code + |z_c|):
    |y - y_oracle| <= (2^-17 + C * 2^-22) * S + 2^-21 * (|bias| + |y_oracle|).
Where every product and partial sum is an integer below 2^24 the result must be exact."""
import numpy as np
import pytest
import torch

from gpu_util import Guarded
from oracle import granq_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2503_18339_b200 import binding
    binding.lib()
    return binding


def packed_words(codes: np.ndarray, bits: int) -> torch.Tensor:
    """The oracle's bit string of the codes (in the order given), padded to whole 32-bit words, on the device."""
    by = orc.pack_codes(codes, bits)
    pad = (-by.size) % 4
    by = np.concatenate([by, np.zeros(pad, np.uint8)])
    return torch.from_numpy(by.view(np.int32).copy()).cuda()


def run(b, codes_nchw, bits, s, z, w, channels_last, flags=0):
    n, c, h, wd = codes_nchw.shape
    o = w.shape[0]
    src = np.ascontiguousarray(codes_nchw.transpose(0, 2, 3, 1)) if channels_last else codes_nchw
    g = Guarded()
    y = g.empty((n, h, wd, o) if channels_last else (n, o, h, wd), torch.float32)
    got, ws = b.granq_accumulate_codes(packed_words(src, bits), src.shape, bits, torch.from_numpy(s).cuda(),
                                       torch.from_numpy(z).cuda(), torch.from_numpy(w).cuda(),
                                       channel_axis=3 if channels_last else 1, y=y, flags=flags)
    assert b.workspace_status(ws) == b.OK
    g.check()
    got = got.cpu().numpy().astype(np.float64)
    return got.transpose(0, 3, 1, 2) if channels_last else got


def bound(codes, s, z, w):
    ws = np.abs(w.astype(np.float64) * s.astype(np.float64))
    S = np.einsum("oc,nchw->nohw", ws, codes.astype(np.float64)) + (ws @ np.abs(z.astype(np.float64))).reshape(1, -1, 1, 1)
    bias = np.abs((w.astype(np.float64) * s.astype(np.float64)) @ z.astype(np.float64)).reshape(1, -1, 1, 1)
    return S, bias


SHAPES = [   # (N, C, H, W, O)
    (2, 64, 7, 7, 64),        # one K block, one tile per sample with 49 of 128 rows used
    (3, 96, 14, 14, 100),     # C not a multiple of 64 (second K block half empty), O not a multiple of the tile
    (2, 20, 5, 6, 24),        # C padded to 24, tiny everything
    (1, 256, 28, 28, 200),    # 4 K blocks (one full turn of the ring), 7 pixel tiles, 2 channel tiles
    (2, 384, 14, 14, 72),     # 6 K blocks: the ring wraps
    (5, 128, 7, 7, 512),      # tiles that straddle samples, 4 channel tiles
    (32, 64, 56, 56, 64),     # 784 pixel tiles: a persistent CTA takes five or six, both accumulators and every
                              # stage of the ring come round several times
    (9, 72, 28, 28, 40),      # 56 tiles, 2 K blocks each (the second one 8 channels wide)
    (40, 128, 56, 56, 128),   # 980 tiles with the 128-channel tile: only two accumulators, which the two epilogue
                              # groups take in turn six or seven times per CTA (a wait that mistook an earlier
                              # completion of a barrier for the one it needs would read a stale accumulator here)
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("channels_last", [False, True], ids=["nchw", "nhwc"])
def test_accumulate_matches_the_oracle_within_the_derived_bound(b, shape, channels_last):
    n, c, h, wd, o = shape
    rng = np.random.default_rng(sum(shape))
    x = (rng.standard_normal((n, c, h, wd)) * np.exp(rng.standard_normal((1, c, 1, 1)))).astype(np.float32)
    bits = 2 + sum(shape) % 7
    res = orc.fused(x, bits)                                       # codes, s, z by the oracle (signed data: z != 0)
    w = (rng.standard_normal((o, c)) / np.sqrt(c)).astype(np.float32)
    ref = orc.accumulate(res.codes, res.s, res.z, w)
    S, bias = bound(res.codes, res.s, res.z, w)
    tol = (2.0 ** -17 + c * 2.0 ** -22) * S + 2.0 ** -21 * (bias + np.abs(ref))
    for flags in (0, b.FLAG_FORCE_TWO_PASS):       # the persistent kernel (where the weights fit), one tile per CTA
        got = run(b, res.codes, bits, res.s, res.z, w, channels_last, flags)
        err = np.abs(got - ref)
        assert np.all(err <= tol), f"max err/tol {np.max(err / np.maximum(tol, 1e-300)):.3f} (flags {flags})"
        assert np.max(err / np.maximum(tol, 1e-300)) < 0.5            # and in practice well inside it
    # a dropped K block, a transposed operand or a missing bias would be far outside: the error is not trivially small
    assert np.max(np.abs(ref)) > 100 * np.max(tol)


@pytest.mark.parametrize("channels_last", [False, True], ids=["nchw", "nhwc"])
def test_accumulate_is_exact_on_small_integers(b, channels_last):
    """Integer weights in [-8, 8], scales that are powers of two, integer zero-points: every product and every
    partial sum is an integer far below 2^24, so the tensor-core result must equal the oracle bit for bit."""
    n, c, h, wd, o = 3, 160, 9, 11, 130
    rng = np.random.default_rng(5)
    bits = 5
    codes = rng.integers(0, 2 ** bits, (n, c, h, wd), dtype=np.uint8)
    s = (2.0 ** rng.integers(-2, 3, c)).astype(np.float32)
    z = rng.integers(0, 2 ** bits, c).astype(np.float32)
    w = rng.integers(-8, 9, (o, c)).astype(np.float32)
    ref = orc.accumulate(codes, s, z, w)
    for flags in (0, b.FLAG_FORCE_TWO_PASS):
        got = run(b, codes, bits, s, z, w, channels_last, flags)
        assert np.array_equal(got, ref)
    # one-hot weights select the pre-scaled activation of one channel
    onehot = np.zeros((c, c), np.float32)
    onehot[np.arange(c), (np.arange(c) * 7) % c] = 1
    got = run(b, codes, bits, s, z, onehot, channels_last)
    want = (s.reshape(1, c, 1, 1) * (codes.astype(np.float32) - z.reshape(1, c, 1, 1)))[:, (np.arange(c) * 7) % c]
    assert np.array_equal(got, want.astype(np.float64))


def test_accumulate_from_the_library_s_own_packed_codes(b):
    """Whole chain on the GPU: range -> packed codes, scale, zero-point -> accumulation, against the oracle's chain."""
    n, c, h, wd, o = 4, 64, 14, 14, 64
    rng = np.random.default_rng(9)
    x = np.maximum(rng.standard_normal((n, c, h, wd)) * np.exp(rng.standard_normal((1, c, 1, 1))), 0).astype(np.float32)
    w = (rng.standard_normal((o, c)) / 8).astype(np.float32)
    res = orc.fused(x, 4)
    ref = orc.accumulate(res.codes, res.s, res.z, w)
    xd = torch.from_numpy(x).cuda()
    lo, hi = b.granq_range(xd)
    q = b.granq_quantize_packed(xd, 4, lo, hi)
    got, ws = b.granq_accumulate_codes(q.packed_codes, x.shape, 4, q.s, q.z, torch.from_numpy(w).cuda())
    assert b.workspace_status(ws) == b.OK
    S, bias = bound(res.codes, res.s, res.z, w)
    tol = (2.0 ** -17 + c * 2.0 ** -22) * S + 2.0 ** -21 * (bias + np.abs(ref))
    assert np.all(np.abs(got.cpu().numpy().astype(np.float64) - ref) <= tol)


def test_accumulate_argument_errors(b):
    x = torch.zeros(4, dtype=torch.int32, device="cuda")
    f = torch.zeros(8, device="cuda")
    w = torch.zeros(8, 8, device="cuda")
    with pytest.raises(b.GranqError) as err:
        b.granq_accumulate_codes(x, (1, 8, 2, 2), 9, f, f, w)
    assert err.value.status == b.ERR_INVALID_ARG
    with pytest.raises(b.GranqError) as err:
        b.granq_accumulate_codes(x, (1, 8, 2, 2), 4, f, f, w, workspace=torch.zeros(256, dtype=torch.uint8, device="cuda"))
    assert err.value.status == b.ERR_WORKSPACE
    assert b.accumulate_workspace_bytes((1, 8, 2, 2), 2, 8) == 0          # channel axis must be 1 or 3
