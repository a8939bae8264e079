"""GPU parity of the packed integer codes (Eq. 1 -> bit string -> Eq. 6) against the CPU oracle:
the bit string byte for byte, scale / zero-point and the dequantized tensor bit for bit."""
import numpy as np
import pytest
import torch

from oracle import granq_oracle as orc
from paper_2503_18339_b200 import workloads as wl
from test_parity_gpu import b, make_case, same_bits, to_dev, to_np  # noqa: F401

pytestmark = pytest.mark.gpu

SHAPES = [(2, 2, 2, 2), (1, 1, 1, 9), (3, 5, 7, 7), (4, 16, 14, 14), (16, 32, 7, 7), (9, 24, 12, 12), (5, 7, 3, 11),
          (2, 3, 64, 67)]


def padded(p: np.ndarray, nbytes: int) -> np.ndarray:
    out = np.zeros(nbytes, np.uint8)
    out[:p.size] = p
    return out


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_quantize_packed_then_dequantize_packed(b, shape, dtype):
    x, _ = make_case(shape, seed=sum(shape) + 9, dtype=dtype)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    for mode in (orc.GROUP_CHANNEL, orc.GROUP_SAMPLE_CHANNEL, orc.GROUP_TENSOR):
        lo, hi = orc.range_(x, group_mode=mode)
        lo2 = (lo + 0.1 * (hi - lo)).astype(np.float32)          # a stale range: both clamp sides are live
        hi2 = (lo + 0.8 * (hi - lo)).astype(np.float32)
        for bits in range(1, 9):
            ref = orc.fakequant(x, bits, lo2, hi2, group_mode=mode)
            want = orc.pack_codes(ref.codes, bits)
            got = b.granq_quantize_packed(to_dev(x), bits, to_dev(lo2), to_dev(hi2), group=mode, want_y=(bits % 2 == 0))
            nbytes = b.packed_codes_bytes(shape, bits)
            assert nbytes == (x.size * bits + 31) // 32 * 4
            assert np.array_equal(got.packed_codes.cpu().numpy().view(np.uint8), padded(want, nbytes)), \
                f"bit string differs (mode {mode}, b = {bits})"
            assert same_bits(to_np(got.s), ref.s) and same_bits(to_np(got.z), ref.z)
            if got.y is not None:
                assert same_bits(to_np(got.y), ref.y)
            y = b.granq_dequantize_packed(got.packed_codes, shape, tdt, bits, got.s, got.z, group=mode)
            assert same_bits(to_np(y), ref.y), f"dequantized tensor differs (mode {mode}, b = {bits})"
            assert same_bits(to_np(y), orc.dequant_packed(want, shape, bits, ref.s, ref.z, dtype=x.dtype, group_mode=mode))


@pytest.mark.parametrize("spec", [wl.config_tensors(3)[1], wl.config_tensors(3)[4], wl.config_tensors(4)[3]],
                         ids=lambda s: s.name)
def test_packed_codes_full_size(b, spec):
    """Every element of three benchmarked tensors (56x56, 7x7 and 28x28 planes) at the paper's bit-widths."""
    x = wl.make_activation(spec)
    lo, hi = orc.range_(x)
    for bits in (3, 4, 5):
        ref = orc.fakequant(x, bits, lo, hi)
        got = b.granq_quantize_packed(to_dev(x), bits, to_dev(lo), to_dev(hi))
        want = orc.pack_codes(ref.codes, bits)
        assert np.array_equal(got.packed_codes.cpu().numpy().view(np.uint8)[:want.size], want)
        y = b.granq_dequantize_packed(got.packed_codes, x.shape, torch.float32, bits, got.s, got.z)
        assert same_bits(to_np(y), ref.y)


def test_packed_codes_reject_bad_arguments(b):
    x = to_dev(make_case((2, 4, 4, 4), seed=1)[0])
    lo, hi = torch.zeros(4, device="cuda"), torch.ones(4, device="cuda")
    buf = torch.empty(b.packed_codes_bytes(x.shape, 4) + 4, dtype=torch.uint8, device="cuda")
    with pytest.raises(b.GranqError) as err:
        b.granq_quantize_packed(x, 4, lo, hi, packed_codes=buf[1:])
    assert err.value.status == b.ERR_INVALID_ARG
    assert b.packed_codes_bytes((1, 1, 1, 33), 3) == 16 and b.packed_codes_bytes((1, 1, 1, 32), 9) == 0


FUSED_SHAPES = [(2, 2, 2, 2), (3, 5, 7, 7), (4, 16, 14, 14), (16, 32, 7, 7), (16, 8, 7, 7), (9, 24, 12, 12), (8, 4, 8, 8),
                (32, 6, 40, 28), (5, 7, 3, 11), (12, 10, 16, 16)]


@pytest.mark.parametrize("shape", FUSED_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_quantize_packed_fused(b, shape, dtype):
    """Range of the tensor itself -> parameters -> packed codes in one call, on every plan that takes the geometry
    (cluster-local kernel, column walk, range pass + flat pass), every bit-width, both group modes with planes."""
    x, _ = make_case(shape, seed=sum(shape) + 21, dtype=dtype, relu=(shape[1] % 2 == 0))
    taken = set()
    for mode in (orc.GROUP_CHANNEL, orc.GROUP_SAMPLE_CHANNEL):
        for bits in range(1, 9):
            ref = orc.fused(x, bits, group_mode=mode, want_codes=True)
            want = padded(orc.pack_codes(ref.codes, bits), b.packed_codes_bytes(shape, bits))
            for flags in (0, b.FLAG_FORCE_TWO_PASS, b.FLAG_FORCE_COLWALK, b.FLAG_FORCE_CLUSTER):
                try:
                    got = b.granq_quantize_packed_fused(to_dev(x), bits, group=mode, flags=flags)
                except b.GranqError as err:
                    assert flags in (b.FLAG_FORCE_COLWALK, b.FLAG_FORCE_CLUSTER) and err.status == b.ERR_UNSUPPORTED
                    continue
                taken.add(flags)
                assert b.workspace_status(got.workspace) == b.OK
                assert np.array_equal(got.packed_codes.cpu().numpy().view(np.uint8), want), \
                    f"bit string differs (mode {mode}, b = {bits}, flags {flags})"
                assert same_bits(to_np(got.lo), ref.lo) and same_bits(to_np(got.hi), ref.hi)
                assert same_bits(to_np(got.s), ref.s) and same_bits(to_np(got.z), ref.z)
    e = int(np.prod(shape))
    if e % 32 == 0 and (shape[1] * shape[2] * shape[3]) % 8 == 0 and shape[2] * shape[3] >= 8:
        assert b.FLAG_FORCE_CLUSTER in taken, "the cluster-local kernel must take whole groups of 8 codes"
        if shape[0] >= 8:
            assert b.FLAG_FORCE_COLWALK in taken


@pytest.mark.parametrize("spec", [wl.config_tensors(3)[1], wl.config_tensors(3)[4], wl.config_tensors(4)[3]],
                         ids=lambda s: s.name)
def test_quantize_packed_fused_full_size(b, spec):
    """Every code of three benchmarked tensors (column walk, cluster-local with 7x7 planes, cluster-local with 28x28)."""
    x = wl.make_activation(spec)
    for bits in (3, 4, 5):
        ref = orc.fused(x, bits, want_codes=True)
        got = b.granq_quantize_packed_fused(to_dev(x), bits)
        want = orc.pack_codes(ref.codes, bits)
        assert b.workspace_status(got.workspace) == b.OK
        assert np.array_equal(got.packed_codes.cpu().numpy().view(np.uint8)[:want.size], want)
        assert same_bits(to_np(got.s), ref.s) and same_bits(to_np(got.z), ref.z)
