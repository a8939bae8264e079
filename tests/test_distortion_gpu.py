"""GPU parity of the distortion statistics of Table 2 (Section 4.1) against the CPU oracle.

Tolerance: the kernels sum the terms of one 16-byte pack (4 fp32 or 8 bf16 elements) in fp32 and
everything else in fp64, the oracle sums everything in fp64.  Every term of three of the sums is
non-negative and x*q is non-negative wherever x and q have the same sign, so a sum differs from the
oracle's by at most about 8 roundings of 2^-24 of its own size: 1e-6 relative is asserted (the
x*q sum is compared against sum |x*q|)."""
import numpy as np
import pytest
import torch

from oracle import granq_oracle as orc
from paper_2503_18339_b200 import workloads as wl
from test_parity_gpu import assert_parity, b, knobs, make_case, to_dev, to_np, widen  # noqa: F401

pytestmark = pytest.mark.gpu

RTOL = 1e-6
SHAPES = [(2, 2, 2, 2), (1, 1, 1, 9), (3, 5, 7, 7), (16, 32, 7, 7), (9, 24, 12, 12), (33, 6, 40, 28), (5, 7, 3, 11)]


def close(got: np.ndarray, ref: np.ndarray, x: np.ndarray, q: np.ndarray) -> bool:
    scale = ref.copy()
    scale[2] = float(np.abs(widen(x).astype(np.float64) * widen(q).astype(np.float64)).sum())
    return bool(np.all(np.abs(got - ref) <= RTOL * scale + 1e-300))


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_distortion_of_a_given_pair(b, shape, dtype):
    x, other = make_case(shape, seed=sum(shape) + 5, dtype=dtype)
    ref_q = orc.fused(x, 3).y
    for q in (ref_q, other, x):                     # a quantization, an unrelated tensor, the identity
        got = b.granq_distortion(to_dev(x), to_dev(q)).cpu().numpy()
        assert close(got, orc.distortion_sums(x, q), x, q)
    # unaligned views take the scalar path
    flat_x, flat_q = to_dev(x).reshape(1, 1, 1, -1), to_dev(ref_q).reshape(1, 1, 1, -1)
    if flat_x.shape[-1] > 3:
        got = b.granq_distortion(flat_x[..., 1:].clone()[..., 1:], flat_q[..., 1:].clone()[..., 1:]).cpu().numpy()
        xs, qs = x.reshape(1, 1, 1, -1)[..., 2:], ref_q.reshape(1, 1, 1, -1)[..., 2:]
        assert close(got, orc.distortion_sums(xs, qs), xs, qs)


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fused_stats_every_grouping_and_plan(b, knobs, shape, dtype):
    x, _ = make_case(shape, seed=sum(shape) + 6, dtype=dtype, spread=1.5)
    bits = 2 + sum(shape) % 4
    for mode in (orc.GROUP_CHANNEL, orc.GROUP_SAMPLE_CHANNEL, orc.GROUP_TENSOR):
        ref = orc.fused(x, bits, group_mode=mode)
        ref_sums = orc.distortion_sums(x, ref.y)
        for flags, wave_kb in ((0, 0), (b.FLAG_FORCE_TWO_PASS, 0), (b.FLAG_FORCE_COLWALK, 1), (b.FLAG_FORCE_CLUSTER, 0)):
            knobs(l2_wave_kb=wave_kb)
            try:
                got = b.granq_fakequant_fused_stats(to_dev(x), bits, group=mode, want_params=True, flags=flags)
            except b.GranqError as err:
                assert flags in (b.FLAG_FORCE_COLWALK, b.FLAG_FORCE_CLUSTER) and err.status == b.ERR_UNSUPPORTED
                continue
            assert b.workspace_status(got.workspace) == b.OK
            assert_parity(got, ref, shape, 1, mode, backward=False)
            sums = got.sums.cpu().numpy()
            assert close(sums, ref_sums, x, ref.y), f"sums differ (mode {mode}, flags {flags})"
            cos, rel = b.distortion_from_sums(sums)
            rcos, rrel = orc.distortion(ref_sums)
            assert cos == pytest.approx(rcos, rel=2e-6, abs=1e-12) and rel == pytest.approx(rrel, rel=2e-6, abs=1e-12)


@pytest.mark.parametrize("spec", [wl.config_tensors(1)[0]] + wl.config_tensors(3)[1:3], ids=lambda s: s.name)
def test_channel_wise_distorts_less_than_layer_wise_at_3_bits(b, spec):
    """Table 2 in kind on the synthetic sets: with per-channel spread the channel-wise method has the
    higher cosine similarity and the lower relative error; both against the oracle at full size."""
    x = wl.make_activation(spec)
    out = {}
    for mode in (orc.GROUP_CHANNEL, orc.GROUP_TENSOR):
        got = b.granq_fakequant_fused_stats(to_dev(x), 3, group=mode)
        ref = orc.fused(x, 3, group_mode=mode, want_codes=False)
        sums = got.sums.cpu().numpy()
        assert np.array_equal(to_np(got.y).view(np.uint32), ref.y.view(np.uint32))
        assert close(sums, orc.distortion_sums(x, ref.y), x, ref.y)
        out[mode] = b.distortion_from_sums(sums)
    assert out[orc.GROUP_CHANNEL][0] > out[orc.GROUP_TENSOR][0]
    assert out[orc.GROUP_CHANNEL][1] < out[orc.GROUP_TENSOR][1]


def test_stats_reject_bad_arguments(b):
    x = to_dev(make_case((2, 4, 4, 4), seed=1)[0])
    buf = torch.empty(40, dtype=torch.uint8, device="cuda")
    with pytest.raises(b.GranqError) as err:      # sums not on an 8-byte boundary
        b.granq_distortion(x, x, sums=buf[4:36])
    assert err.value.status == b.ERR_INVALID_ARG
