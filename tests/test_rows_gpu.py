"""Channels-last tensors ([N, H, W, C], channel_axis = 3) and planes of one element ([N, C, 1, 1]) through the
plan made for them (a range launch and a quantize launch, one 16-byte unit column per thread) against the CPU
oracle: small and adversarial shapes, and two tensors of the benchmark's activation sets transposed to
channels-last at full size; every output between guard bands."""
import numpy as np
import pytest
import torch

from gpu_util import Guarded, assert_parity, guarded_out, make_case, to_dev
from oracle import granq_oracle as orc
from paper_2503_18339_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2503_18339_b200 import binding
    binding.lib()
    for k in range(binding.N_KNOBS):
        binding.tune(k, 0)
    return binding


def run(b, x, gy, bits, axis):
    shape = x.shape
    ref = orc.fused(x, bits, gy=gy, channel_axis=axis)
    xd = to_dev(x)
    g = Guarded()
    out = guarded_out(b, g, xd, shape[axis], backward=gy is not None)
    dt = b.BF16 if x.dtype == np.uint16 else b.F32
    assert b.fused_plan(dt, shape, channel_axis=axis)[0] == b.PLAN_ROWS
    got = b.granq_fakequant_fused(xd, bits, gy=None if gy is None else to_dev(gy), channel_axis=axis, out=out,
                                  want_codes=True, want_mask=True, want_params=True)
    assert b.workspace_status(got.workspace) == b.OK
    assert_parity(got, ref, shape, axis, orc.GROUP_CHANNEL, backward=gy is not None)
    g.check()


def nhwc_case(shape, seed, dtype):
    """make_case() draws a per-channel spread along axis 1; move that axis last."""
    n, h, w, c = shape
    x, gy = make_case((n, c, h, w), seed, "f32", relu=(seed % 2 == 0))
    x, gy = np.ascontiguousarray(x.transpose(0, 2, 3, 1)), np.ascontiguousarray(gy.transpose(0, 2, 3, 1))
    return (wl.to_bf16_bits(x), wl.to_bf16_bits(gy)) if dtype == "bf16" else (x, gy)


SHAPES = [(2, 5, 7, 8), (3, 4, 4, 64), (1, 1, 1, 16), (5, 9, 3, 96), (2, 3, 3, 2048), (7, 1, 13, 24), (2, 2, 2, 4096),
          (300, 1, 1, 8), (1, 33, 17, 40)]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_channels_last_small(b, shape, dtype):
    x, gy = nhwc_case(shape, seed=sum(shape), dtype=dtype)
    bits = 2 + sum(shape) % 7
    run(b, x, gy, bits, 3)
    run(b, x, None, bits, 3)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_planes_of_one_element(b, dtype):
    """[N, C, 1, 1] with the usual channel axis is the same matrix [N, C]."""
    x, gy = make_case((37, 24, 1, 1), seed=3, dtype=dtype)
    run(b, x, gy, 4, 1)


def test_geometries_the_plan_does_not_take(b):
    assert b.fused_plan(b.F32, (2, 3, 3, 6), channel_axis=3)[0] == b.PLAN_TWO_PASS       # rows of 24 bytes
    assert b.fused_plan(b.BF16, (2, 3, 3, 4), channel_axis=3)[0] == b.PLAN_TWO_PASS      # rows of 8 bytes
    assert b.fused_plan(b.F32, (2, 3, 3, 8192), channel_axis=3)[0] == b.PLAN_TWO_PASS    # more channels than the table holds
    x, gy = nhwc_case((2, 3, 3, 6), 1, "f32")
    ref = orc.fused(x, 4, gy=gy, channel_axis=3)
    got = b.granq_fakequant_fused(to_dev(x), 4, gy=to_dev(gy), channel_axis=3, want_codes=True, want_mask=True,
                                  want_params=True)
    assert_parity(got, ref, x.shape, 3, orc.GROUP_CHANNEL, backward=True)


@pytest.mark.parametrize("index", [3, 4], ids=["cfg3.3", "cfg3.4"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_channels_last_at_full_size(b, index, dtype):
    """[128, 256, 14, 14] and [128, 512, 7, 7] of the ResNet-18-shaped set, stored channels-last."""
    spec = wl.config_tensors(3)[index]
    x = np.ascontiguousarray(wl.make_activation(spec).transpose(0, 2, 3, 1))
    gy = np.ascontiguousarray(wl.make_upstream_grad(spec).transpose(0, 2, 3, 1))
    if dtype == "bf16":
        x, gy = wl.to_bf16_bits(x), wl.to_bf16_bits(gy)
    run(b, x, gy, spec.bits[0], 3)
