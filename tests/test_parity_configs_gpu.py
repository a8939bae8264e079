"""Parity on the five synthetic activation sets at their full sizes, in the launch
configuration the benchmark times (default plan, fused forward + backward), every element
compared with the CPU oracle: min / max, codes and STE mask bit-exact, y within
1e-6 * scale (asserted bit-exact as well, which is what the arithmetic delivers).  Both
group modes (per channel over the batch; Eq. 4 per sample) run on every tensor of every
config, and every output sits between guard bands that must come back untouched."""
import numpy as np
import pytest
import torch

from gpu_util import Guarded, guarded_out, same_bits, to_dev, to_np
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


def widen64(a):
    return (wl.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a).astype(np.float64)


def expected_plan(b, dt, shape, mode, backward):
    """The default plan per geometry: the cluster-local kernel where a run of channels fits the shared memory
    of one cluster (except forward-only bf16 tensors of 48 MB and more, measured faster on the column walk),
    else the column walk over the batch (channel groups) or the L2-resident waves."""
    if (dt == b.BF16 and not backward and mode == orc.GROUP_CHANNEL and shape[0] >= 8
            and 2 * int(np.prod(shape, dtype=np.int64)) >= 48 << 20):
        return b.PLAN_COLWALK          # the measured exception: long forward-only bf16 tensors
    if b.cluster_geometry(dt, shape, group=mode, with_backward=backward) is not None:
        return b.PLAN_CLUSTER
    return b.PLAN_COLWALK if mode == orc.GROUP_CHANNEL else b.PLAN_L2WAVE


def check(b, x, gy, bits, mode, with_codes, flags=0, offset=0):
    dt = b.F32 if x.dtype == np.float32 else b.BF16
    if flags == 0:
        plan, _ = b.fused_plan(dt, x.shape, group=mode, with_backward=gy is not None)
        assert plan == expected_plan(b, dt, x.shape, mode, gy is not None), "not the plan the benchmark launches"
    ref = orc.fused(x, bits, gy=gy, group_mode=mode, want_codes=with_codes)
    xd = to_dev(x)
    g = Guarded()
    out = guarded_out(b, g, xd, b.num_groups(x.shape, 1, mode), backward=gy is not None, codes=with_codes,
                      offset=offset)
    got = b.granq_fakequant_fused(xd, bits, gy=None if gy is None else to_dev(gy), group=mode, out=out,
                                  want_codes=with_codes, want_mask=with_codes, want_params=True, flags=flags)
    assert b.workspace_status(got.workspace) == b.OK
    assert same_bits(to_np(got.lo), ref.lo) and same_bits(to_np(got.hi), ref.hi)
    assert same_bits(to_np(got.s), ref.s) and same_bits(to_np(got.z), ref.z)
    y = to_np(got.y)
    n, c = x.shape[0], x.shape[1]
    s_of = ref.s.astype(np.float64)
    tol = 1e-6 * (s_of.reshape(1, c, 1, 1) if mode == orc.GROUP_CHANNEL else s_of.reshape(n, c, 1, 1))
    assert np.all(np.abs(widen64(y) - widen64(ref.y)) <= tol)
    assert same_bits(y, ref.y)
    if with_codes:
        assert np.array_equal(to_np(got.codes), ref.codes)
    if gy is not None:
        assert same_bits(to_np(got.gx), ref.gx)
        if with_codes:
            assert np.array_equal(to_np(got.mask), ref.mask)
    g.check()
    return ref


def distinct(specs):
    seen, out = set(), []
    for s in specs:
        if s.shape not in seen:
            seen.add(s.shape)
            out.append(s)
    return out


def test_config1_resnet20_first_layer(b):
    spec = wl.config_tensors(1)[0]
    x, gy = wl.make_activation(spec), wl.make_upstream_grad(spec)
    ref = check(b, x, gy, 3, orc.GROUP_CHANNEL, True)
    assert (ref.lo == 0).all() and (ref.z == 0).all()          # post-ReLU: every channel starts at 0
    check(b, x, gy, 3, orc.GROUP_SAMPLE_CHANNEL, True)
    # the 'conventional' per-channel loop (three launches per channel) and every other plan, at full size
    for flags in (b.FLAG_FORCE_NAIVE, b.FLAG_FORCE_TWO_PASS, b.FLAG_FORCE_COLWALK, b.FLAG_FORCE_L2WAVE,
                  b.FLAG_FORCE_STAGED, b.FLAG_FORCE_CLUSTER):
        assert b.fused_plan(b.F32, spec.shape, flags=flags)[0] >= 0      # every plan takes this tensor
        check(b, x, gy, 3, orc.GROUP_CHANNEL, True, flags=flags)
    check(b, x, gy, 3, orc.GROUP_SAMPLE_CHANNEL, True, flags=b.FLAG_FORCE_NAIVE)


@pytest.mark.parametrize("spec", distinct(wl.config_tensors(2)), ids=lambda s: s.name)
def test_config2_resnet20_cifar_set(b, spec):
    x, gy = wl.make_activation(spec), wl.make_upstream_grad(spec)
    dead = np.flatnonzero(wl.channel_sigma(spec) == 0)
    for bits in spec.bits:
        ref = check(b, x, gy, bits, orc.GROUP_CHANNEL, True)
        assert (ref.codes[:, dead] == 0).all() and (ref.y[:, dead] == 0).all()
    check(b, x, gy, 3, orc.GROUP_SAMPLE_CHANNEL, True)
    check(b, x, gy, 4, orc.GROUP_CHANNEL, True, flags=b.FLAG_FORCE_NAIVE)


@pytest.mark.parametrize("spec", wl.config_tensors(3) + wl.config_tensors(4), ids=lambda s: s.name)
def test_config3_4_imagenet_shaped(b, spec):
    x, gy = wl.make_activation(spec), wl.make_upstream_grad(spec)
    check(b, x, gy, spec.bits[0], orc.GROUP_CHANNEL, True)
    check(b, x, gy, spec.bits[1], orc.GROUP_CHANNEL, False)     # exactly what the benchmark launches
    check(b, x, gy, spec.bits[0], orc.GROUP_SAMPLE_CHANNEL, True)
    if b.cluster_geometry(b.F32, spec.shape) is not None:       # the thin-plane tensors also through the column walk
        check(b, x, gy, spec.bits[1], orc.GROUP_CHANNEL, False, flags=b.FLAG_FORCE_COLWALK)


CFG5_BITS = {   # (fused bits, forward-only bits) per tensor and dtype: bits 2..8 all appear both ways
    (0, "f32"): (2, 8), (0, "bf16"): (3, 7), (1, "f32"): (4, 6), (1, "bf16"): (5, 2),
    (2, "f32"): (6, 3), (2, "bf16"): (7, 4), (3, "f32"): (8, 5), (3, "bf16"): (2, 8),
}


@pytest.mark.parametrize("spec", wl.config_tensors(5), ids=lambda s: s.name)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_config5_bandwidth_sweep(b, spec, dtype):
    x, gy = wl.make_activation(spec), wl.make_upstream_grad(spec)
    if dtype == "bf16":
        x, gy = wl.to_bf16_bits(x), wl.to_bf16_bits(gy)
    fused_bits, fwd_bits = CFG5_BITS[(spec.index, dtype)]
    ref = check(b, x, gy, fused_bits, orc.GROUP_CHANNEL, True)
    assert (ref.z != 0).any()                                     # signed data: the zero-point path is live
    check(b, x, None, fwd_bits, orc.GROUP_CHANNEL, False)
    check(b, x, gy, fwd_bits, orc.GROUP_SAMPLE_CHANNEL, False)    # Eq. 4 per sample, at full size
