"""Parity of the cluster-local plan (a run of channels staged once in the shared memory of one
thread-block cluster) with the CPU oracle: every cut the planner can make - clusters of 1, 2, 4
and 8 CTAs, every way of staging (per-thread asynchronous copies, bulk copies, plain loads; gy staged or not), several thread counts, ragged 7x7 planes, a last run
with fewer channels, odd batches that do not split evenly over a cluster, per-sample groups -
with guard bands around every output."""
import numpy as np
import pytest
import torch

from gpu_util import Guarded, assert_parity, guarded_out, make_case, to_dev
from oracle import granq_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2503_18339_b200 import binding
    binding.lib()
    yield binding
    for k in range(binding.N_KNOBS):
        binding.tune(k, 0)


@pytest.fixture()
def knobs(b):
    def set_(**kw):
        names = {"tile_kb": b.KNOB_CLUSTER_TILE_KB, "ctas": b.KNOB_CLUSTER_CTAS, "threads": b.KNOB_CLUSTER_THREADS,
                 "load": b.KNOB_CLUSTER_LOAD, "prefetch": b.KNOB_CLUSTER_PREFETCH, "kmul": b.KNOB_CLUSTER_KMUL, "spin_limit": b.KNOB_SPIN_LIMIT,
                 "extra_arrivals": b.KNOB_TEST_EXTRA_ARRIVALS}
        for k, v in kw.items():
            b.tune(names[k], v)
    yield set_
    for k in range(b.N_KNOBS):
        b.tune(k, 0)


def run_and_check(b, x, gy, bits, mode, offset=0):
    shape = x.shape
    ref = orc.fused(x, bits, gy=gy, group_mode=mode)
    xd = to_dev(x)
    g = Guarded()
    out = guarded_out(b, g, xd, b.num_groups(shape, 1, mode), backward=gy is not None, offset=offset)
    got = b.granq_fakequant_fused(xd, bits, gy=None if gy is None else to_dev(gy), group=mode, out=out,
                                  want_codes=True, want_mask=True, want_params=True, flags=b.FLAG_FORCE_CLUSTER)
    assert b.workspace_status(got.workspace) == b.OK
    assert_parity(got, ref, shape, 1, mode, backward=gy is not None)
    g.check()


SHAPES = [
    (3, 8, 7, 7),        # 7x7 planes: a 16-byte pack straddles two channels, runs of 4 channels
    (4, 16, 14, 14),     # 196-element planes
    (5, 6, 32, 32),      # more columns than threads: several column tiles
    (2, 4, 56, 56),
    (13, 24, 7, 7),      # odd batch: uneven shares inside a cluster
    (9, 10, 7, 7),       # ... and a last run of 2 channels (10 = 4 + 4 + 2) - 98 elements: not whole packs -> refused
    (9, 12, 20, 20),
    (16, 20, 7, 7),      # 5 runs of 4
    (37, 8, 3, 4),       # planes of 12 elements
    (1, 16, 14, 14),     # one slab
    (128, 8, 7, 7),      # a real group: 25 KB
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", [orc.GROUP_CHANNEL, orc.GROUP_SAMPLE_CHANNEL])
def test_cluster_plan_every_cut(b, knobs, shape, dtype, mode):
    dt = b.BF16 if dtype == "bf16" else b.F32
    if b.cluster_geometry(dt, shape, group=mode) is None:
        pack = 8 if dtype == "bf16" else 4
        assert (shape[1] * shape[2] * shape[3]) % pack != 0 or shape[2] * shape[3] < pack
        with pytest.raises(b.GranqError) as err:
            b.granq_fakequant_fused(to_dev(make_case(shape, 1, dtype)[0]), 4, group=mode, flags=b.FLAG_FORCE_CLUSTER)
        assert err.value.status == b.ERR_UNSUPPORTED
        return
    x, gy = make_case(shape, seed=sum(shape) + 5 * mode, dtype=dtype, relu=(shape[0] % 2 == 0))
    bits = 2 + (sum(shape) + mode) % 7
    slabs = shape[0] if mode == orc.GROUP_CHANNEL else 1
    for ctas in (0, 1, 2, 4, 8):
        if ctas > slabs:
            continue
        for load, threads, tile_kb, kmul in ((0, 0, 0, 0), (1, 0, 0, 0), (2, 0, 0, 0), (3, 0, 0, 0), (4, 0, 0, 0),
                                             (1, 128, 0, 2), (2, 96, 8, 0), (1, 512, 2, 0), (3, 160, 0, 3),
                                             (3, 64, 4, 0), (5, 96, 6, 0), (4, 320, 0, 2), (5, 512, 0, 5)):
            knobs(ctas=ctas, load=load, threads=threads, tile_kb=tile_kb, kmul=kmul)
            if b.cluster_geometry(dt, shape, group=mode) is None:      # the forced cut does not fit the tile limit
                continue
            run_and_check(b, x, gy, bits, mode)
    knobs(ctas=0, load=0, threads=0, tile_kb=0, kmul=0)
    run_and_check(b, x, None, bits, mode)                               # forward only


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_cluster_plan_real_group_sizes(b, knobs, dtype):
    """Groups of 100 KB and 401 KB (fp32): one CTA, clusters of 2, 4 and 8, both ways of staging."""
    for shape in ((128, 6, 14, 14), (128, 3, 28, 28), (64, 8, 7, 7)):
        x, gy = make_case(shape, seed=shape[1], dtype=dtype, relu=True)
        for ctas, load in ((0, 0), (0, 1), (0, 2), (0, 3), (0, 4), (8, 1), (4, 2), (2, 1), (8, 3), (4, 3), (8, 5), (4, 4), (2, 5)):
            knobs(ctas=ctas, load=load)
            if b.cluster_geometry(b.BF16 if dtype == "bf16" else b.F32, shape) is None:
                continue
            run_and_check(b, x, gy, 4, orc.GROUP_CHANNEL)


def test_cluster_plan_degenerate_groups(b):
    shape = (8, 8, 14, 14)
    x, gy = make_case(shape, seed=3, relu=True)
    x[:, 0] = 0.0                  # dead channel: s floored at 1e-8
    x[:, 1] = 3.7                  # non-zero constant channel
    x[:, 2] = -100.0
    x[:, 3] = np.minimum(x[:, 3] * 50, 6.0)     # saturating channel: many ties at the maximum
    x[1, 4, 2, 3] = 3.0e38         # huge outlier: this group takes IEEE division
    x[:, 5] *= np.float32(1e-30)   # tiny values
    for bits in (1, 3, 8):
        run_and_check(b, x, gy, bits, orc.GROUP_CHANNEL)


def test_cluster_plan_unaligned_outputs_are_refused_or_exact(b):
    """y / gx that do not start on a 16-byte boundary: the plan is not taken (the default falls back)."""
    shape = (4, 8, 14, 14)
    x, gy = make_case(shape, seed=4)
    xd = to_dev(x)
    g = Guarded()
    out = guarded_out(b, g, xd, 8, backward=True, offset=4)
    with pytest.raises(b.GranqError) as err:
        b.granq_fakequant_fused(xd, 4, gy=to_dev(gy), out=out, flags=b.FLAG_FORCE_CLUSTER)
    assert err.value.status == b.ERR_UNSUPPORTED
    got = b.granq_fakequant_fused(xd, 4, gy=to_dev(gy), out=out, want_codes=True, want_mask=True, want_params=True)
    assert_parity(got, orc.fused(x, 4, gy=gy), shape, 1, orc.GROUP_CHANNEL, backward=True)
    g.check()


def test_cluster_plan_bounded_wait_reports_timeout(b, knobs):
    """The wait on the CTA's own bulk copies is bounded: told to wait, after its tile has landed, for a
    barrier phase that never completes, the kernel stops by itself, reports GRANQ_ERR_TIMEOUT and leaves
    the context usable."""
    shape = (8, 16, 14, 14)
    x, gy = make_case(shape, seed=2)
    for load in (1, 3):
        knobs(extra_arrivals=1, spin_limit=2000, load=load)
        got = b.granq_fakequant_fused(to_dev(x), 4, gy=to_dev(gy), flags=b.FLAG_FORCE_CLUSTER)
        assert b.workspace_status(got.workspace) == b.ERR_TIMEOUT
    knobs(extra_arrivals=0, spin_limit=0, load=0)
    run_and_check(b, x, gy, 4, orc.GROUP_CHANNEL)


def test_cluster_plan_keeps_a_zeroed_workspace_zeroed(b):
    shape = (16, 24, 14, 14)
    x, gy = make_case(shape, seed=11)
    ws = b.make_workspace(to_dev(x), zeroed=True)
    for bits in (4, 3):
        got = b.granq_fakequant_fused(to_dev(x), bits, gy=to_dev(gy), out=b.FakeQuantOut(workspace=ws),
                                      want_codes=True, want_mask=True, want_params=True,
                                      flags=b.FLAG_WORKSPACE_ZEROED | b.FLAG_FORCE_CLUSTER)
        assert b.workspace_status(ws) == b.OK
        assert_parity(got, orc.fused(x, bits, gy=gy), shape, 1, orc.GROUP_CHANNEL, backward=True)
        assert int(ws.view(torch.int32).abs().sum().item()) == 0
