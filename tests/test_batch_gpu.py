"""granq_fakequant_fused_batch: a list of tensors in one host call.  Every tensor must come out bit for bit as the
oracle computes it (and as the single call does); a bad descriptor stops the batch at its index."""
import numpy as np
import pytest
import torch

from gpu_util import assert_parity, make_case, same_bits, to_dev, to_np
from oracle import granq_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2503_18339_b200 import binding
    binding.lib()
    return binding


SHAPES = [(4, 16, 32, 32), (4, 32, 16, 16), (8, 64, 8, 8), (3, 20, 7, 7), (16, 8, 14, 14), (2, 3, 5, 5)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("backward", [True, False], ids=["fwd+bwd", "fwd"])
def test_batch_matches_the_oracle_and_the_single_calls(b, dtype, backward):
    cases = [make_case(s, seed=100 + i, dtype=dtype, relu=(i % 2 == 0)) for i, s in enumerate(SHAPES)]
    bits = [2 + (i * 3) % 7 for i in range(len(SHAPES))]
    xs = [to_dev(x) for x, _ in cases]
    gys = [to_dev(gy) if backward else None for _, gy in cases]
    batch = b.FusedBatch(list(zip(xs, bits, gys)), want_params=True)
    outs = batch.run()
    torch.cuda.synchronize()
    for i, ((x, gy), o) in enumerate(zip(cases, outs)):
        ref = orc.fused(x, bits[i], gy=gy if backward else None)
        assert b.workspace_status(o.workspace) == b.OK
        assert_parity(o, ref, SHAPES[i], 1, orc.GROUP_CHANNEL, backward=backward)
        single = b.granq_fakequant_fused(xs[i], bits[i], gy=gys[i], want_params=True)
        assert same_bits(to_np(single.y), to_np(o.y)) and same_bits(to_np(single.lo), to_np(o.lo))
        if backward:
            assert same_bits(to_np(single.gx), to_np(o.gx))
    # a second run over the same descriptors (workspaces are left as they were found)
    outs = batch.run()
    torch.cuda.synchronize()
    for i, ((x, gy), o) in enumerate(zip(cases, outs)):
        assert same_bits(to_np(o.y), orc.fused(x, bits[i]).y)


def test_batch_per_sample_groups(b):
    x, gy = make_case((6, 10, 9, 9), seed=7)
    batch = b.FusedBatch([(to_dev(x), 4, to_dev(gy))], group=b.GROUP_SAMPLE_CHANNEL, want_params=True)
    o = batch.run()[0]
    assert_parity(o, orc.fused(x, 4, gy=gy, group_mode=orc.GROUP_SAMPLE_CHANNEL), x.shape, 1, orc.GROUP_SAMPLE_CHANNEL,
                  backward=True)


def test_batch_stops_at_the_bad_descriptor(b):
    xs = [to_dev(make_case(s, seed=i)[0]) for i, s in enumerate(SHAPES[:3])]
    batch = b.FusedBatch([(x, 4, None) for x in xs])
    batch._descs[1].bits = 9                       # out of range: tensor 0 runs, tensor 1 is refused, tensor 2 is not reached
    before = to_np(batch.outs[2].y.fill_(-7.0)).copy()
    with pytest.raises(b.GranqError) as err:
        batch.run()
    assert err.value.status == b.ERR_INVALID_ARG and "tensor 1" in str(err.value)
    torch.cuda.synchronize()
    assert same_bits(to_np(batch.outs[2].y), before)
    assert same_bits(to_np(batch.outs[0].y), orc.fused(to_np(xs[0]), 4).y)
