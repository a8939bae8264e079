"""GPU parity of the mask-carrying split of forward and backward (Section 2.1) against the CPU
oracle: the packed 1-bit mask bit for bit, y within 1e-6 * s (asserted bit-exact), gx bit for bit."""
import numpy as np
import pytest
import torch

from oracle import granq_oracle as orc
from paper_2503_18339_b200 import workloads as wl
from test_parity_gpu import assert_parity, b, knobs, make_case, same_bits, to_dev, to_np  # noqa: F401

pytestmark = pytest.mark.gpu

SHAPES = [
    (2, 2, 2, 2),        # 16 elements: half a mask word
    (1, 1, 1, 9),        # scalar path, one partial word
    (3, 5, 7, 7),        # 735 elements, ragged planes, scalar path
    (4, 16, 14, 14),     # vector path
    (16, 8, 7, 7),       # 7x7 planes, slab of 392 elements = 49 bytes of mask: cluster plan, else two-pass
    (3, 8, 7, 7),        # the same with a last mask word that is half padding
    (16, 32, 7, 7),      # 7x7 planes, slab of 1568 = 49 words: column walk with 32-channel waves
    (9, 24, 12, 12),     # column walk, aligned planes
    (8, 3, 4, 4),        # 48 elements per slab
    (33, 6, 40, 28),     # long planes, odd batch
    (5, 7, 3, 11),       # nothing aligned
]


def packed_ref(mask: np.ndarray) -> np.ndarray:
    """The oracle's packed mask padded with zero bytes to whole 32-bit words."""
    p = orc.pack_mask(mask)
    out = np.zeros((mask.size + 31) // 32 * 4, np.uint8)
    out[:p.size] = p
    return out


def packed_np(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint8)


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fwd_packmask_then_bwd_packmask(b, shape, dtype):
    """Stale, narrower range so both clamp sides are live; every grouping mode."""
    x, gy = make_case(shape, seed=sum(shape) + 1, dtype=dtype)
    for mode in (orc.GROUP_CHANNEL, orc.GROUP_SAMPLE_CHANNEL, orc.GROUP_TENSOR):
        bits = 2 + (sum(shape) + mode) % 7
        lo, hi = orc.range_(x, group_mode=mode)
        lo2 = (lo + 0.2 * (hi - lo)).astype(np.float32)
        hi2 = (lo + 0.7 * (hi - lo)).astype(np.float32)
        ref = orc.fakequant(x, bits, lo2, hi2, gy=gy, group_mode=mode)
        if x.size > 64:
            assert 0 < ref.mask.sum() < ref.mask.size
        got = b.granq_fakequant_fwd_packmask(to_dev(x), bits, to_dev(lo2), to_dev(hi2), group=mode, want_params=True)
        assert_parity(got, ref, shape, 1, mode, backward=False)
        assert np.array_equal(packed_np(got.packed_mask), packed_ref(ref.mask)), "packed mask differs"
        gx = b.granq_fakequant_bwd_packmask(to_dev(gy), got.packed_mask)
        assert same_bits(to_np(gx), ref.gx), "gx from the packed mask differs"
        assert same_bits(to_np(gx), orc.bwd_packed(gy, orc.pack_mask(ref.mask)))


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fused_fwd_packmask(b, knobs, shape, dtype):
    """Range of the tensor itself (mask all ones except at ties), both plans, small waves."""
    x, gy = make_case(shape, seed=sum(shape) + 2, dtype=dtype, relu=(shape[0] % 2 == 0))
    bits = 2 + sum(shape) % 7
    ref = orc.fused(x, bits, gy=gy)
    expect = packed_ref(ref.mask)
    dt = b.BF16 if dtype == "bf16" else b.F32
    for flags, wave_kb in ((0, 0), (b.FLAG_FORCE_TWO_PASS, 0), (b.FLAG_FORCE_COLWALK, 1), (b.FLAG_FORCE_COLWALK, 0),
                           (b.FLAG_FORCE_CLUSTER, 0), (b.FLAG_FORCE_CLUSTER, 2)):
        knobs(l2_wave_kb=wave_kb)
        if flags == b.FLAG_FORCE_CLUSTER:
            b.tune(b.KNOB_CLUSTER_CTAS, wave_kb)          # the cluster plan: automatic cut, then clusters of 2
        try:
            got = b.granq_fakequant_fused_fwd_packmask(to_dev(x), bits, want_params=True, flags=flags)
        except b.GranqError as err:
            assert flags in (b.FLAG_FORCE_COLWALK, b.FLAG_FORCE_CLUSTER) and err.status == b.ERR_UNSUPPORTED
            continue
        finally:
            b.tune(b.KNOB_CLUSTER_CTAS, 0)
        assert b.workspace_status(got.workspace) == b.OK
        assert_parity(got, ref, shape, 1, orc.GROUP_CHANNEL, backward=False)
        assert np.array_equal(packed_np(got.packed_mask), expect), f"packed mask differs (flags {flags})"
        gx = b.granq_fakequant_bwd_packmask(to_dev(gy), got.packed_mask)
        assert same_bits(to_np(gx), ref.gx)
    # the column walk must really be taken where slabs and waves are whole mask words, the cluster plan where
    # slabs are whole bytes of mask
    wide = shape[2] * shape[3] >= (8 if dtype == "bf16" else 4)
    if shape[0] >= 8 and (shape[1] * shape[2] * shape[3]) % 32 == 0 and wide:
        b.granq_fakequant_fused_fwd_packmask(to_dev(x), bits, flags=b.FLAG_FORCE_COLWALK)
    if (shape[1] * shape[2] * shape[3]) % 8 == 0 and wide:
        b.granq_fakequant_fused_fwd_packmask(to_dev(x), bits, flags=b.FLAG_FORCE_CLUSTER)


def test_packmask_rejects_bad_arguments(b):
    x = to_dev(make_case((2, 4, 4, 4), seed=1)[0])
    lo = torch.zeros(4, device="cuda")
    hi = torch.ones(4, device="cuda")
    pm = torch.empty(b.packmask_bytes(x.shape) + 4, dtype=torch.uint8, device="cuda")
    with pytest.raises(b.GranqError) as err:      # packed mask not on a 4-byte boundary
        b.granq_fakequant_fwd_packmask(x, 4, lo, hi, packed_mask=pm[1:])
    assert err.value.status == b.ERR_INVALID_ARG
    with pytest.raises(b.GranqError) as err:      # gx on top of gy
        b.granq_fakequant_bwd_packmask(x, b.make_packed_mask(x), gx=x)
    assert err.value.status == b.ERR_INVALID_ARG
    assert b.packmask_bytes((2, 4, 4, 4)) == 16 and b.packmask_bytes((1, 1, 1, 33)) == 8


@pytest.mark.parametrize("spec", wl.config_tensors(3) + wl.config_tensors(4), ids=lambda s: s.name)
def test_packmask_configs_3_4_full_size(b, spec):
    """Every element of the benchmarked tensors: fused forward with packed mask, then backward from it."""
    x, gy = wl.make_activation(spec), wl.make_upstream_grad(spec)
    bits = spec.bits[0]
    ref = orc.fused(x, bits, gy=gy)
    got = b.granq_fakequant_fused_fwd_packmask(to_dev(x), bits, want_params=True)
    assert b.workspace_status(got.workspace) == b.OK
    assert same_bits(to_np(got.lo), ref.lo) and same_bits(to_np(got.hi), ref.hi)
    assert same_bits(to_np(got.s), ref.s) and same_bits(to_np(got.z), ref.z)
    assert same_bits(to_np(got.y), ref.y)
    assert np.array_equal(packed_np(got.packed_mask), packed_ref(ref.mask))
    gx = b.granq_fakequant_bwd_packmask(to_dev(gy), got.packed_mask)
    assert same_bits(to_np(gx), ref.gx)


def test_wave_cut_of_the_packed_mask_call_is_its_own(b):
    """The planner remembers wave cuts per geometry; the cut of a call with a packed mask (waves of whole
    mask words) must not be the one remembered for a call without (waves of whole 16-byte packs).
    [256,1024,14,14]: several waves, 196-element planes, so the two cuts differ."""
    spec = wl.config_tensors(5)[2]
    x, gy = wl.make_activation(spec), wl.make_upstream_grad(spec)
    ref = orc.fused(x, 4, gy=gy, want_codes=True)
    dx = to_dev(x)
    first = b.granq_fakequant_fused(dx, 4, gy=to_dev(gy))                     # remembers the plain cut
    assert same_bits(to_np(first.y), ref.y)
    got = b.granq_fakequant_fused_fwd_packmask(dx, 4, flags=b.FLAG_FORCE_COLWALK)
    assert b.workspace_status(got.workspace) == b.OK
    assert same_bits(to_np(got.y), ref.y)
    assert np.array_equal(packed_np(got.packed_mask), packed_ref(ref.mask))



def test_batch_sharded_step_on_one_rank_equals_the_fused_path(b):
    """data_parallel.fakequant_forward / fakequant_backward (range -> exchange -> forward with packed mask,
    backward from the mask) with a single rank, where the exchange is a no-op: the fused path's results."""
    from paper_2503_18339_b200 import data_parallel as dp
    shape = (16, 24, 14, 14)
    x, gy = make_case(shape, seed=31)
    ref = orc.fused(x, 4, gy=gy)
    fwd = dp.fakequant_forward(to_dev(x), 4)
    assert same_bits(to_np(fwd.lo), ref.lo) and same_bits(to_np(fwd.hi), ref.hi) and same_bits(to_np(fwd.y), ref.y)
    assert same_bits(to_np(dp.fakequant_backward(to_dev(gy), fwd.packed_mask)), ref.gx)
    # the same on a stream that is not the current one (the exchange is ordered on that stream too)
    import torch
    st = torch.cuda.Stream()
    xd, gyd = to_dev(x), to_dev(gy)
    torch.cuda.synchronize()
    fwd = dp.fakequant_forward(xd, 4, stream=st)
    gx = dp.fakequant_backward(gyd, fwd.packed_mask, stream=st)
    st.synchronize()
    assert same_bits(to_np(fwd.lo), ref.lo) and same_bits(to_np(fwd.y), ref.y) and same_bits(to_np(gx), ref.gx)
