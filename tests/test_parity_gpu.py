"""Parity of the CUDA library with the CPU oracle, through the C ABI, on the same seeded inputs.

Bar: per-group min / max bit-exact, integer codes and STE mask bit-exact, dequantized
outputs within 1e-6 * scale of the oracle's (s, z bit-exact; in practice y and gx are
bit-exact too and the tests say so where that is expected)."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import granq_oracle as orc
from paper_2503_18339_b200 import workloads as wl

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.fixture(scope="module")
def b():
    from paper_2503_18339_b200 import binding
    binding.lib()
    yield binding
    for k in range(binding.N_KNOBS):
        binding.tune(k, 0)


@pytest.fixture()
def knobs(b):
    """Planner overrides that are always reset afterwards."""
    def set_(**kw):
        names = {"depth": b.KNOB_STAGED_DEPTH, "max_buf_units": b.KNOB_STAGED_MAX_BUF_UNITS,
                 "grid": b.KNOB_STAGED_GRID, "spin_limit": b.KNOB_SPIN_LIMIT,
                 "extra_arrivals": b.KNOB_TEST_EXTRA_ARRIVALS, "l2_wave_kb": b.KNOB_L2_WAVE_KB,
                 "l2_upl": b.KNOB_L2_UPL, "l2_ctas_per_sm": b.KNOB_L2_CTAS_PER_SM, "l2_lag": b.KNOB_L2_LAG}
        for k, v in kw.items():
            b.tune(names[k], v)
    yield set_
    for k in range(b.N_KNOBS):
        b.tune(k, 0)


# ---- marshalling helpers -----------------------------------------------------------------------
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
    v = np.uint16 if a.dtype == np.uint16 else np.uint32
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
    """got: binding.FakeQuantOut on the device; ref: oracle FakeQuantResult."""
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


SMALL_SHAPES = [
    (2, 3, 5, 7),        # odd everything, inner % 4 != 0: scalar fallback
    (3, 8, 7, 7),        # 7x7 planes: a 16-byte pack straddles two channels
    (4, 16, 14, 14),     # 196-element planes
    (5, 6, 32, 32),      # several tiles per channel
    (2, 4, 56, 56),
    (1, 1, 1, 37),       # single group, ragged
    (3, 5, 1, 4),        # one pack per plane
    (2, 130, 8, 8),      # many channels
    (9, 12, 20, 20),     # ragged tail inside the last tile
]
MODES = [orc.GROUP_CHANNEL, orc.GROUP_SAMPLE_CHANNEL, orc.GROUP_TENSOR]


# ---- 1. fused entry point, every plan, small and adversarial tensors ---------------------------------
@pytest.mark.parametrize("shape", SMALL_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fused_small_all_plans(b, shape, mode, dtype):
    bits = 2 + (sum(shape) + mode) % 7
    x, gy = make_case(shape, seed=sum(shape) * 7 + mode, dtype=dtype, relu=(shape[0] % 2 == 0))
    ref = orc.fused(x, bits, gy=gy, group_mode=mode)
    for flags in (0, b.FLAG_FORCE_TWO_PASS, b.FLAG_FORCE_NAIVE, b.FLAG_FORCE_L2WAVE, b.FLAG_FORCE_COLWALK,
                  b.FLAG_FORCE_CLUSTER):
        if flags == b.FLAG_FORCE_NAIVE and b.num_groups(shape, 1, mode) > 300:
            continue
        try:
            got = b.granq_fakequant_fused(to_dev(x), bits, gy=to_dev(gy), group=mode, want_codes=True,
                                          want_mask=True, want_params=True, flags=flags)
        except b.GranqError as err:      # the persistent plans do not take every geometry
            assert flags in (b.FLAG_FORCE_L2WAVE, b.FLAG_FORCE_COLWALK, b.FLAG_FORCE_CLUSTER)
            assert err.status == b.ERR_UNSUPPORTED
            continue
        assert b.workspace_status(got.workspace) == b.OK
        assert_parity(got, ref, shape, 1, mode, backward=True)
    # forward only
    ref_f = orc.fused(x, bits, group_mode=mode)
    got = b.granq_fakequant_fused(to_dev(x), bits, group=mode, want_codes=True, want_params=True)
    assert_parity(got, ref_f, shape, 1, mode, backward=False)


@pytest.mark.parametrize("axis", [0, 1, 2, 3])
@pytest.mark.parametrize("mode", MODES)
def test_fused_every_channel_axis(b, axis, mode):
    shape = (6, 5, 8, 12)
    x, gy = make_case(shape, seed=40 + axis)
    ref = orc.fused(x, 4, gy=gy, channel_axis=axis, group_mode=mode)
    for flags in (0, b.FLAG_FORCE_TWO_PASS):
        got = b.granq_fakequant_fused(to_dev(x), 4, gy=to_dev(gy), channel_axis=axis, group=mode, want_codes=True,
                                      want_mask=True, want_params=True, flags=flags)
        assert_parity(got, ref, shape, axis, mode, backward=True)


# ---- 2. the staged plan cut into many waves, every pipeline depth ---------------------------------------
@pytest.mark.parametrize("shape", [(4, 16, 14, 14), (3, 8, 7, 7), (6, 12, 32, 32), (2, 40, 56, 56), (5, 24, 7, 7)],
                         ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("depth", [1, 2, 3])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_staged_multiwave(b, knobs, shape, depth, dtype):
    if dtype == "bf16" and (shape[1] * shape[2] * shape[3]) % 8 != 0:
        pytest.skip("slab not a whole number of 16-byte packs")
    x, gy = make_case(shape, seed=sum(shape), dtype=dtype)
    bits = 3 + depth
    ref = orc.fused(x, bits, gy=gy)
    elt = 4 if dtype == "f32" else 2
    plane_units = max(1, shape[2] * shape[3] * elt // 16)
    grids = (5, 148) if depth > 1 else (148,)
    for grid in grids:
        if depth == 1:
            knobs(depth=1, max_buf_units=0, grid=grid)
        else:
            # buffers so small that the tensor needs many waves (a wave = a few channels)
            per_cta = max(64, shape[0] * plane_units * 4 // grid + 8)
            knobs(depth=depth, max_buf_units=per_cta, grid=grid)
        dt = b.F32 if dtype == "f32" else b.BF16
        plan, _ = b.fused_plan(dt, shape, flags=b.FLAG_FORCE_STAGED)
        assert plan == b.PLAN_STAGED
        got = b.granq_fakequant_fused(to_dev(x), bits, gy=to_dev(gy), want_codes=True, want_mask=True,
                                      want_params=True, flags=b.FLAG_FORCE_STAGED)
        assert b.workspace_status(got.workspace) == b.OK
        assert_parity(got, ref, shape, 1, orc.GROUP_CHANNEL, backward=True)


@pytest.mark.parametrize("shape", [(4, 16, 14, 14), (3, 8, 7, 7), (6, 12, 32, 32), (2, 40, 56, 56), (5, 24, 7, 7)],
                         ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("upl", [2, 4])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_l2wave_multiwave(b, knobs, shape, upl, dtype):
    """The L2-resident-wave plan cut into many small waves (a few channels each)."""
    if dtype == "bf16" and (shape[1] * shape[2] * shape[3]) % 8 != 0:
        pytest.skip("slab not a whole number of 16-byte packs")
    x, gy = make_case(shape, seed=sum(shape) + upl, dtype=dtype)
    bits = 2 + upl
    ref = orc.fused(x, bits, gy=gy)
    ref_f = orc.fused(x, bits)
    for wave_kb, cap in ((1, 1), (8, 0), (0, 0)):
        knobs(l2_wave_kb=wave_kb, l2_upl=upl, l2_ctas_per_sm=cap)
        got = b.granq_fakequant_fused(to_dev(x), bits, gy=to_dev(gy), want_codes=True, want_mask=True,
                                      want_params=True, flags=b.FLAG_FORCE_L2WAVE)
        assert b.workspace_status(got.workspace) == b.OK
        assert_parity(got, ref, shape, 1, orc.GROUP_CHANNEL, backward=True)
        got = b.granq_fakequant_fused(to_dev(x), bits, flags=b.FLAG_FORCE_L2WAVE)      # forward only, no extras
        assert_parity(got, ref_f, shape, 1, orc.GROUP_CHANNEL, backward=False)


def test_l2wave_bounded_wait_reports_timeout(b, knobs):
    shape = (4, 16, 14, 14)
    x, gy = make_case(shape, seed=2)
    knobs(extra_arrivals=1, spin_limit=2000)
    got = b.granq_fakequant_fused(to_dev(x), 4, gy=to_dev(gy), flags=b.FLAG_FORCE_L2WAVE)
    assert b.workspace_status(got.workspace) == b.ERR_TIMEOUT
    knobs(extra_arrivals=0, spin_limit=0)
    got = b.granq_fakequant_fused(to_dev(x), 4, gy=to_dev(gy), want_codes=True, want_mask=True, want_params=True,
                                  flags=b.FLAG_FORCE_L2WAVE)
    assert b.workspace_status(got.workspace) == b.OK
    assert_parity(got, orc.fused(x, 4, gy=gy), shape, 1, orc.GROUP_CHANNEL, backward=True)


@pytest.mark.parametrize("shape", [(8, 16, 14, 14), (9, 8, 7, 7), (16, 12, 32, 32), (8, 40, 56, 56), (13, 24, 7, 7),
                                   (300, 8, 5, 5), (8, 3, 4, 4), (40, 72, 3, 3)],
                         ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_colwalk_multiwave(b, knobs, shape, dtype):
    """The column-walk plan cut into many small waves, every lag, few and many CTAs."""
    if dtype == "bf16" and ((shape[1] * shape[2] * shape[3]) % 8 != 0 or shape[2] * shape[3] < 8):
        pytest.skip("slab not a whole number of 16-byte packs, or planes shorter than a pack")
    x, gy = make_case(shape, seed=sum(shape) + 3, dtype=dtype)
    bits = 2 + sum(shape) % 7
    ref = orc.fused(x, bits, gy=gy)
    ref_f = orc.fused(x, bits)
    for wave_kb, cap, lag in ((1, 1, 1), (1, 0, 2), (8, 0, 3), (0, 0, 0), (2, 2, 1)):
        knobs(l2_wave_kb=wave_kb, l2_ctas_per_sm=cap, l2_lag=lag)
        assert b.fused_plan(b.BF16 if dtype == "bf16" else b.F32, shape, flags=b.FLAG_FORCE_COLWALK)[0] == b.PLAN_COLWALK
        got = b.granq_fakequant_fused(to_dev(x), bits, gy=to_dev(gy), want_codes=True, want_mask=True,
                                      want_params=True, flags=b.FLAG_FORCE_COLWALK)
        assert b.workspace_status(got.workspace) == b.OK
        assert_parity(got, ref, shape, 1, orc.GROUP_CHANNEL, backward=True)
        got = b.granq_fakequant_fused(to_dev(x), bits, flags=b.FLAG_FORCE_COLWALK)      # forward only, no extras
        assert_parity(got, ref_f, shape, 1, orc.GROUP_CHANNEL, backward=False)


def test_colwalk_needs_slabs_to_walk(b):
    """Too few slabs (or the sample-channel / tensor views, which have one): left to the other plans."""
    with pytest.raises(b.GranqError) as err:
        b.granq_fakequant_fused(to_dev(make_case((2, 8, 8, 8), seed=1)[0]), 4, flags=b.FLAG_FORCE_COLWALK)
    assert err.value.status == b.ERR_UNSUPPORTED
    # defaults: groups that fit the shared memory of a cluster go to the cluster-local kernel; larger ones to
    # the column walk when the batch has slabs to walk, else to the L2-resident waves
    assert b.fused_plan(b.F32, (2, 8, 8, 8))[0] == b.PLAN_CLUSTER
    assert b.fused_plan(b.F32, (64, 8, 8, 8), group=b.GROUP_SAMPLE_CHANNEL)[0] == b.PLAN_CLUSTER
    assert b.fused_plan(b.F32, (64, 8, 112, 112))[0] == b.PLAN_COLWALK
    assert b.fused_plan(b.F32, (2, 8, 512, 512))[0] == b.PLAN_L2WAVE
    assert b.fused_plan(b.F32, (64, 8, 2, 2, ))[0] == b.PLAN_CLUSTER


def test_colwalk_workspace_stays_zeroed(b, knobs):
    """FLAG_WORKSPACE_ZEROED: a cleared workspace serves call after call without being cleared again,
    also when plans, shapes sharing the workspace size, bit-widths and wave cuts alternate."""
    shape = (16, 24, 14, 14)
    x, gy = make_case(shape, seed=11)
    x2, gy2 = make_case(shape, seed=12)
    ws = b.make_workspace(to_dev(x), zeroed=True)
    for k, (xx, gg, bits, extra, wave_kb) in enumerate([(x, gy, 4, 0, 0), (x2, gy2, 3, 0, 1), (x, None, 5, 0, 4),
                                                        (x2, gy2, 6, b.FLAG_FORCE_TWO_PASS, 0),
                                                        (x, gy, 2, b.FLAG_FORCE_L2WAVE, 0), (x2, gy2, 8, 0, 2)]):
        knobs(l2_wave_kb=wave_kb)
        out = b.FakeQuantOut(workspace=ws)
        got = b.granq_fakequant_fused(to_dev(xx), bits, gy=None if gg is None else to_dev(gg), out=out,
                                      want_codes=True, want_mask=True, want_params=True,
                                      flags=b.FLAG_WORKSPACE_ZEROED | extra)
        assert b.workspace_status(ws) == b.OK
        assert_parity(got, orc.fused(xx, bits, gy=gg), shape, 1, orc.GROUP_CHANNEL, backward=gg is not None)
        assert int(ws.view(torch.int32).abs().sum().item()) == 0, f"call {k} left the workspace dirty"


def test_colwalk_bounded_wait_reports_timeout(b, knobs):
    shape = (8, 16, 14, 14)
    x, gy = make_case(shape, seed=2)
    knobs(extra_arrivals=1, spin_limit=2000)
    got = b.granq_fakequant_fused(to_dev(x), 4, gy=to_dev(gy), flags=b.FLAG_FORCE_COLWALK)
    assert b.workspace_status(got.workspace) == b.ERR_TIMEOUT
    knobs(extra_arrivals=0, spin_limit=0)
    got = b.granq_fakequant_fused(to_dev(x), 4, gy=to_dev(gy), want_codes=True, want_mask=True, want_params=True,
                                  flags=b.FLAG_FORCE_COLWALK)
    assert b.workspace_status(got.workspace) == b.OK
    assert_parity(got, orc.fused(x, 4, gy=gy), shape, 1, orc.GROUP_CHANNEL, backward=True)


def test_staged_geometry_really_has_many_waves(b, knobs):
    knobs(depth=3, max_buf_units=1000, grid=5)      # 5 CTAs x 1000 units hold 3 of the 12 channels
    geo = b.staged_geometry(b.F32, (6, 12, 32, 32), sm_count=5)
    assert geo is not None and geo["nwaves"] >= 4 and geo["depth"] == 3


# ---- 3. hand-worked cases straight through the GPU ---------------------------------------------------------
with open(os.path.join(HERE, "golden", "hand_cases.json")) as fh:
    HAND = json.load(fh)["cases"]
MODE_OF = {"channel": orc.GROUP_CHANNEL, "sample_channel": orc.GROUP_SAMPLE_CHANNEL, "tensor": orc.GROUP_TENSOR}


@pytest.mark.parametrize("case", HAND, ids=[c["name"] for c in HAND])
def test_hand_cases_on_gpu(b, case):
    f32 = lambda v: np.asarray(v, np.float64).astype(np.float32)
    x = f32(case["x"]).reshape(case["shape"])
    gy = (np.arange(x.size, dtype=np.float32) + 1).reshape(x.shape)
    mode = MODE_OF[case["group_mode"]]
    if case.get("given_range"):
        lo, hi = to_dev(f32(case["lo"])), to_dev(f32(case["hi"]))
        fw = b.granq_fakequant_fwd(to_dev(x), case["bits"], lo, hi, group=mode, want_codes=True, want_params=True)
        bw = b.granq_fakequant_bwd(to_dev(gy), to_dev(x), case["bits"], lo, hi, group=mode, want_mask=True)
        y, codes, s, z, gx, mask = fw.y, fw.codes, fw.s, fw.z, bw.gx, bw.mask
    else:
        o = b.granq_fakequant_fused(to_dev(x), case["bits"], gy=to_dev(gy), group=mode, want_codes=True,
                                    want_mask=True, want_params=True)
        assert same_bits(to_np(o.lo), f32(case["lo"])) and same_bits(to_np(o.hi), f32(case["hi"]))
        y, codes, s, z, gx, mask = o.y, o.codes, o.s, o.z, o.gx, o.mask
    assert same_bits(to_np(s), f32(case["s"])) and same_bits(to_np(z), f32(case["z"]))
    assert to_np(codes).ravel().tolist() == case["codes"]
    assert to_np(mask).ravel().tolist() == case["mask"]
    assert same_bits(to_np(y).ravel(), f32(case["y"]))
    assert same_bits(to_np(gx).ravel(), np.where(np.array(case["mask"]) == 1, gy.ravel(), np.float32(0)))


# ---- 4. stand-alone entry points with a stale range (both clamp sides active) --------------------------------
@pytest.mark.parametrize("shape", [(3, 8, 7, 7), (4, 6, 32, 32), (2, 3, 5, 7)], ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_range_fwd_bwd_with_stale_range(b, shape, mode, dtype):
    x, gy = make_case(shape, seed=11 + mode, dtype=dtype)
    other, _ = make_case(shape, seed=99, dtype=dtype)
    lo_ref, hi_ref = orc.range_(other, group_mode=mode)
    lo, hi = b.granq_range(to_dev(other), group=mode)
    assert same_bits(to_np(lo), lo_ref) and same_bits(to_np(hi), hi_ref)
    # a narrower range than the data: plenty of clamped elements on both sides
    lo_n = (lo_ref * np.float32(0.5)).astype(np.float32)
    hi_n = (hi_ref * np.float32(0.5)).astype(np.float32)
    ref = orc.fakequant(x, 3, lo_n, hi_n, gy=gy, group_mode=mode)
    assert 0 < ref.mask.mean() < 1
    fw = b.granq_fakequant_fwd(to_dev(x), 3, to_dev(lo_n), to_dev(hi_n), group=mode, want_codes=True, want_params=True)
    bw = b.granq_fakequant_bwd(to_dev(gy), to_dev(x), 3, to_dev(lo_n), to_dev(hi_n), group=mode, want_mask=True)
    fw.lo = fw.hi = None
    assert_parity(fw, ref, shape, 1, mode, backward=False)
    assert np.array_equal(to_np(bw.mask), ref.mask) and same_bits(to_np(bw.gx), ref.gx)


# ---- 5. misaligned base pointers, degenerate groups, extremes ----------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_unaligned_base_pointers(b, dtype):
    shape = (3, 4, 8, 8)
    x, gy = make_case(shape, seed=5, dtype=dtype)
    ref = orc.fused(x, 4, gy=gy)

    def shifted(a):     # same values one element past a 16-byte boundary
        t = to_dev(np.concatenate([a.ravel()[:1], a.ravel()]))
        return t[1:].view(shape)

    xd, gyd = shifted(x), shifted(gy)
    assert xd.data_ptr() % 16 != 0
    out = b.FakeQuantOut(y=shifted(np.zeros_like(x)), gx=shifted(np.zeros_like(x)))
    got = b.granq_fakequant_fused(xd, 4, gy=gyd, out=out, want_codes=True, want_mask=True, want_params=True)
    assert_parity(got, ref, shape, 1, orc.GROUP_CHANNEL, backward=True)


def test_constant_zero_and_outlier_groups(b):
    shape = (4, 8, 14, 14)
    x, gy = make_case(shape, seed=3, relu=True)
    x[:, 0] = 0.0                  # dead channel: s floored at 1e-8
    x[:, 1] = 3.7                  # non-zero constant channel
    x[:, 2] = -100.0
    x[:, 3] = np.minimum(x[:, 3] * 50, 6.0)     # saturating channel: many ties at the maximum
    x[1, 4, 2, 3] = 3.0e38         # huge outlier
    x[:, 5] *= np.float32(1e-30)   # tiny values
    for bits in (1, 3, 8):
        ref = orc.fused(x, bits, gy=gy)
        for flags in (0, b.FLAG_FORCE_TWO_PASS, b.FLAG_FORCE_NAIVE):
            got = b.granq_fakequant_fused(to_dev(x), bits, gy=to_dev(gy), want_codes=True, want_mask=True,
                                          want_params=True, flags=flags)
            assert_parity(got, ref, shape, 1, orc.GROUP_CHANNEL, backward=True)


def test_results_are_deterministic(b):
    shape = (8, 32, 28, 28)
    x, gy = make_case(shape, seed=8)
    xd, gyd = to_dev(x), to_dev(gy)
    first = b.granq_fakequant_fused(xd, 4, gy=gyd)
    y0, g0 = first.y.clone(), first.gx.clone()
    for _ in range(5):
        again = b.granq_fakequant_fused(xd, 4, gy=gyd)
        assert torch.equal(again.y, y0) and torch.equal(again.gx, g0)


def test_non_default_stream(b):
    shape = (4, 16, 14, 14)
    x, gy = make_case(shape, seed=9)
    ref = orc.fused(x, 5, gy=gy)
    st = torch.cuda.Stream()
    xd, gyd = to_dev(x), to_dev(gy)
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        got = b.granq_fakequant_fused(xd, 5, gy=gyd, want_codes=True, want_mask=True, want_params=True, stream=st)
    st.synchronize()
    assert_parity(got, ref, shape, 1, orc.GROUP_CHANNEL, backward=True)


def test_more_than_2_to_the_31_elements(b):
    """Index arithmetic beyond 32 bits: a bf16 tensor of 2^31 + 2^21 elements through the range,
    forward and fused entry points, every element compared with the oracle."""
    shape = (2, 4, 16384, 16400)
    n = int(np.prod(shape, dtype=np.int64))
    assert n > 2 ** 31
    rng = np.random.default_rng(31)
    # bf16 bit patterns of finite values in about [-4, 4): sign + exponent 120..128 + 7 mantissa bits
    xb = (rng.integers(120, 129, n, dtype=np.uint16) << 7) | rng.integers(0, 128, n, dtype=np.uint16)
    xb |= rng.integers(0, 2, n, dtype=np.uint16) << 15
    xb = xb.reshape(shape)
    xd = to_dev(xb)
    lo_ref, hi_ref = orc.range_(xb)
    lo, hi = b.granq_range(xd)
    assert same_bits(to_np(lo), lo_ref) and same_bits(to_np(hi), hi_ref)
    ref = orc.fakequant(xb, 4, lo_ref, hi_ref)
    fw = b.granq_fakequant_fwd(xd, 4, lo, hi, want_codes=True)
    assert np.array_equal(to_np(fw.codes), ref.codes) and same_bits(to_np(fw.y), ref.y)
    del fw
    got = b.granq_fakequant_fused(xd, 4, want_codes=True)
    assert b.workspace_status(got.workspace) == b.OK
    assert same_bits(to_np(got.lo), lo_ref) and same_bits(to_np(got.hi), hi_ref)
    assert np.array_equal(to_np(got.codes), ref.codes) and same_bits(to_np(got.y), ref.y)


# ---- 6. the bounded device-side wait gives up cleanly ------------------------------------------------------------
def test_bounded_wait_reports_timeout_and_context_survives(b, knobs):
    """A wave is told to wait for one arrival more than the grid can provide, with a short
    iteration limit: the kernel must stop by itself, report GRANQ_ERR_TIMEOUT, and leave the
    context usable."""
    shape = (4, 16, 14, 14)
    x, gy = make_case(shape, seed=2)
    knobs(extra_arrivals=1, spin_limit=2000)
    got = b.granq_fakequant_fused(to_dev(x), 4, gy=to_dev(gy), flags=b.FLAG_FORCE_STAGED)
    assert b.workspace_status(got.workspace) == b.ERR_TIMEOUT
    knobs(extra_arrivals=0, spin_limit=0)
    ref = orc.fused(x, 4, gy=gy)
    got = b.granq_fakequant_fused(to_dev(x), 4, gy=to_dev(gy), want_codes=True, want_mask=True, want_params=True,
                                  flags=b.FLAG_FORCE_STAGED)
    assert b.workspace_status(got.workspace) == b.OK
    assert_parity(got, ref, shape, 1, orc.GROUP_CHANNEL, backward=True)


# ---- 6b. the staged kernel's division is IEEE division ---------------------------------------------------------
def test_reciprocal_division_matches_ieee_division(b):
    for seed in range(4):
        assert b.selftest_division(1 << 30, seed) == 0


# ---- 7. host-buffer entry point --------------------------------------------------------------------------------------
def test_fused_host_entry_point(b):
    shape = (8, 16, 14, 14)
    x, gy = make_case(shape, seed=13)
    ref = orc.fused(x, 4, gy=gy)
    xh, gyh = torch.from_numpy(x).pin_memory(), torch.from_numpy(gy).pin_memory()
    yh, gxh = torch.empty_like(xh).pin_memory(), torch.empty_like(xh).pin_memory()
    lo, hi, s, z = (torch.empty(16).pin_memory() for _ in range(4))
    arena = torch.empty(b.host_arena_bytes(b.F32, shape), dtype=torch.uint8, device="cuda")
    b.granq_fakequant_fused_host(xh, 4, gyh, yh, gxh, lo, hi, arena, s=s, z=z)
    assert same_bits(lo.numpy(), ref.lo) and same_bits(hi.numpy(), ref.hi)
    assert same_bits(s.numpy(), ref.s) and same_bits(z.numpy(), ref.z)
    assert same_bits(yh.numpy(), ref.y) and same_bits(gxh.numpy(), ref.gx)
