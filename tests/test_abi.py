"""Host-only checks of the C ABI: the library builds, loads, exports every symbol that
include/granq.h declares, rejects bad arguments before anything is launched, and plans the
staged kernel's waves within the shared-memory budget."""
import ctypes
import os
import random
import re

import pytest

from paper_2503_18339_b200 import build as granq_build
from paper_2503_18339_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    granq_build.build()
    from paper_2503_18339_b200 import binding
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "granq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(granq_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2503_18339_b200 import binding
    names = declared_functions()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_status_strings(lib):
    from paper_2503_18339_b200 import binding
    seen = {binding.status_string(i) for i in range(6)}
    assert len(seen) == 6 and binding.status_string(99) == "unknown status"


def test_geometry_queries(lib):
    from paper_2503_18339_b200 import binding as b
    shape = (8, 16, 7, 7)
    assert b.num_groups(shape, 1, b.GROUP_CHANNEL) == 16
    assert b.num_groups(shape, 1, b.GROUP_SAMPLE_CHANNEL) == 128
    assert b.num_groups(shape, 1, b.GROUP_TENSOR) == 1
    assert b.num_groups(shape, 0, b.GROUP_CHANNEL) == 8
    assert b.workspace_bytes(b.F32, shape) % 256 == 0 and b.workspace_bytes(b.F32, shape) >= 256 + 16 * 12
    assert b.workspace_bytes(7, shape) == 0
    with pytest.raises(ValueError):
        b.num_groups((8, 0, 7, 7))
    with pytest.raises(ValueError):
        b.num_groups((8, 16, 7, 7), channel_axis=4)
    with pytest.raises(ValueError):
        b.num_groups((1 << 20, 1 << 20, 2, 1))       # more than 2^40 elements


def test_argument_errors_are_detected_before_any_launch(lib):
    """Null pointers, bad bit-widths, bad enums and a missing workspace never reach the GPU
    (this runs on a machine without one)."""
    from paper_2503_18339_b200 import binding as b
    dims = (ctypes.c_int64 * 4)(2, 3, 4, 4)
    fake = ctypes.c_void_p(256 * 1024)                # never dereferenced on the host
    far = ctypes.c_void_p(256 * 1024 * 1024)
    r = lib.granq_range(None, b.F32, dims, 1, 0, fake, fake, fake, 4096, 0, None)
    assert r == b.ERR_INVALID_ARG
    r = lib.granq_range(fake, b.F32, dims, 1, 0, fake, fake, None, 0, 0, None)
    assert r == b.ERR_WORKSPACE
    r = lib.granq_range(fake, b.F32, dims, 1, 0, fake, fake, ctypes.c_void_p(256 * 1024 + 8), 4096, 0, None)
    assert r == b.ERR_WORKSPACE                       # misaligned workspace
    r = lib.granq_range(fake, b.F32, dims, 1, 0, fake, fake, fake, 64, 0, None)
    assert r == b.ERR_WORKSPACE                       # too small
    for bits in (0, 9, -1):
        r = lib.granq_fakequant_fwd(fake, b.F32, dims, 1, 0, bits, fake, fake, far, None, None, None, 0, None)
        assert r == b.ERR_INVALID_ARG
    r = lib.granq_fakequant_fwd(fake, 5, dims, 1, 0, 4, fake, fake, far, None, None, None, 0, None)
    assert r == b.ERR_INVALID_ARG                     # bad dtype
    r = lib.granq_fakequant_fwd(fake, b.F32, dims, 1, 3, 4, fake, fake, far, None, None, None, 0, None)
    assert r == b.ERR_INVALID_ARG                     # bad group mode
    r = lib.granq_fakequant_fwd(fake, b.F32, dims, 1, 0, 4, fake, fake, fake, None, None, None, 0, None)
    assert r == b.ERR_INVALID_ARG                     # y overlaps x
    r = lib.granq_fakequant_bwd(fake, far, b.F32, dims, 1, 0, 4, fake, fake, None, None, 0, None)
    assert r == b.ERR_INVALID_ARG                     # gx missing
    # fused: gy without gx, mask without gy
    r = lib.granq_fakequant_fused(fake, far, b.F32, dims, 1, 0, 4, ctypes.c_void_p(3 << 28), None, fake, fake,
                                  None, None, None, None, fake, 4096, 0, None)
    assert r == b.ERR_INVALID_ARG
    r = lib.granq_fakequant_fused(fake, None, b.F32, dims, 1, 0, 4, far, None, fake, fake,
                                  None, fake, None, None, fake, 4096, 0, None)
    assert r == b.ERR_INVALID_ARG
    assert lib.granq_tune(99, 0) == b.ERR_INVALID_ARG
    assert lib.granq_workspace_status(None, None) == b.ERR_INVALID_ARG
    # the later entry points: missing outputs, misaligned buffers, bad bit-widths
    odd = ctypes.c_void_p(3 << 28 | 2)
    r = lib.granq_fakequant_fwd_packmask(fake, b.F32, dims, 1, 0, 4, fake, fake, far, None, None, None, 0, None)
    assert r == b.ERR_INVALID_ARG                     # packed mask missing
    r = lib.granq_fakequant_fwd_packmask(fake, b.F32, dims, 1, 0, 4, fake, fake, far, odd, None, None, 0, None)
    assert r == b.ERR_INVALID_ARG                     # packed mask not on a 4-byte boundary
    r = lib.granq_fakequant_bwd_packmask(fake, ctypes.c_void_p(3 << 28), b.F32, dims, fake, 0, None)
    assert r == b.ERR_INVALID_ARG                     # gx on top of gy
    r = lib.granq_fakequant_fused_fwd_packmask(fake, b.F32, dims, 1, 0, 4, far, ctypes.c_void_p(3 << 28), fake, fake,
                                               None, None, None, 0, 0, None)
    assert r == b.ERR_WORKSPACE
    r = lib.granq_distortion(fake, far, b.F32, dims, odd, 0, None)
    assert r == b.ERR_INVALID_ARG                     # sums not on an 8-byte boundary
    r = lib.granq_fakequant_fused_stats(fake, b.F32, dims, 1, 0, 4, far, fake, fake, None, None, None, fake, 4096, 0,
                                        None)
    assert r == b.ERR_INVALID_ARG                     # sums missing
    r = lib.granq_quantize_packed(fake, b.F32, dims, 1, 0, 9, fake, fake, far, None, fake, fake, 0, None)
    assert r == b.ERR_INVALID_ARG                     # 9 bits
    r = lib.granq_quantize_packed(fake, b.F32, dims, 1, 0, 4, fake, fake, far, None, None, fake, 0, None)
    assert r == b.ERR_INVALID_ARG                     # scale output missing
    r = lib.granq_dequantize_packed(far, b.F32, dims, 1, 0, 4, fake, None, fake, 0, None)
    assert r == b.ERR_INVALID_ARG                     # zero-point missing
    assert b.packmask_bytes((2, 3, 4, 4)) == 12 and b.packed_codes_bytes((2, 3, 4, 4), 3) == 36
    desc = (b.WeightDesc * 1)(b.WeightDesc(256 * 1024, None, 3 << 28, None, 256 * 1024, 256 * 1024, None, None, 4, 8,
                                           0, 0))
    assert lib.granq_fakequant_weights(desc, 1, b.F32, fake, 4096, 0, None) == b.ERR_INVALID_ARG      # 0 bits
    desc[0].bits = 4
    assert lib.granq_fakequant_weights(desc, 1, b.F32, None, 0, 0, None) == b.ERR_WORKSPACE
    assert lib.granq_fakequant_weights(desc, 0, b.F32, fake, 4096, 0, None) == b.ERR_INVALID_ARG
    assert lib.granq_host_arena_status(b.F32, dims, 1, 0, 1, None, None) == b.ERR_INVALID_ARG


def test_binding_refuses_cpu_tensors(lib):
    import torch
    from paper_2503_18339_b200 import binding as b
    x = torch.zeros(2, 3, 4, 4)
    with pytest.raises(ValueError):
        b.granq_fakequant_fused(x, 4, out=b.FakeQuantOut(
            y=torch.empty_like(x), lo=torch.empty(3), hi=torch.empty(3), workspace=torch.empty(4096, dtype=torch.uint8)))


def _check_geometry(shape, dt, grp, geo):
    n, c, h, w = shape
    V = 4 if dt == 0 else 8
    outer, groups = (n, c) if grp == 0 else (1, n * c)
    inner = h * w
    cw, cu, nw = geo["cw"], geo["cu"], geo["nwaves"]
    assert geo["smem_bytes"] <= 232448 and 1 <= geo["depth"] <= 3
    assert (nw - 1) * cw < groups <= nw * cw
    if nw > 1:
        assert (cw * inner) % V == 0                       # every wave's slab starts on a 16-byte boundary
    for ch in ({cw, groups - (nw - 1) * cw} if nw > 1 else {groups}):
        units = ch * inner // V
        cps = -(-units // cu)
        nk = -(-outer * cps // geo["grid"])
        assert nk * cu <= geo["buf_units"], (shape, geo, nk)


def test_staged_plan_fits_the_shared_memory_budget_for_every_workload(lib):
    from paper_2503_18339_b200 import binding as b
    for cfg in range(1, 6):
        for spec in wl.config_tensors(cfg):
            for dt in ([b.F32, b.BF16] if cfg == 5 else [b.F32]):
                for grp in (b.GROUP_CHANNEL, b.GROUP_SAMPLE_CHANNEL):
                    geo = b.staged_geometry(dt, spec.shape, 1, grp)
                    assert geo is not None, (spec.name, dt, grp)
                    _check_geometry(spec.shape, dt, grp, geo)


def test_staged_plan_under_forced_small_buffers(lib):
    from paper_2503_18339_b200 import binding as b
    rnd = random.Random(1)
    planned = 0
    try:
        for _ in range(1500):
            shape = (rnd.randint(1, 9), rnd.randint(1, 40), rnd.choice([1, 2, 4, 7, 8, 14, 28]),
                     rnd.choice([4, 7, 8, 14, 16]))
            dt = rnd.choice([0, 1])
            V = 4 if dt == 0 else 8
            b.tune(b.KNOB_STAGED_DEPTH, rnd.choice([0, 1, 2, 3]))
            b.tune(b.KNOB_STAGED_MAX_BUF_UNITS, rnd.choice([0, 64, 100, 500]))
            grid = rnd.choice([3, 5, 148])
            geo = b.staged_geometry(dt, shape, sm_count=grid)
            if (shape[1] * shape[2] * shape[3]) % V or shape[2] * shape[3] < V:
                assert geo is None
                continue
            if geo is not None:
                planned += 1
                _check_geometry(shape, dt, 0, geo)
    finally:
        for k in range(b.N_KNOBS):
            b.tune(k, 0)
    assert planned > 500


def test_distortion_stats_against_the_oracle_and_closed_forms(lib):
    """Table 2's two statistics from the four sums: the C entry point against the oracle's and against
    closed forms (Q = X, Q = 0, a 3-4-5 pair), and its degenerate cases."""
    from oracle import granq_oracle as orc
    from paper_2503_18339_b200 import binding as b
    assert b.distortion_from_sums([4.0, 4.0, 4.0, 0.0]) == (1.0, 0.0)               # Q = X
    assert b.distortion_from_sums([4.0, 0.0, 0.0, 4.0]) == (0.0, 1.0)               # Q = 0
    assert b.distortion_from_sums([0.0, 0.0, 0.0, 0.0]) == (0.0, 0.0)               # X = 0
    cos, rel = b.distortion_from_sums([9.0, 16.0, 0.0, 25.0])                       # X = (3, 0), Q = (0, 4)
    assert cos == 0.0 and abs(rel - 5.0 / 3.0) < 1e-15
    rnd = random.Random(3)
    for _ in range(50):
        sxx, sqq = rnd.uniform(0.1, 1e6), rnd.uniform(0.1, 1e6)
        sxq = rnd.uniform(-1, 1) * (sxx * sqq) ** 0.5
        sums = [sxx, sqq, sxq, sxx + sqq - 2 * sxq]
        got, want = b.distortion_from_sums(sums), orc.distortion(sums)
        assert abs(got[0] - want[0]) <= 1e-15 * max(1.0, abs(want[0])) and abs(got[1] - want[1]) <= 1e-15 * max(1.0, want[1])
    assert lib.granq_distortion_stats(None, None, None) == b.ERR_INVALID_ARG


def test_cluster_plan_cuts_within_its_limits(lib):
    """Host-only: whatever the cluster-local planner answers respects its own invariants - a run is a whole
    number of 16-byte units in every slab, a CTA's tiles fit the shared memory of an SM twice over (or the
    forced limit), the cluster size is a portable power of two no larger than the number of slabs."""
    from paper_2503_18339_b200 import binding as b
    rnd = random.Random(11)
    planned = 0
    try:
        for _ in range(3000):
            shape = (rnd.choice([1, 2, 3, 8, 13, 64, 128, 256]), rnd.randint(1, 600),
                     rnd.choice([1, 2, 4, 7, 8, 14, 28, 56]), rnd.choice([1, 4, 7, 8, 14, 16, 28, 56]))
            dt, mode, bwd = rnd.choice([0, 1]), rnd.choice([0, 1]), rnd.choice([False, True])
            V, esize = (4, 4) if dt == 0 else (8, 2)
            b.tune(b.KNOB_CLUSTER_CTAS, rnd.choice([0, 0, 0, 1, 2, 4, 8]))
            b.tune(b.KNOB_CLUSTER_TILE_KB, rnd.choice([0, 0, 8, 32, 200]))
            b.tune(b.KNOB_CLUSTER_LOAD, rnd.choice([0, 0, 1, 2, 3, 4, 5]))
            b.tune(b.KNOB_CLUSTER_KMUL, rnd.choice([0, 0, 0, 2, 5]))
            geo = b.cluster_geometry(dt, shape, group=mode, with_backward=bwd)
            inner = shape[2] * shape[3]
            outer, C = (shape[0], shape[1]) if mode == 0 else (1, shape[0] * shape[1])
            if (C * inner) % V or inner < V:
                assert geo is None
                continue
            if geo is None:
                continue
            planned += 1
            k, R = geo["channels_per_run"], geo["cluster"]
            assert (k * inner) % V == 0 and k >= 1
            assert R in (1, 2, 4, 8) and R <= outer
            assert geo["grid"] == -(-C // k) * R
            assert geo["tile_bytes"] == -(-outer // R) * min(k, C if k > C else k) * inner * esize or k > C
            tiles = 2 if geo["staging"] in (2, 4) else 1
            assert tiles == 1 or bwd
            assert geo["smem_bytes"] >= tiles * geo["tile_bytes"] and geo["smem_bytes"] <= 227 * 1024
            assert geo["threads"] % 32 == 0 and 32 <= geo["threads"] <= 512
    finally:
        for k in range(b.N_KNOBS):
            b.tune(k, 0)
    assert planned > 300
