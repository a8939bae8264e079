"""Pins for the CPU oracle: every expected value here comes from the paper's equations
worked by hand, a closed form, exact rational arithmetic or an invariant - never from
running the oracle (or any other implementation) to produce it."""
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import granq_oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))
MODES = {"channel": orc.GROUP_CHANNEL, "sample_channel": orc.GROUP_SAMPLE_CHANNEL, "tensor": orc.GROUP_TENSOR}


def f32(v):
    return np.asarray(v, dtype=np.float64).astype(np.float32)


def bits_eq(a, b):
    a = np.ascontiguousarray(a, np.float32).view(np.uint32)
    b = np.ascontiguousarray(b, np.float32).view(np.uint32)
    return np.array_equal(a, b)


# --------------------------------------------------------------------------------------
# 1. hand-worked cases (tests/golden/hand_cases.json; derivations are in the file)
# --------------------------------------------------------------------------------------
with open(os.path.join(HERE, "golden", "hand_cases.json")) as fh:
    HAND = json.load(fh)["cases"]


@pytest.mark.parametrize("case", HAND, ids=[c["name"] for c in HAND])
def test_hand_case(case):
    x = f32(case["x"]).reshape(case["shape"])
    mode = MODES[case["group_mode"]]
    gy = (np.arange(x.size, dtype=np.float32) + 1).reshape(x.shape)   # distinct, non-zero
    if case.get("given_range"):
        res = orc.fakequant(x, case["bits"], f32(case["lo"]), f32(case["hi"]), gy=gy,
                            channel_axis=case["channel_axis"], group_mode=mode)
    else:
        res = orc.fused(x, case["bits"], gy=gy, channel_axis=case["channel_axis"], group_mode=mode)
        assert bits_eq(res.lo, f32(case["lo"])) and bits_eq(res.hi, f32(case["hi"]))
    assert bits_eq(res.s, f32(case["s"]))
    assert bits_eq(res.z, f32(case["z"]))
    assert res.codes.ravel().tolist() == case["codes"]
    assert res.mask.ravel().tolist() == case["mask"]
    assert bits_eq(res.y.ravel(), f32(case["y"])), (res.y.ravel(), case["y"])
    want_gx = np.where(np.array(case["mask"]) == 1, gy.ravel(), np.float32(0))
    assert bits_eq(res.gx.ravel(), want_gx)


# --------------------------------------------------------------------------------------
# 2. closed forms for Eq. 2 / Eq. 5
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("bits", range(1, 9))
@pytest.mark.parametrize("k", [-6, -1, 0, 3])
def test_params_closed_form(bits, k):
    qmax = (1 << bits) - 1
    step = 2.0 ** k
    m = np.array([0, 1, 5, 17, 100], dtype=np.float64)
    lo = f32(-m * step)
    hi = f32(-m * step + qmax * step)        # exactly representable: small integers x power of two
    s, z = orc.params(lo, hi, bits)
    assert bits_eq(s, f32(np.full(m.size, step)))
    assert bits_eq(z, f32(m))


def test_params_degenerate_range_is_floored():
    lo = f32([0.0, 3.7, -100.0, -0.0])
    s, z = orc.params(lo, lo.copy(), 3)
    assert bits_eq(s, f32([1e-8] * 4))
    assert z[0] == 0 and not np.signbit(z[0])
    assert z[3] == 0 and not np.signbit(z[3])
    # z = round(-lo / 1e-8): the quotient is already an integer-valued float
    assert z[1] == np.float32(-3.7) / np.float32(1e-8)
    assert z[2] == np.float32(100.0) / np.float32(1e-8)


@pytest.mark.parametrize("c", [3.7, -100.0, 1e-3, 250.0])
def test_constant_group_reconstructs_itself(c):
    x = np.full((2, 1, 3, 3), c, np.float32)
    res = orc.fused(x, 3)
    assert (res.codes == 0).all() and (res.mask == 1).all()
    ulp = np.spacing(np.float32(abs(c)))
    assert np.all(np.abs(res.y - np.float32(c)) <= 2 * ulp)


# --------------------------------------------------------------------------------------
# 3. exact rational arithmetic with explicit IEEE rounding (an independent evaluator)
# --------------------------------------------------------------------------------------
def rne_f32(q: Fraction) -> Fraction:
    """Round an exact rational to the nearest fp32 (ties to even); normal range only."""
    if q == 0:
        return Fraction(0)
    sign = -1 if q < 0 else 1
    a = abs(q)
    e = math.floor(math.log2(a))
    while Fraction(2) ** e > a:
        e -= 1
    while Fraction(2) ** (e + 1) <= a:
        e += 1
    assert -126 <= e <= 127
    ulp = Fraction(2) ** (e - 23)
    n = a / ulp
    fl = n.numerator // n.denominator
    rem = n - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return sign * fl * ulp


def rne_int(q: Fraction) -> int:
    fl = q.numerator // q.denominator
    rem = q - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return fl


def exact_reference(x, groups, bits, lo_hi=None):
    """Eq. 1, 2, 4, 6 over python Fractions; x: list of exact fp32 values; groups: list of index lists."""
    qmax = (1 << bits) - 1
    out = {}
    for g, idx in enumerate(groups):
        vals = [Fraction(float(x[i])) for i in idx]
        lo, hi = (min(vals), max(vals)) if lo_hi is None else (Fraction(float(lo_hi[0][g])), Fraction(float(lo_hi[1][g])))
        s = rne_f32(rne_f32(hi - lo) / qmax)
        s = max(s, Fraction(float(np.float32(1e-8))))
        z = Fraction(rne_int(rne_f32(-lo / s)))
        for i, v in zip(idx, vals):
            u = rne_f32(rne_f32(v / s) + z)
            r = rne_int(u)
            code = min(max(r, 0), qmax)
            y = rne_f32(s * rne_f32(code - z))
            out[i] = (code, int(0 <= r <= qmax), y, lo, hi, s, z, g)
    return out


def groups_of(shape, axis, mode):
    outer = int(np.prod(shape[:axis], dtype=np.int64))
    C = shape[axis]
    inner = int(np.prod(shape[axis + 1:], dtype=np.int64))
    G = {orc.GROUP_CHANNEL: C, orc.GROUP_SAMPLE_CHANNEL: outer * C, orc.GROUP_TENSOR: 1}[mode]
    groups = [[] for _ in range(G)]
    for o in range(outer):
        for c in range(C):
            g = {orc.GROUP_CHANNEL: c, orc.GROUP_SAMPLE_CHANNEL: o * C + c, orc.GROUP_TENSOR: 0}[mode]
            groups[g].extend(range((o * C + c) * inner, (o * C + c + 1) * inner))
    return groups


@pytest.mark.parametrize("mode", list(MODES.values()))
@pytest.mark.parametrize("axis", [0, 1, 2])
@pytest.mark.parametrize("bits", [1, 2, 3, 5, 8])
def test_exact_rational_small_tensors(mode, axis, bits):
    rng = np.random.default_rng(100 * bits + 10 * axis + mode)
    shape = (3, 4, 2, 5)
    x = (rng.standard_normal(shape) * np.exp(rng.standard_normal((1, 4, 1, 1)))).astype(np.float32)
    if bits == 3:
        x = np.maximum(x, 0) + np.float32(0)
    gy = rng.standard_normal(shape).astype(np.float32)
    res = orc.fused(x, bits, gy=gy, channel_axis=axis, group_mode=mode)
    ref = exact_reference(x.ravel(), groups_of(shape, axis, mode), bits)
    for i, (code, mask, y, lo, hi, s, z, g) in ref.items():
        assert Fraction(float(res.lo[g])) == lo and Fraction(float(res.hi[g])) == hi
        assert Fraction(float(res.s[g])) == s and Fraction(float(res.z[g])) == z
        assert int(res.codes.ravel()[i]) == code
        assert int(res.mask.ravel()[i]) == mask
        assert Fraction(float(res.y.ravel()[i])) == y
        assert res.gx.ravel()[i] == (gy.ravel()[i] if mask else 0.0)


def test_exact_rational_stale_range_hits_both_clamp_sides():
    rng = np.random.default_rng(7)
    shape = (2, 3, 4, 4)
    x = rng.standard_normal(shape).astype(np.float32)
    lo0, hi0 = orc.range_(x)
    lo = (lo0 + np.float32(0.3) * (hi0 - lo0)).astype(np.float32)
    hi = (lo0 + np.float32(0.6) * (hi0 - lo0)).astype(np.float32)
    gy = rng.standard_normal(shape).astype(np.float32)
    res = orc.fakequant(x, 3, lo, hi, gy=gy)
    ref = exact_reference(x.ravel(), groups_of(shape, 1, orc.GROUP_CHANNEL), 3, lo_hi=(lo, hi))
    masks = []
    for i, (code, mask, y, *_rest) in ref.items():
        assert int(res.codes.ravel()[i]) == code and int(res.mask.ravel()[i]) == mask
        assert Fraction(float(res.y.ravel()[i])) == y
        masks.append(mask)
    assert 0 < sum(masks) < len(masks)
    assert (res.codes[res.mask == 0] == 0).any() and (res.codes[res.mask == 0] == 7).any()


# --------------------------------------------------------------------------------------
# 4. invariants of the definition
# --------------------------------------------------------------------------------------
def _spread_tensor(seed, shape=(4, 6, 7, 7), relu=True):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal(shape) * np.exp(rng.standard_normal((1, shape[1], 1, 1)))
    x = x.astype(np.float32)
    return (np.maximum(x, 0) + np.float32(0)) if relu else x


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("relu", [True, False])
def test_invariants(bits, relu):
    qmax = (1 << bits) - 1
    x = _spread_tensor(bits, relu=relu)
    gy = np.random.default_rng(1).standard_normal(x.shape).astype(np.float32)
    res = orc.fused(x, bits, gy=gy)
    C = x.shape[1]
    assert res.codes.max() <= qmax
    for c in range(C):
        xc, cc, yc = x[:, c].ravel(), res.codes[:, c].ravel(), res.y[:, c].ravel()
        s, z = float(res.s[c]), float(res.z[c])
        assert res.lo[c] == xc.min() and res.hi[c] == xc.max()
        # the minimum always lands on code 0; the maximum on the top code (or one below at a tie in z)
        assert cc[np.argmin(xc)] == 0
        top = cc[np.argmax(xc)]
        assert top == qmax if relu else top in (qmax - 1, qmax)
        # monotone: sorting by x sorts the codes
        order = np.argsort(xc, kind="stable")
        assert np.all(np.diff(cc[order].astype(np.int32)) >= 0)
        # y = s * k for an integer k, at most qmax + 1 distinct values
        assert len(np.unique(yc)) <= qmax + 1
        # rounding error at most half a step wherever the clamp was inactive
        inside = res.mask[:, c].ravel() == 1
        assert np.all(np.abs(yc[inside].astype(np.float64) - xc[inside]) <= 0.5 * s * (1 + 1e-5) + 1e-30)
        assert np.all(np.abs(yc.astype(np.float64) - xc) <= s * (1 + 1e-5) + 1e-30)
    # backward: pass-through or zero, and zero exactly where the mask is zero
    assert np.array_equal(res.gx, np.where(res.mask == 1, gy, np.float32(0)))
    # idempotence with the same (lo, hi): quantizing y again returns y
    again = orc.fakequant(res.y, bits, res.lo, res.hi)
    assert bits_eq(again.y, res.y) and np.array_equal(again.codes, res.codes)


def test_mask_is_clamp_inactive_and_both_sides_seen():
    x = _spread_tensor(3, relu=False)
    lo0, hi0 = orc.range_(x)
    lo = (lo0 * np.float32(0.25)).astype(np.float32)
    hi = (hi0 * np.float32(0.25)).astype(np.float32)
    res = orc.fakequant(x, 4, lo, hi, gy=np.ones_like(x))
    for c in range(x.shape[1]):
        s, z = np.float64(res.s[c]), np.float64(res.z[c])
        u = x[:, c].astype(np.float64) / s + z
        far_low, far_high = u < -0.51, u > 15.51       # clearly outside: mask must be 0
        inner = (u > 0.51) & (u < 14.49)               # clearly inside: mask must be 1
        m = res.mask[:, c]
        assert (m[far_low] == 0).all() and (m[far_high] == 0).all() and (m[inner] == 1).all()
        assert (res.codes[:, c][far_low] == 0).all() and (res.codes[:, c][far_high] == 15).all()
        assert far_low.any() and far_high.any()
    assert np.array_equal(res.gx, res.mask.astype(np.float32))


def test_range_is_permutation_invariant_and_handles_signed_zero():
    x = _spread_tensor(11, relu=False)
    rng = np.random.default_rng(0)
    xp = x.copy()
    for c in range(x.shape[1]):                     # shuffle the members of every channel group
        v = xp[:, c].ravel()
        rng.shuffle(v)
        xp[:, c] = v.reshape(xp[:, c].shape)
    lo, hi = orc.range_(x)
    lop, hip = orc.range_(xp)
    assert bits_eq(lo, lop) and bits_eq(hi, hip)
    zeros = np.array([-0.0, 0.0, -0.0, -0.0], np.float32).reshape(1, 1, 2, 2)
    lo, hi = orc.range_(zeros)
    assert not np.signbit(lo[0]) and not np.signbit(hi[0])
    one = np.array([5.5], np.float32).reshape(1, 1, 1, 1)
    lo, hi = orc.range_(one)
    assert lo[0] == hi[0] == np.float32(5.5)


def test_non_finite_input_is_rejected():
    x = np.zeros((1, 2, 2, 2), np.float32)
    x[0, 1, 0, 1] = np.inf
    with pytest.raises(RuntimeError):
        orc.range_(x)


# --------------------------------------------------------------------------------------
# 5. layer-wise special case and group geometry
# --------------------------------------------------------------------------------------
def test_tensor_mode_is_channel_mode_with_one_channel():
    x = _spread_tensor(5, relu=False)
    t = orc.fused(x, 4, group_mode=orc.GROUP_TENSOR)
    flat = x.reshape(1, 1, 1, -1)
    c1 = orc.fused(flat, 4, group_mode=orc.GROUP_CHANNEL)
    assert bits_eq(t.y.ravel(), c1.y.ravel()) and np.array_equal(t.codes.ravel(), c1.codes.ravel())
    assert t.lo[0] == x.min() and t.hi[0] == x.max()


def test_channel_mode_equals_tensor_mode_when_ranges_coincide():
    rng = np.random.default_rng(2)
    x = rng.uniform(-1, 1, (3, 4, 5, 5)).astype(np.float32)
    x[0, :, 0, 0] = -2.0           # every channel gets the same extremes
    x[1, :, 1, 1] = 3.0
    ch = orc.fused(x, 3, group_mode=orc.GROUP_CHANNEL)
    te = orc.fused(x, 3, group_mode=orc.GROUP_TENSOR)
    assert bits_eq(ch.y, te.y) and np.array_equal(ch.codes, te.codes)
    assert np.all(ch.s == te.s[0]) and np.all(ch.z == te.z[0])


def test_sample_channel_mode_is_channel_mode_on_the_folded_batch():
    x = _spread_tensor(8, relu=False)
    n, c, h, w = x.shape
    sc = orc.fused(x, 5, group_mode=orc.GROUP_SAMPLE_CHANNEL)
    folded = orc.fused(x.reshape(1, n * c, h, w), 5, group_mode=orc.GROUP_CHANNEL)
    assert bits_eq(sc.y.ravel(), folded.y.ravel()) and bits_eq(sc.lo, folded.lo) and bits_eq(sc.hi, folded.hi)
    # and its range is the per-plane min / max
    assert np.array_equal(sc.lo.reshape(n, c), x.min(axis=(2, 3)))
    assert np.array_equal(sc.hi.reshape(n, c), x.max(axis=(2, 3)))


def test_channel_axis_zero_is_a_transposed_view():
    x = _spread_tensor(9, shape=(5, 3, 2, 4), relu=False)
    a0 = orc.fused(x, 4, channel_axis=0)                       # groups = dim 0 (weight tensors)
    xt = np.ascontiguousarray(x.transpose(1, 0, 2, 3))        # same values with dim 0 moved to axis 1
    a1 = orc.fused(xt, 4, channel_axis=1)
    assert bits_eq(a0.lo, a1.lo) and bits_eq(a0.hi, a1.hi)
    assert bits_eq(a0.y, np.ascontiguousarray(a1.y.transpose(1, 0, 2, 3)))


def test_channel_wise_distortion_not_worse_than_layer_wise():
    """Table 2's statistics on a tensor with a wide per-channel spread: the channel-wise
    relative error must not exceed the layer-wise one (the direction the paper reports)."""
    x = _spread_tensor(21, shape=(8, 16, 8, 8), relu=True)
    ch = orc.fused(x, 3, group_mode=orc.GROUP_CHANNEL).y.astype(np.float64)
    te = orc.fused(x, 3, group_mode=orc.GROUP_TENSOR).y.astype(np.float64)
    xd = x.astype(np.float64)
    rel = lambda q: np.linalg.norm(xd - q) / np.linalg.norm(xd)
    cos = lambda q: float((xd * q).sum() / (np.linalg.norm(xd) * np.linalg.norm(q)))
    assert rel(ch) < rel(te) and cos(ch) > cos(te)


# --------------------------------------------------------------------------------------
# 6. bf16 storage: exact widening, round-to-nearest-even narrowing
# --------------------------------------------------------------------------------------
def test_bf16_identity_quantizer_round_trips_all_small_integers():
    # range [0, 255], b = 8 -> s = 1, z = 0: y must equal x for integer x (all exactly representable in bf16)
    vals = np.arange(256, dtype=np.float32)
    bits16 = (vals.view(np.uint32) >> 16).astype(np.uint16).reshape(1, 1, 16, 16)
    res = orc.fused(bits16, 8)
    assert np.array_equal(res.y, bits16) and res.codes.ravel().tolist() == list(range(256))
    assert res.lo[0] == 0 and res.hi[0] == 255 and res.s[0] == 1 and res.z[0] == 0


def test_bf16_output_is_rounded_to_nearest_even():
    # lo = 0, hi = 3 * 1.00390625 (b = 2): s = 1.00390625 = 0x3F808000 (a bf16 tie) exactly, since
    # hi is built as 3 * s in exact arithmetic below and (hi - 0) / 3 divides back exactly.
    s = 1.00390625
    hi = 3 * s                                    # 3.01171875 = 0x4040C000: also a bf16 tie
    x32 = np.array([0.0, 1.0, 2.0, 3.0], np.float32)          # bf16-exact members, codes 0,1,2,3
    xb = (x32.view(np.uint32) >> 16).astype(np.uint16).reshape(1, 1, 2, 2)
    res = orc.fakequant(xb, 2, f32([0.0]), f32([hi]))
    assert res.s[0] == np.float32(s) and res.z[0] == 0
    assert res.codes.ravel().tolist() == [0, 1, 2, 3]
    # fp32 y = [0, 1.00390625, 2.0078125, 3.01171875]
    #   1.00390625 = 0x3F808000 -> tie, keep even 0x3F80 (1.0)
    #   2.0078125  = 0x40008000 -> tie, keep even 0x4000 (2.0)
    #   3.01171875 = 0x4040C000 -> above the tie, round up to 0x4041
    assert res.y.ravel().tolist() == [0x0000, 0x3F80, 0x4000, 0x4041]


def test_bf16_backward_passes_bits_through():
    rng = np.random.default_rng(3)
    xb = (rng.standard_normal((2, 3, 4, 4)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    gb = (rng.standard_normal((2, 3, 4, 4)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    res = orc.fused(xb, 4, gy=gb)
    assert np.array_equal(res.gx, np.where(res.mask == 1, gb, np.uint16(0)))
    # ranges are the exact widened extremes
    wide = (xb.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(res.lo, wide.min(axis=(0, 2, 3))) and np.array_equal(res.hi, wide.max(axis=(0, 2, 3)))


# --------------------------------------------------------------------------------------
# 9. mask-carrying split of forward and backward (Section 2.1): the packed 1-bit mask
# --------------------------------------------------------------------------------------
def test_packed_mask_hand_case():
    """The stale-range hand case: mask [0,0,1,0,1,1,1,0 | 1], least significant bit first ->
    byte 0 = 4 + 16 + 32 + 64 = 0x74, byte 1 = 0x01; the backward keeps gy at elements 2, 4, 5, 6, 8."""
    case = next(c for c in HAND if c["name"] == "H6_stale_range")
    x = f32(case["x"]).reshape(case["shape"])
    res = orc.fakequant(x, case["bits"], f32(case["lo"]), f32(case["hi"]))
    packed = orc.pack_mask(res.mask)
    assert packed.tolist() == [0x74, 0x01]
    gy = f32([10, 20, 30, 40, 50, 60, 70, 80, 90]).reshape(case["shape"])
    assert orc.bwd_packed(gy, packed).ravel().tolist() == [0, 0, 30, 0, 50, 60, 70, 0, 90]


@pytest.mark.parametrize("n", [0, 1, 7, 8, 9, 15, 16, 17, 63, 64, 65, 1000, 4099])
def test_packed_mask_matches_numpy_bit_packing(n):
    rng = np.random.default_rng(n)
    m = (rng.random(n) < 0.7).astype(np.uint8)
    packed = np.full((n + 7) // 8, 0xFF, np.uint8)          # pre-filled: the last partial byte must come out clean
    packed[:] = orc.pack_mask(m)
    assert np.array_equal(packed, np.packbits(m, bitorder="little"))
    assert np.array_equal(np.unpackbits(packed, bitorder="little")[:n], m)
    assert int(sum(bin(b).count("1") for b in packed.tolist())) == int(m.sum())
    # any non-zero byte counts as set
    assert np.array_equal(orc.pack_mask(m * 200), packed)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_backward_from_packed_mask_equals_backward_from_x(dtype):
    """With the forward pass's own mask the split backward is the STE backward of the fused path,
    for a range that clips on both sides; and gx is bitwise gy or +0."""
    rng = np.random.default_rng(5)
    shape = (3, 5, 7, 7)                                       # 735 elements: a last partial byte
    x = rng.standard_normal(shape).astype(np.float32)
    gy = rng.standard_normal(shape).astype(np.float32)
    gy[0, 0, 0, :3] = [-0.0, 0.0, -1.5]
    if dtype == "bf16":
        x = (x.view(np.uint32) >> 16).astype(np.uint16)
        gy = (gy.view(np.uint32) >> 16).astype(np.uint16)
    lo = np.full(5, -0.5, np.float32)
    hi = np.full(5, 0.8, np.float32)
    ref = orc.fakequant(x, 3, lo, hi, gy=gy)
    assert 0 < ref.mask.sum() < ref.mask.size
    packed = orc.pack_mask(ref.mask)
    gx = orc.bwd_packed(gy, packed)
    u = np.uint16 if dtype == "bf16" else np.uint32
    assert np.array_equal(gx.view(u), ref.gx.view(u))
    bits = np.unpackbits(packed, bitorder="little")[:x.size].reshape(shape).astype(bool)
    assert np.array_equal(gx.view(u), np.where(bits, gy.view(u), u(0)))


# --------------------------------------------------------------------------------------
# 10. distortion statistics (Section 4.1, Table 2): cosine similarity and relative error
# --------------------------------------------------------------------------------------
def test_distortion_closed_forms():
    x = f32([3, 4, 0, 0]).reshape(1, 1, 1, 4)
    cases = [
        (x, (1.0, 0.0)),                                            # Q = X
        (2 * x, (1.0, 1.0)),                                        # Q = 2X: same direction, |X - Q| = |X|
        (f32([0, 0, 5, 0]).reshape(1, 1, 1, 4), (0.0, math.sqrt(2))),   # orthogonal, |X - Q|^2 = 25 + 25
        (f32([4, 3, 0, 0]).reshape(1, 1, 1, 4), (24 / 25, math.sqrt(2) / 5)),
        (-x, (-1.0, 2.0)),
        (0 * x, (0.0, 1.0)),                                        # |Q| = 0: cosine reported as 0
    ]
    for q, (cos, rel) in cases:
        sums = orc.distortion_sums(x, q)
        got = orc.distortion(sums)
        assert got[0] == pytest.approx(cos, abs=1e-15) and got[1] == pytest.approx(rel, abs=1e-15)
    assert orc.distortion_sums(x, f32([4, 3, 0, 0]).reshape(1, 1, 1, 4)).tolist() == [25.0, 25.0, 24.0, 2.0]
    assert orc.distortion(np.zeros(4)) == (0.0, 0.0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_distortion_sums_match_float64_dot_products(dtype):
    rng = np.random.default_rng(8)
    x = (rng.standard_normal((3, 5, 7, 7)) * 10).astype(np.float32)
    if dtype == "bf16":
        xb = (x.view(np.uint32) >> 16).astype(np.uint16)
        res = orc.fused(xb, 4)
        xw = (xb.astype(np.uint32) << 16).view(np.float32).astype(np.float64).ravel()
        qw = (res.y.astype(np.uint32) << 16).view(np.float32).astype(np.float64).ravel()
        sums = orc.distortion_sums(xb, res.y)
    else:
        res = orc.fused(x, 4)
        xw, qw = x.astype(np.float64).ravel(), res.y.astype(np.float64).ravel()
        sums = orc.distortion_sums(x, res.y)
    want = [math.fsum(xw * xw), math.fsum(qw * qw), math.fsum(xw * qw), math.fsum((xw - qw) ** 2)]
    assert np.allclose(sums, want, rtol=1e-13, atol=0)
    cos, rel = orc.distortion(sums)
    assert cos == pytest.approx(np.dot(xw, qw) / (np.linalg.norm(xw) * np.linalg.norm(qw)), rel=1e-12)
    assert rel == pytest.approx(np.linalg.norm(xw - qw) / np.linalg.norm(xw), rel=1e-12)
    assert 0.9 < cos <= 1.0 and 0.0 < rel < 0.2


# --------------------------------------------------------------------------------------
# 11. integer codes as a packed bit string (Eq. 1 -> Eq. 6)
# --------------------------------------------------------------------------------------
def test_packed_codes_hand_case():
    """Hand case H1, channel 0, b = 2: codes [0,1,2,3 | 0,2,2,0] -> 0 + 1*4 + 2*16 + 3*64 = 0xE4 and
    0 + 2*4 + 2*16 + 0 = 0x28; b = 3 of [5, 2, 7]: 5 + 2*8 + 7*64 = 469 = 0x01D5 -> bytes D5 01."""
    assert orc.pack_codes(np.array([0, 1, 2, 3, 0, 2, 2, 0], np.uint8), 2).tolist() == [0xE4, 0x28]
    assert orc.pack_codes(np.array([5, 2, 7], np.uint8), 3).tolist() == [0xD5, 0x01]
    y = orc.dequant_packed(np.array([0xD5, 0x01], np.uint8), (1, 1, 1, 3), 3, f32([0.5]), f32([2]))
    assert y.ravel().tolist() == [1.5, 0.0, 2.5]                       # 0.5 * ([5, 2, 7] - 2)


@pytest.mark.parametrize("bits", range(1, 9))
@pytest.mark.parametrize("n", [1, 7, 32, 33, 1000])
def test_packed_codes_match_big_integer_packing(bits, n):
    rng = np.random.default_rng(bits * 100 + n)
    codes = rng.integers(0, 1 << bits, n).astype(np.uint8)
    big = 0
    for e, c in enumerate(codes.tolist()):                  # the bit string as one Python integer
        big |= c << (e * bits)
    want = np.frombuffer(big.to_bytes((n * bits + 7) // 8, "little"), np.uint8)
    assert np.array_equal(orc.pack_codes(codes, bits), want)
    with pytest.raises(RuntimeError):                        # a code that needs more than b bits
        if bits < 8:
            orc.pack_codes(np.array([1 << bits], np.uint8), bits)
        else:
            raise RuntimeError


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", [orc.GROUP_CHANNEL, orc.GROUP_SAMPLE_CHANNEL, orc.GROUP_TENSOR])
def test_dequantizing_the_packed_codes_gives_the_fake_quantized_tensor(dtype, mode):
    rng = np.random.default_rng(12)
    x = rng.standard_normal((3, 5, 7, 7)).astype(np.float32)
    if dtype == "bf16":
        x = (x.view(np.uint32) >> 16).astype(np.uint16)
    for bits in (3, 5, 8):
        ref = orc.fused(x, bits, group_mode=mode)
        y = orc.dequant_packed(orc.pack_codes(ref.codes, bits), x.shape, bits, ref.s, ref.z, dtype=x.dtype,
                               group_mode=mode)
        assert np.array_equal(y.view(x.dtype), ref.y.view(x.dtype))



# ---- the accumulation over the pre-scaled activations (Eq. 6 left-hand side, Algorithm 1 output step) ----
def test_accumulate_hand_case_from_the_first_hand_case():
    """Codes, scales and zero-points of hand case H1 (channel mode, b = 2): channel 0 has s = 1, z = 0 and codes
    [0,1,2,3 | 0,2,2,0], channel 1 has s = 1, z = 1 and codes [0,1,2,3 | 1,2,3,1], so the pre-scaled activations are
    [0,1,2,3 | 0,2,2,0] and [-1,0,1,2 | 0,1,2,0].  With w = [[2, -1], [0.5, 0.25]] (all products exact):
    y[o=0] = 2 A0 - A1 = [1,2,3,4 | 0,3,2,0],  y[o=1] = A0 / 2 + A1 / 4 = [-.25,.5,1.25,2 | 0,1.25,1.5,0]."""
    codes = np.array([[[[0, 1], [2, 3]], [[0, 1], [2, 3]]], [[[0, 2], [2, 0]], [[1, 2], [3, 1]]]], np.uint8)
    s, z = np.array([1, 1], np.float32), np.array([0, 1], np.float32)
    w = np.array([[2, -1], [0.5, 0.25]], np.float32)
    want = np.array([[[1, 2, 3, 4], [-0.25, 0.5, 1.25, 2.0]], [[0, 3, 2, 0], [0, 1.25, 1.5, 0]]], np.float64)
    for inloop in (False, True):
        y = orc.accumulate(codes, s, z, w, inloop=inloop)
        assert y.shape == (2, 2, 2, 2) and np.array_equal(y.reshape(2, 2, 4), want)
        ycl = orc.accumulate(np.ascontiguousarray(codes.transpose(0, 2, 3, 1)), s, z, w, channels_last=True, inloop=inloop)
        assert np.array_equal(ycl.transpose(0, 3, 1, 2), y)


def test_accumulate_special_weights_and_library_contraction():
    rng = np.random.default_rng(77)
    n, c, h, wd, o = 3, 13, 5, 7, 6
    x = (rng.standard_normal((n, c, h, wd)) * np.exp(rng.standard_normal((1, c, 1, 1)))).astype(np.float32)
    res = orc.fused(x, 4)
    w = rng.standard_normal((o, c)).astype(np.float32)
    # zero weights give zero, one-hot weights pick the pre-scaled activation of one channel (the fake-quantized tensor)
    assert not orc.accumulate(res.codes, res.s, res.z, np.zeros((o, c), np.float32)).any()
    onehot = np.zeros((c, c), np.float32)
    onehot[np.arange(c), np.arange(c)[::-1]] = 1
    y1 = orc.accumulate(res.codes, res.s, res.z, onehot)
    assert np.array_equal(y1, res.y[:, ::-1].astype(np.float64))
    # a library contraction in float64 over the fake-quantized tensor (Eq. 6 read as a matrix product)
    y = orc.accumulate(res.codes, res.s, res.z, w)
    lib = np.einsum("oc,nchw->nohw", w.astype(np.float64), res.y.astype(np.float64))
    scale = np.einsum("oc,nchw->nohw", np.abs(w).astype(np.float64), np.abs(res.y).astype(np.float64))
    assert np.all(np.abs(y - lib) <= 1e-13 * scale + 1e-300)
    # Eq. 3 (scale inside the loop) is the same real number: equal up to the fp32 rounding of the pre-scaled value
    y3 = orc.accumulate(res.codes, res.s, res.z, w, inloop=True)
    assert np.all(np.abs(y - y3) <= 2.0 ** -23 * scale + 1e-300) and not np.array_equal(y, y3)
    # and Eq. 3 against its own float64 contraction: w * s folded into the weights, the zero-point as a rank-one term
    ws = w.astype(np.float64) * res.s.astype(np.float64)
    alt = np.einsum("oc,nchw->nohw", ws, res.codes.astype(np.float64)) - (ws @ res.z.astype(np.float64)).reshape(1, o, 1, 1)
    assert np.all(np.abs(y3 - alt) <= 1e-12 * (scale + np.abs(ws @ res.z.astype(np.float64)).reshape(1, o, 1, 1)))
