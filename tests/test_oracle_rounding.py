"""Pins for the oracle's rounding steps: E2M1 element rounding and Round_SF of Eq. 1 / Eq. 2,
against ml_dtypes casts (an independent library routine) and exact rational arithmetic."""
import os
from fractions import Fraction as F

import ml_dtypes
import numpy as np
import pytest

import exact_ref as ex
from oracle import mxq_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
f32 = np.float32


def _neigh(x):
    x = f32(x)
    return [np.nextafter(x, f32(-np.inf)), x, np.nextafter(x, f32(np.inf))]


# ------------------------------------------------------------------------------------------------
# E2M1 element rounding
# ------------------------------------------------------------------------------------------------
def test_e2m1_hand_listed_ties_and_saturation():
    # round-to-nearest-even on the grid: each midpoint goes to the neighbour with the even index
    want = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0,
            6.0: 6.0, 7.0: 6.0, 100.0: 6.0, float("inf"): 6.0, 0.0: 0.0, 5.000001: 6.0, 4.999999: 4.0}
    for t, q in want.items():
        assert orc.e2m1_value(orc.e2m1_index(t)) == q, t
        assert orc.e2m1_index(-t) == orc.e2m1_index(t)


def test_e2m1_rounding_equals_ml_dtypes_cast():
    rng = np.random.default_rng(11)
    pts = [f32(0)]
    for m in (0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0, 7.0):
        pts += _neigh(m)
    pts += list(rng.uniform(0, 8, 4000).astype(f32)) + list(np.ldexp(rng.random(500), rng.integers(-40, 3, 500)).astype(f32))
    pts = np.array(pts, dtype=f32)
    lib = pts.astype(ml_dtypes.float4_e2m1fn).astype(f32)
    grid = ex.e2m1_magnitudes()
    for t, want in zip(pts, lib):
        assert orc.e2m1_value(orc.e2m1_index(t)) == want, float(t)
        assert orc.e2m1_index(t) == ex.nearest_even_index(ex.frac(t), grid) or t >= 6


# ------------------------------------------------------------------------------------------------
# Round_SF for the FP8 scale formats (Eq. 2: rounded to nearest even and clipped to the format's range)
# ------------------------------------------------------------------------------------------------
def _boundary_points(fmt):
    tab = ex.TABLES[fmt]()
    pts = []
    for a, b in zip(tab, tab[1:]):
        mid = (F(a) + F(b)) / 2
        m32 = ex.f32_round(mid)
        if ex.frac(m32) == mid:
            pts += _neigh(m32)
        pts += [f32(a)]
    pts += _neigh(tab[-1]) + [f32(tab[-1] * 1.03), f32(tab[-1] * 1.07), f32(tab[-1] * 4), f32(np.inf)]
    return [p for p in pts if p >= 0]


def test_ue4m3_rne_hand_listed():
    r = lambda w: orc.round_scale(orc.UE4M3, w)
    assert r(2.0 ** -10) == 0            # tie between 0 and 2^-9 -> even code 0
    assert r(np.nextafter(f32(2.0 ** -10), f32(1))) == 1
    assert r(1.5 * 2.0 ** -9) == 2       # tie between codes 1 and 2 -> 2
    assert r(2.5 * 2.0 ** -9) == 2       # tie between codes 2 and 3 -> 2
    assert r(1.0) == 0x38 and r(448.0) == 0x7E
    assert r(464.0) == 0x7E and r(1e9) == 0x7E and r(np.inf) == 0x7E   # clip: never the NaN code
    assert r(0.0) == 0


def test_ue4m3_rne_equals_ml_dtypes_cast():
    rng = np.random.default_rng(12)
    pts = _boundary_points(orc.UE4M3) + list(np.ldexp(rng.random(3000) + 1, rng.integers(-14, 10, 3000)).astype(f32))
    for w in pts:
        lib_code = int(np.minimum(f32(w), f32(448.0)).astype(ml_dtypes.float8_e4m3fn).view(np.uint8))  # ml_dtypes does not clip
        assert orc.round_scale(orc.UE4M3, w) == lib_code, float(w)


@pytest.mark.parametrize("fmt", [orc.UE4M3, orc.UE5M3])
def test_fp8_scale_rne_equals_exact_nearest(fmt):
    rng = np.random.default_rng(13 + fmt)
    lo, hi = (-14, 10) if fmt == orc.UE4M3 else (-22, 18)
    pts = _boundary_points(fmt) + list(np.ldexp(rng.random(1500) + 1, rng.integers(lo, hi, 1500)).astype(f32))
    tab = ex.TABLES[fmt]()
    for w in pts:
        want = len(tab) - 1 if not np.isfinite(w) else ex.nearest_even_index(ex.frac(w), tab)
        assert orc.round_scale(fmt, w) == want, float(w)


def test_ue4m3_zero_scale_threshold_closed_form():
    # abs-max target amax/6 rounds to code 0 exactly when amax/6 <= 2^-10, i.e. amax <= 6*2^-10
    thr = f32(6 * 2.0 ** -10)
    assert thr == f32(0.005859375)
    for amax in _neigh(thr) + [f32(1e-4), f32(0.0058), f32(0.0059), f32(0.01)]:
        w = f32(amax) / f32(6.0)
        assert (orc.round_scale(orc.UE4M3, w) == 0) == (F(float(amax)) / 6 <= F(1, 1024)), float(amax)
    assert orc.round_scale(orc.UE4M3, f32(0.0058) / f32(6)) == 0
    assert orc.round_scale(orc.UE4M3, f32(0.0059) / f32(6)) == 1


# ------------------------------------------------------------------------------------------------
# Eq. 1: power-of-two floor rule
# ------------------------------------------------------------------------------------------------
def test_mx_scale_hand_worked_blocks():
    with open(os.path.join(GOLDEN, "mx_scale_worked.txt")) as f:
        rows = [l.split("#")[0].split() for l in f if l.split("#")[0].strip()]
    assert len(rows) >= 10
    for amax, k in rows:
        amax, k = f32(float(amax)), int(k)
        # a block whose largest magnitude is amax
        x = np.array([amax * f32(0.3), -amax, amax * f32(0.01), 0], dtype=f32)
        _, scales, _ = orc.quantize(x, 4, orc.UE8M0, orc.ABSMAX)
        assert int(scales[0]) - 127 == k, (float(amax), k)
        assert orc.scale_value(orc.UE8M0, int(scales[0])) == 2.0 ** k


def test_mx_scale_is_largest_power_with_6S_le_amax():
    rng = np.random.default_rng(14)
    for amax in np.ldexp(rng.random(400) + 1, rng.integers(-30, 30, 400)).astype(f32):
        w = f32(amax) / f32(6.0)
        c = orc.round_scale(orc.UE8M0, w)
        k = c - 127
        # exact statement of floor(log2(amax/6)): 6*2^k <= amax < 6*2^(k+1)  (up to the one
        # float rounding of amax/6, which cannot cross a power of two from below)
        assert 6 * F(2) ** k <= ex.frac(amax) * (1 + F(1, 2 ** 23))
        assert ex.frac(amax) < 6 * F(2) ** (k + 1)
    assert orc.round_scale(orc.UE8M0, 0.0) == 0
    assert orc.round_scale(orc.UE8M0, 1e-45) == 0
    assert orc.round_scale(orc.UE8M0, 3e38) == 254
    assert orc.round_scale(orc.UE8M0, 2.0 ** 127) == 254
    assert orc.round_scale(orc.UE8M0, np.nextafter(f32(1.0), f32(0))) == 126
    assert orc.round_scale(orc.UE8M0, 1.0) == 127


def test_ue5m3_rounding_equals_a_scaled_ue4m3_rounding():
    """The UE5M3 value set is the UE4M3 value set times 2^-8 (codes 0..0x7E), the UE4M3 normals themselves
    (codes + 0x40) and the UE4M3 normals times 2^8 (codes + 0x80), so rounding onto UE5M3 is rounding a
    scaled number onto UE4M3 plus a code offset: below 1 scale by 256, from 1 to 256 by 1, above by 1/256,
    with saturation at 448 standing for saturation at 114688.  The lean kernels round both 4-over-6 targets
    this way with one hardware E4M3 conversion, choosing the stretch by the larger target.  Checked against
    the oracle's UE5M3 rounding on every mantissa pattern near the stretch boundaries, on a sample of all
    other binades, and for the smaller target w / 1.5 rounded in the stretch that w selects."""
    import ml_dtypes

    rng = np.random.default_rng(53)
    ws = [np.float32(0.0)]
    for e in (-19, -18, -17, -15, -14, -9, -1, 0, 7, 8, 15, 16, 17):          # whole binades, every 64th mantissa
        ws += list((np.arange(0, 1 << 23, 64, dtype=np.uint32) | np.uint32((e + 127) << 23)).view(np.float32))
    for e in range(-30, 30):
        ws += list((rng.integers(0, 1 << 23, 600).astype(np.uint32) | np.uint32((e + 127) << 23)).view(np.float32))
    for c in range(0, 254):                                                   # the midpoints between codes, and their neighbours
        mid = np.float32((orc.scale_value(orc.UE5M3, c) + orc.scale_value(orc.UE5M3, c + 1)) / 2)
        ws += [mid, np.nextafter(mid, np.float32(0)), np.nextafter(mid, np.float32(np.inf))]
    ws = np.array(ws, dtype=np.float32)

    def via_e4m3(w, chooser):
        low, high = chooser < 1.0, chooser >= 256.0
        s = np.where(low, 256.0, np.where(high, 1.0 / 256.0, 1.0)).astype(np.float32)
        off = np.where(low, 0, np.where(high, 0x80, 0x40))
        t = np.minimum((w * s).astype(np.float32), np.float32(448.0))         # the conversion saturates
        return t.astype(ml_dtypes.float8_e4m3fn).view(np.uint8).astype(np.int64) + off

    want = np.array([orc.round_scale(orc.UE5M3, float(w)) for w in ws])
    assert np.array_equal(via_e4m3(ws, ws), want)
    w6 = (ws / np.float32(1.5)).astype(np.float32)
    want6 = np.array([orc.round_scale(orc.UE5M3, float(w)) for w in w6])
    assert np.array_equal(via_e4m3(w6, ws), want6)
