"""Pins for the oracle's analysis outputs: clipping-only SSE, entry / scale histograms and the
segment MSE of the numerical study (CPU only)."""
from fractions import Fraction

import numpy as np
import pytest

import exact_ref as ex
from oracle import mxq_oracle as orc


def test_clipping_sse_hand_worked_block():
    # UE4M3 code 0x38 is S = 1: elements above 6 are cut to 6, the others contribute nothing
    v = np.array([7.0, -9.0, 6.0, 5.9, 0.3, -6.0, 6.5, -0.0], dtype=np.float32)
    clip = orc.block_clip_sse(v, np.array([0x38], dtype=np.uint8), 8, orc.UE4M3)
    assert clip[0] == np.float32(1.0 + 9.0 + 0.25)
    # with a scale of 2 nothing exceeds 6 * 2
    clip = orc.block_clip_sse(v, np.array([0x40], dtype=np.uint8), 8, orc.UE4M3)
    assert clip[0] == 0.0
    # a zero scale clips nothing: its error is underflow
    clip = orc.block_clip_sse(v, np.array([0], dtype=np.uint8), 8, orc.UE4M3)
    assert clip[0] == 0.0


def test_clipping_sse_against_exact_rational_arithmetic():
    rng = np.random.default_rng(5)
    for fmt, g in ((orc.UE4M3, 1.0), (orc.UE4M3, 0.0131), (orc.UE5M3, 1.0), (orc.UE8M0, 0.7)):
        for trial in range(40):
            B = int(rng.choice([2, 4, 8, 16]))
            v = (rng.standard_normal(B) * np.exp2(rng.integers(-6, 3))).astype(np.float32)
            code = int(rng.integers(1, orc.num_codes(fmt)))
            if fmt != orc.UE8M0:
                # keep the scale near the data so that some elements clip and some do not
                w = np.float32(np.abs(v).max() / g / rng.choice([6.0, 9.0, 14.0, 30.0]))
                code = max(1, orc.round_scale(fmt, w))
            else:
                code = int(np.clip(127 + np.floor(np.log2(np.abs(v).max() / g / rng.choice([6.0, 12.0, 40.0]))), 1, 254))
            got = orc.block_clip_sse(v, np.array([code], dtype=np.uint8), B, fmt, g)[0]
            want = ex.clip_sse_exact(v, fmt, code, g)
            assert np.float32(got).view(np.uint32) == np.float32(want).view(np.uint32), (fmt, g, code, v)


def test_clipping_sse_is_part_of_the_block_sse_and_vanishes_without_clipping():
    rng = np.random.default_rng(9)
    x = (rng.standard_normal(4096) * 0.02).astype(np.float32)
    for B in (4, 16):
        for recipe in (orc.ABSMAX, orc.ABSMAX_PZ, orc.R4O6, orc.BRUTE):
            codes, scales, sse = orc.quantize(x, B, orc.UE4M3, recipe)
            clip = orc.block_clip_sse(x, scales, B, orc.UE4M3)
            assert np.all(clip <= sse)          # a subsequence of the same non-negative terms
            # blocks whose largest quotient stays within 6 have no clipping error
            S = np.array([orc.scale_value(orc.UE4M3, int(c)) for c in scales], dtype=np.float32)
            amax = np.abs(x.reshape(-1, B)).max(axis=1)
            inside = (S > 0) & (np.float32(amax) / np.where(S > 0, S, 1) <= 6.0)
            assert np.all(clip[inside] == 0.0)
            assert np.any(clip > 0) or recipe in (orc.R4O6, orc.BRUTE)


def test_histograms_count_every_entry_once():
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(2048) * 0.3).astype(np.float32)
    codes, scales, _ = orc.quantize(x, 16, orc.UE4M3, orc.ABSMAX)
    ch, sh = orc.histograms(codes, scales, x.size, 16)
    assert int(ch.sum()) == x.size and int(sh.sum()) == x.size // 16
    nib = np.stack([codes & 15, codes >> 4], axis=1).reshape(-1)
    assert np.array_equal(ch, np.bincount(nib, minlength=16).astype(np.uint64))
    assert np.array_equal(sh, np.bincount(scales, minlength=256).astype(np.uint64))
    # every block of an abs-max quantization holds an entry of magnitude 4 or 6 (the maximum maps to ~6)
    mags = (nib & 7).reshape(-1, 16).max(axis=1)
    assert np.all(mags >= 6)
    # the sign bit of the code is the sign of the input
    assert np.array_equal((nib >> 3).astype(bool), np.signbit(x))


def test_segment_mse_is_the_tensor_mse_of_each_segment():
    rng = np.random.default_rng(4)
    sse = (rng.random(7 * 50) * np.exp2(rng.integers(-20, 2, 350))).astype(np.float32)
    out = orc.segment_mse(sse, 50, 50 * 16)
    for s in range(7):
        seg = sse[s * 50:(s + 1) * 50]
        assert out[s] == orc.tensor_mse(seg, 50 * 16)
        exact = sum(Fraction(float(v)) for v in seg) / (50 * 16)
        assert abs(Fraction(out[s]) - exact) <= exact * Fraction(1, 10 ** 14)


def test_ocp_power_of_two_rule_hand_worked_and_against_eq1():
    # S = 2^(floor(log2 amax) - 2): amax 1 -> 2^-2, 3.9 -> 2^-1, 4 -> 1, 6 -> 1, 7.99 -> 1, 8 -> 2
    for amax, code in ((1.0, 125), (3.9, 126), (4.0, 127), (6.0, 127), (7.99, 127), (8.0, 128), (0.75, 124)):
        assert orc.ocp_code(amax) == code, amax
    assert orc.ocp_code(0.0) == 0
    assert orc.ocp_code(1.0, 0.25) == orc.ocp_code(4.0)          # the tensor scale divides the maximum first
    rng = np.random.default_rng(12)
    for a in np.exp2(rng.uniform(-20, 20, 2000)).astype(np.float32):
        c_ocp, c_eq1 = orc.ocp_code(a), orc.round_scale(orc.UE8M0, np.float32(a) / np.float32(6.0))
        assert c_ocp - c_eq1 in (0, 1)                           # same scale, or twice the one of Eq. 1
        q = Fraction(float(a)) / Fraction(2) ** (c_ocp - 127)
        assert 4 <= q < 8                                        # the maximum lands in [4, 8)
    x = (rng.standard_normal(1024) * 0.3).astype(np.float32)
    codes, scales, sse = orc.quantize(x, 32, orc.UE8M0, orc.ABSMAX_OCP)
    amax = np.abs(x.reshape(-1, 32)).max(axis=1)
    assert np.array_equal(scales, np.array([orc.ocp_code(a) for a in amax], dtype=np.uint8))
    for b in range(4):
        s_b, _ = orc.block_sse(x[b * 32:(b + 1) * 32], orc.UE8M0, int(scales[b]))
        assert s_b == sse[b]


def test_clip7_power_of_two_rule_hand_worked_and_against_eq1():
    # S = 2^floor(log2(amax / 3.5)): the maximum lands in [3.5, 7) and is clipped above 6 (Background)
    for amax, code in ((3.5, 127), (6.0, 127), (6.99, 127), (7.0, 128), (3.49, 126), (1.0, 125), (0.875, 125),
                       (0.874, 124), (14.0, 129), (1.75, 126), (1.74, 125)):
        assert orc.clip7_code(amax) == code, amax
    assert orc.clip7_code(0.0) == 0
    assert orc.clip7_code(1.0, 0.25) == orc.clip7_code(4.0)
    assert orc.clip7_code(3.0e38, 1.0e-3) == 254                 # amax / g overflows: the largest scale
    rng = np.random.default_rng(14)
    for a in np.exp2(rng.uniform(-20, 20, 2000)).astype(np.float32):
        c7, c_eq1 = orc.clip7_code(a), orc.round_scale(orc.UE8M0, np.float32(a) / np.float32(6.0))
        q = Fraction(float(a)) / Fraction(2) ** (c7 - 127)
        assert Fraction(7, 2) <= q < 7
        # Eq. 1 takes the largest power of two <= fl(a / 6); on a binade edge the rounding of a / 6 may lift it
        assert c7 - c_eq1 in (0, 1)
    # the bottom of the code range: maxima below 3.5 * 2^-127 clamp to code 0
    assert orc.clip7_code(np.float32(2.0 ** -126)) == 0 and orc.clip7_code(np.float32(3.5 * 2.0 ** -126)) == 1
    x = (rng.standard_normal(1024) * 0.3).astype(np.float32)
    codes, scales, sse = orc.quantize(x, 32, orc.UE8M0, orc.ABSMAX_CLIP7)
    amax = np.abs(x.reshape(-1, 32)).max(axis=1)
    assert np.array_equal(scales, np.array([orc.clip7_code(a) for a in amax], dtype=np.uint8))
    for b in range(4):
        s_b, _ = orc.block_sse(x[b * 32:(b + 1) * 32], orc.UE8M0, int(scales[b]))
        assert s_b == sse[b]
    with pytest.raises(Exception):
        orc.quantize(x, 32, orc.UE4M3, orc.ABSMAX_CLIP7)


def test_fake_quantize_is_dequantize_of_quantize():
    rng = np.random.default_rng(13)
    x = (rng.standard_normal(512) * 0.1).astype(np.float32)
    for fmt, recipe, g in ((orc.UE4M3, orc.R4O6, 1.0), (orc.UE5M3, orc.ABSMAX_PZ, 0.37), (orc.UE8M0, orc.ABSMAX_OCP, 1.0)):
        xh = orc.fake_quantize(x, 16, fmt, recipe, g)
        codes, scales, sse = orc.quantize(x, 16, fmt, recipe, g)
        # the block SSE is the squared distance between x and its fake-quantized copy (up to one rounding per term)
        err = ((x.astype(np.float64) - xh.astype(np.float64)) ** 2).reshape(-1, 16).sum(axis=1)
        assert np.allclose(err, sse, rtol=1e-5, atol=1e-30)
        # every value is a grid value times the decode scale of its block
        S = np.array([orc.scale_value(fmt, int(c)) for c in scales], dtype=np.float32) * np.float32(g)
        ratio = np.abs(xh.reshape(-1, 16)) / S[:, None]
        assert np.all(np.isin(np.round(ratio * 2) / 2, [0, .5, 1, 1.5, 2, 3, 4, 6]))


def test_mask_interval_definition():
    x = np.array([0.0, -0.0, 0.01, -0.01, 0.02, 0.0199999, -0.035, 0.5, 1e-30], dtype=np.float32)
    out = orc.mask_interval(x, 0.01, 0.02)
    assert np.array_equal(out, np.array([0.0, -0.0, 0.0, 0.0, 0.02, 0.0, -0.035, 0.5, 1e-30], dtype=np.float32))
    assert np.array_equal(orc.mask_interval(x, 0.0, 0.0), x)                       # empty interval
    assert np.count_nonzero(orc.mask_interval(x, 0.0, 1.0)) == 0                   # everything below 1 goes
    rng = np.random.default_rng(1)
    y = (rng.standard_normal(4096) * 0.02).astype(np.float32)
    lo, hi = 0.005, 0.015
    m = orc.mask_interval(y, lo, hi)
    inside = (np.abs(y) >= lo) & (np.abs(y) < hi)
    assert np.count_nonzero(m) == y.size - inside.sum() and np.array_equal(m[~inside], y[~inside])
    # bf16 bit patterns in, bf16 bit patterns out
    yb = (y.view(np.uint32) >> 16).astype(np.uint16)
    mb = orc.mask_interval(yb, lo, hi)
    yf = (yb.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(mb == 0, ((np.abs(yf) >= lo) & (np.abs(yf) < hi)) | (yb == 0))
