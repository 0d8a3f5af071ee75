"""Pins for the oracle's number formats: the values the paper prints, exhaustive tables against
ml_dtypes bit patterns, and the structure of the UE5M3 reading."""
import os

import ml_dtypes
import numpy as np
import pytest

from oracle import mxq_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_rows(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append(line.split())
    return rows


def test_e2m1_values_match_paper_list():
    # Experimental Setup: +-{0, 0.5, 1, 1.5, 2, 3, 4, 6}
    mags = [float(r[0]) for r in _read_rows("e2m1_values.txt")]
    assert len(mags) == 8
    for i, m in enumerate(mags):
        assert orc.e2m1_value(i) == m
        assert orc.e2m1_value(8 | i) == -m
    assert np.signbit(np.float32(orc.e2m1_value(8)))  # -0 keeps its sign


def test_e2m1_codes_match_ml_dtypes_bit_patterns():
    dec = np.arange(16, dtype=np.uint8).view(ml_dtypes.float4_e2m1fn).astype(np.float32)
    for c in range(16):
        assert orc.e2m1_value(c) == dec[c]


def test_paper_constants():
    k = {r[0]: float(r[1]) for r in _read_rows("paper_constants.txt")}
    # eps_SF = 2^-9 is the smallest nonzero E4M3 value (Eq. 3 text)
    assert orc.scale_value(orc.UE4M3, 1) == k["eps_SF_E4M3"] == 2.0 ** -9
    assert orc.scale_value(orc.UE4M3, 0) == 0.0
    # M_max: the largest E2M1 magnitude
    assert orc.e2m1_value(7) == k["M_max_E2M1"]
    # "clipping in [6,7] is equivalent to rounding in [3,3.5]": both intervals collapse onto one
    # grid point (6 and 3), i.e. the interior rounds down and never reaches the next point.
    for t in np.linspace(k["clip_lo"], k["clip_hi"], 101, dtype=np.float32):
        assert orc.e2m1_value(orc.e2m1_index(t)) == 6.0
    for t in np.linspace(k["round_lo"], k["round_hi"], 101, dtype=np.float32)[:-1]:
        assert orc.e2m1_value(orc.e2m1_index(t)) == 3.0


def test_num_codes():
    assert orc.num_codes(orc.UE8M0) == 255
    assert orc.num_codes(orc.UE4M3) == 127
    assert orc.num_codes(orc.UE5M3) == 255
    assert orc.num_codes(7) == 0


def test_ue4m3_table_equals_ml_dtypes_exhaustive():
    dec = np.arange(0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float32)
    vals = [orc.scale_value(orc.UE4M3, c) for c in range(0x7F)]
    assert np.array_equal(np.array(vals, dtype=np.float32), dec)
    assert all(b > a for a, b in zip(vals, vals[1:]))
    assert vals[7] == 7 * 2.0 ** -9 and vals[8] == 2.0 ** -6 and vals[0x38] == 1.0 and vals[0x7E] == 448.0
    assert np.isnan(orc.scale_value(orc.UE4M3, 0x7F))  # the NaN code is never a scale
    assert np.isnan(ml_dtypes.float8_e4m3fn(np.uint8(0x7F).view(ml_dtypes.float8_e4m3fn)).astype(np.float32))


def test_ue8m0_table_equals_ml_dtypes_exhaustive():
    dec = np.arange(0xFF, dtype=np.uint8).view(ml_dtypes.float8_e8m0fnu).astype(np.float64)
    for c in range(0xFF):
        assert float(orc.scale_value(orc.UE8M0, c)) == dec[c] == 2.0 ** (c - 127)
    assert np.isnan(orc.scale_value(orc.UE8M0, 0xFF))


def test_ue5m3_reading_structure():
    vals = [orc.scale_value(orc.UE5M3, c) for c in range(0xFF)]
    assert vals[0] == 0.0 and vals[1] == 2.0 ** -17 and vals[8] == 2.0 ** -14
    assert vals[0x78] == 1.0 and vals[0xFE] == 1.75 * 2.0 ** 16
    assert all(b > a for a, b in zip(vals, vals[1:]))
    # same mantissa width as E4M3, wider exponent: every UE4M3 value is a UE5M3 value
    s5 = set(vals)
    assert all(orc.scale_value(orc.UE4M3, c) in s5 for c in range(0x7F))
    # three mantissa bits: within a binade eight equally spaced values
    for e in range(1, 31):
        seg = vals[8 * e:8 * e + 8]
        assert all(seg[i] == seg[0] * (1 + i / 8) for i in range(8))
    assert np.isnan(orc.scale_value(orc.UE5M3, 0xFF))


@pytest.mark.parametrize("fmt", [orc.UE8M0, orc.UE4M3, orc.UE5M3])
def test_out_of_range_codes_are_nan(fmt):
    assert np.isnan(orc.scale_value(fmt, -1))
    assert np.isnan(orc.scale_value(fmt, 256))
