"""Exact-rational helpers for pinning the oracle (test-only; imports neither the oracle nor the
CUDA package).

Everything here is computed with ``fractions.Fraction``: IEEE binary32 operations are emulated as
"exact result, then one round-to-nearest-even", and rounding onto a value lattice is a nearest-point
search with ties to the even index.  Value tables come from ``ml_dtypes`` where that library has
the format (E2M1, E4M3, E8M0); UE5M3 has no independent source and is written from its stated
reading (bias 15, subnormals, codes 0..0xFE).
"""
from __future__ import annotations

from fractions import Fraction

import ml_dtypes
import numpy as np

F = Fraction


def frac(x) -> Fraction:
    return F(float(x))  # exact: every float is a dyadic rational


def f32_round(x: Fraction) -> np.float32:
    """One IEEE-754 binary32 round-to-nearest-even of an exact rational (denormals, overflow)."""
    if x == 0:
        return np.float32(0.0)
    sign = -1 if x < 0 else 1
    a = -x if x < 0 else x
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if F(2) ** e > a:
        e -= 1
    assert F(2) ** e <= a < F(2) ** (e + 1)
    e = max(e, -126)
    quantum = F(2) ** (e - 23)
    qn = a / quantum
    n = qn.numerator // qn.denominator
    rem = qn - n
    if rem > F(1, 2) or (rem == F(1, 2) and n % 2 == 1):
        n += 1
    r = n * quantum
    if r >= F(2) ** 128:
        return np.float32(sign * np.inf)
    return np.float32(sign * float(r))


def f32_div(a, b) -> np.float32:
    return f32_round(frac(a) / frac(b))


def f32_mul(a, b) -> np.float32:
    return f32_round(frac(a) * frac(b))


def f32_fma(a, b, c) -> np.float32:
    return f32_round(frac(a) * frac(b) + frac(c))


# ------------------------------------------------------------------------------------------------
# Value tables
# ------------------------------------------------------------------------------------------------
def e2m1_magnitudes():
    """The 8 non-negative E2M1 values in code order, decoded by ml_dtypes from bit patterns 0..7."""
    return [float(v) for v in np.arange(8, dtype=np.uint8).view(ml_dtypes.float4_e2m1fn).astype(np.float32)]


def ue4m3_table():
    """Finite non-negative E4M3 values, bit patterns 0x00..0x7E, decoded by ml_dtypes."""
    return [float(v) for v in np.arange(0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float32)]


def ue8m0_table():
    return [float(v) for v in np.arange(0xFF, dtype=np.uint8).view(ml_dtypes.float8_e8m0fnu).astype(np.float64)]


def ue5m3_table():
    """Stated reading of UE5M3: bias 15, 3 mantissa bits, subnormals m*2^-17, codes 0..0xFE."""
    out = []
    for c in range(0xFF):
        e, m = c >> 3, c & 7
        out.append(float(F(m, 8) * F(2) ** (-14) if e == 0 else (1 + F(m, 8)) * F(2) ** (e - 15)))
    return out


TABLES = {0: ue8m0_table, 1: ue4m3_table, 2: ue5m3_table}


def nearest_even_index(x: Fraction, table) -> int:
    """Index of the lattice point nearest to x >= 0; ties to the even index; clip at the top."""
    best, best_d = None, None
    for i, t in enumerate(table):
        d = abs(x - frac(t))
        if best is None or d < best_d or (d == best_d and i % 2 == 0 and best % 2 == 1):
            best, best_d = i, d
    return best


def floor_pow2_index(x: Fraction, table) -> int:
    """Largest index whose (power-of-two) value is <= x, else 0."""
    lo = 0
    for i, t in enumerate(table):
        if frac(t) <= x:
            lo = i
    return lo


def round_scale_exact(fmt: int, w) -> int:
    tab = TABLES[fmt]()
    x = frac(w)
    if x <= 0:
        return 0
    return floor_pow2_index(x, tab) if fmt == 0 else nearest_even_index(x, tab)


# ------------------------------------------------------------------------------------------------
# Whole-block reference (slow; tiny inputs only)
# ------------------------------------------------------------------------------------------------
def eval_block_exact(v, fmt: int, code: int, g=1.0):
    """(sse float32, list of 4-bit codes) of one block under one scale code, every float operation
    emulated exactly: D = fl(S*g); t = fl(v/D); e = fl(fma(-q, D, v)); sse = fl(fma(e, e, sse))."""
    grid = e2m1_magnitudes()
    S = TABLES[fmt]()[code]
    D = f32_mul(np.float32(S), np.float32(g))
    sse = np.float32(0.0)
    codes = []
    for x in np.asarray(v, dtype=np.float32):
        if D == 0:
            idx = 0
        else:
            t = f32_div(x, D)
            idx = 7 if abs(float(t)) >= 6.0 else nearest_even_index(abs(frac(t)), grid)
        sgn = 8 if np.signbit(x) else 0
        codes.append(sgn | idx)
        q = -grid[idx] if sgn else grid[idx]
        e = f32_fma(-q, D, x)
        sse = f32_fma(e, e, sse)
    return sse, codes


def absmax_code_exact(v, fmt: int, g=1.0, M=6.0, pz=False) -> int:
    amax = np.float32(np.max(np.abs(np.asarray(v, dtype=np.float32))))
    w = f32_div(f32_div(amax, np.float32(g)), np.float32(M))
    c = round_scale_exact(fmt, w)
    if pz and fmt != 0 and c < 1:
        c = 1
    return c


def choose_exact(v, fmt: int, recipe: int, g=1.0):
    """(code, sse) by recipe id 0..5 (abs-max, +pz, 4-over-6, +pz, brute, +pz)."""
    pz = recipe in (1, 3, 5)
    if recipe in (0, 1):
        c = absmax_code_exact(v, fmt, g, 6.0, pz)
        return c, eval_block_exact(v, fmt, c, g)[0]
    if recipe in (2, 3):
        c6 = absmax_code_exact(v, fmt, g, 6.0, pz)
        c4 = absmax_code_exact(v, fmt, g, 4.0, pz)
        s6 = eval_block_exact(v, fmt, c6, g)[0]
        s4 = eval_block_exact(v, fmt, c4, g)[0]
        return (c4, s4) if s4 < s6 else (c6, s6)
    tab = TABLES[fmt]()
    first = 1 if (pz and fmt != 0) else 0
    best = None
    for c in range(first, len(tab)):
        D = f32_mul(np.float32(tab[c]), np.float32(g))
        if not np.isfinite(D):
            continue
        s = eval_block_exact(v, fmt, c, g)[0]
        if best is None or s < best[1]:
            best = (c, s)
    return best


def clip_sse_exact(v, fmt: int, code: int, g=1.0):
    """SSE restricted to the elements whose quotient by the decode scale exceeds 6 in magnitude,
    every float operation emulated exactly (same order as eval_block_exact)."""
    S = TABLES[fmt]()[code]
    D = f32_mul(np.float32(S), np.float32(g))
    sse = np.float32(0.0)
    if D == 0:
        return sse
    for x in np.asarray(v, dtype=np.float32):
        t = f32_div(x, D)
        if abs(frac(t)) > 6:
            q = -6.0 if np.signbit(x) else 6.0
            e = f32_fma(-q, D, x)
            sse = f32_fma(e, e, sse)
    return sse
