"""Do the pins have teeth?  Each case plants ONE plausible mistake in a copy of the oracle's C source
(a wrong tie rule, sign, index, divisor, bias, operand order ...), builds the copy, and runs the
oracle's pin tests against it in a child process: at least one pin must fail.  The mistakes live
in copies on the CPU only; the CUDA path is not involved."""
import concurrent.futures as cf
import os
import subprocess
import sys

import pytest

from oracle import mxq_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PIN_FILES = ["tests/test_oracle_formats.py", "tests/test_oracle_rounding.py", "tests/test_oracle_recipes.py",
             "tests/test_oracle_analysis.py"]

# (name, text in mxq_oracle.c, replacement)
MUTANTS = [
    ("e2m1 ties away from zero", "return (lo % 2 == 0) ? lo : lo + 1;", "return lo + 1;"),
    ("e2m1 grid value 3 -> 2.5", "2.0f, 3.0f, 4.0f, 6.0f};", "2.0f, 2.5f, 4.0f, 6.0f};"),
    ("residual with the wrong sign", "float e = fmaf(-q, D, v[i]);", "float e = fmaf(q, D, v[i]);"),
    ("SSE not fused", "sse = fmaf(e, e, sse);\n    }\n    return sse;", "sse = sse + e * e;\n    }\n    return sse;"),
    ("scale ties always up", "return (lo % 2 == 0) ? lo : hi;", "return hi;"),
    ("scale rounding truncates", "if ((double)w > mid) return hi;", "if ((double)w > mid) return lo;"),
    ("UE4M3 bias 8", "int bias = (fmt == ORC_UE4M3) ? 7 : 15;", "int bias = (fmt == ORC_UE4M3) ? 8 : 15;"),
    ("UE5M3 bias 16", "int bias = (fmt == ORC_UE4M3) ? 7 : 15;", "int bias = (fmt == ORC_UE4M3) ? 7 : 16;"),
    ("subnormal scales one binade low", "return ldexpf((float)m, 1 - bias - 3);", "return ldexpf((float)m, -bias - 3);"),
    ("Eq. 1 excludes the exact power of two", "if (ldexpf(1.0f, c - 127) <= w) lo = c;", "if (ldexpf(1.0f, c - 127) < w) lo = c;"),
    ("4-over-6 tie goes to M = 4", "if (s4 < s6) { best = c4;", "if (s4 <= s6) { best = c4;"),
    ("4-over-6 second divisor 3", "absmax_code(amax, g, 4.0f, fmt, pz)", "absmax_code(amax, g, 3.0f, fmt, pz)"),
    ("prevent-zero clamps to code 2", "c < 1) c = 1;", "c < 1) c = 2;"),
    ("brute-force tie keeps the larger code", "if (best < 0 || s < best_sse) { best = c;", "if (best < 0 || s <= best_sse) { best = c;"),
    ("brute force under prevent-zero keeps code 0", "int first = (pz && fmt != ORC_UE8M0) ? 1 : 0;", "int first = 0;"),
    ("brute force stops one code early", "for (int c = first; c < n; ++c) {", "for (int c = first; c < n - 1; ++c) {"),
    ("two successive divisions", "float t = v[i] / D;", "float t = (v[i] / S) / g;"),
    ("target from one division by g * M", "float w = u / M;", "float w = amax / (g * M);"),
    ("nibbles swapped", "(uint8_t)(c4[i] | (c4[i + 1] << 4))", "(uint8_t)(c4[i + 1] | (c4[i] << 4))"),
    ("negative zero loses its sign", "(signbit(v[i]) ? 8 : 0) | idx", "((v[i] < 0.0f) ? 8 : 0) | idx"),
    ("zero scale not special", "if (D != 0.0f) {", "if (1) {"),
    ("MSE divided by the block count", "return s / (double)n;", "return s / (double)n_blocks;"),
    ("dequantize forgets the tensor scale", "float D = mxq_oracle_scale_value(fmt, sc) * g;", "float D = mxq_oracle_scale_value(fmt, sc);"),
    ("dequantize reads the nibbles in the other order", "int c4 = (codes[i / 2] >> ((i & 1) ? 4 : 0)) & 15;", "int c4 = (codes[i / 2] >> ((i & 1) ? 0 : 4)) & 15;"),
    ("clipping includes the value 6 itself", "if (fabsf(t) > 6.0f) {", "if (fabsf(t) >= 5.0f) {"),
    ("OCP exponent off by one", "int c = 127 + (e - 1) - 2;", "int c = 127 + (e - 1) - 3;"),
    ("[3.5, 7) rule excludes the lower edge", "while ((double)ldexp(3.5, e) > (double)u) --e;", "while ((double)ldexp(3.5, e) >= (double)u) --e;"),
    ("tensor amax without the absolute value", "float a = fabsf(load_elem(x, dtype, i));\n        if (a > amax) amax = a;", "float a = load_elem(x, dtype, i);\n        if (a > amax) amax = a;"),
    ("bf16 output truncated", "u += 0x7FFFu + lsb;", "u += 0u * lsb;"),
    ("segment MSE of the wrong segment", "block_sse[s * blocks_per_segment + b]", "block_sse[b]"),
    ("histogram skips the sign bit", "code_hist[(codes[i / 2] >> ((i & 1) ? 4 : 0)) & 15] += 1;", "code_hist[(codes[i / 2] >> ((i & 1) ? 4 : 0)) & 7] += 1;"),
]


def _run_pins_against(name, old, new, workdir):
    src = open(orc._SRC).read()
    assert src.count(old) >= 1, f"mutant '{name}': the text to replace is not in the oracle source"
    path_c = os.path.join(workdir, f"m{abs(hash(name)) % 10 ** 8}.c")
    path_so = path_c[:-2] + ".so"
    with open(path_c, "w") as f:
        f.write(src.replace(old, new, 1))
    subprocess.run(["gcc", *orc._CFLAGS, "-o", path_so, path_c, "-lm"], check=True)
    env = dict(os.environ, MXQ_ORACLE_LIB=path_so)
    r = subprocess.run([sys.executable, "-m", "pytest", *PIN_FILES, "-x", "-q", "-p", "no:cacheprovider"],
                       cwd=ROOT, env=env, capture_output=True, text=True)
    return name, r.returncode, r.stdout[-600:]


def test_every_planted_mistake_fails_a_pin(tmp_path):
    if os.environ.get("MXQ_ORACLE_LIB"):
        pytest.skip("already running against a replaced oracle build")
    with cf.ThreadPoolExecutor(max_workers=os.cpu_count() or 4) as ex:
        results = list(ex.map(lambda m: _run_pins_against(*m, str(tmp_path)), MUTANTS))
    survived = [name for name, rc, _ in results if rc == 0]
    broken = [(name, rc, out) for name, rc, out in results if rc not in (0, 1)]
    assert not broken, f"pin run did not finish normally: {broken[:2]}"
    assert not survived, f"no pin noticed: {survived}"
