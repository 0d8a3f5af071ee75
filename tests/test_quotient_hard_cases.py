"""The CUDA kernels form fl32(v / D) as a reciprocal multiply with one residual correction.  That is
the IEEE quotient for every pair of binary32 numbers: the argument is in the header of
``quotient_hard_cases.c``, which enumerates every pair whose quotient lies close enough to a rounding
boundary for the last rounding to go wrong, and checks them all on the host (about 6 s)."""
import os
import subprocess


def test_one_correction_quotient_on_every_hard_pair(tmp_path):
    here = os.path.dirname(os.path.abspath(__file__))
    exe = str(tmp_path / "quotient_hard_cases")
    subprocess.run(["gcc", "-O2", "-ffp-contract=off", "-o", exe, os.path.join(here, "quotient_hard_cases.c"), "-lm"], check=True)
    out = subprocess.run([exe], capture_output=True, text=True, check=True).stdout.split()
    tested, failures, uncorrected_wrong = int(out[1]), int(out[3]), int(out[5])
    assert failures == 0
    assert tested > 90_000_000                     # the enumeration found the pairs
    assert uncorrected_wrong > tested // 3         # and they are hard: the uncorrected quotient fails on many


def test_one_multiply_quotient_for_bf16_inputs_and_short_decode_scales():
    """For bf16 elements (8 significant bits) and decode scales of at most 4 significant bits the one-pass
    kernels take the FP4 code of RZ(v * RN(1 / D)) instead of that of fl(v / D).  Checked here for every
    bf16 significand over 30 binades, both signs and all eight scale significands (the claim is invariant
    under powers of two): the product is formed exactly in binary64 and truncated to binary32, the
    reference is the IEEE binary32 quotient; both are rounded onto the FP4 grid by an independent library."""
    import ml_dtypes
    import numpy as np

    sig = np.arange(128, 256, dtype=np.float64) / 128.0
    vals = np.concatenate([sig * 2.0 ** e for e in range(-15, 15)])
    vals = np.concatenate([vals, -vals, [0.0, -0.0]])

    def fp4(t):
        return np.clip(t, -6, 6).astype(np.float32).astype(ml_dtypes.float4_e2m1fn).astype(np.float32)

    def truncate_to_f32(x64):
        f = x64.astype(np.float32)
        over = np.abs(f.astype(np.float64)) > np.abs(x64)
        return np.where(over, np.nextafter(f, np.float32(0)), f).astype(np.float32)

    for m in range(8):
        for e in (-9, -3, 0, 8):
            D = np.float32((1 + m / 8.0) * 2.0 ** e)
            R = np.float32(1.0) / D                                   # RN(1 / D)
            assert np.float64(R) * np.float64(D) >= 1.0              # never below 1 / D for these significands
            want = vals.astype(np.float32) / D
            got = truncate_to_f32(vals * np.float64(R))               # 8 x 24 bits: exact in binary64
            assert np.array_equal(fp4(want), fp4(got)), (m, e)
            assert np.array_equal(np.signbit(want), np.signbit(got)), (m, e)
    # the rounding mode matters: with a round-to-nearest product the significand 1.875 fails on 2.34375 / 1.875 = 1.25
    D, v = np.float32(1.875), np.float32(2.34375)
    assert fp4(np.array([v / D]))[0] == 1.0 and fp4(np.array([v * (np.float32(1) / D)]))[0] == 1.5


def test_per_launch_check_of_the_one_multiply_quotient_for_long_decode_scales():
    """Under a tensor scale the decode scales D = fl(S g) have 24 significant bits, and whether the FP4 code
    of RZ(v * R) is that of fl(v / D) for every bf16 v depends on how the roundings fall next to the FP4
    midpoints.  The kernels find out per launch: for a reciprocal R (RN(1 / D) or one of its two
    neighbours) they compare the two codes on the fourteen bf16 values next to M * D (floor to bf16 and
    the value after it, M the seven rounding midpoints of the FP4 grid) and use R only if all agree.
    This test models that check in numpy and compares its verdict with the truth, found by trying EVERY
    positive normal bf16 value: the verdicts must coincide (a passing reciprocal is right everywhere, a
    failing one is wrong somewhere), on scales from random tensor scales, on scales built to sit next to
    (bf16 value) / midpoint, and on the scales of g = amax / 2688 for every bf16 amax significand, where
    it also counts how often some candidate passes in all eight significand classes."""
    import ml_dtypes
    import numpy as np

    f32 = np.float32
    mids = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]
    every_bf16 = (np.arange(0x0080, 0x7F80, dtype=np.uint32) << 16).view(f32)       # positive normal bf16 values

    def fp4(t):
        return np.minimum(t, f32(6)).astype(f32).astype(ml_dtypes.float4_e2m1fn).astype(f32)

    def mul_rz(v, R):
        p = v.astype(np.float64) * np.float64(R)                                    # exact
        with np.errstate(over="ignore"):
            f = p.astype(f32)
        f = np.where(np.isinf(f), np.finfo(f32).max, f)
        return np.where(f.astype(np.float64) > p, np.nextafter(f, f32(0)), f).astype(f32)

    def codes_agree(v, D, R):
        with np.errstate(over="ignore"):
            want = (v / D).astype(f32)
        return fp4(want) == fp4(mul_rz(v, R))

    def launch_check(D, R):
        ok = True
        for m in mids:
            p = np.float64(m) * np.float64(D)
            f = f32(p)
            if np.float64(f) > p:
                f = np.nextafter(f, f32(0))
            b0 = np.array([f]).view(np.uint32) & np.uint32(0xFFFF0000)
            pair = np.concatenate([b0, b0 + np.uint32(0x10000)]).view(f32)
            ok = ok and bool(np.all(codes_agree(pair, D, R)))
        return ok

    def candidates(D):
        R = f32(1) / D
        return [R, np.nextafter(R, f32(np.inf)), np.nextafter(R, f32(0))]

    rng = np.random.default_rng(2605)
    scales = []
    ue4m3 = [(1 + (c & 7) / 8) * 2.0 ** ((c >> 3) - 7) if c >= 8 else (c & 7) * 2.0 ** -9 for c in range(1, 127)]
    for _ in range(2):                                                              # every UE4M3 code under random tensor scales
        g = f32(np.exp(rng.uniform(np.log(1e-5), np.log(10.0))))
        scales += [f32(f32(s) * g) for s in ue4m3]
    for _ in range(300):                                                            # scales next to (bf16 value) / midpoint
        v = every_bf16[int(rng.integers(0x3000 - 0x80, 0x4F00 - 0x80))]
        D = f32(np.float64(v) / mids[int(rng.integers(0, 7))])
        for _k in range(int(rng.integers(0, 4))):
            D = np.nextafter(D, f32(np.inf) if rng.integers(0, 2) else f32(0))
        scales.append(D)
    passed = failed = 0
    for D in scales:
        for R in candidates(D)[:1 + int(rng.integers(0, 3))]:
            verdict = launch_check(D, R)
            truth = bool(np.all(codes_agree(every_bf16, D, R)))
            assert verdict == truth, (float(D), float(R), verdict, truth)
            passed += int(verdict)
            failed += int(not verdict)
    assert passed > 600 and failed > 50                                             # both kinds were seen

    # hierarchical scaling of bf16 tensors: g = fl(amax / 2688), the eight significand classes fl((1 + m / 8) g)
    plain = rescued = 0
    for s in range(128, 256):
        g = f32(f32(s / 128.0) / f32(2688.0))
        ok_plain = ok_any = True
        for m in range(8):
            D = f32(f32(1 + m / 8) * g)
            verdicts = [launch_check(D, R) for R in candidates(D)]
            if s % 16 == 0:                                                         # spot-check these against the truth too
                for R, verdict in zip(candidates(D), verdicts):
                    assert verdict == bool(np.all(codes_agree(every_bf16, D, R)))
            ok_plain = ok_plain and verdicts[0]
            ok_any = ok_any and any(verdicts)
        plain += int(ok_plain)
        rescued += int(ok_any)
    assert plain < 64 and rescued >= 120, (plain, rescued)                          # RN(1 / D) alone fails for most amax; a neighbour nearly always works
