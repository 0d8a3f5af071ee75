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
