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
