"""Writes tests/golden/exp_softplus_kat.txt: known answers (input bits -> output bits) of the two fixed binary32
routines the decode step feeds back through the recurrence, exp_spec and softplus_spec.

Run from the repository root: python tests/golden/make_spec_kat.py
Calls only the CPU oracle.  The table freezes today's bits, so that a later change that moved the oracle AND the
kernels together would still fail a test; the routines themselves are pinned by accuracy against float64 elsewhere.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402


def points(lo, hi, extra, seed):
    rng = np.random.default_rng(seed)
    z = np.concatenate([np.float32(extra), rng.uniform(lo, hi, 20).astype(np.float32),
                        (rng.uniform(-1, 1, 6) * np.float32(2.0) ** rng.integers(-30, -3, 6)).astype(np.float32)])
    return z.astype(np.float32)


def main():
    ze = points(-87.0, 5.0, [0.0, -0.0, -87.0, -100.0, 88.0, 100.0, -0.6931472, 0.6931472, -1.0, 1.0, -1e-10, -86.99999], 1)
    zs = points(-30.0, 25.0, [0.0, -0.0, 20.0, 20.000002, 19.999998, -20.0, 1.0, -1.0, 100.0, -100.0, 1e-8, -1e-8], 2)
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "exp_softplus_kat.txt")
    with open(out, "w") as f:
        f.write("# function  input bits  output bits   (binary32, hexadecimal)\n")
        f.write("# written by tests/golden/make_spec_kat.py from the CPU oracle; the decay a = exp(A dt) of Eq. 1 / Appendix B\n")
        f.write("# \"Runners\" and the step size dt = softplus(dt_raw + dt_bias) are fixed operation sequences in this build\n")
        for name, z, fn in (("exp_spec", ze, oracle.exp_spec), ("softplus_spec", zs, oracle.softplus_spec)):
            y = fn(z)
            for a, b in zip(z.view(np.uint32), y.view(np.uint32)):
                f.write(f"{name} {int(a):08x} {int(b):08x}\n")
    print(out)


if __name__ == "__main__":
    main()
