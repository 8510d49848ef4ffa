"""Writes tests/golden/tiny_cycles.txt: per-cycle error-vs-serial and residual norms of the fp64 oracle on the
tiny configuration (T=64, B=2, I=16, H=32, c_f=4, two levels, implicit cell; seed 0, inputs NOT rounded to
fp32).  Calls only oracle/ and NumPy.  The file is a regression fixture for the oracle's finite-cycle iterates,
which have no closed form and which the paper does not print (parity unpinned).
Run:  python tests/golden/make_golden.py"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import mgrit_gru_oracle as O  # noqa: E402


def tiny_fp64():
    rng = np.random.default_rng(0)
    H, I, B, T = 32, 16, 2, 64
    k = 1 / np.sqrt(H)
    Wi = rng.uniform(-k, k, (3 * H, I)); Wh = rng.uniform(-k, k, (3 * H, H))
    bi = rng.uniform(-k, k, 3 * H); bh = rng.uniform(-k, k, 3 * H)
    x = rng.standard_normal((T, B, I))
    return (Wi, Wh, bi, bh), x, np.zeros((B, H))


def rows():
    P, x, h0 = tiny_fp64()
    hs = O.serial_forward(*P, x, h0)
    out = []
    for relax in (O.RELAX_F, O.RELAX_FCF):
        for it in (1, 2, 3, 4):
            h, res = O.mgrit_forward(*P, x, h0, 4, 2, it, relax_fine=relax)
            out.append((relax, it, float(np.max(np.abs(h - hs))), res[-1]))
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_cycles.txt")
    with open(path, "w") as f:
        f.write("# written by tests/golden/make_golden.py from oracle/ only: relax(0=F,1=FCF) cycles max|h-h_serial| residual_of_last_cycle\n")
        for r in rows():
            f.write("%d %d %.10e %.10e\n" % r)
    print(open(path).read())
