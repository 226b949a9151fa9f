"""Writes the stored expected values under tests/golden/ by calling only the CPU oracle.

    python tests/golden/make_golden.py

cfg1_oracle_out.txt: every 8th output row of benchmark configuration 1 (B=1, H=1, n=64, d=16,
r=8, eps=0.1, T=50, seed 0), float64.  The paper prints no worked numeric example, so this
file pins the oracle against accidental change, not against the paper; the paper-derived pins
(closed forms, marginals, rank) live in tests/test_oracle_pins.py.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import lot_oracle as O                      # noqa: E402
from paper_2509_23436_b200 import synth                 # noqa: E402


def main():
    x = synth.config(1)
    d = x.f64()
    out = O.attention_fwd(d["q"], d["k"], d["v"], d["z"], d["beta"], x.eps, x.iters)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg1_oracle_out.txt")
    np.savetxt(path, out[0, 0, ::8, :], fmt="%.17e",
               header="oracle float64, config 1 (seed 0), rows 0,8,...,56 of out[0,0]; written by make_golden.py")
    print("wrote", path)


if __name__ == "__main__":
    main()
