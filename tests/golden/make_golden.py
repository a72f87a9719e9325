"""Writes the stored expected values under tests/golden/.  Calls only oracle/ (and the seeded
input generator, which holds no arithmetic of the method).  Run from the repository root:

    python tests/golden/make_golden.py

tiny_fp32_rows.txt: rows of the operator's output on the tiny fp32 workload (B=1, 2 heads of
64, 4 frames of 8x8, chunk 1, overlap 1), evaluated by the direct form of Eq. 5-9 with the
causal sets of Eq. 13.  The paper itself prints no numeric example of the operator, so there
is no fixture that quotes it.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import rehyat_oracle as orc                      # noqa: E402
from paper_2601_04342_b200 import synth                      # noqa: E402

ROWS = [0, 1, 63, 64, 65, 127, 128, 191, 192, 200, 255]


def main():
    wl = synth.CONFIGS["tiny_fp32"]
    x = synth.to_f64(synth.make_inputs(wl))
    y = orc.hybrid_direct(x["q"], x["k"], x["v"], x["phi_q"], x["phi_k"], wl.T, wl.HW, wl.Tc, wl.To)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_fp32_rows.txt")
    with open(path, "w") as f:
        f.write("# head row then 64 output values; oracle direct form (Eq. 5-9, sets of Eq. 13), "
                "c = row max\n")
        for h in range(wl.n_heads):
            for r in ROWS:
                f.write(f"{h} {r} " + " ".join(f"{val:.17e}" for val in y[0, h, r]) + "\n")
    print("wrote", path)


if __name__ == "__main__":
    main()
