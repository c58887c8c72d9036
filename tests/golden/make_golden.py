"""Writes the stored expected values under tests/golden/ that come from the oracle.

Calls only the CPU oracle and the seeded input generators. Run from the repo root:
    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2507_08771_b200 import inputs as I  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))


def main():
    sh, seed = I.SHAPES[0], I.config_seed(0)
    w = I.make_layer(sh, seed)
    x = I.make_x(sh.d, sh.L, seed)
    r = oracle.layer_forward(x, w["W_r"], w["gain"], w["U"], w["D"])
    with open(os.path.join(HERE, "tiny_layer_oracle.txt"), "w") as f:
        f.write("# tiny configuration (d=256, E=16, d_e=64, L=4, router on), seed 0xB10CFF:\n")
        f.write("# token, column, FFN output (Eq. 1-3) as computed by oracle/ in float64\n")
        for t in range(sh.L):
            for c in (0, 1, 37, 128, 255):
                f.write(f"{t} {c} {r.out[t, c]!r}\n".replace("np.float64(", "").replace(")", ""))
    with open(os.path.join(HERE, "tiny_layer_union.txt"), "w") as f:
        f.write("# union expert ids of the same chunk (Sec. 3.3), ascending\n")
        f.write(" ".join(str(int(i)) for i in r.union_ids[:r.n_union]) + "\n")


if __name__ == "__main__":
    main()
