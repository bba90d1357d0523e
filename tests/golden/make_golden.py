"""Writes the stored expected values under tests/golden/.  Calls only the CPU oracle.

    python tests/golden/make_golden.py

The paper prints no numeric example of the path (no entry of A, C or an update appears in it),
so these files freeze the generator definition this project adopted for Algorithm 1's
"A_W <- N_{s_W}(0, 1/r)": a change of a constant, of the counter layout or of the rounding
order shows up as a diff here.
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
from oracle import flora_oracle as orc  # noqa: E402


def main():
    with open(os.path.join(HERE, "projection_seed42_r8_m24.txt"), "w") as f:
        f.write("# A = N_seed(0, 1/r) for seed 42, r 8, m 24 (Algorithm 1, line 'A_W <- N_{s_W}(0,1/r)'):\n")
        f.write("# one row of A per line, fp32 bit patterns in hex; written by make_golden.py from the CPU oracle\n")
        A = orc.materialize_A(42, 8, 24)
        for row in A.view(np.uint32):
            f.write(" ".join(f"{int(x):08x}" for x in row) + "\n")
    with open(os.path.join(HERE, "philox_blocks.txt"), "w") as f:
        f.write("# Philox4x32-10 blocks: c0 c1 c2 c3 k0 k1 -> x0 x1 x2 x3 (hex); written by make_golden.py from the CPU oracle\n")
        for ctr, key in (([0, 0, 0, 0], [0, 0]), ([1, 2, 0, 0], [42, 0]), ([0xFFFFFFFF] * 4, [0xFFFFFFFF] * 2),
                         ([2751, 255, 0, 0], [0x9ABCDEF0, 0x12345678])):
            out = orc.philox4x32_10(ctr, key)
            f.write(" ".join(f"{int(x):08x}" for x in list(ctr) + list(key)) + " -> " +
                    " ".join(f"{int(x):08x}" for x in out) + "\n")


if __name__ == "__main__":
    main()
