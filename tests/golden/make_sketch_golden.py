"""Writes tests/golden/sketch_v1_bits.txt from the oracle alone (never from the CUDA path).

Run from the repository root:  python tests/golden/make_sketch_golden.py
The file freezes a few bit patterns of the "Gaussian v1" sketch so that an accidental change to
oracle/sketch.py shows up as a failing CPU test.
"""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from oracle import sketch as sk  # noqa: E402

CASES = [(0, 256, 16), (42, 896, 64), (0xDEADBEEFCAFEF00D, 3072, 128), (7, 8192, 256)]
PICKS = [(0, 0), (0, 1), (0, 2), (0, 3), (1, 0), (5, 7), (-1, -1), (-3, 9)]


def main():
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "sketch_v1_bits.txt")
    with open(out, "w") as f:
        f.write("# seed d_in r i j fp32_bits bf16_bits   (written by make_sketch_golden.py from oracle/sketch.py)\n")
        for seed, d_in, r in CASES:
            s = sk.sketch(seed, d_in, r)
            b = sk.round_to_bf16(s)
            for (i, j) in PICKS:
                i, j = i % d_in, j % r
                f.write("%x %d %d %d %d %08x %04x\n" % (seed, d_in, r, i, j, s[i:i + 1, j].view(np.uint32)[0],
                                                       b[i:i + 1, j].view(np.uint32)[0] >> 16))
            f.write("%x %d %d sum_fp32_bits_xor - %08x -\n" % (seed, d_in, r, np.bitwise_xor.reduce(s.view(np.uint32).ravel())))


if __name__ == "__main__":
    main()
