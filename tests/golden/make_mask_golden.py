"""Writes tests/golden/mask_10_tokens.txt: the mask of Eq. 2 for a ten-token input as the oracle
computes it (a regression golden, not a value the paper prints: the paper's mask figure is an
image).  Run from the repository root: python tests/golden/make_mask_golden.py"""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.join(os.path.dirname(__file__), "..", ".."))
from oracle import sepllm_oracle as orc  # noqa: E402

# ten tokens, separators at positions 3 and 7 (a comma and a full stop in a short sentence)
FLAGS = np.array([0, 0, 0, 1, 0, 0, 0, 1, 0, 0], dtype=bool)
A, N = 1, 2

if __name__ == "__main__":
    M = orc.mask_matrix(FLAGS, A, N)
    out = os.path.join(os.path.dirname(__file__), "mask_10_tokens.txt")
    with open(out, "w") as f:
        f.write("# Eq. 2 for 10 tokens, separators at 3 and 7, n_init = 1, n_neighbor = 2; rows = queries\n")
        for row in M:
            f.write("".join("1" if x else "." for x in row) + "\n")
    print(open(out).read())
