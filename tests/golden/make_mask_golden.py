"""Writes tests/golden/mask_10_tokens.txt: the mask of Eq. 2 for a ten-token input as the oracle
computes it (a regression golden, not a value the paper prints: the paper's mask figure is an
image).  Run from the repository root: python tests/golden/make_mask_golden.py"""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.join(os.path.dirname(__file__), "..", ".."))
from oracle import sepllm_oracle as orc  # noqa: E402

# The ten-token input of the paper's mask figure caption, "ABC,DE.FG\n": the comma, the full stop
# and the newline (positions 3, 6, 9) are separators.
TEXT = "ABC,DE.FG\n"
FLAGS = np.array([ch in ",.\n" for ch in TEXT], dtype=bool)
A, N = 1, 2

if __name__ == "__main__":
    M = orc.mask_matrix(FLAGS, A, N)
    out = os.path.join(os.path.dirname(__file__), "mask_10_tokens.txt")
    with open(out, "w") as f:
        f.write("# Eq. 2 for the caption input ABC,DE.FG\\n (separators at 3, 6, 9), n_init = 1, n_neighbor = 2; rows = queries\n")
        for row in M:
            f.write("".join("1" if x else "." for x in row) + "\n")
    print(open(out).read())
