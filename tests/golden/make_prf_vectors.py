#!/usr/bin/env python
"""Writes tests/golden/prf_vectors.txt: stored outputs of the oracle's integer hash and of the two shared-PRF
masks (Section 3.1, M = g(layer, step, tokens, features)), so that a silent change of a constant, a shift or the
bit layout shows up as a failing pin.  Imports only oracle/; run from the repository root:

    python tests/golden/make_prf_vectors.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import spectral_oracle as so  # noqa: E402

HASH_INPUTS = [0, 1, 2, 3, 0xFFFFFFFF, 0x80000000, 0x7FFFFFFF, 0x9E3779B9, 0xDEADBEEF, 0x12345678, 1 << 16, 65535,
               1000003, 0xA5A5A5A5, 0x0F0F0F0F, 42]
MASK_ARGS = dict(seed=0x5EED, layer=3, step=17, tokens=4, features=16)


def bits(row):
    return "".join("1" if x else "0" for x in row)


def main():
    out = ["# Written by tests/golden/make_prf_vectors.py from oracle/ alone (regression pins, not paper values).",
           "# lowbias32 of 16 inputs, hexadecimal"]
    h = so.lowbias32(np.array(HASH_INPUTS, np.uint32))
    out += ["lowbias32 %08x %08x" % (x, int(y)) for x, y in zip(HASH_INPUTS, h)]
    out.append("# prf_keep_mask(seed=0x5EED, layer=3, step=17, tokens=4, features=16, keep=0.5): one row per token")
    for row in so.prf_keep_mask(keep=0.5, **MASK_ARGS):
        out.append("keep_mask " + bits(row))
    out.append("# prf_exact_k_mask(same arguments, keep=0.25): exactly 4 ones per row")
    for row in so.prf_exact_k_mask(keep=0.25, **MASK_ARGS):
        out.append("exact_k_mask " + bits(row))
    with open(os.path.join(ROOT, "tests", "golden", "prf_vectors.txt"), "w") as f:
        f.write("\n".join(out) + "\n")


if __name__ == "__main__":
    main()
