"""Writes tests/golden/oracle_seed0.txt from the oracle alone (run from the repo root).

The file is a regression fixture of the oracle's own seeded output: the first
eight Philox words of stream 0 under seed 0, and the 4 x 4 orthogonal mixing
matrix of seed 0.  The paper prints no worked numeric example, so no value in
it comes from the paper; the words are additionally checked in the tests
against an independent Philox4x32-10 implementation.
"""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
import oracle  # noqa: E402

here = os.path.dirname(os.path.abspath(__file__))
w = oracle.philox_words(0, 0, 0, 0, 8)
A, _ = oracle.sample_mixing(4, 0, seed=0)
with open(os.path.join(here, "oracle_seed0.txt"), "w") as f:
    f.write("# written by tests/golden/make_golden.py from oracle/ only\n")
    f.write("# Philox4x32-10, key = seed 0, counter = (block, 0, stream 0, attempt 0): words of elements 0..7\n")
    f.write("philox_words_seed0_stream0: " + " ".join(f"{int(x):08x}" for x in w) + "\n")
    f.write("# Section 3.2 step 1.2 with the orthogonal construction: Q of QR(G0), diag(R) > 0, row-major\n")
    f.write("orthogonal_A_m4_seed0: " + " ".join(repr(float(x)) for x in A.ravel()) + "\n")
