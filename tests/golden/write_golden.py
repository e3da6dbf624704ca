"""Writes the stored expected values under tests/golden/ by calling the CPU oracle only.

Run from the repository root:  python tests/golden/write_golden.py

codebook_dynamic_tree.txt : the 256 fp32 codes as hex bit patterns, one per line, plus the
                            SHA-256 of their 1024 little-endian bytes.  Definition: the
                            dynamic-tree 8-bit map over [-1, 1] (sign bit, decade chosen by
                            the exponent field, linear fraction), used for the "dynamic
                            blockwise quantization" of the paper's section "Compression
                            techniques", item 1.
thresholds_round_down.txt : the 255 midpoints between neighbouring codes, each rounded
                            toward -inf to fp32 (hex), plus their SHA-256.

These files are REGRESSION pins: they hold what the oracle produced when they were written, so
they catch a later change of the oracle, not a mistake it had from the start.  The checks of the
codebook against its definition are elsewhere (tests/test_oracle_codebook.py): the rebuild of all
256 values in exact rational arithmetic, the decoding of the eight bit fields, and the mirror /
sum / decade invariants.
"""
import hashlib
import os
import struct
import sys
from fractions import Fraction

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402


def hexf(v) -> str:
    return "0x%08x" % struct.unpack("<I", struct.pack("<f", float(v)))[0]


def main() -> None:
    cb = oracle.make_codebook()
    with open(os.path.join(HERE, "codebook_dynamic_tree.txt"), "w") as f:
        f.write("# dynamic-tree codebook, fp32 bit patterns, index ascending (regression pin: written by write_golden.py from oracle/; the definition is checked by the exact-rational rebuild in test_oracle_codebook.py)\n")
        for v in cb:
            f.write(hexf(v) + "\n")
        f.write("sha256 " + hashlib.sha256(cb.astype("<f4").tobytes()).hexdigest() + "\n")
    # midpoints, rounded down, from the oracle's codes in exact rational arithmetic
    down = []
    for j in range(255):
        t = (Fraction(float(cb[j])) + Fraction(float(cb[j + 1]))) / 2
        g = np.float32(float(t))
        if Fraction(float(g)) > t:
            g = np.nextafter(g, np.float32(-np.inf))
        down.append(g)
    down = np.array(down, np.float32)
    with open(os.path.join(HERE, "thresholds_round_down.txt"), "w") as f:
        f.write("# midpoints between neighbouring codes, rounded toward -inf to fp32 (regression pin: written by write_golden.py from the oracle's codes in exact rationals)\n")
        for v in down:
            f.write(hexf(v) + "\n")
        f.write("sha256 " + hashlib.sha256(down.astype("<f4").tobytes()).hexdigest() + "\n")


if __name__ == "__main__":
    main()
