"""Writes fma_pairs.txt: cases where a*b+c rounded once differs from rounding a*b then adding.

Exact rational arithmetic only (fractions + a local round-to-nearest-even to binary32);
calls neither the oracle nor the CUDA library.
"""
import os
import struct
from fractions import Fraction

import numpy as np


def rn32(q: Fraction) -> float:
    """Round an exact rational to binary32, nearest even (normal range only)."""
    if q == 0:
        return 0.0
    s = -1 if q < 0 else 1
    a = abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    if Fraction(2) ** (e + 1) <= a:
        e += 1
    quantum = Fraction(2) ** (e - 23)
    n = a / quantum
    fl = n.numerator // n.denominator
    rem = n - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return float(s * fl * quantum)


def bits(x: float) -> int:
    return struct.unpack("<I", struct.pack("<f", x))[0]


def main():
    rng = np.random.default_rng(12345)
    rows = []
    # the two hand-picked cases: w - lr*g and mu*v + g
    fixed = [("sub", 0.5, float(np.float32(0.01)), 2.69921875),
             ("add", 0.140625, float(np.float32(0.9)), 0.300048828125)]
    cands = list(fixed)
    for _ in range(4000):
        w = float(np.float32(rng.standard_normal()))
        g = float(np.float16(rng.standard_normal() * 3))
        cands.append(("sub", w, float(np.float32(0.01)), g))
        v = float(np.float32(rng.standard_normal() * 0.2))
        cands.append(("add", v, float(np.float32(0.9)), g))
    for kind, x, c, g in cands:
        X, C, G = Fraction(x), Fraction(c), Fraction(g)
        if kind == "sub":      # x - c*g
            sep = rn32(X - Fraction(rn32(C * G)))
            fused = rn32(X - C * G)
        else:                  # c*x + g
            sep = rn32(Fraction(rn32(C * X)) + G)
            fused = rn32(C * X + G)
        if sep != fused:
            rows.append((kind, bits(x), bits(c), bits(g), bits(sep), bits(fused)))
        if len(rows) >= 40:
            break
    here = os.path.dirname(os.path.abspath(__file__))
    with open(os.path.join(here, "fma_pairs.txt"), "w") as f:
        f.write("# kind x c g separately_rounded fused   (binary32 bit patterns, hex)\n")
        f.write("# kind sub: x - c*g ; kind add: c*x + g.  IEEE 754; written by make_fma_pairs.py\n")
        for r in rows:
            f.write("%s %08x %08x %08x %08x %08x\n" % r)


if __name__ == "__main__":
    main()
