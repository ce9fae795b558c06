"""Writes the stored expected values under tests/golden/ by calling only the CPU oracle.

Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402


def main():
    cases = [(0, 0, 0), (0, 0, 1), (0, 1, 0), (1, 0, 0), (4, 9, 7), (2**32, 2**33, 31),
             (2**64 - 1, 2**64 - 1, 2**64 - 1), (123456789, 987654321, 5)]
    cases += [(s, t, w) for s in (3, 4) for t in (0, 19) for w in (0, 15)]
    with open(os.path.join(HERE, "rng_kat.txt"), "w") as f:
        f.write("# counter RNG known answers: seed step worker hash64(hex) uniform(hex float)\n")
        f.write("# hash = three chained SplitMix64 output rounds (the method's level draw, Alg. 2 'Sample l ~ p^l',\n")
        f.write("# needs one uniform per worker per step; the generator itself is this build's choice)\n")
        for s, t, w in cases:
            f.write(f"{s} {t} {w} {oracle.hash64(s, t, w):016x} {oracle.uniform(s, t, w).hex()}\n")


if __name__ == "__main__":
    main()
