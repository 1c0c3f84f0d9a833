"""Rewrites hash_vectors.txt from the CPU oracle (and nothing else).

Run from the repository root:  python tests/golden/make_hash_vectors.py
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import oracle  # noqa: E402

CASES = [(0, 0, 0), (7, 0, 0), (7, 3, 12345), (3, 0, 2 ** 30 - 1), (0, 0, 1), (0, 1, 0),
         (1, 0, 0), (2 ** 64 - 1, 2 ** 32, 2 ** 40 + 17), (7, 39, 36863), (123456789, 5, 4095)]


def main():
    path = os.path.join(HERE, "hash_vectors.txt")
    header = [l for l in open(path) if l.startswith("#")]
    with open(path, "w") as f:
        f.writelines(header)
        for s, l, i in CASES:
            f.write(f"{s} {l} {i} {oracle.hash24(s, l, i)}\n")


if __name__ == "__main__":
    main()
