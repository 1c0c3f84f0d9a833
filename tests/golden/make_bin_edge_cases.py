"""Writes tests/golden/bin_edge_cases.txt: values at bin edges where the order and
precision of the bin arithmetic decide the bin.

    python tests/golden/make_bin_edge_cases.py

The shared bins (Sec. 3.3, the EDF at resolution r) are evaluated as separate fp32
operations: w = hi - lo; scale = r / w; t = v - lo; u = t * scale; floor; clamp.  This
script walks the fp32 neighbours of every interior edge of a few (lo, hi, r) and keeps
the values for which another plausible evaluation - the product left unrounded, a
division first, everything in double, the real-number definition - gives a different
bin.  The stored expected bin is the ORACLE's (adapt_oracle_bin_index); the integer
model of tests/f32_model.py only selects the rows and records what each other
evaluation would have given.  Nothing here calls the CUDA library.
"""
import os
import struct
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import oracle as O  # noqa: E402
from tests import f32_model as M  # noqa: E402

CASES = [  # (lo, hi, n_bins)
    (-0.731, 0.694, 2048), (-1.3, 2.7, 64), (0.0, 4.2113953, 512), (-0.21, 0.19, 100),
    (1000.0, 1000.01, 37), (-3.0e-4, 2.5e-4, 150), (-123456.0, -123392.0, 256), (0.5, 1.0, 50),
]
MAX_ROWS_PER_VARIANT = 12


def bits(x):
    return struct.unpack("<I", struct.pack("<f", float(x)))[0]


def main():
    rows, per_variant = [], {k: 0 for k in M.VARIANTS}
    for lo, hi, nb in CASES:
        lo, hi = np.float32(lo), np.float32(hi)
        flo, fhi = M.frac_of_f32(lo), M.frac_of_f32(hi)
        for b in range(1, nb):
            centre = np.float32(float(flo + (fhi - flo) * b / nb))
            v = centre
            for _ in range(6):
                v = np.nextafter(v, np.float32(-np.inf))
            for _ in range(13):
                fv = M.frac_of_f32(v)
                want = M.bin_separate_fp32_ops(fv, flo, fhi, nb)
                other = {k: f(fv, flo, fhi, nb) for k, f in M.VARIANTS.items()}
                differing = [k for k in other if other[k] != want]
                if differing and any(per_variant[k] < MAX_ROWS_PER_VARIANT for k in differing):
                    for k in differing:
                        per_variant[k] += 1
                    expected = O.bin_index(v, lo, hi, nb)       # the stored value is the oracle's
                    rows.append("%08x %08x %08x %d %d %s" % (
                        bits(v), bits(lo), bits(hi), nb, expected,
                        " ".join("%s=%d" % (k, other[k]) for k in sorted(other))))
                v = np.nextafter(v, np.float32(np.inf))
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "bin_edge_cases.txt")
    with open(out, "w") as f:
        f.write("# Values next to bin edges where the evaluation order of the bin index matters.\n"
                "# Shared bins of Sec. 3.3 (EDF at resolution r), evaluated as separate fp32 operations\n"
                "# w = hi - lo; scale = r / w; t = v - lo; u = t * scale; floor; clamp.\n"
                "# Columns: v lo hi (fp32 bit patterns, hex)  r  bin by the oracle  then the bin each\n"
                "# other evaluation would give (integer model).  Written by make_bin_edge_cases.py.\n")
        f.write("\n".join(rows) + "\n")
    print(len(rows), "rows", per_variant)


if __name__ == "__main__":
    main()
