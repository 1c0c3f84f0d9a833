"""Pin of the oracle's bin index AT the bin edges (shared bins of Sec. 3.3).

Every histogram, divergence and chosen format hangs on which side of an edge a value
falls, and that is decided by the order and precision of five fp32 operations:
w = hi - lo; scale = r / w; t = v - lo; u = t * scale; floor.  An integer model of fp32
rounding on exact rationals (tests/f32_model.py) evaluates that sequence without the
machine's float unit; the oracle must agree with it at, below and above every edge.
The stored cases are values where another plausible sequence (product left unrounded,
division first, all in double, the real-number definition) lands in the other bin.
CPU only."""
import os
import struct
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle as O
from tests import f32_model as M

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "bin_edge_cases.txt")


def f32_from_bits(h):
    return np.float32(struct.unpack("<f", struct.pack("<I", int(h, 16)))[0])


def test_integer_model_reproduces_ieee_single_operations():
    """The model itself, against the hardware's fp32 add / multiply / divide."""
    rng = np.random.default_rng(314)
    a = (rng.standard_normal(400) * np.exp2(rng.integers(-20, 20, 400))).astype(np.float32)
    b = (rng.standard_normal(400) * np.exp2(rng.integers(-20, 20, 400))).astype(np.float32)
    for x, y in zip(a, b):
        fx, fy = M.frac_of_f32(x), M.frac_of_f32(y)
        assert M.rn32(fx - fy) == Fraction(float(np.float32(x - y)))
        assert M.rn32(fx * fy) == Fraction(float(np.float32(x * y)))
        if y != 0:
            assert M.rn32(fx / fy) == Fraction(float(np.float32(x / y)))
            assert M.rn64(fx / fy) == Fraction(float(x) / float(y))
    # ties go to even, also in the subnormal range
    assert M.rn32(Fraction(1) + Fraction(1, 1 << 24)) == 1
    assert M.rn32(Fraction(1) + Fraction(3, 1 << 24)) == Fraction(1) + Fraction(1, 1 << 22)
    assert M.rn32(Fraction(3, 1 << 150)) == Fraction(1, 1 << 148)
    assert M.rn32(Fraction(1, 1 << 150)) == 0


@pytest.mark.parametrize("lo,hi,n_bins", [
    (-0.731, 0.694, 2048), (-1.3, 2.7, 64), (0.0, 4.2113953, 512), (-0.21, 0.19, 100),
    (1000.0, 1000.01, 37), (-3.0e-4, 2.5e-4, 150), (-7.5, -1.25, 3), (2.0 ** -130, 2.0 ** -120, 16),
])
def test_oracle_follows_the_separate_fp32_operations_at_every_edge(lo, hi, n_bins):
    lo, hi = np.float32(lo), np.float32(hi)
    flo, fhi = M.frac_of_f32(lo), M.frac_of_f32(hi)
    disagree_with_exact = 0
    for b in range(1, n_bins):
        v = np.float32(float(flo + (fhi - flo) * b / n_bins))
        for _ in range(5):
            v = np.nextafter(v, np.float32(-np.inf))
        seen = []
        for _ in range(11):
            fv = M.frac_of_f32(v)
            want = M.bin_separate_fp32_ops(fv, flo, fhi, n_bins)
            assert O.bin_index(v, lo, hi, n_bins) == want, (float(v), b)
            disagree_with_exact += want != M.bin_exact(fv, flo, fhi, n_bins)
            seen.append(want)
            v = np.nextafter(v, np.float32(np.inf))
        assert seen == sorted(seen) and seen[0] <= b <= seen[-1] + 1     # monotone, around bin b
    # the two ends and values outside the range
    for v in (lo, hi, np.nextafter(lo, np.float32(-np.inf)), np.nextafter(hi, np.float32(np.inf)),
              np.nextafter(hi, np.float32(-np.inf))):
        assert O.bin_index(v, lo, hi, n_bins) == M.bin_separate_fp32_ops(M.frac_of_f32(v), flo, fhi, n_bins)
    if n_bins >= 100:
        assert disagree_with_exact > 0     # the sweep did reach values where rounding decides


def test_stored_edge_cases_where_other_evaluations_differ():
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 20
    differs = {k: 0 for k in M.VARIANTS}
    for v_h, lo_h, hi_h, nb, expected, *others in rows:
        v, lo, hi, nb, expected = f32_from_bits(v_h), f32_from_bits(lo_h), f32_from_bits(hi_h), int(nb), int(expected)
        fv, flo, fhi = M.frac_of_f32(v), M.frac_of_f32(lo), M.frac_of_f32(hi)
        assert O.bin_index(v, lo, hi, nb) == expected
        assert M.bin_separate_fp32_ops(fv, flo, fhi, nb) == expected
        stored = dict(o.split("=") for o in others)
        wrong = 0
        for name, fn in M.VARIANTS.items():
            got = fn(fv, flo, fhi, nb)
            assert got == int(stored[name])
            if got != expected:
                differs[name] += 1
                wrong += 1
        assert wrong >= 1
    assert all(n > 0 for n in differs.values()), differs


def test_histogram_of_edge_values_matches_the_model():
    """The tensor-level histogram uses the same rule: a tensor made of edge neighbours."""
    lo, hi, nb = np.float32(-0.731), np.float32(0.694), 256
    flo, fhi = M.frac_of_f32(lo), M.frac_of_f32(hi)
    vals = [lo, hi]
    for b in range(1, nb):
        v = np.float32(float(flo + (fhi - flo) * b / nb))
        vals += [np.nextafter(v, np.float32(-np.inf)), v, np.nextafter(v, np.float32(np.inf))]
    vals = np.array(vals, dtype=np.float32)
    want = np.zeros(nb, dtype=np.uint64)
    for v in vals:
        want[M.bin_separate_fp32_ops(M.frac_of_f32(v), flo, fhi, nb)] += 1
    assert np.array_equal(O.histogram(vals, lo, hi, nb), want)
