"""Property tests (hypothesis) of the oracle against exact arithmetic and invariants. CPU only."""
import math
from fractions import Fraction

import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import oracle as O
from tests.test_oracle_quantize import exact_code, nearest_f32

f32s = st.floats(width=32, allow_nan=False, allow_infinity=False,
                 min_value=-(2.0 ** 63), max_value=2.0 ** 63)
formats = st.integers(2, 32).flatmap(lambda w: st.tuples(st.just(w), st.integers(0, w - 1)))


@settings(max_examples=300, deadline=None)
@given(x=f32s, fmt=formats, k=st.integers(0, 2 ** 24 - 1), mode=st.sampled_from([0, 1]))
def test_quantize_matches_exact_rational_arithmetic(x, fmt, k, mode):
    wl, fl = fmt
    code = O.quantize_one(x, wl, fl, mode, k)
    assert code == exact_code(float(np.float32(x)), wl, fl, mode, k)
    assert -(1 << (wl - 1)) <= code <= (1 << (wl - 1)) - 1
    assert O.dequantize_one(code, fl) == nearest_f32(Fraction(code, 1 << fl))


@settings(max_examples=200, deadline=None)
@given(vals=st.lists(f32s.filter(lambda v: abs(v) < 1e6), min_size=2, max_size=40),
       n_bins=st.integers(1, 300))
def test_bins_are_monotone_and_histograms_keep_every_element(vals, n_bins):
    x = np.sort(np.float32(vals))
    lo, hi, bad = O.value_range(x)
    assert bad == 0 and lo == x[0] and hi == x[-1]
    bins = [O.bin_index(v, lo, hi, n_bins) for v in x]
    assert all(0 <= b < n_bins for b in bins)
    assert bins == sorted(bins) and bins[0] == 0
    if hi > lo and np.isfinite(np.float32(n_bins) / (hi - lo)):
        assert bins[-1] == n_bins - 1
    h = O.histogram(x, lo, hi, n_bins)
    assert h.sum() == x.size
    assert np.array_equal(h, np.bincount(bins, minlength=n_bins).astype(np.uint64))


@settings(max_examples=200, deadline=None)
@given(data=st.data(), n_bins=st.integers(1, 64))
def test_divergence_is_a_divergence(data, n_bins):
    q = np.array(data.draw(st.lists(st.integers(0, 10 ** 6), min_size=n_bins, max_size=n_bins)))
    perm = data.draw(st.permutations(list(range(n_bins))))
    p = q[perm]                                    # same total, different placement
    d = O.kld(p, q)
    assert d >= 0.0
    if np.array_equal(p, q):
        assert d == 0.0
    elif ((p > 0) & (q == 0)).any():
        assert math.isinf(d)
    else:
        assert 0.0 < d < math.inf
        # against the textbook sum in double (no cancellation problem at these sizes)
        n = q.sum()
        m = p > 0
        ref = float((p[m] / n * np.log2(p[m] / q[m])).sum())
        assert abs(d - ref) <= 1e-9 * max(1.0, abs(ref)) + 1e-12
