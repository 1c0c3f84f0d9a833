"""Pins of the oracle's binning, divergence, selection and whole-search steps
against exact rational arithmetic, high-precision decimals, library routines
(numpy.histogram, scipy.stats.entropy), closed forms and invariants.  CPU only."""
import math
import os
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle as O
from paper_2107_13490_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def exact_u(v, lo, hi, n_bins):
    return (Fraction(float(v)) - Fraction(float(lo))) * n_bins / (Fraction(float(hi)) - Fraction(float(lo)))


# ---- bins -------------------------------------------------------------------

def test_bin_index_matches_exact_rational_away_from_edges():
    rng = np.random.default_rng(4)
    x = rng.standard_normal(3000).astype(np.float32) * np.float32(0.05)
    lo, hi = x.min(), x.max()
    for n_bins in (1, 2, 50, 64, 150, 2048):
        checked = 0
        for v in x[:600]:
            u = exact_u(v, lo, hi, n_bins)
            fl_u = math.floor(u)
            if min(u - fl_u, fl_u + 1 - u) < Fraction(1, 1000) and n_bins > 1:
                continue  # within rounding distance of an edge: fp32 may fall either side
            want = min(max(fl_u, 0), n_bins - 1)
            assert O.bin_index(v, lo, hi, n_bins) == want
            checked += 1
        assert checked > 400


def test_bin_index_is_close_to_exact_everywhere_and_monotone():
    rng = np.random.default_rng(6)
    x = np.sort(rng.laplace(0, 0.02, 4000).astype(np.float32))
    lo, hi = x[0], x[-1]
    n_bins = 256
    bins = [O.bin_index(v, lo, hi, n_bins) for v in x]
    assert all(b1 <= b2 for b1, b2 in zip(bins, bins[1:]))
    for v, b in zip(x[::40], bins[::40]):
        u = float(exact_u(v, lo, hi, n_bins))
        assert abs(min(max(math.floor(u), 0), n_bins - 1) - b) <= 1
        assert b - 1e-3 <= u <= b + 1 + 1e-3 or b in (0, n_bins - 1)
    # walk the fp32 neighbours across one interior edge: index steps once, never back
    edge = np.float32(lo + (hi - lo) * np.float32(37.0 / 256))
    v = edge
    for _ in range(40):
        v = np.nextafter(v, np.float32(-np.inf))
    seq = []
    for _ in range(80):
        seq.append(O.bin_index(v, lo, hi, n_bins))
        v = np.nextafter(v, np.float32(np.inf))
    assert seq == sorted(seq) and seq[-1] - seq[0] == 1


def test_bin_edges_and_clamping():
    lo, hi = np.float32(-1.0), np.float32(3.0)
    assert O.bin_index(lo, lo, hi, 64) == 0
    assert O.bin_index(hi, lo, hi, 64) == 63            # right edge is inclusive
    assert O.bin_index(np.float32(3.5), lo, hi, 64) == 63  # above range -> last bin
    assert O.bin_index(np.float32(-7.0), lo, hi, 64) == 0  # below range -> first bin
    assert O.bin_index(np.float32(1.0), lo, hi, 4) == 2
    assert O.bin_index(np.float32(0.999999), lo, hi, 4) == 1
    # degenerate range: everything in bin 0
    assert O.bin_index(np.float32(5.0), np.float32(5.0), np.float32(5.0), 16) == 0
    assert O.bin_index(np.float32(9.0), np.float32(5.0), np.float32(5.0), 16) == 0
    # subnormal width: scale overflows to inf, (v - lo) = 0 gives 0*inf = NaN -> bin 0
    tiny = np.float32(1e-45)
    assert O.bin_index(np.float32(0.0), np.float32(0.0), tiny, 8) == 0
    assert O.bin_index(tiny, np.float32(0.0), tiny, 8) == 7


def test_histogram_matches_numpy_histogram_away_from_edges():
    rng = np.random.default_rng(9)
    x = rng.standard_normal(50000).astype(np.float32)
    lo, hi, bad = O.value_range(x)
    assert bad == 0 and lo == x.min() and hi == x.max()
    n_bins = 128
    u = (x.astype(np.float64) - float(lo)) * n_bins / (float(hi) - float(lo))
    safe = np.abs(u - np.rint(u)) > 1e-3
    safe |= (x == hi)
    h = O.histogram(x[safe], lo, hi, n_bins)
    ref, _ = np.histogram(x[safe].astype(np.float64), bins=n_bins, range=(float(lo), float(hi)))
    assert np.array_equal(h.astype(np.int64), ref)
    assert O.histogram(x, lo, hi, n_bins).sum() == x.size
    # out-of-range values are counted in the edge bins, so the total is kept
    y = np.concatenate([x, np.float32([hi + 1, lo - 1, hi * 2])])
    hy = O.histogram(y, lo, hi, n_bins)
    assert hy.sum() == y.size
    hx = O.histogram(x, lo, hi, n_bins)
    assert hy[-1] == hx[-1] + 2 and hy[0] == hx[0] + 1


def test_range_flags_nonfinite():
    x = np.float32([1.0, -2.0, 3.0])
    assert O.value_range(x) == (np.float32(-2.0), np.float32(3.0), 0)
    for bad in (np.nan, np.inf, -np.inf):
        y = x.copy()
        y[1] = bad
        assert O.value_range(y)[2] == 1


# ---- divergence -------------------------------------------------------------

def test_hand_worked_divergences():
    for line in open(os.path.join(GOLDEN, "kld_hand.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, q, val = line.split(";")
        base, *p = head.split()
        p = [int(t) for t in p]
        q = [int(t) for t in q.split()]
        b = math.e if base == "e" else float(base)
        got = O.kld(p, q, log_base=b)
        want = float(val)
        if math.isinf(want):
            assert math.isinf(got) and got > 0
        else:
            assert got == pytest.approx(want, rel=1e-12, abs=1e-15), line


def decimal_kld(p, q, base=2):
    getcontext().prec = 60
    n = Decimal(int(sum(p)))
    s = Decimal(0)
    for a, b in zip(p, q):
        if a == 0:
            continue
        pa, qb = Decimal(int(a)) / n, Decimal(int(b)) / n
        s += pa * (pa / qb).ln()
    return s / Decimal(base).ln()


def test_divergence_matches_textbook_sum_in_high_precision():
    rng = np.random.default_rng(10)
    for n_bins in (2, 7, 64, 300):
        q = rng.integers(1, 10 ** 6, n_bins)
        shift = rng.integers(-50, 51, n_bins)
        shift[-1] -= shift.sum()
        p = q + shift
        assert p.min() >= 0 and p.sum() == q.sum()
        want = decimal_kld(p, q)
        got = O.kld(p, q)
        assert got == pytest.approx(float(want), rel=1e-9)


def test_divergence_survives_cancellation_in_well_filled_bins():
    # 10^7 counts per bin, one count moved: KL ~ 1/(q N ln 2), far below the
    # rounding error of a naive p*log(p/q) sum in double precision.
    q = np.full(100, 10 ** 7, dtype=np.int64)
    p = q.copy()
    p[3] += 1
    p[60] -= 1
    want = float(decimal_kld(p, q))
    assert want > 0
    assert O.kld(p, q) == pytest.approx(want, rel=1e-7)


def test_divergence_matches_scipy_entropy():
    from scipy.stats import entropy
    rng = np.random.default_rng(13)
    q = rng.integers(1, 5000, 90)
    p = rng.permutation(q)
    assert O.kld(p, q) == pytest.approx(entropy(p, q, base=2), rel=1e-10)
    assert O.kld(p, q, log_base=math.e) == pytest.approx(entropy(p, q), rel=1e-10)
    assert O.kld(q, p) != pytest.approx(O.kld(p, q), rel=1e-3)  # direction matters


def test_divergence_properties():
    rng = np.random.default_rng(14)
    for _ in range(50):
        q = rng.integers(0, 40, 32)
        p = rng.permutation(q)
        d = O.kld(p, q)
        assert d >= 0.0                                    # Gibbs
        if np.array_equal(p, q):
            assert d == 0.0
        elif ((p > 0) & (q == 0)).any():
            assert math.isinf(d)
        else:
            assert d > 0.0
    h = rng.integers(0, 10 ** 9, 512)
    assert O.kld(h, h) == 0.0                              # exactly zero
    assert O.kld([0, 0, 0], [0, 0, 0]) == 0.0              # empty tensor
    # pseudo-count removes the infinity and stays a valid divergence
    d = O.kld([3, 1], [4, 0], alpha=0.5)
    want = (3.5 * math.log2(3.5 / 4.5) + 1.5 * math.log2(1.5 / 0.5)) / 5.0
    assert d == pytest.approx(want, rel=1e-12)


# ---- selection --------------------------------------------------------------

def test_select_lowest_candidate_meeting_eps():
    wl, fl = W.candidate_grid([4, 8])
    k = np.full(wl.size, 0.5)
    i84 = int(np.where((wl == 8) & (fl == 4))[0][0])
    i86 = int(np.where((wl == 8) & (fl == 6))[0][0])
    k[i84] = 0.0
    k[i86] = 0.0
    assert list(O.select(k, wl, fl, 0.0)) == [8, 4, i84, 1]
    k[int(np.where((wl == 4) & (fl == 3))[0][0])] = 1e-4
    assert list(O.select(k, wl, fl, 1e-3))[:2] == [4, 3]
    assert list(O.select(k, wl, fl, 0.0))[:2] == [8, 4]
    # order of the arrays does not matter, only (WL, FL)
    perm = np.random.default_rng(0).permutation(wl.size)
    out = O.select(k[perm], wl[perm], fl[perm], 0.0)
    assert list(out[:2]) == [8, 4] and perm[out[2]] == i84


def test_select_fallbacks():
    wl, fl = W.candidate_grid([2, 3])          # (2,0) (2,1) (3,0) (3,1) (3,2)
    k = np.array([0.7, 0.2, 0.9, 0.2, 0.4])
    assert list(O.select(k, wl, fl, 0.0)) == [2, 1, 1, 0]     # argmin, first among ties
    k = np.array([np.inf, np.inf, 0.3, np.inf, np.inf])
    assert list(O.select(k, wl, fl, 0.0)) == [3, 0, 2, 0]     # inf loses to finite
    k = np.full(5, np.inf)
    assert list(O.select(k, wl, fl, 0.0)) == [3, 2, 4, 0]     # all inf: last in order


def test_select_descent_from_current_format():
    # order: (2,0) (2,1) (3,0) (3,1) (3,2) (4,0) (4,1) (4,2) (4,3)
    wl, fl = W.candidate_grid([2, 3, 4])
    k = np.array([0.5, 0.0, 0.3, 0.0, 0.0, 0.0, 0.0, 0.2, 0.0])
    # from <4,1>: (4,1) ok, (4,0) ok, (3,2) ok, (3,1) ok, (3,0) loses information -> stop at (3,1)
    assert list(O.select_descent(k, wl, fl, 4, 1)) == [3, 1, 3, 1]
    # from <4,3>: (4,2) already loses information -> stays
    assert list(O.select_descent(k, wl, fl, 4, 3)) == [4, 3, 8, 1]
    # the start itself loses information: returned with the flag cleared
    assert list(O.select_descent(k, wl, fl, 4, 2)) == [4, 2, 7, 0]
    # a descent can end above the global lowest admissible format (2,1)
    assert list(O.select(k, wl, fl, 0.0))[:2] == [2, 1]
    # eps widens what counts as lossless: 0.3 admitted, the walk reaches (2,1)
    assert list(O.select_descent(k, wl, fl, 4, 1, eps=0.3))[:2] == [2, 1]
    # walking to the very first candidate, and a start outside the grid
    assert list(O.select_descent(np.zeros(9), wl, fl, 4, 3)) == [2, 0, 0, 1]
    assert list(O.select_descent(k, wl, fl, 5, 1)) == [5, 1, -1, 0]
    # array order does not matter
    perm = np.random.default_rng(1).permutation(9)
    out = O.select_descent(k[perm], wl[perm], fl[perm], 4, 1)
    assert list(out[:2]) == [3, 1] and perm[out[2]] == 3


# ---- the whole search -------------------------------------------------------

def _by_definition(x, wl, fl, n_bins, mode, seed, layer):
    """The search re-assembled from the separately pinned steps."""
    lo, hi, _ = O.value_range(x)
    qh = O.histogram(x, lo, hi, n_bins)
    _, xhat = O.quantize(x, wl, fl, mode, seed, layer)
    ph = O.histogram(xhat, lo, hi, n_bins)
    return qh, ph


@pytest.mark.parametrize("mode", [O.ROUND_RNE, O.ROUND_STOCHASTIC])
def test_search_outputs_are_consistent(mode):
    w = W.WORKLOADS["single4k"]
    x = W.generate(w)[0]
    wl, fl = w.grid()
    r = O.precision_search_layer(x, wl, fl, w.n_bins, mode, seed=7, layer=2, want_hist=True)
    assert r["nonfinite"] == 0
    assert (r["hist"].sum(axis=1) == x.size).all()
    assert (r["kld"] >= 0).all()
    for c in (0, 5, 17, 39):
        qh, ph = _by_definition(x, int(wl[c]), int(fl[c]), w.n_bins, mode, 7, 2)
        assert np.array_equal(r["hist"][0], qh) and np.array_equal(r["hist"][c + 1], ph)
        assert r["kld"][c] == O.kld(ph, qh)
        codes, _ = O.quantize(x, int(wl[c]), int(fl[c]), mode, 7, 2)
        assert r["zeros"][c] == (codes == 0).sum()
    same = [(r["hist"][c + 1] == r["hist"][0]).all() for c in range(wl.size)]
    assert [(k == 0.0) for k in r["kld"]] == same
    assert list(r["best"]) == list(O.select(r["kld"], wl, fl, 0.0))
    if mode == O.ROUND_RNE:
        for f in range(16):  # zero count does not depend on WL
            assert len({int(z) for z, ff in zip(r["zeros"], fl) if ff == f}) == 1


def test_search_saturation_folds_unsaturated_histogram():
    # For one FL the rounded value is the same for all WL; WL only clamps, and
    # the bin function is monotone, so the clamped histogram is the unclamped
    # one with both tails folded into the bins of the two saturation values.
    rng = np.random.default_rng(31)
    x = (rng.standard_normal(6000) * 3).astype(np.float32)
    n_bins = 100
    lo, hi, _ = O.value_range(x)
    for fl in (0, 2, 5):
        _, xu = O.quantize(x, 32, fl, O.ROUND_RNE)
        u = O.histogram(xu, lo, hi, n_bins).astype(np.int64)
        for wl in range(fl + 1, fl + 6):
            if wl < 2:
                continue
            _, xs = O.quantize(x, wl, fl, O.ROUND_RNE)
            h = O.histogram(xs, lo, hi, n_bins).astype(np.int64)
            bh = O.bin_index(O.dequantize_one((1 << (wl - 1)) - 1, fl), lo, hi, n_bins)
            bl = O.bin_index(O.dequantize_one(-(1 << (wl - 1)), fl), lo, hi, n_bins)
            want = np.zeros(n_bins, dtype=np.int64)
            for b in range(n_bins):
                want[min(max(b, bl), bh)] += u[b]
            assert np.array_equal(h, want), (wl, fl)


@pytest.mark.parametrize("mode", [O.ROUND_RNE, O.ROUND_STOCHASTIC])
def test_search_on_grid_tensor_loses_nothing(mode):
    rng = np.random.default_rng(40)
    codes0 = rng.integers(-128, 128, 5000)
    x = (codes0 * 2.0 ** -4).astype(np.float32)       # exactly on the <8,4> grid
    wl, fl = W.candidate_grid(range(2, 17))
    r = O.precision_search_layer(x, wl, fl, 150, mode, seed=3, layer=0)
    for c in range(wl.size):
        if fl[c] >= 4 and wl[c] - fl[c] >= 4:            # finer grid, at least the range
            assert r["kld"][c] == 0.0
    assert r["best"][3] & 1
    assert (r["best"][0], r["best"][1]) <= (8, 4)


def test_search_degenerate_cases():
    wl, fl = W.candidate_grid([2, 4, 8])
    r = O.precision_search_layer(np.full(100, 0.3, np.float32), wl, fl, 50)
    assert (r["kld"] == 0).all() and list(r["best"]) == [2, 0, 0, 3]
    r = O.precision_search_layer(np.zeros(0, np.float32), wl, fl, 50)
    assert (r["kld"] == 0).all() and (r["zeros"] == 0).all() and list(r["best"]) == [2, 0, 0, 3]
    r = O.precision_search_layer(np.float32([0.1, 0.7, -0.4]), wl, fl, 1)     # one bin
    assert (r["kld"] == 0).all()
    r = O.precision_search_layer(np.float32([0.1, np.nan]), wl, fl, 8)
    assert r["nonfinite"] == 1


def test_search_reaches_zero_once_quantum_is_below_every_margin():
    x = np.float32([0.1, 0.22, 0.37, 0.41, 0.58, 0.73, 0.9])
    wl, fl = W.candidate_grid([24])
    r = O.precision_search_layer(x, wl, fl, 8)
    assert (r["kld"][12:] == 0.0).all()        # 2^-13 is far below all bin-edge margins
    assert r["kld"][0] > 0                      # FL = 0 collapses everything onto {0, 1}


def test_threaded_farm_equals_sequential():
    w = W.WORKLOADS["resnet20_weights_grads"]
    xs = W.generate(w)
    pick = [0, 1, 20, 39]
    ts = [xs[i] for i in pick]
    wl, fl = W.candidate_grid([2, 5, 9])
    a = O.precision_search(ts, wl, fl, 64, O.ROUND_STOCHASTIC, 7, threads=1, want_hist=True)
    b = O.precision_search(ts, wl, fl, 64, O.ROUND_STOCHASTIC, 7, threads=4, want_hist=True)
    for ra, rb in zip(a, b):
        assert np.array_equal(ra["kld"], rb["kld"]) and np.array_equal(ra["zeros"], rb["zeros"])
        assert np.array_equal(ra["best"], rb["best"]) and np.array_equal(ra["hist"], rb["hist"])
