"""Pins of the oracle's other number formats (block floating point, floating point <E,M>).

Checked against things other than the oracle itself: hand-worked values (golden file), exact
rational arithmetic over an enumerated grid of representable values, IEEE half precision as
numpy casts it, bfloat16 and the 8-bit float types as torch casts them, and the fixed-point
oracle (pinned on its own) where a block-floating-point format coincides with <WL,FL>.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "formats_hand.txt")
KIND = {"fixed": O.FMT_FIXED, "bfp": O.FMT_BFP, "float": O.FMT_FLOAT}


def _rows(tag):
    with open(GOLDEN) as fh:
        for line in fh:
            parts = line.split()
            if parts and parts[0] == tag:
                yield parts[1:]


def test_golden_scales():
    n = 0
    for lo, hi, wl, s in _rows("scale"):
        assert O.bfp_scale(float(lo), float(hi), int(wl)) == int(s), (lo, hi, wl)
        n += 1
    assert n >= 10


def test_golden_values():
    n = 0
    for x, kind, a, b, mode, k, want in _rows("value"):
        got = O.format_value_one(float(x), KIND[kind], int(a), int(b),
                                 O.ROUND_RNE if mode == "rne" else O.ROUND_STOCHASTIC, int(k))
        assert got == float(want), (x, kind, a, b, mode, k, got)
        n += 1
    assert n >= 30


def _exact_scale(lo, hi, wl):
    """Largest s with hi*2^s <= UB+1/2 and -lo*2^s <= -LB+1/2, in rational arithmetic."""
    ub = Fraction(2 ** (wl - 1) - 1) + Fraction(1, 2)
    lb = Fraction(2 ** (wl - 1)) + Fraction(1, 2)
    lims = []
    if hi > 0:
        lims.append(ub / Fraction(float(hi)))
    if lo < 0:
        lims.append(lb / -Fraction(float(lo)))
    if not lims:
        return 0
    ratio = min(lims)
    s = 0
    while Fraction(2) ** (s + 1) <= ratio:
        s += 1
    while Fraction(2) ** s > ratio:
        s -= 1
    return max(-100, min(100, s))


def test_bfp_scale_against_rational_arithmetic():
    rng = np.random.default_rng(11)
    for _ in range(400):
        mag = 10.0 ** rng.uniform(-12, 12)
        lo = np.float32(-mag * rng.uniform(0, 1)) if rng.random() < 0.8 else np.float32(0)
        hi = np.float32(mag * rng.uniform(0, 1)) if rng.random() < 0.8 else np.float32(0)
        if lo > hi:
            lo, hi = hi, lo
        wl = int(rng.integers(2, 33))
        assert O.bfp_scale(lo, hi, wl) == _exact_scale(lo, hi, wl), (lo, hi, wl)
    # extremes on the boundary: hi = (UB + 0.5) * 2^-s exactly
    for wl in (2, 4, 8, 12):
        for s in (-5, 0, 7):
            hi = np.float32((2 ** (wl - 1) - 0.5) * 2.0 ** -s)
            assert O.bfp_scale(np.float32(0), hi, wl) == s
            assert O.bfp_scale(np.float32(0), np.nextafter(hi, np.float32(np.inf)), wl) == s - 1


def test_bfp_uses_the_word_and_equals_fixed_point():
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(5000) * 0.3).astype(np.float32)
    lo, hi, _ = O.value_range(x)
    for wl in (2, 3, 5, 8, 12, 16):
        s = O.bfp_scale(lo, hi, wl)
        v = O.format_quantize(x, O.FMT_BFP, wl, s)
        codes = v.astype(np.float64) * 2.0 ** s
        assert np.all(codes == np.rint(codes))
        assert codes.max() <= 2 ** (wl - 1) - 1 and codes.min() >= -(2 ** (wl - 1))
        # "maximum utilisation" of the word (Sec. 2.2): one more bit of scale would not fit
        top = max(hi * 2.0 ** (s + 1) / (2 ** (wl - 1) - 0.5), -lo * 2.0 ** (s + 1) / (2 ** (wl - 1) + 0.5))
        assert top > 1.0
        if 0 <= s <= wl - 1:
            _, xhat = O.quantize(x, wl, s)
            assert np.array_equal(v, xhat)


def _grid(e_bits, m_bits):
    """Every non-negative representable value of <E,M> as (Fraction, mantissa code)."""
    bias = 2 ** (e_bits - 1) - 1
    emin, emax = 1 - bias, bias
    vals = []
    for m in range(2 ** m_bits):                       # subnormals and zero
        vals.append((Fraction(m, 2 ** m_bits) * Fraction(2) ** emin, m))
    for e in range(emin, emax + 1):
        for m in range(2 ** m_bits):
            vals.append(((1 + Fraction(m, 2 ** m_bits)) * Fraction(2) ** e, m))
    return vals


def _nearest_even(xf, vals):
    """Nearest grid value to |x|; ties to the even mantissa code; beyond the top: the top."""
    ax = abs(xf)
    best = None
    for i, (v, m) in enumerate(vals):
        d = abs(v - ax)
        if best is None or d < best[0] or (d == best[0] and m % 2 == 0 and vals[best[1]][1] % 2 == 1):
            best = (d, i)
    v = vals[best[1]][0]
    return -v if xf < 0 else v


@pytest.mark.parametrize("e_bits,m_bits", [(2, 1), (3, 2), (4, 3), (3, 4), (5, 2)])
def test_float_format_against_enumerated_grid(e_bits, m_bits):
    vals = _grid(e_bits, m_bits)
    top = float(vals[-1][0])
    rng = np.random.default_rng(e_bits * 100 + m_bits)
    xs = np.concatenate([
        (rng.standard_normal(150) * top / 3).astype(np.float32),
        (rng.standard_normal(150) * float(vals[1][0]) * 4).astype(np.float32),
        np.array([float(v) for v, _ in vals[:40]], dtype=np.float32),          # on the grid
        np.array([float((vals[i][0] + vals[i + 1][0]) / 2) for i in range(0, min(40, len(vals) - 1))],
                 dtype=np.float32),                                            # exact ties
        np.array([top, -top, top * 1.01, top * 4, 0.0], dtype=np.float32)])
    got = O.format_quantize(xs, O.FMT_FLOAT, e_bits, m_bits)
    for x, g in zip(xs, got):
        want = _nearest_even(Fraction(float(x)), vals)
        assert Fraction(float(g)) == want, (float(x), float(g), float(want))


def _mixed_magnitudes(seed, n=20000):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal(n) * 10.0 ** rng.uniform(-9, 4.5, n)).astype(np.float32)


def test_half_precision_matches_numpy():
    x = _mixed_magnitudes(1)
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).astype(np.float32)
    got = O.format_quantize(x, O.FMT_FLOAT, 5, 10)
    fin = np.isfinite(want)
    assert fin.sum() > 15000 and (want == 0).sum() > 100
    assert np.array_equal(got[fin], want[fin])
    assert np.all(np.abs(got[~fin]) == 65504.0)          # overflow saturates


def test_bfloat16_and_float8_match_torch():
    x = _mixed_magnitudes(2)
    t = torch.from_numpy(x)
    want = t.to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O.format_quantize(x, O.FMT_FLOAT, 8, 7), want)
    # e5m2 is the IEEE-like <5,2>; e4m3fn has <4,3>'s grid up to 240 (it gives up infinities
    # for one more binade, so only values that stay below 240 are compared)
    x8 = (x * np.float32(1e-2)).astype(np.float32)
    w52 = torch.from_numpy(x8).to(torch.float8_e5m2).to(torch.float32).numpy()
    g52 = O.format_quantize(x8, O.FMT_FLOAT, 5, 2)
    fin = np.isfinite(w52)
    assert np.array_equal(g52[fin], w52[fin])
    small = np.abs(x8) < 200.0
    w43 = torch.from_numpy(x8[small]).to(torch.float8_e4m3fn).to(torch.float32).numpy()
    assert np.array_equal(O.format_quantize(x8[small], O.FMT_FLOAT, 4, 3), w43)


def test_full_width_float_is_the_identity():
    x = _mixed_magnitudes(3)
    assert np.array_equal(O.format_quantize(x, O.FMT_FLOAT, 8, 23), x)
    sub = np.array([1e-45, -3e-42, 1.1754942e-38], dtype=np.float32)   # subnormal inputs
    assert np.array_equal(O.format_quantize(sub, O.FMT_FLOAT, 8, 23), sub)


def test_stochastic_rounding_on_the_local_grid():
    """SR(x) of Sec. 3.2 on the format's grid: the result is one of the two neighbours, the
    upper one iff P < (x - lower) / quantum, in exact arithmetic."""
    e_bits, m_bits = 4, 3
    vals = sorted({v for v, _ in _grid(e_bits, m_bits)} | {-v for v, _ in _grid(e_bits, m_bits)})
    rng = np.random.default_rng(9)
    xs = (rng.standard_normal(300) * 3).astype(np.float32)
    checked = 0
    for i, x in enumerate(xs):
        xf = Fraction(float(x))
        lower = max(v for v in vals if v <= xf)
        upper = min(v for v in vals if v > xf)
        q = upper - lower
        if lower < 0 and lower + q > 0:
            continue      # the quantum changes across zero only for the lowest cell; skip it
        k = int(rng.integers(0, 1 << 24))
        got = Fraction(O.format_value_one(x, O.FMT_FLOAT, e_bits, m_bits, O.ROUND_STOCHASTIC, k))
        want = upper if Fraction(k, 1 << 24) < (xf - lower) / q else lower
        assert got == want, (float(x), k)
        checked += 1
    assert checked > 250
    # the tensor form draws k from the counter hash of (seed, layer, index)
    v = O.format_quantize(xs, O.FMT_FLOAT, e_bits, m_bits, O.ROUND_STOCHASTIC, seed=7, layer=2)
    for i in (0, 17, 299):
        assert v[i] == O.format_value_one(xs[i], O.FMT_FLOAT, e_bits, m_bits, O.ROUND_STOCHASTIC,
                                          O.hash24(7, 2, i))


def test_format_search_steps():
    rng = np.random.default_rng(4)
    x = (rng.standard_normal(4000) * 0.05).astype(np.float32)
    kinds = [O.FMT_BFP, O.FMT_FLOAT, O.FMT_FIXED, O.FMT_BFP, O.FMT_FLOAT, O.FMT_FLOAT]
    a = [4, 4, 8, 8, 5, 8]
    b = [0, 3, 6, 0, 10, 23]
    r = O.format_search_layer(x, kinds, a, b, 64)
    lo, hi, _ = O.value_range(x)
    q = O.histogram(x, lo, hi, 64)
    for c in range(len(kinds)):
        bc = O.bfp_scale(lo, hi, a[c]) if kinds[c] == O.FMT_BFP else b[c]
        assert r["b"][c] == bc
        v = O.format_quantize(x, kinds[c], a[c], bc)
        assert r["zeros"][c] == int((v == 0).sum())
        assert r["kld"][c] == O.kld(O.histogram(v, lo, hi, 64), q)
    # the fixed-point candidate agrees with the fixed-point search
    fx = O.precision_search_layer(x, [8], [6], 64)
    assert r["kld"][2] == fx["kld"][0] and r["zeros"][2] == fx["zeros"][0]
    # the identity format loses nothing, so with eps = 0 the first lossless one is chosen
    assert r["kld"][5] == 0.0
    first = int(np.argmax(r["kld"] <= 0.0))
    assert r["best"][2] == first and r["best"][3] & 1
    # with an unreachable eps the least divergence wins, first among ties
    r2 = O.format_search_layer(x, kinds[:4], a[:4], b[:4], 64, eps=-1.0)
    assert r2["best"][2] == int(np.argmin(r2["kld"])) and not (r2["best"][3] & 1)
    assert r2["best"][0] == a[r2["best"][2]] and r2["best"][1] == r2["b"][r2["best"][2]]
