"""Pins of the oracle's quantizer against things other than itself:
hand-worked values, exact rational arithmetic (Python Fraction / big ints),
closed forms and invariants.  CPU only."""
import math
import os
import struct
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f32(x):
    return float(np.float32(x))


def frac_of_f32(x):
    """Exact rational value of an fp32 number, from its bit pattern."""
    bits = struct.unpack("<I", struct.pack("<f", x))[0]
    sign = -1 if bits >> 31 else 1
    e = (bits >> 23) & 0xFF
    m = bits & 0x7FFFFF
    if e == 0:
        return sign * Fraction(m, 1 << 149)
    return sign * Fraction((1 << 23) | m, 1) * Fraction(2) ** (e - 150)


def nearest_f32(q: Fraction) -> float:
    """Round a rational to the nearest fp32 (ties to even) with integer arithmetic."""
    if q == 0:
        return 0.0
    s = -1 if q < 0 else 1
    a = abs(q)
    e = math.floor(math.log2(a)) if a >= 1 else -math.ceil(math.log2(1 / a))
    while Fraction(2) ** e > a:
        e -= 1
    while Fraction(2) ** (e + 1) <= a:
        e += 1
    e = max(e, -126)
    ulp = Fraction(2) ** (e - 23)
    k = a / ulp
    lo = k.numerator // k.denominator
    rem = k - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (lo & 1)):
        lo += 1
    return float(s * lo * ulp)


def rne_int(q: Fraction) -> int:
    return round(q)  # Fraction.__round__ rounds halves to even


def exact_code(x: float, wl: int, fl: int, mode: int, k24: int) -> int:
    """The definition in exact arithmetic: scale, round, saturate."""
    y = frac_of_f32(x) * (1 << fl)
    if mode == O.ROUND_RNE:
        r = rne_int(y)
    else:
        f = math.floor(y)
        frac = nearest_f32(y - f)  # the one inexact step of the rule: an fp32 subtraction
        r = f + (1 if Fraction(k24, 1 << 24) < Fraction(frac) else 0)
    top = 1 << (wl - 1)
    return max(-top, min(top - 1, r))


def read_rows(name):
    rows = []
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append(line)
    return rows


def test_hand_worked_quantizations():
    for row in read_rows("quantize_hand.txt"):
        x, wl, fl, mode, k, code, xhat = row.split()
        m = O.ROUND_RNE if mode == "rne" else O.ROUND_STOCHASTIC
        got = O.quantize_one(float(x), int(wl), int(fl), m, int(k))
        assert got == int(code), row
        assert O.dequantize_one(got, int(fl)) == float(xhat), row


def test_nearest_f32_helper_matches_numpy():
    rng = np.random.default_rng(5)
    for v in rng.standard_normal(200) * 10.0 ** rng.integers(-8, 8, 200):
        assert nearest_f32(Fraction(float(v))) == f32(v)


def _sample_floats(rng, n):
    mant = rng.standard_normal(n).astype(np.float32)
    expo = rng.integers(-36, 34, n)
    x = (mant * np.exp2(expo).astype(np.float32)).astype(np.float32)
    special = np.array([0.0, -0.0, 0.5, -0.5, 1.5, 2.5, -2.5, 2 ** -32, -2 ** -33, 2 ** -31 * 1.5,
                        2 ** 30, -2 ** 31, 2 ** 31, 1e-45, -1e-45, 16777216.0, 16777217.0,
                        8388607.5, -8388608.5, 0.49999997, 0.50000006], dtype=np.float32)
    return np.concatenate([x, special])


def test_rne_codes_match_exact_rational_bruteforce():
    rng = np.random.default_rng(11)
    xs = _sample_floats(rng, 160)
    for wl in (2, 3, 4, 8, 12, 16, 24, 25, 26, 31, 32):
        for fl in sorted({0, 1, wl // 2, wl - 1}):
            codes, xhat = O.quantize(xs, wl, fl, O.ROUND_RNE)
            for x, c, xh in zip(xs, codes, xhat):
                assert c == exact_code(float(x), wl, fl, O.ROUND_RNE, 0), (x, wl, fl)
                assert float(xh) == nearest_f32(Fraction(int(c), 1 << fl)), (x, wl, fl)


def test_stochastic_codes_match_exact_rational_bruteforce():
    rng = np.random.default_rng(12)
    xs = _sample_floats(rng, 120)
    seed, layer = 99, 4
    for wl, fl in ((2, 1), (4, 3), (8, 4), (16, 7), (16, 15), (32, 0), (32, 31), (27, 20)):
        codes, _ = O.quantize(xs, wl, fl, O.ROUND_STOCHASTIC, seed, layer)
        for i, (x, c) in enumerate(zip(xs, codes)):
            k = O.hash24(seed, layer, i)
            assert c == exact_code(float(x), wl, fl, O.ROUND_STOCHASTIC, k), (x, wl, fl, k)


def test_stochastic_rule_thresholds():
    # y = 2.25 at FL = 2 for x = 0.5625: rounds up exactly when P < 0.25.
    for k, want in ((0, 3), (4194303, 3), (4194304, 2), (16777215, 2)):
        assert O.quantize_one(0.5625, 16, 2, O.ROUND_STOCHASTIC, k) == want
    # exactly representable values never move, whatever P is
    for k in (0, 1, 8388608, 16777215):
        assert O.quantize_one(-1.75, 16, 2, O.ROUND_STOCHASTIC, k) == -7
    # expected value of SR over all P equals the unrounded value (unbiasedness)
    x = 0.3
    y = frac_of_f32(f32(x)) * 16
    ks = np.arange(0, 1 << 24, 4099)
    ups = sum(O.quantize_one(x, 16, 4, O.ROUND_STOCHASTIC, int(k)) == 5 for k in ks)
    assert abs(ups / len(ks) - float(y - 4)) < 2e-3


def test_unsaturated_rne_equals_library_rint():
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(5000) * 1000).astype(np.float32)
    codes, xhat = O.quantize(x, 32, 0, O.ROUND_RNE)
    assert np.array_equal(codes, np.rint(x).astype(np.int32))
    assert np.array_equal(xhat, np.rint(x))
    codes, xhat = O.quantize(x, 32, 6, O.ROUND_RNE)
    assert np.array_equal(codes, np.rint(x.astype(np.float64) * 64).astype(np.int32))


@pytest.mark.parametrize("mode", [O.ROUND_RNE, O.ROUND_STOCHASTIC])
def test_codes_in_range_and_error_bound(mode):
    rng = np.random.default_rng(8)
    x = (rng.standard_normal(4000) * np.exp2(rng.integers(-20, 12, 4000))).astype(np.float32)
    for wl in (2, 5, 8, 13, 16, 32):
        for fl in (0, wl // 2, wl - 1):
            codes, xhat = O.quantize(x, wl, fl, mode, seed=1, layer=2)
            top = 1 << (wl - 1)
            assert codes.min() >= -top and codes.max() <= top - 1
            inside = (x.astype(np.float64) * 2.0 ** fl < top - 1) & (x.astype(np.float64) * 2.0 ** fl > -top)
            err = np.abs(xhat.astype(np.float64) - x.astype(np.float64))[inside]
            bound = 2.0 ** -(fl + 1) if mode == O.ROUND_RNE else 2.0 ** -fl
            assert (err <= bound).all()


@pytest.mark.parametrize("mode", [O.ROUND_RNE, O.ROUND_STOCHASTIC])
def test_on_grid_inputs_are_reproduced_bitwise(mode):
    rng = np.random.default_rng(21)
    wl, fl = 12, 7
    codes0 = rng.integers(-(1 << (wl - 1)), 1 << (wl - 1), 3000).astype(np.int32)
    x = (codes0.astype(np.float32) * np.float32(2.0 ** -fl)).astype(np.float32)
    for wl2, fl2 in ((12, 7), (13, 8), (20, 12), (32, 27)):  # same or finer grid, enough range
        codes, xhat = O.quantize(x, wl2, fl2, mode, seed=5, layer=1)
        assert np.array_equal(xhat.view(np.uint32), x.view(np.uint32))
        assert np.array_equal(codes, codes0 << (fl2 - fl))


def test_rne_zero_count_closed_form_and_wl_independence():
    rng = np.random.default_rng(2)
    x = (rng.laplace(0, 0.02, 20000)).astype(np.float32)
    x[::17] = 0.0
    x[5] = 2.0 ** -9   # exactly half a quantum at FL = 8: ties to even -> 0
    x[6] = -2.0 ** -9
    prev = None
    for fl in range(0, 16):
        counts = set()
        for wl in range(max(2, fl + 1), 33, 5):
            codes, _ = O.quantize(x, wl, fl, O.ROUND_RNE)
            counts.add(int((codes == 0).sum()))
        assert len(counts) == 1
        z = counts.pop()
        assert z == int((np.abs(x.astype(np.float64)) <= 2.0 ** -(fl + 1)).sum())
        if prev is not None:
            assert z <= prev
        prev = z


def test_hash_vectors_and_statistics():
    for row in read_rows("hash_vectors.txt"):
        s, l, i, k = (int(t) for t in row.split())
        assert O.hash24(s, l, i) == k
    n = 1 << 16
    ks = np.array([O.hash24(7, 3, i) for i in range(n)], dtype=np.float64)
    assert ks.min() >= 0 and ks.max() < 2 ** 24
    p = ks / 2 ** 24
    assert abs(p.mean() - 0.5) < 0.01
    assert abs(p.var() * 12 - 1.0) < 0.03
    hist = np.bincount((ks // 2 ** 16).astype(int), minlength=256)
    chi2 = ((hist - n / 256) ** 2 / (n / 256)).sum()
    assert 150 < chi2 < 380  # 255 degrees of freedom
    other = np.array([O.hash24(7, 4, i) for i in range(n)], dtype=np.float64) / 2 ** 24
    assert abs(np.corrcoef(p, other)[0, 1]) < 0.02
    assert abs(np.corrcoef(p[:-1], p[1:])[0, 1]) < 0.02
