"""Pins of the oracle's PushUp step (Sec. 3.3 "The PushUp Operation", the strategy
equation, and the buffer bits of "Dealing with Fixed-Points Limited Range") against
hand-worked values, exact rational arithmetic and invariants.  CPU only."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "pushup_hand.txt")
STRATEGY = {"min": O.STRATEGY_MIN, "mean": O.STRATEGY_MEAN, "max": O.STRATEGY_MAX}


def test_hand_worked_pushups():
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 20
    seen = set()
    for d, wl_min, fl_min, st, buff, *want in rows:
        got = O.pushup(float(d), int(wl_min), int(fl_min), STRATEGY[st], int(buff))
        assert list(got) == [int(v) for v in want], (d, wl_min, fl_min, st, buff)
        seen.add(st)
    assert seen == {"min", "mean", "max"}


def exact_pushup(d: Fraction, wl_min: int, fl_min: int, st: str, buff: int):
    """The same paragraph in exact rational arithmetic (d given as a rational)."""
    s1 = s2 = 0
    s = 1
    if d > 0:
        if d == 1:
            s1 = 32
        else:
            s1 = min(max(math.ceil(1 / (d - 1)), 1), 32)
        s2 = min(max(math.ceil(min(32 * d * d - 1, Fraction(32))) - fl_min, 1), 32)
        s = {"min": min(s1, s2), "mean": math.ceil(Fraction(s1 + s2, 2)), "max": max(s1, s2)}[st]
    fl = min(fl_min + s, 32)
    wl = min(max(wl_min, fl) + 1, 32)
    fl = min(fl, 32 - buff)
    wl = max(min(fl + buff, 32), wl)
    fl = min(fl, wl - 1)
    return [wl, fl, s1, s2, s]


def test_against_exact_rationals_on_a_dyadic_grid():
    # d = k / 64 is exact in double, and so are d - 1, d * d and 32 d^2 - 1: the double
    # evaluation must give the rational result everywhere, including at d = 1 and around the
    # points where a ceiling steps
    formats = [(2, 0), (8, 4), (6, 2), (16, 12), (16, 15), (24, 3), (32, 0), (32, 31)]
    for k in range(-16, 260):
        d = Fraction(k, 64)
        for wl_min, fl_min in formats:
            for st in STRATEGY:
                for buff in (0, 4, 8):
                    want = exact_pushup(d, wl_min, fl_min, st, buff)
                    got = list(O.pushup(float(d), wl_min, fl_min, STRATEGY[st], buff))
                    assert got == want, (k, wl_min, fl_min, st, buff)


def test_invariants():
    rng = np.random.default_rng(12)
    for _ in range(3000):
        d = float(rng.choice([rng.normal(0.8, 0.8), rng.random() * 3, 1.0, 0.0]))
        wl_min = int(rng.integers(2, 33))
        fl_min = int(rng.integers(0, wl_min))
        buff = int(rng.choice([0, 1, 4, 8]))
        res = {st: O.pushup(d, wl_min, fl_min, STRATEGY[st], buff) for st in STRATEGY}
        for st, (wl, fl, s1, s2, s) in res.items():
            assert 2 <= wl <= 32 and 0 <= fl <= wl - 1          # a valid fixed-point format
            assert wl >= min(wl_min, 32) and s >= 1
            assert fl >= min(fl_min + 1, 32 - buff, wl - 1)      # precision goes up unless a cap binds
            if buff:
                assert wl - fl >= min(buff, wl - fl_min) or wl == 32   # the buffer bits are there
        # the strategies are ordered
        assert res["min"][4] <= res["mean"][4] <= res["max"][4]
        assert res["min"][1] <= res["mean"][1] <= res["max"][1]
        if d <= 0:
            assert all(r[4] == 1 and r[2] == 0 and r[3] == 0 for r in res.values())


def test_log_form_of_the_diversity_feeds_pushup():
    """The chain the switch uses: gradients -> diversity (log form) -> new format."""
    g = [np.float32([1, 0, 0, 0]), np.float32([0, 1, 0, 0]), np.float32([0, 0, 1, 0]),
         np.float32([0, 0, 0, 1])]
    div = O.gradient_diversity(g)               # 4 / 2 = 2, log form ln 2 = 0.693...
    assert div[2] == 2.0 and abs(div[3] - math.log(2.0)) < 1e-15
    # s1 = max(ceil(1/(0.693-1)), 1) = 1; s2 = max(ceil(32*0.4805-1) - 4, 1) = ceil(14.37) - 4 = 11
    assert list(O.pushup(div[3], 8, 4, O.STRATEGY_MAX, 4)) == [19, 15, 1, 11, 11]
    # cancelling gradients: delta_s infinite, log form 1
    div = O.gradient_diversity([np.float32([1, -1]), np.float32([-1, 1])])
    assert div[3] == 1.0
    assert list(O.pushup(div[3], 8, 4, O.STRATEGY_MIN, 4)) == [32, 28, 32, 27, 27]
