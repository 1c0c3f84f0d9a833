"""The library's PushUp step (adapt_pushup, host arithmetic behind the C ABI) against the
oracle's: identical integers for every strategy, buffer width and starting format, over a
sweep of diversities that includes the branch points.  Needs no GPU: the call launches nothing."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2107_13490_b200 import workloads as W


@pytest.fixture(scope="module")
def B():
    from paper_2107_13490_b200 import binding
    binding.lib()
    return binding


def test_pushup_matches_the_oracle(B):
    rng = np.random.default_rng(2107)
    d = np.concatenate([np.arange(-8, 200) / 64.0, rng.normal(0.9, 0.7, 400), rng.random(200) * 4,
                        [1.0, 0.0, -0.0, 1.0 + 2.0 ** -40, 1.0 - 2.0 ** -40, 1e-300, 50.0, 1e300,
                         np.nextafter(1.0, 2.0), np.sqrt(33.0 / 32.0)]])
    wl, fl = W.candidate_grid(range(2, 33))
    pick = rng.integers(0, wl.size, d.size)
    div = np.zeros((d.size, 4))
    div[:, 3] = d
    best = np.zeros((d.size, 4), dtype=np.int32)
    best[:, 0], best[:, 1] = wl[pick], fl[pick]
    for st in (B.STRATEGY_MIN, B.STRATEGY_MEAN, B.STRATEGY_MAX):
        for buff in (0, 1, 4, 8, 31):
            got, sug = B.adapt_pushup(div, best, st, buff, want_suggestions=True)
            for l in range(d.size):
                want = O.pushup(d[l], best[l, 0], best[l, 1], st, buff)
                assert list(got[l]) == list(want[:2]), (d[l], best[l, :2], st, buff)
                assert list(sug[l]) == list(want[2:]), (d[l], best[l, :2], st, buff)


def test_pushup_argument_errors(B):
    div = np.zeros((2, 4)); best = np.array([[8, 4, 0, 1], [16, 12, 0, 1]], dtype=np.int32)
    for bad in (dict(strategy=3), dict(strategy=-1), dict(buff=-1), dict(buff=32)):
        kw = dict(strategy=0, buff=4); kw.update(bad)
        with pytest.raises(B.AdaptError) as e:
            B.adapt_pushup(div, best, kw["strategy"], kw["buff"])
        assert e.value.status == B.ERR_INVALID_ARG
    for row in ([1, 0, 0, 0], [33, 2, 0, 0], [8, 8, 0, 0], [8, -1, 0, 0]):
        with pytest.raises(B.AdaptError):
            B.adapt_pushup(div, np.array([[8, 4, 0, 1], row], dtype=np.int32), 0, 4)
