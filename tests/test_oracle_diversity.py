"""Pins of the oracle's gradient-diversity reduction: hand-worked values, closed forms
(identical / orthogonal / cancelling gradients), numpy.linalg.norm.  CPU only."""
import math
import os

import numpy as np
import pytest

from oracle import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_hand_worked_diversities():
    for line in open(os.path.join(GOLDEN, "diversity_hand.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        vecs, ds, lg = line.split("|")
        grads = [np.float32([float(t) for t in v.split()]) for v in vecs.split(";")]
        out = O.gradient_diversity(grads)
        want = float(ds)
        if math.isnan(want):
            assert math.isnan(out[2])
        elif math.isinf(want):
            assert math.isinf(out[2]) and out[2] > 0
        else:
            assert out[2] == pytest.approx(want, rel=1e-14)
        assert out[3] == pytest.approx(float(lg), rel=1e-13, abs=1e-15)


def test_closed_forms():
    rng = np.random.default_rng(1)
    g = rng.standard_normal(5000).astype(np.float32)
    for k in (1, 2, 7, 25):
        out = O.gradient_diversity([g] * k)             # identical gradients: exactly aligned
        assert out[2] == pytest.approx(1.0, rel=1e-14) and abs(out[3]) < 1e-13
    # K orthogonal gradients of equal norm: Delta s = sqrt(K)
    for k in (2, 5, 16):
        grads = []
        for j in range(k):
            v = np.zeros(64, np.float32)
            v[j * 3] = 2.5
            grads.append(v)
        out = O.gradient_diversity(grads)
        assert out[2] == pytest.approx(math.sqrt(k), rel=1e-14)
        assert out[3] == pytest.approx(0.5 * math.log(k), rel=1e-13)
    # scaling all gradients by a power of two changes nothing; reordering changes nothing
    gs = [rng.standard_normal(3000).astype(np.float32) for _ in range(6)]
    a = O.gradient_diversity(gs)
    b = O.gradient_diversity([x * np.float32(8.0) for x in gs])
    c = O.gradient_diversity(gs[::-1])
    assert b[2] == pytest.approx(a[2], rel=1e-14) and c[2] == pytest.approx(a[2], rel=1e-13)
    assert a[2] >= 1.0 - 1e-12                              # triangle inequality


def test_matches_numpy_norms():
    rng = np.random.default_rng(2)
    gs = [(rng.laplace(0, 1e-4, 40000) * (rng.random(40000) > 0.05)).astype(np.float32)
          for _ in range(25)]
    out = O.gradient_diversity(gs)
    g64 = [x.astype(np.float64) for x in gs]
    sum_norms = sum(np.linalg.norm(x) for x in g64)
    norm_sum = np.linalg.norm(np.sum(g64, axis=0))
    assert out[0] == pytest.approx(sum_norms, rel=1e-12)
    assert out[1] == pytest.approx(norm_sum, rel=1e-12)
    assert out[2] == pytest.approx(sum_norms / norm_sum, rel=1e-12)
    assert out[3] == pytest.approx(math.log(sum_norms / norm_sum), rel=1e-11)


def test_normalized_gradient_pins():
    """g / ||g||_2 (Sec. 3.3): hand-worked 3-4-5 triangle, unit norm, exact invariance under a
    power-of-two scale and a sign flip, exact rational quotients, the all-zero gradient."""
    from fractions import Fraction
    out = O.normalize_gradient(np.float32([3.0, 4.0]))
    assert out[0] == np.float32(0.6) and out[1] == np.float32(0.8)
    out = O.normalize_gradient(np.float32([0.0, -2.0, 0.0]))
    assert list(out) == [0.0, -1.0, 0.0]
    rng = np.random.default_rng(5)
    g = (rng.standard_normal(10001) * 1e-3).astype(np.float32)
    out = O.normalize_gradient(g)
    assert abs(np.linalg.norm(out.astype(np.float64)) - 1.0) < 1e-7
    assert np.array_equal(O.normalize_gradient(g * np.float32(1024.0)), out)     # exact scaling
    assert np.array_equal(O.normalize_gradient(-g), -out)
    want = (g.astype(np.float64) / np.linalg.norm(g.astype(np.float64))).astype(np.float32)
    assert np.max(np.abs(out.view(np.int32).astype(np.int64) - want.view(np.int32))) <= 1
    # small case against exact rational arithmetic: squares sum to 49 = 7^2
    h = np.float32([2.0, 3.0, 6.0])
    out = O.normalize_gradient(h)
    for o, x in zip(out, h):
        assert o == np.float32(float(Fraction(int(x), 7)))
    z = np.zeros(17, dtype=np.float32)
    assert np.array_equal(O.normalize_gradient(z), z)
    assert O.normalize_gradient(np.zeros(0, dtype=np.float32)).size == 0
