"""GPU parity of the gradient-diversity reduction against the CPU oracle (both accumulate in
double; only the summation order differs, so the tolerance is 1e-10 relative)."""
import math

import numpy as np
import pytest

from oracle import oracle as O
from paper_2107_13490_b200 import workloads as W

pytestmark = pytest.mark.gpu
RTOL = 1e-10


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2107_13490_b200 import binding
    binding.lib()
    return binding


def _close(got, want):
    for a, b in zip(got, want):
        if math.isnan(b):
            assert math.isnan(a)
        elif math.isinf(b):
            assert a == b
        else:
            assert a == pytest.approx(b, rel=RTOL, abs=1e-300)


def _grads(shape_n, k, seed, layer):
    spec = W.LayerSpec("g", (shape_n,), "laplace", 1e-4, zero_frac=0.05)
    return [W.generate_layer(spec, seed, layer * 1000 + j, threads=1) for j in range(k)]


def test_resnet20_gradient_sets(B):
    import torch
    shapes = [s for _, s in W._resnet20_shapes()]
    k = 25                                           # the paper's smallest lookback
    host = [_grads(int(np.prod(s)), k, 7, l) for l, s in enumerate(shapes)]
    dev = [[torch.from_numpy(g).cuda() for g in gl] for gl in host]
    out = B.adapt_gradient_diversity(dev).cpu().numpy()
    for l, gl in enumerate(host):
        _close(out[l], O.gradient_diversity(gl))
    assert (out[:, 2] >= 1.0).all()                  # triangle inequality


@pytest.mark.parametrize("n,k", [(1, 1), (5, 3), (2047, 2), (2048, 4), (2049, 7), (100003, 16),
                                 (3000, 256)])
def test_ragged_sizes_misaligned_and_many_gradients(B, n, k):
    import torch
    rng = np.random.default_rng(n + k)
    host = [(rng.standard_normal(n) * 10.0 ** rng.integers(-4, 3)).astype(np.float32) for _ in range(k)]
    dev = []
    for j, g in enumerate(host):
        buf = torch.zeros(n + 4, dtype=torch.float32, device="cuda")
        buf[j % 4:j % 4 + n] = torch.from_numpy(g).cuda()
        dev.append(buf[j % 4:j % 4 + n])
    out = B.adapt_gradient_diversity([dev]).cpu().numpy()
    _close(out[0], O.gradient_diversity(host))


def test_degenerate_cases_and_errors(B):
    import torch
    z = torch.zeros(1000, dtype=torch.float32, device="cuda")
    a = torch.linspace(-1, 1, 1000, dtype=torch.float32, device="cuda")
    e = torch.zeros(0, dtype=torch.float32, device="cuda")
    out = B.adapt_gradient_diversity([[z, z], [a, -a], [a, a], [e, e]]).cpu().numpy()
    assert math.isnan(out[0][2]) and out[0][3] == 1.0          # 0/0
    assert math.isinf(out[1][2]) and out[1][3] == 1.0          # gradients cancel
    assert out[2][2] == pytest.approx(1.0, rel=1e-14) and abs(out[2][3]) < 1e-13
    assert math.isnan(out[3][2]) and out[3][3] == 1.0          # empty layer
    with pytest.raises(B.AdaptError):
        B.adapt_gradient_diversity([[a] * 257])


def test_large_multi_tile(B):
    import torch
    n, k = (1 << 22) + 77, 6
    host = _grads(n, k, 11, 0)
    dev = [torch.from_numpy(g).cuda() for g in host]
    out = B.adapt_gradient_diversity([dev]).cpu().numpy()
    _close(out[0], O.gradient_diversity(host))


def test_gradient_normalisation_matches_the_oracle(B):
    """g / ||g||_2 per layer (Sec. 3.3).  The norm's summation order differs (sequential on the
    CPU, tree on the GPU): its relative error stays below n * 2^-53, far inside half an fp32 ulp
    of every quotient except at rounding boundaries - so at most one ulp of fp32 per element,
    and the sums of squares agree to 1e-12."""
    import torch
    rng = np.random.default_rng(11)
    host = [(rng.laplace(0, 1e-4, n)).astype(np.float32) for n in (1, 5, 2047, 2048, 2049, 70001, 1 << 20)]
    host.append(np.zeros(300, dtype=np.float32))            # zero norm: copied
    host.append(np.zeros(0, dtype=np.float32))              # empty layer
    host.append(np.float32([3.0, 4.0]))
    dev = []
    for j, h in enumerate(host):                              # odd phases: scalar path too
        b = torch.zeros(h.size + 4, dtype=torch.float32, device="cuda")
        b[j % 4:j % 4 + h.size] = torch.from_numpy(h).cuda()
        dev.append(b[j % 4:j % 4 + h.size])
    out, sumsq = B.adapt_normalize_gradients(dev, want_sumsq=True)
    torch.cuda.synchronize()
    sumsq = sumsq.cpu().numpy()
    for j, h in enumerate(host):
        want = O.normalize_gradient(h)
        got = out[j].cpu().numpy()
        assert got.shape == want.shape
        if h.size:
            d = np.abs(got.view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
            assert d.max() <= 1, (j, int(d.max()))
            ss = float(np.sum(h.astype(np.float64) ** 2))
            assert sumsq[j] == pytest.approx(ss, rel=1e-12, abs=0.0)
    assert list(out[-1].cpu().numpy()) == [np.float32(0.6), np.float32(0.8)]
    # in place
    ref = [o.clone() for o in out]
    B.adapt_normalize_gradients(dev, out=dev)
    torch.cuda.synchronize()
    for a, b in zip(dev, ref):
        assert torch.equal(a, b)


def test_precision_switch_chain_search_diversity_pushup(B):
    """One precision switch of a few layers as Algorithm 2 strings it together: PushDown (the
    search on the weights), the gradient diversity over the lookback, PushUp - every stage through
    the C ABI, the chosen formats against the same chain on the oracle."""
    import torch
    shapes = [s for _, s in W._resnet20_shapes()][:6]
    k = 25
    wl, fl = W.candidate_grid(range(2, 17))
    weights = [W.generate_layer(W._kaiming("w", s), 7, l, threads=1) for l, s in enumerate(shapes)]
    grads = [_grads(int(np.prod(s)), k, 9, l) for l, s in enumerate(shapes)]
    res = B.adapt_precision_search_ex([torch.from_numpy(w).cuda() for w in weights], B.Grid(wl, fl), 100)
    div = B.adapt_gradient_diversity([[torch.from_numpy(g).cuda() for g in gl] for gl in grads])
    torch.cuda.synchronize()
    ora = O.precision_search(weights, wl, fl, 100)
    for st in (B.STRATEGY_MIN, B.STRATEGY_MEAN, B.STRATEGY_MAX):
        got = B.adapt_pushup(div, res.best, st, 4)
        for l in range(len(shapes)):
            d = O.gradient_diversity(grads[l])[3]
            want = O.pushup(d, ora[l]["best"][0], ora[l]["best"][1], st, 4)
            assert list(got[l]) == list(want[:2]), (l, st)
