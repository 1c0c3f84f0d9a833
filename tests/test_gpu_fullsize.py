"""Parity at the full size of the benchmark workload (2^30 elements, 527 candidates,
2048 bins), in the launch configuration bench.py times: sampled candidates are checked
against the oracle in full (zero count, whole histogram, divergence), every candidate
against properties that hold at any size."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2107_13490_b200 import workloads as W
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

# low word lengths as training meets them, plus one candidate in every four fraction lengths up to
# the finest: the keyed kernel treats a level by where it lies against the cells' and the
# sub-cells' levels, so the sample walks across all of them
SAMPLED = [(2, 1), (6, 3), (8, 4), (12, 9), (16, 15), (20, 6),
           (32, 0), (32, 12), (32, 17), (32, 19), (32, 21), (32, 23), (32, 25), (32, 27), (32, 29), (32, 31)]


def test_stress_1g_sampled_candidates_and_invariants():
    import torch
    from paper_2107_13490_b200 import binding as B
    B.lib()
    w = W.WORKLOADS["stress_1g"]
    wl, fl = w.grid()
    x = W.generate(w)[0]
    n = x.size
    xd = torch.from_numpy(x).cuda()
    grid = B.Grid(wl, fl)
    ws = torch.empty(B.adapt_search_workspace_bytes([n], grid, w.n_bins), dtype=torch.uint8,
                     device="cuda")
    res = B.adapt_precision_search_ex([xd], grid, w.n_bins, workspace=ws, want_hist=True,
                                      want_range=True)
    torch.cuda.synchronize()
    kld = res.kld.cpu().numpy()[0]
    zeros = res.zeros.cpu().numpy()[0]
    hist = res.hist.cpu().numpy()[0].view(np.uint32).astype(np.uint64)
    best = res.best.cpu().numpy()[0]
    rng = res.range.cpu().numpy()[0]
    del xd, ws

    # properties that hold at any size
    assert rng[0] == x.min() and rng[1] == x.max()
    assert (hist.sum(axis=1) == n).all()                       # every histogram holds all elements
    assert (kld >= 0).all()
    for f in (0, 5, 11, 17, 25, 31):                            # RNE zero count, closed form
        want = int((np.abs(x) <= np.float32(2.0 ** -(f + 1))).sum())
        got = {int(z) for z, ff in zip(zeros, fl) if ff == f}
        assert got == {want}
    same = (hist[1:] == hist[0]).all(axis=1)
    assert np.array_equal(kld == 0.0, same)                     # KLD is 0 exactly for identical histograms
    assert list(best) == list(O.select(kld, wl, fl, 0.0))       # the choice follows from the divergences

    # sampled candidates, in full, against the oracle
    idx = [int(np.where((wl == a) & (fl == b))[0][0]) for a, b in SAMPLED]
    ora = O.precision_search([x], wl[idx], fl[idx], w.n_bins, threads=len(idx), want_hist=True)[0]
    assert np.array_equal(ora["hist"][0], hist[0])
    for j, c in enumerate(idx):
        assert zeros[c] == ora["zeros"][j], SAMPLED[j]
        assert np.array_equal(hist[c + 1], ora["hist"][j + 1]), SAMPLED[j]
    G.assert_kld_close(kld[idx], ora["kld"], "stress_1g sampled")
