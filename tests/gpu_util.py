"""Helpers shared by the GPU parity tests: run the library through its C ABI
(via the ctypes binding) and the oracle on the same seeded inputs, compare."""
import math
import os

import numpy as np

from oracle import oracle as O

KLD_RTOL = 1e-5  # relative tolerance of the divergence; everything else is bit-exact


def host_threads():
    return max(1, min(64, os.cpu_count() or 1))


def to_device(arrays, device="cuda"):
    import torch
    return [torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device) for a in arrays]


def assert_kld_close(got, want, where=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape
    exact = (want == 0.0) | np.isinf(want)
    if exact.any():
        bad = np.where(exact & (got != want))[0]
        assert bad.size == 0, f"{where}: KLD must equal the oracle's 0/inf exactly at {bad[:8]}: " \
                              f"{got[bad[:8]]} vs {want[bad[:8]]}"
    rest = ~exact
    if rest.any():
        err = np.abs(got[rest] - want[rest]) / np.abs(want[rest])
        worst = float(err.max())
        assert worst <= KLD_RTOL, f"{where}: KLD relative error {worst:.3e} > {KLD_RTOL}"


def compare_search(res, oracle_results, n_layers, where="", check_hist=False, check_range=False):
    """res: binding.SearchResult (device or host tensors); oracle_results: list of dicts."""
    kld = res.kld.cpu().numpy()
    zeros = res.zeros.cpu().numpy()
    best = res.best.cpu().numpy()
    hist = res.hist.cpu().numpy().view(np.uint32) if (check_hist and res.hist is not None) else None
    rng = res.range.cpu().numpy() if (check_range and res.range is not None) else None
    for l in range(n_layers):
        o = oracle_results[l]
        tag = f"{where} layer {l}"
        assert np.array_equal(zeros[l], o["zeros"]), f"{tag}: zero counts differ"
        if hist is not None:
            assert np.array_equal(hist[l].astype(np.uint64), o["hist"]), f"{tag}: histograms differ"
        assert_kld_close(kld[l], o["kld"], tag)
        assert list(best[l]) == list(o["best"]), f"{tag}: best {best[l]} vs oracle {o['best']}"
        if rng is not None:
            assert rng[l][0] == o["range"][0] and rng[l][1] == o["range"][1], f"{tag}: range"


ALGORITHMS = (0, 1, 2)   # auto, keyed wherever it can serve, direct everywhere


def run_and_compare(B, tensors_np, wl, fl, n_bins, round_mode=0, seed=0, layer_base=0, eps=0.0,
                    pseudo_count=0.0, log_base=0.0, check_hist=True, threads=None, where="",
                    algorithms=ALGORITHMS):
    """B = the binding module.  Runs the library once per kernel form and compares each
    run with one oracle run.  Returns (last gpu result, oracle results)."""
    import torch
    grid = B.Grid(wl, fl)
    dev = to_device(tensors_np)
    ora = O.precision_search(tensors_np, wl, fl, n_bins, round_mode, seed, layer_base, eps,
                             pseudo_count, 2.0 if log_base == 0.0 else log_base,
                             want_hist=check_hist, threads=threads or host_threads())
    res = None
    for algo in algorithms:
        res = B.adapt_precision_search_ex(dev, grid, n_bins, round_mode=round_mode, seed=seed,
                                          layer_base=layer_base, eps=eps,
                                          pseudo_count=pseudo_count, log_base=log_base,
                                          want_hist=check_hist, want_range=True, algorithm=algo)
        torch.cuda.synchronize()
        compare_search(res, ora, len(tensors_np), f"{where} [algorithm {algo}]",
                       check_hist=check_hist, check_range=True)
    return res, ora
