"""The allocation-free search entry point (adapt_precision_search_static).

It is meant for hosts that cannot let the library call cudaMalloc (all device
memory already handed to a pool, a fixed audited budget, or a step loop that
cannot afford cudaMalloc's device-wide stall), so its scratch is a fixed array
inside the library.  The array is shared by all calls and keeps the previous
call's contents; these tests call it several times in a row, through the C ABI, on
different inputs and compare every output with the regular entry point's and with
the CPU oracle's, and check that the free device memory does not move across a call.
This file sorts last on purpose: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2107_13490_b200 import workloads as W
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

KLD_RTOL = 1e-5   # same tolerance as the parity tests; everything else must be identical


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2107_13490_b200 import binding
    binding.lib()
    return binding


def _outputs(B, n_layers, n_cand):
    import torch
    return B.SearchResult(torch.full((n_layers, n_cand), -1.0, dtype=torch.float64, device="cuda"),
                          torch.full((n_layers, n_cand), -1, dtype=torch.int64, device="cuda"),
                          torch.full((n_layers, 4), -1, dtype=torch.int32, device="cuda"))


def _same(a, b):
    ka, kb = a.kld.cpu().numpy(), b.kld.cpu().numpy()
    assert np.array_equal(a.zeros.cpu().numpy(), b.zeros.cpu().numpy())
    assert np.array_equal(a.best.cpu().numpy(), b.best.cpu().numpy())
    exact = (kb == 0) | ~np.isfinite(kb)
    assert np.array_equal(ka[exact], kb[exact])
    assert (np.abs(ka[~exact] - kb[~exact]) <= KLD_RTOL * np.abs(kb[~exact])).all()


def test_two_calls_in_a_row_match_the_regular_entry_point(B):
    import torch
    rng = np.random.default_rng(2024)
    wl, fl = W.candidate_grid(range(2, 33))
    grid = B.Grid(wl, fl)
    # first call: several layers, many elements, the most bins allowed
    first = [(rng.standard_normal(300001) * 0.1).astype(np.float32),
             np.maximum(rng.standard_normal(70000), 0).astype(np.float32),
             (rng.laplace(0, 1e-4, 12345)).astype(np.float32),
             np.zeros(0, np.float32),
             np.full(77, 0.25, np.float32)]
    # second call: fewer, smaller layers and fewer bins - stale counts of the first call
    # left in the shared scratch would show up here
    second = [(rng.standard_normal(999) * 3.0).astype(np.float32),
              (rng.standard_normal(40000) * 0.02).astype(np.float32)]
    for xs, n_bins in ((first, B.STATIC_MAX_BINS), (second, 50), (first, 128)):
        dev = [torch.from_numpy(x).cuda() for x in xs]
        got = _outputs(B, len(xs), len(grid))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        launches_before = B.adapt_kernel_launch_count()
        B.adapt_precision_search_static(dev, grid, n_bins, got)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before      # nothing was allocated or freed
        assert B.adapt_kernel_launch_count() > launches_before
        want = B.adapt_precision_search(dev, grid, n_bins)
        torch.cuda.synchronize()
        _same(got, want)
        ora = O.precision_search(xs, wl, fl, n_bins, threads=G.host_threads())
        G.compare_search(got, ora, len(xs), f"static call, {n_bins} bins")


def test_at_the_limits_of_the_fixed_scratch(B):
    """Exactly the most layers, candidates and bins the fixed array has room for."""
    import torch
    rng = np.random.default_rng(99)
    wl, fl = W.candidate_grid(range(2, 33))
    reps = -(-B.STATIC_MAX_CAND // wl.size)
    wl = np.tile(wl, reps)[:B.STATIC_MAX_CAND]
    fl = np.tile(fl, reps)[:B.STATIC_MAX_CAND]
    grid = B.Grid(wl, fl)
    xs = [(rng.standard_normal(3000 + 517 * l) * 2.0 ** (-l)).astype(np.float32)
          for l in range(B.STATIC_MAX_LAYERS)]
    dev = [torch.from_numpy(x).cuda() for x in xs]
    for _ in range(2):
        got = _outputs(B, len(xs), len(grid))
        B.adapt_precision_search_static(dev, grid, B.STATIC_MAX_BINS, got)
        torch.cuda.synchronize()
        ora = O.precision_search(xs, wl, fl, B.STATIC_MAX_BINS, threads=G.host_threads())
        G.compare_search(got, ora, len(xs), "static call at its limits")


def test_sizes_beyond_the_fixed_scratch_are_rejected(B):
    import torch
    x = torch.zeros(100, dtype=torch.float32, device="cuda")
    wl, fl = W.candidate_grid([8])
    out = _outputs(B, B.STATIC_MAX_LAYERS + 1, len(wl))
    for tensors, grid, n_bins in (
            ([x], B.Grid(wl, fl), B.STATIC_MAX_BINS + 1),
            ([x] * (B.STATIC_MAX_LAYERS + 1), B.Grid(wl, fl), 64),
            ([x], B.Grid(np.full(B.STATIC_MAX_CAND + 1, 8), np.full(B.STATIC_MAX_CAND + 1, 4)), 64)):
        with pytest.raises(B.AdaptError) as e:
            B.adapt_precision_search_static(tensors, grid, n_bins, out)
        assert e.value.status == B.ERR_WORKSPACE
        assert "at most" in str(e.value)
    torch.cuda.synchronize()
    assert (out.best.cpu().numpy() == -1).all()      # nothing was written
