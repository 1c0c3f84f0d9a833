"""GPU parity of the precision-switch search against the CPU oracle, through the
C ABI: zero counts, histograms and the chosen <WL,FL> bit-exact, divergences to
1e-5 relative (exactly where the oracle gives 0 or inf)."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2107_13490_b200 import workloads as W
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2107_13490_b200 import binding
    binding.lib()  # fails loudly when the CUDA library has not been built
    return binding


def test_single4k_all_candidates(B):
    w = W.WORKLOADS["single4k"]
    wl, fl = w.grid()
    G.run_and_compare(B, W.generate(w), wl, fl, w.n_bins, where="single4k")
    # the named call (RNE, eps 0, bits) gives the same answer
    import torch
    dev = G.to_device(W.generate(w))
    r = B.adapt_precision_search(dev, B.Grid(wl, fl), w.n_bins)
    torch.cuda.synchronize()
    ora = O.precision_search(W.generate(w), wl, fl, w.n_bins)
    G.compare_search(r, ora, 1, "single4k named call")


def test_resnet20_weights_grads_stochastic(B):
    w = W.WORKLOADS["resnet20_weights_grads"]
    wl, fl = w.grid()
    G.run_and_compare(B, W.generate(w), wl, fl, w.n_bins, round_mode=w.round_mode, seed=w.seed,
                      where="resnet20")


def test_alexnet_weights_full_grid(B):
    w = W.WORKLOADS["alexnet_weights"]
    wl, fl = w.grid()
    G.run_and_compare(B, W.generate(w), wl, fl, w.n_bins, where="alexnet")


def test_resnet18_weights_acts_full_grid(B):
    w = W.WORKLOADS["resnet18_weights_acts"]
    wl, fl = w.grid()
    G.run_and_compare(B, W.generate(w), wl, fl, w.n_bins, where="resnet18")


def test_stress_scaled_full_grid(B):
    # same distribution, grid and bins as the 2^30 stress case, several hundred tiles, ragged tail
    w = W.scaled(W.WORKLOADS["stress_1g"], (1 << 22) + 4099)
    wl, fl = w.grid()
    G.run_and_compare(B, W.generate(w), wl, fl, w.n_bins, where="stress scaled")
    G.run_and_compare(B, W.generate(w), wl, fl, w.n_bins, round_mode=O.ROUND_STOCHASTIC, seed=3,
                      where="stress scaled SR")


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 31, 32, 33, 127, 1023, 1024, 1025, 4093, 4095, 4096,
                               4097, 8191, 8193, 12289])
def test_ragged_sizes_and_misaligned_pointers(B, n):
    import torch
    rng = np.random.default_rng(n)
    wl, fl = W.candidate_grid([2, 3, 7, 12, 20, 32])
    grid = B.Grid(wl, fl)
    for mis in range(4):
        buf = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
        x = (rng.standard_normal(n) * 0.3).astype(np.float32)
        buf[mis:mis + n] = torch.from_numpy(x).cuda()
        view = buf[mis:mis + n]
        for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
            ora = O.precision_search([x], wl, fl, 37, mode, 11, 2, want_hist=True)
            for algo in G.ALGORITHMS:
                res = B.adapt_precision_search_ex([view], grid, 37, round_mode=mode, seed=11,
                                                  layer_base=2, want_hist=True, want_range=True,
                                                  algorithm=algo)
                torch.cuda.synchronize()
                G.compare_search(res, ora, 1, f"n={n} mis={mis} mode={mode} algo={algo}", True, True)


def test_many_layers_with_empty_and_degenerate_ones(B):
    rng = np.random.default_rng(77)
    xs = [np.zeros(0, np.float32),
          (rng.standard_normal(5000) * 0.1).astype(np.float32),
          np.full(300, 0.37, np.float32),                     # max == min
          np.zeros(0, np.float32),
          (-np.abs(rng.standard_normal(4096))).astype(np.float32),   # negative only
          np.float32([1e-40, -1e-41, 3e-39, 0.0]),            # subnormals
          np.float32([5.0]),
          (rng.standard_normal(9000) * 1e4).astype(np.float32),      # saturates most formats
          np.zeros(100, np.float32),
          np.zeros(0, np.float32)]
    wl, fl = W.candidate_grid(range(2, 33))
    for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
        res, ora = G.run_and_compare(B, xs, wl, fl, 50, round_mode=mode, seed=5,
                                     where=f"mixed layers mode={mode}")
        best = res.best.cpu().numpy()
        for l in (0, 2, 3, 6, 8, 9):
            assert best[l][3] & B.FLAG_DEGENERATE
        assert not (best[1][3] & B.FLAG_DEGENERATE)


def test_thousands_of_small_layers_share_ctas(B):
    """More layers than the direct kernel has CTAs: every CTA walks several layers in a row and
    must hand each one clean private counters (round-to-nearest-even zero classes included)."""
    rng = np.random.default_rng(4242)
    sizes = rng.integers(1, 1500, 3000)
    xs = []
    for l, n in enumerate(sizes):
        x = (rng.standard_normal(n) * 2.0 ** rng.integers(-12, 2)).astype(np.float32)
        x[rng.random(n) < 0.2] = 0.0
        xs.append(x)
    wl, fl = W.candidate_grid([4, 9, 14])
    for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
        G.run_and_compare(B, xs, wl, fl, 32, round_mode=mode, seed=21, where=f"3000 layers mode={mode}",
                          algorithms=(0, 2))


def test_hundreds_of_keyed_layers_of_uneven_size(B):
    """More keyed layers than the counting kernel has CTAs, sizes from just above the keyed
    threshold to a few hundred thousand elements, several value classes: the CTAs' tile ranges
    (balanced by cost, several layers per CTA, large layers cut over many CTAs) must cover every
    tile once, and the slices and roles of the expand kernel must add up."""
    rng = np.random.default_rng(909)
    xs = []
    for l in range(220):
        n = int(rng.choice([32768, 33001, 40000, 65537, 131072, 300000], p=[.3, .3, .2, .1, .07, .03]))
        kind = l % 4
        if kind == 0:
            x = rng.standard_normal(n) * 2.0 ** rng.integers(-8, 3)
        elif kind == 1:
            x = np.maximum(rng.standard_normal(n), 0) * 0.7
        elif kind == 2:
            x = rng.laplace(0, 0.02, n) * np.where(rng.random(n) < 0.01, 50.0, 1.0)
        else:
            x = rng.integers(-100, 100, n) * 2.0 ** -5          # on a grid: keyed by value
        xs.append(x.astype(np.float32))
    wl, fl = W.candidate_grid([5, 11, 18])
    G.run_and_compare(B, xs, wl, fl, 96, where="220 keyed layers", algorithms=(0,))


def test_options_eps_pseudocount_base_and_grid_order(B):
    rng = np.random.default_rng(3)
    xs = [(rng.laplace(0, 0.02, 20000)).astype(np.float32),
          (rng.standard_normal(7777) * 0.5).astype(np.float32)]
    wl, fl = W.candidate_grid([4, 6, 8, 10, 16])
    perm = rng.permutation(wl.size)
    wl_p = np.concatenate([wl[perm], wl[:5]])       # shuffled, with duplicates
    fl_p = np.concatenate([fl[perm], fl[:5]])
    G.run_and_compare(B, xs, wl_p, fl_p, 150, eps=1e-3, where="eps")
    G.run_and_compare(B, xs, wl_p, fl_p, 150, pseudo_count=0.5, where="pseudo-count")
    G.run_and_compare(B, xs, wl_p, fl_p, 150, log_base=float(np.e), where="nats")
    G.run_and_compare(B, xs, wl_p, fl_p, 1, where="one bin")
    G.run_and_compare(B, xs, [8], [4], 64, where="single candidate")
    G.run_and_compare(B, xs, wl_p, fl_p, 16384, where="max bins")


def test_adversarial_value_patterns(B):
    """Inputs built to sit on the places where the keyed kernel's shortcuts could
    go wrong: bin edges, cell boundaries, rounding ties, powers of two around zero,
    subnormals, ranges far from zero, very wide and very narrow ranges."""
    rng = np.random.default_rng(123)
    n = 40000
    cases = {}
    base = (rng.standard_normal(n) * 0.25).astype(np.float32)
    # values on and next to the exact bin edges of a 100-bin histogram of `base`
    lo, hi = base.min(), base.max()
    edges = (lo + (hi - lo) * np.arange(1, 100, dtype=np.float32) / np.float32(100)).astype(np.float32)
    near = np.concatenate([edges, np.nextafter(edges, np.float32(np.inf)),
                           np.nextafter(edges, np.float32(-np.inf))])
    cases["bin_edges"] = np.concatenate([base, np.tile(near, 20)]).astype(np.float32)
    # multiples of 2^-k: every element is a tie at some coarser level
    cases["ties"] = (rng.integers(-4000, 4000, n) * 2.0 ** -9 + 2.0 ** -10).astype(np.float32)
    cases["on_grid_mixed"] = np.where(rng.random(n) < 0.5, np.round(base * 1024) / 1024, base).astype(np.float32)
    # powers of two and their neighbours around zero (zero-count ties), subnormals, exact zeros
    p2 = np.float32(2.0) ** np.arange(-40, 2, dtype=np.float32)
    p2 = np.concatenate([p2, -p2, np.nextafter(p2, np.float32(0)), np.nextafter(p2, np.float32(4)),
                         np.float32([0.0, -0.0, 1e-45, -1e-45, 1e-39])])
    cases["pow2_near_zero"] = np.concatenate([np.tile(p2, 100), base[:5000] * np.float32(1e-3)]).astype(np.float32)
    cases["half_zero"] = np.maximum(rng.standard_normal(n), 0).astype(np.float32)
    cases["far_from_zero"] = (1000.0 + rng.random(n) * 0.01).astype(np.float32)
    cases["far_negative"] = (-123456.0 - rng.random(n) * 64).astype(np.float32)
    cases["wide"] = (rng.standard_normal(n) * 1e6).astype(np.float32)
    cases["very_wide"] = (rng.standard_normal(n) * 1e15).astype(np.float32)
    cases["tiny"] = (rng.standard_normal(n) * 1e-9).astype(np.float32)
    cases["narrow_offset"] = (0.75 + rng.integers(0, 50, n) * 2.0 ** -24).astype(np.float32)
    cases["two_values"] = np.where(rng.random(n) < 0.3, 0.1, -0.7).astype(np.float32)
    cases["integers"] = rng.integers(-300, 300, n).astype(np.float32)
    # the counting loop's forms: a handful of exact zeros among values off and on the cell grid
    # (the form without zero steering, whose element handler takes the zeros out again), a
    # positive range away from zero with few zero significand bits to go by, and one with many
    few = base.copy()
    few[rng.integers(0, n, 6)] = np.float32([0.0, -0.0, 0.0, 0.0, -0.0, 0.0])
    cases["few_zeros"] = few
    grid_few = (rng.integers(1, 4000, n) * rng.choice([-1.0, 1.0], n) * 2.0 ** -9).astype(np.float32)
    grid_few[rng.integers(0, n, 4)] = 0.0
    cases["few_zeros_on_grid"] = grid_few
    off100 = (100.0 + rng.random(n)).astype(np.float32)
    off100[::7] = (100.0 + rng.integers(0, 2048, off100[::7].size) * 2.0 ** -11).astype(np.float32)
    cases["offset_100"] = off100
    cases["half_to_one"] = (0.5 + 0.5 * rng.random(n)).astype(np.float32)
    # points of grids finer than the cells but coarser than (or equal to) the sub-cells of the edge
    # cells: rounding ties at levels between the two, many of them inside edge cells
    fine = rng.integers(-(1 << 13), 1 << 13, n).astype(np.float64)
    cases["fine_grid_15"] = (fine * 2.0 ** -15 + 2.0 ** -16).astype(np.float32)
    cases["fine_grid_mixed"] = np.where(rng.random(n) < 0.5, fine * 2.0 ** -15,
                                        rng.integers(-(1 << 15), 1 << 15, n) * 2.0 ** -17).astype(np.float32)
    # tensors on a fixed-point grid (the table is keyed by value), and such tensors with a few
    # elements off the grid at places the range scan's sample does not look at
    for name, spec in W.distribution_sweep(n):
        if name.startswith("on_grid"):
            cases[name] = W.generate_layer(spec, 5, 0)
    stray = (rng.integers(-2000, 2000, n) * 2.0 ** -6).astype(np.float32)
    for at in (700, 1000, 4095, 5000, 20000, n - 1):
        stray[at] = np.float32(rng.standard_normal() * 3.0)
    stray[30000] = 0.0
    cases["on_grid_with_strays"] = stray
    cases["on_grid_far_from_zero"] = (300.0 + rng.integers(0, 3000, n) * 2.0 ** -3).astype(np.float32)
    cases["on_grid_negative_powers"] = (rng.integers(-9, 9, n) * 2.0 ** -20).astype(np.float32)
    wl, fl = W.candidate_grid(range(2, 33))
    for name, x in cases.items():
        for n_bins in (100, 2048):
            G.run_and_compare(B, [x], wl, fl, n_bins, where=f"{name} B={n_bins}",
                              algorithms=(1, 2))


def test_per_layer_resolutions(B):
    """Each layer with its own number of bins (the paper's per-layer resolution r^l) in one call."""
    import torch
    rng = np.random.default_rng(17)
    xs = [(rng.standard_normal(60000) * 0.1).astype(np.float32),
          (rng.laplace(0, 1e-3, 40000)).astype(np.float32),
          np.maximum(rng.standard_normal(70001), 0).astype(np.float32),
          (rng.standard_normal(333) * 5).astype(np.float32),
          (rng.standard_normal(50000) * 0.02).astype(np.float32),
          np.zeros(0, np.float32)]
    bins = [50, 150, 97, 2048, 1, 64]
    wl, fl = W.candidate_grid(range(2, 33))
    grid = B.Grid(wl, fl)
    dev = G.to_device(xs)
    ora = [O.precision_search_layer(x, wl, fl, b, want_hist=True) for x, b in zip(xs, bins)]
    for algo in G.ALGORITHMS:
        res = B.adapt_precision_search_ex(dev, grid, 7, n_bins_per_layer=bins, want_hist=True,
                                          want_range=True, algorithm=algo)
        torch.cuda.synchronize()
        hist = res.hist.cpu().numpy().view(np.uint32)
        assert hist.shape[2] == max(bins)
        for l, b in enumerate(bins):
            assert np.array_equal(hist[l][:, :b].astype(np.uint64), ora[l]["hist"]), (algo, l)
            assert not hist[l][:, b:].any()
            assert np.array_equal(res.zeros.cpu().numpy()[l], ora[l]["zeros"])
            G.assert_kld_close(res.kld.cpu().numpy()[l], ora[l]["kld"], f"layer {l} algo {algo}")
            assert list(res.best.cpu().numpy()[l]) == list(ora[l]["best"])
    with pytest.raises(B.AdaptError):
        B.adapt_precision_search_ex(dev, grid, 7, n_bins_per_layer=[50, 0, 97, 2048, 1, 64])


def test_pushdown_as_a_descent_from_the_current_format(B):
    import torch
    w = W.WORKLOADS["resnet20_weights_grads"]
    xs = W.generate(w)[:8]
    wl, fl = W.candidate_grid(range(2, 17))
    grid = B.Grid(wl, fl)
    dev = G.to_device(xs)
    ora = O.precision_search(xs, wl, fl, 100, threads=G.host_threads())
    starts = [(8, 4), (16, 15), (16, 8), (2, 0), (12, 11), (16, 12), (9, 3), (17, 1)]
    for eps in (0.0, 1e-3):
        res = B.adapt_precision_search_ex(dev, grid, 100, eps=eps, start_wl_fl=starts)
        torch.cuda.synchronize()
        best = res.best.cpu().numpy()
        for l, (a, b) in enumerate(starts):
            want = O.select_descent(ora[l]["kld"], wl, fl, a, b, eps)
            assert list(best[l][:3]) == list(want[:3]), (l, eps)
            assert (best[l][3] & 1) == want[3]
    # without start formats the answer is the lowest admissible format of the whole grid
    res = B.adapt_precision_search_ex(dev, grid, 100)
    assert [list(r) for r in res.best.cpu().numpy()] == [list(o["best"]) for o in ora]


def test_on_grid_tensor_is_lossless(B):
    rng = np.random.default_rng(40)
    x = (rng.integers(-128, 128, 50000) * 2.0 ** -4).astype(np.float32)
    wl, fl = W.candidate_grid(range(2, 17))
    for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
        res, _ = G.run_and_compare(B, [x], wl, fl, 150, round_mode=mode, seed=9, where="on grid")
        kld = res.kld.cpu().numpy()[0]
        ok = (fl >= 4) & (wl - fl >= 4)
        assert (kld[ok] == 0.0).all()
        assert tuple(res.best.cpu().numpy()[0][:2]) <= (8, 4)


def test_nonfinite_and_out_of_range_layers_are_flagged(B):
    import torch
    rng = np.random.default_rng(2)
    good = (rng.standard_normal(6000)).astype(np.float32)
    bad_nan = good.copy(); bad_nan[4097] = np.nan
    bad_inf = good.copy(); bad_inf[17] = -np.inf
    bad_big = good.copy(); bad_big[5000] = 3e19            # |x| >= 2^64
    wl, fl = W.candidate_grid([4, 8])
    grid = B.Grid(wl, fl)
    dev = G.to_device([good, bad_nan, bad_inf, bad_big, good])
    res = B.adapt_precision_search_ex(dev, grid, 64, want_hist=True, want_status=True)
    torch.cuda.synchronize()
    assert list(res.status.cpu().numpy()) == [B.OK, B.ERR_NONFINITE, B.ERR_NONFINITE, B.ERR_RANGE, B.OK]
    flags = res.best.cpu().numpy()[:, 3]
    assert not flags[0] & (B.FLAG_NONFINITE | B.FLAG_RANGE)
    assert flags[1] & B.FLAG_NONFINITE and flags[2] & B.FLAG_NONFINITE
    assert flags[3] & B.FLAG_RANGE
    ora = O.precision_search([good], wl, fl, 64, want_hist=True)
    for l in (0, 4):   # the clean layers are unaffected by their neighbours
        assert np.array_equal(res.zeros.cpu().numpy()[l], ora[0]["zeros"])
        G.assert_kld_close(res.kld.cpu().numpy()[l], ora[0]["kld"])
    assert O.value_range(bad_nan)[2] == 1 and O.value_range(bad_inf)[2] == 1
    # the host-buffer form returns the data error as its status
    with pytest.raises(B.AdaptError) as e:
        B.adapt_precision_search_host([torch.from_numpy(bad_nan)], grid, 64)
    assert e.value.status == B.ERR_NONFINITE
    with pytest.raises(B.AdaptError) as e:
        B.adapt_precision_search_host([torch.from_numpy(bad_big)], grid, 64)
    assert e.value.status == B.ERR_RANGE


def test_caller_workspace_and_argument_errors(B):
    import torch
    rng = np.random.default_rng(8)
    x = (rng.standard_normal(10000) * 0.2).astype(np.float32)
    wl, fl = W.candidate_grid([3, 9])
    grid = B.Grid(wl, fl)
    dev = G.to_device([x])
    need = B.adapt_search_workspace_bytes([x.size], grid, 100)
    assert need > 0
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    res = B.adapt_precision_search_ex(dev, grid, 100, workspace=ws, want_hist=True, want_range=True)
    torch.cuda.synchronize()
    G.compare_search(res, O.precision_search([x], wl, fl, 100, want_hist=True), 1, "workspace",
                     True, True)
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.AdaptError) as e:
        B.adapt_precision_search_ex(dev, grid, 100, workspace=small)
    assert e.value.status == B.ERR_WORKSPACE
    for bad_bins in (0, -3, 16385):
        with pytest.raises(B.AdaptError) as e:
            B.adapt_precision_search_ex(dev, grid, bad_bins)
        assert e.value.status == B.ERR_INVALID_ARG
    for bw, bf in (([1], [0]), ([33], [0]), ([8], [8]), ([8], [-1])):
        with pytest.raises(B.AdaptError) as e:
            B.adapt_precision_search_ex(dev, B.Grid(bw, bf), 10)
        assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.AdaptError):
        B.adapt_precision_search_ex(dev, grid, 10, round_mode=7)
    with pytest.raises(B.AdaptError):
        B.adapt_precision_search_ex(dev, grid, 10, eps=-1.0)
    assert B.adapt_search_workspace_bytes([-1], grid, 10) == 0


def test_host_buffer_form_matches(B):
    import torch
    w = W.WORKLOADS["resnet20_weights_grads"]
    xs = W.generate(w)[:6] + W.generate(w)[20:24]
    wl, fl = w.grid()
    host = [torch.from_numpy(x).pin_memory() for x in xs]
    res = B.adapt_precision_search_host(host, B.Grid(wl, fl), w.n_bins, round_mode=w.round_mode,
                                        seed=w.seed)
    ora = O.precision_search(xs, wl, fl, w.n_bins, w.round_mode, w.seed, threads=G.host_threads())
    G.compare_search(res, ora, len(xs), "host form")
    # search + re-quantisation of every layer from one upload
    res2, codes = B.adapt_precision_switch_host(host, B.Grid(wl, fl), w.n_bins,
                                                round_mode=w.round_mode, seed=w.seed)
    G.compare_search(res2, ora, len(xs), "switch host form")
    for l, x in enumerate(xs):
        want, _ = O.quantize(x, int(ora[l]["best"][0]), int(ora[l]["best"][1]), w.round_mode, w.seed, l)
        assert np.array_equal(codes[l].numpy(), want), l


def test_host_switch_with_packed_codes_in_slices(B):
    """Packed codes through the host-buffer switch: layers larger than a download slice, many
    small ones, both rounding modes; a word length that does not fit is reported, not written."""
    import torch
    rng = np.random.default_rng(31)
    xs = [(rng.standard_normal((1 << 24) + 12345) * 0.05).astype(np.float32),      # two slices
          (rng.integers(-100, 100, 70000) * 2.0 ** -3).astype(np.float32),          # fits 8 bits
          np.zeros(0, np.float32),
          (rng.standard_normal(5000) * 0.3).astype(np.float32),
          (rng.integers(-20000, 20000, 40000) * 2.0 ** -2).astype(np.float32)]      # needs 17 bits
    wl, fl = W.candidate_grid(range(2, 21))
    host = [torch.from_numpy(x).pin_memory() for x in xs]
    for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
        ora = O.precision_search(xs, wl, fl, 64, mode, 9, threads=G.host_threads())
        for bits, dt in ((8, np.int8), (16, np.int16), (32, np.int32)):
            sentinel = [torch.full((x.size,), -77, dtype={8: torch.int8, 16: torch.int16, 32: torch.int32}[bits])
                        for x in xs]
            res, codes, unfit = B.adapt_precision_switch_host_packed(host, B.Grid(wl, fl), 64, bits,
                                                                    round_mode=mode, seed=9, codes_out=sentinel)
            G.compare_search(res, ora, len(xs), f"packed switch {bits} bits mode {mode}")
            for l, x in enumerate(xs):
                w_sel, f_sel = int(ora[l]["best"][0]), int(ora[l]["best"][1])
                if w_sel > bits:
                    assert unfit[l] == w_sel and (codes[l].numpy() == -77).all(), (l, bits)
                    continue
                assert unfit[l] == 0
                want, _ = O.quantize(x, w_sel, f_sel, mode, 9, l)
                assert np.array_equal(codes[l].numpy(), want.astype(dt)), (l, bits, mode)


def test_stochastic_rounding_large_layers_keyed_and_direct(B):
    """Stochastic rounding on layers large enough for its keyed kernel (cells for the fine
    levels, tables of rounded values for the coarse ones), against the oracle, next to the
    direct form: smooth data, many exact zeros, values on grids, ranges far from zero (left to
    the direct kernel by the plan), tiny and wide ranges, several layers in one call."""
    rng = np.random.default_rng(777)
    n = 50000
    base = (rng.standard_normal(n) * 0.25).astype(np.float32)
    cases = {
        "normal": base,
        "laplace_outliers": W.generate_layer(W.LayerSpec("t", (n,), "laplace_outliers", 0.02,
                                                         outlier_frac=0.01, outlier_gain=50.0), 3, 0),
        "half_zero": np.maximum(base, 0),
        "on_grid": (rng.integers(-2000, 2000, n) * 2.0 ** -6).astype(np.float32),
        "ties": (rng.integers(-4000, 4000, n) * 2.0 ** -9 + 2.0 ** -10).astype(np.float32),
        "far_from_zero": (1000.0 + rng.random(n) * 0.01).astype(np.float32),
        "far_negative": (-123456.0 - rng.random(n) * 64).astype(np.float32),
        "wide": (rng.standard_normal(n) * 1e6).astype(np.float32),
        "tiny": (rng.standard_normal(n) * 1e-9).astype(np.float32),
        "tiny_negative_fractions": (-np.abs(rng.standard_normal(n)) * 2.0 ** -30).astype(np.float32),
        "integers": rng.integers(-300, 300, n).astype(np.float32),
        "positive_only": (0.5 + 0.5 * rng.random(n)).astype(np.float32),
    }
    wl, fl = W.candidate_grid(range(2, 33))
    for name, x in cases.items():
        for n_bins in (100, 2048):
            G.run_and_compare(B, [x], wl, fl, n_bins, round_mode=O.ROUND_STOCHASTIC, seed=13, layer_base=2,
                              where=f"SR {name} B={n_bins}", algorithms=(0, 1, 2))
    # several layers, large and small, ragged and misaligned, in one call
    xs = [base[1:40001], cases["half_zero"][:33000], base[:100], np.zeros(0, np.float32),
          cases["far_from_zero"], cases["on_grid"][3:45000], np.full(40000, 0.37, np.float32)]
    G.run_and_compare(B, [np.ascontiguousarray(x) for x in xs], wl, fl, 128, round_mode=O.ROUND_STOCHASTIC,
                      seed=7, where="SR layers", algorithms=(0, 1, 2))
    # a layer large enough for the automatic choice to take the keyed route by itself
    big = W.generate_layer(W.LayerSpec("t", ((1 << 22) + 777,), "laplace_outliers", 0.02,
                                       outlier_frac=0.01, outlier_gain=50.0), 5, 0)
    wl2, fl2 = W.candidate_grid((6, 12, 20, 32))
    G.run_and_compare(B, [big, base], wl2, fl2, 256, round_mode=O.ROUND_STOCHASTIC, seed=21,
                      where="SR automatic route", algorithms=(0,))
