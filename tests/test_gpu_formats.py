"""GPU parity of the format search and the format quantize kernel against the CPU oracle:
values, zero counts, block scales and choices bit-exact; divergences within 1e-5 relative."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2107_13490_b200 import workloads as W
from tests.gpu_util import assert_kld_close, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2107_13490_b200 import binding
    binding.lib()
    return binding


def mixed_formats():
    """Block floating point at every word length up to 16, a ladder of float formats, and a
    few fixed-point formats (which share histograms with each other by FL)."""
    f = [(O.FMT_BFP, wl, 0) for wl in range(2, 17)]
    f += [(O.FMT_FLOAT, e, m) for e, m in ((2, 1), (3, 2), (4, 3), (5, 2), (5, 10), (8, 7), (6, 9),
                                           (8, 23))]
    f += [(O.FMT_FIXED, wl, fl) for wl, fl in ((4, 3), (8, 3), (8, 7), (16, 12), (16, 15))]
    return f


def run_and_compare(B, tensors_np, formats, n_bins, round_mode=0, seed=0, layer_base=0, eps=0.0,
                    pseudo_count=0.0, where=""):
    import torch
    dev = to_device(tensors_np)
    res = B.adapt_format_search(dev, formats, n_bins, round_mode=round_mode, seed=seed,
                                layer_base=layer_base, eps=eps, pseudo_count=pseudo_count,
                                want_range=True, want_hist=True)
    torch.cuda.synchronize()
    hist = res.hist.cpu().numpy().view(np.uint32)
    kld, zeros = res.kld.cpu().numpy(), res.zeros.cpu().numpy()
    b, best, rng = res.b.cpu().numpy(), res.best.cpu().numpy(), res.range.cpu().numpy()
    kind = [f[0] for f in formats]
    a = [f[1] for f in formats]
    bb = [f[2] for f in formats]
    for l, t in enumerate(tensors_np):
        o = O.format_search_layer(t, kind, a, bb, n_bins, round_mode, seed, layer_base + l, eps,
                                  pseudo_count)
        tag = f"{where} layer {l}"
        assert rng[l][0] == o["range"][0] and rng[l][1] == o["range"][1], tag
        assert np.array_equal(b[l], o["b"]), f"{tag}: scales {b[l]} vs {o['b']}"
        assert np.array_equal(zeros[l], o["zeros"]), f"{tag}: zero counts differ"
        assert_kld_close(kld[l], o["kld"], tag)
        assert list(best[l]) == list(o["best"]), f"{tag}: best {best[l]} vs {o['best']}"
        if t.size == 0 or o["nonfinite"]:
            continue
        # every format's histogram bin by bin: the oracle's values of the format through the
        # oracle's own histogram step, on the float tensor's range
        lo, hi = o["range"]
        assert np.array_equal(hist[l][0].astype(np.uint64), O.histogram(t, lo, hi, n_bins)), tag
        for c, (k, fa, _) in enumerate(formats):
            vals = O.format_quantize(t, k, fa, int(o["b"][c]), round_mode, seed, layer_base + l)
            assert np.array_equal(hist[l][c + 1].astype(np.uint64), O.histogram(vals, lo, hi, n_bins)), \
                f"{tag}: histogram of format {formats[c]} differs"
    return res


def test_single4k_mixed_formats_both_modes(B):
    w = W.WORKLOADS["single4k"]
    x = W.generate(w)
    for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
        run_and_compare(B, x, mixed_formats(), w.n_bins, round_mode=mode, seed=7, where=f"mode {mode}")


def test_layers_of_many_scales_ragged_and_misaligned(B):
    rng = np.random.default_rng(21)
    base = (rng.standard_normal(70000)).astype(np.float32)
    tensors = [
        base[:4097] * np.float32(1e-3),
        base[1:9000] * np.float32(300.0),                 # misaligned view, block scale < 0
        np.abs(base[2:30003]) * np.float32(0.1),          # one-sided: only the upper extreme
        -np.abs(base[3:5004]) * np.float32(2e-6),         # one-sided negative, tiny
        np.zeros(100, dtype=np.float32),                  # all zero: scale 0, one bin
        base[:1] * np.float32(0.5),                       # a single element
        np.float32([1e-40, -3e-41, 5e-39, 0.0, 2e-38]),   # subnormal inputs
        base[5:65541] * np.float32(1e4),
        np.zeros(0, dtype=np.float32),                    # empty layer
    ]
    tensors = [np.ascontiguousarray(t) for t in tensors]
    for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
        run_and_compare(B, tensors, mixed_formats(), 128, round_mode=mode, seed=3, layer_base=4,
                        where=f"mode {mode}")
    run_and_compare(B, tensors, mixed_formats(), 128, eps=1e-3, pseudo_count=0.5, where="eps")


def test_weights_and_gradients_workload(B):
    """The ResNet-20 weight and gradient tensors: 40 layers, many more rules than fit in one
    group at 2048 bins, so the rule groups are exercised."""
    w = W.WORKLOADS["resnet20_weights_grads"]
    x = W.generate(w)
    formats = [(O.FMT_BFP, wl, 0) for wl in range(2, 33)] + \
              [(O.FMT_FLOAT, e, m) for e in (2, 3, 4, 5, 8) for m in (1, 2, 3, 5, 7, 10)]
    run_and_compare(B, x, formats, 2048, where="resnet20 rne")
    run_and_compare(B, x, formats[:20], 128, round_mode=O.ROUND_STOCHASTIC, seed=7,
                    where="resnet20 sr")


def test_fixed_point_candidates_agree_with_the_grid_search(B):
    """The same fixed-point candidates through both search calls give the same numbers."""
    import torch
    w = W.WORKLOADS["single4k"]
    x = W.generate(w)
    wl, fl = w.grid()
    dev = to_device(x)
    formats = [(O.FMT_FIXED, a, f) for a, f in zip(wl.tolist(), fl.tolist())]
    r1 = B.adapt_format_search(dev, formats, w.n_bins)
    r2 = B.adapt_precision_search_ex(dev, B.Grid(wl, fl), w.n_bins)
    torch.cuda.synchronize()
    assert torch.equal(r1.zeros, r2.zeros)
    assert torch.allclose(r1.kld, r2.kld, rtol=1e-12, atol=0.0)
    assert torch.equal(r1.best, r2.best)     # the grid is listed in (WL, FL) order


def _specials():
    return np.float32([0.0, -0.0, 0.5, -0.5, 1.5, 2.5, -2.5, 0.3, 1e-45, -1e-45, 2 ** -32, 3e9,
                       -3e9, 65504.0, 65520.0, 65519.9, -65520.0, 5.9604645e-08, 2.9802322e-08,
                       2.9802326e-08, 1e-40, 1.1754944e-38, 1e30, -1e30, 2.0 ** 63, 0.9375,
                       3.3895314e38, 240.0, 248.0, 1.00390625, 1.01171875])


def test_format_quantize_values(B):
    import torch
    rng = np.random.default_rng(8)
    x = np.concatenate([
        (rng.standard_normal(50001) * 10.0 ** rng.uniform(-9, 4.5, 50001)).astype(np.float32),
        _specials()])
    x = x[np.abs(x) < 2.0 ** 64]
    xd = torch.from_numpy(x).cuda()
    cases = [(O.FMT_FLOAT, e, m) for e, m in ((2, 1), (3, 2), (4, 3), (5, 2), (5, 10), (8, 7),
                                              (8, 23), (7, 23), (6, 1))]
    cases += [(O.FMT_BFP, 4, 3), (O.FMT_BFP, 8, -7), (O.FMT_BFP, 16, 30), (O.FMT_BFP, 32, 5),
              (O.FMT_BFP, 2, -100), (O.FMT_BFP, 12, 100), (O.FMT_FIXED, 8, 4), (O.FMT_FIXED, 32, 31)]
    for kind, a, b in cases:
        for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
            got = B.adapt_format_quantize(xd, kind, a, b, mode, seed=5, layer=2).cpu().numpy()
            want = O.format_quantize(x, kind, a, b, mode, seed=5, layer=2)
            bad = np.where(got != want)[0]
            assert bad.size == 0, (kind, a, b, mode, x[bad[:5]], got[bad[:5]], want[bad[:5]])


def test_format_search_rejects_bad_arguments(B):
    import torch
    x = [torch.zeros(16, device="cuda")]
    for bad in ([(O.FMT_FLOAT, 9, 3)], [(O.FMT_FLOAT, 5, 0)], [(O.FMT_BFP, 1, 0)], [(O.FMT_FIXED, 8, 8)],
                [(7, 8, 3)], []):
        with pytest.raises(B.AdaptError) as e:
            B.adapt_format_search(x, bad, 16)
        assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.AdaptError):
        B.adapt_format_quantize(x[0], O.FMT_BFP, 8, 101)
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.AdaptError) as e:
        B.adapt_format_search(x, [(O.FMT_BFP, 8, 0)], 16, workspace=ws)
    assert e.value.status == B.ERR_WORKSPACE
    need = B.adapt_format_search_workspace_bytes([16], [(O.FMT_BFP, 8, 0)], 16)
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    off = (-ws.data_ptr()) % 256
    r = B.adapt_format_search(x, [(O.FMT_BFP, 8, 0)], 16, workspace=ws[off:off + need])
    torch.cuda.synchronize()
    assert r.best.cpu().numpy()[0].tolist()[2] == 0
