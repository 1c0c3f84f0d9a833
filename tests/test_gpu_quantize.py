"""GPU parity of the stand-alone Quantize kernel against the CPU oracle (bit-exact codes)."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2107_13490_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2107_13490_b200 import binding
    binding.lib()
    return binding


def _specials():
    return np.float32([0.0, -0.0, 0.5, -0.5, 1.5, 2.5, -2.5, 0.3, 1e-45, -1e-45, 2 ** -32, 3e9, -3e9,
                       2 ** 31, -2 ** 31, 2 ** 30, 16777217.0, 8388607.5, -8388608.5, 0.49999997,
                       127.5, -128.5, 32767.5, 1e30, -1e30, 2.0 ** 63, 0.9375])


def test_single4k_every_candidate_both_modes(B):
    import torch
    w = W.WORKLOADS["single4k"]
    x = np.concatenate([W.generate(w)[0], _specials()])
    xd = torch.from_numpy(x).cuda()
    wl, fl = w.grid()
    for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
        for a, f in zip(wl.tolist(), fl.tolist()):
            got = B.adapt_quantize(xd, a, f, mode, seed=7)
            want, _ = O.quantize(x, a, f, mode, seed=7, layer=0)
            assert np.array_equal(got.cpu().numpy(), want), (a, f, mode)


@pytest.mark.parametrize("bits", [8, 16, 32])
def test_code_widths_layers_and_alignment(B, bits):
    import torch
    rng = np.random.default_rng(bits)
    dt = {8: np.int8, 16: np.int16, 32: np.int32}[bits]
    for n in (0, 1, 3, 4, 5, 255, 1024, 4099, 100003):
        for mis in (0, 1, 3):
            x = np.concatenate([(rng.standard_normal(n) * 20).astype(np.float32)])
            buf = torch.zeros(n + 4, dtype=torch.float32, device="cuda")
            buf[mis:mis + n] = torch.from_numpy(x).cuda()
            out = torch.full((n + 4,), -1, dtype=getattr(torch, f"int{bits}"), device="cuda")
            for wl, fl in ((2, 0), (bits, bits // 2), (bits, bits - 1), (min(bits, 7), 3)):
                for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
                    view = out[mis:mis + n]
                    B.adapt_quantize_ex(buf[mis:mis + n], wl, fl, mode, seed=5, layer=3,
                                        code_bits=bits, codes_out=view)
                    torch.cuda.synchronize()
                    want, _ = O.quantize(x, wl, fl, mode, seed=5, layer=3)
                    assert np.array_equal(view.cpu().numpy(), want.astype(dt)), (n, mis, wl, fl, mode)
                    # nothing is written outside [0, n)
                    assert (out[:mis] == -1).all() and (out[mis + n:] == -1).all()


def test_quantize_large_multi_wave(B):
    import torch
    w = W.scaled(W.WORKLOADS["stress_1g"], (1 << 24) + 3)
    x = W.generate(w)[0]
    xd = torch.from_numpy(x).cuda()
    for wl, fl, mode in ((8, 4, O.ROUND_RNE), (16, 10, O.ROUND_STOCHASTIC), (32, 20, O.ROUND_RNE)):
        got = B.adapt_quantize_ex(xd, wl, fl, mode, seed=3, layer=0, code_bits=32)
        want, _ = O.quantize(x, wl, fl, mode, seed=3, layer=0)
        assert np.array_equal(got.cpu().numpy(), want)


def test_quantize_at_device_resident_selection(B):
    import torch
    rng = np.random.default_rng(1)
    x = (rng.standard_normal(50001) * 0.4).astype(np.float32)
    xd = torch.from_numpy(x).cuda()
    wl, fl = W.candidate_grid(range(2, 17))
    res = B.adapt_precision_search_ex([xd], B.Grid(wl, fl), 100)
    got = B.adapt_quantize_selected(xd, res.best[0], O.ROUND_RNE)
    torch.cuda.synchronize()
    ora = O.precision_search_layer(x, wl, fl, 100)
    want, _ = O.quantize(x, int(ora["best"][0]), int(ora["best"][1]))
    assert np.array_equal(got.cpu().numpy(), want)


def test_batched_quantize_at_device_resident_selections(B):
    import torch
    w = W.WORKLOADS["resnet20_weights_grads"]
    xs = W.generate(w)
    pick = [0, 3, 10, 19, 20, 25, 39]
    wl, fl = w.grid()
    for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
        bufs = []
        for j, i in enumerate(pick):     # odd phases: some layers take the scalar path
            b = torch.zeros(xs[i].size + 4, dtype=torch.float32, device="cuda")
            b[j % 4:j % 4 + xs[i].size] = torch.from_numpy(xs[i]).cuda()
            bufs.append(b[j % 4:j % 4 + xs[i].size])
        bufs.append(torch.zeros(0, dtype=torch.float32, device="cuda"))       # an empty layer
        res = B.adapt_precision_search_ex(bufs, B.Grid(wl, fl), w.n_bins, round_mode=mode, seed=7,
                                          layer_base=2)
        codes = B.adapt_quantize_selected_batch(bufs, res.best, mode, seed=7, layer_base=2)
        torch.cuda.synchronize()
        ora = O.precision_search([xs[i] for i in pick], wl, fl, w.n_bins, mode, 7, 2)
        for j, i in enumerate(pick):
            want, _ = O.quantize(xs[i], int(ora[j]["best"][0]), int(ora[j]["best"][1]), mode, 7, 2 + j)
            assert np.array_equal(codes[j].cpu().numpy(), want), (mode, i)
        assert codes[-1].numel() == 0
        # packed codes: a layer whose selected word length exceeds the code width is reported
        # and left untouched, the others hold the oracle's codes
        sel = [int(ora[j]["best"][0]) for j in range(len(pick))]
        for bits, dt in ((8, np.int8), (16, np.int16), (32, np.int32)):
            outs = [torch.full((b.numel() + 3,), 77, dtype={8: torch.int8, 16: torch.int16, 32: torch.int32}[bits],
                               device="cuda")[(j % 3):(j % 3) + b.numel()] for j, b in enumerate(bufs)]
            packed, unfit = B.adapt_quantize_selected_batch_packed(bufs, res.best, bits, mode, seed=7,
                                                                   layer_base=2, codes_out=outs)
            torch.cuda.synchronize()
            unfit = unfit.cpu().numpy()
            for j, i in enumerate(pick):
                if sel[j] > bits:
                    assert unfit[j] == sel[j] and (packed[j] == 77).all(), (mode, bits, i)
                else:
                    want, _ = O.quantize(xs[i], sel[j], int(ora[j]["best"][1]), mode, 7, 2 + j)
                    assert unfit[j] == 0 and np.array_equal(packed[j].cpu().numpy(), want.astype(dt)), (mode, bits, i)
            assert unfit[-1] == 0
        # the same loop with dequantized fp32 values as output, to new tensors and in place
        vals = B.adapt_requantize_selected_batch(bufs, res.best, mode, seed=7, layer_base=2)
        torch.cuda.synchronize()
        for j, i in enumerate(pick):
            _, xhat = O.quantize(xs[i], int(ora[j]["best"][0]), int(ora[j]["best"][1]), mode, 7, 2 + j)
            assert np.array_equal(vals[j].cpu().numpy().view(np.uint32), xhat.view(np.uint32)), (mode, i)
        B.adapt_requantize_selected_batch(bufs, res.best, mode, seed=7, layer_base=2, values_out=bufs)
        torch.cuda.synchronize()
        for j in range(len(pick)):
            assert torch.equal(bufs[j], vals[j]), (mode, j)


def test_batched_quantize_repeats_and_changes_its_layer_list(B):
    """The library keeps the layer table of the call before: the same list again (no upload), a
    different list, the first list once more, and the same tensors with new formats must each
    give the oracle's codes."""
    import torch
    rng = np.random.default_rng(31)
    xs = [(rng.standard_normal(n) * 0.3).astype(np.float32) for n in (5000, 70001, 333)]
    dev = [torch.from_numpy(x).cuda() for x in xs]
    fmt_a = np.array([[8, 4, 0, 1], [12, 9, 0, 1], [5, 2, 0, 1]], dtype=np.int32)
    fmt_b = np.array([[16, 12, 0, 1], [4, 1, 0, 1], [9, 8, 0, 1]], dtype=np.int32)

    def check(tensors, hosts, fmt):
        best = torch.from_numpy(fmt[:len(tensors)].copy()).cuda()
        codes = B.adapt_quantize_selected_batch(tensors, best, O.ROUND_RNE, seed=0, layer_base=0)
        torch.cuda.synchronize()
        for j, x in enumerate(hosts):
            want, _ = O.quantize(x, int(fmt[j][0]), int(fmt[j][1]), O.ROUND_RNE, 0, j)
            assert np.array_equal(codes[j].cpu().numpy(), want), j
        return codes

    outs = [torch.empty(x.size, dtype=torch.int32, device="cuda") for x in xs]

    def check_into(fmt):
        best = torch.from_numpy(fmt.copy()).cuda()
        B.adapt_quantize_selected_batch(dev, best, O.ROUND_RNE, seed=0, layer_base=0, codes_out=outs)
        torch.cuda.synchronize()
        for j, x in enumerate(xs):
            want, _ = O.quantize(x, int(fmt[j][0]), int(fmt[j][1]), O.ROUND_RNE, 0, j)
            assert np.array_equal(outs[j].cpu().numpy(), want), j

    check_into(fmt_a)            # uploads the table
    check_into(fmt_a)            # same tensors, same outputs: the table is reused
    check_into(fmt_b)            # same table, other formats on the device
    check(dev[:2], xs[:2], fmt_b)    # a different list (new output tensors)
    check_into(fmt_a)            # the first list again


def test_quantize_argument_errors_and_host_form(B):
    import torch
    x = torch.zeros(16, dtype=torch.float32, device="cuda")
    for wl, fl, bits in ((1, 0, 32), (33, 0, 32), (8, 8, 32), (9, 0, 8), (17, 3, 16), (8, 4, 12)):
        with pytest.raises(B.AdaptError) as e:
            B.adapt_quantize_ex(x, wl, fl, code_bits=bits)
        assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.AdaptError):
        B.adapt_quantize_ex(x, 8, 4, round_mode=5)
    rng = np.random.default_rng(4)
    h = (rng.standard_normal(70001) * 3).astype(np.float32)
    got = B.adapt_quantize_host(torch.from_numpy(h), 8, 3, O.ROUND_STOCHASTIC, seed=2, layer=1,
                                code_bits=8)
    want, _ = O.quantize(h, 8, 3, O.ROUND_STOCHASTIC, seed=2, layer=1)
    assert np.array_equal(got.numpy(), want.astype(np.int8))
