"""The seeded input generators: shapes, counts, determinism, value classes. CPU only."""
import numpy as np

from paper_2107_13490_b200 import workloads as W


def test_workload_sizes_and_grids():
    sizes = {k: (len(W.WORKLOADS[k].layers), W.WORKLOADS[k].numel, W.WORKLOADS[k].grid()[0].size)
             for k in W.WORKLOAD_ORDER}
    assert sizes["single4k"] == (1, 4096, 40)
    assert sizes["alexnet_weights"] == (8, 23262912, 527)
    assert sizes["resnet20_weights_grads"] == (40, 2 * 268336, 135)
    assert sizes["resnet18_weights_acts"] == (25, 11164352 + 15728640, 527)
    assert sizes["stress_1g"] == (1, 1 << 30, 527)
    wl, fl = W.candidate_grid(range(2, 33))
    assert wl.size == 527 and (fl < wl).all() and fl.min() == 0
    order = list(zip(wl.tolist(), fl.tolist()))
    assert order == sorted(order)


def test_generation_is_deterministic_and_chunk_addressable():
    spec = W.scaled(W.WORKLOADS["stress_1g"], 3 * W.CHUNK + 12345).layers[0]
    a = W.generate_layer(spec, 3, 0, threads=1)
    b = W.generate_layer(spec, 3, 0, threads=4)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    c = np.zeros_like(a)
    W.generate_layer(spec, 3, 0, out=c, chunks=[2])
    assert np.array_equal(c[2 * W.CHUNK:3 * W.CHUNK], a[2 * W.CHUNK:3 * W.CHUNK])
    assert not c[:2 * W.CHUNK].any()
    d = W.generate_layer(spec, 4, 0, threads=4)
    assert not np.array_equal(a, d)
    assert np.isfinite(a).all()


def test_value_classes():
    w = W.WORKLOADS["resnet20_weights_grads"]
    xs = W.generate(w)
    g = np.concatenate(xs[20:])
    assert 0.04 < (g == 0).mean() < 0.06
    assert 0.5e-4 < np.abs(g[g != 0]).mean() < 1.5e-4       # Laplace(0, 1e-4): E|x| = b
    conv = xs[1]                                              # [16,16,3,3]: std = sqrt(2/144)
    assert abs(conv.std() - np.sqrt(2 / 144)) < 0.01
    acts = W.generate_layer(W.LayerSpec("a", (1 << 18,), "relu_normal", 1.0), 4, 21)
    assert 0.48 < (acts == 0).mean() < 0.52 and acts.min() == 0
    s = W.generate(W.scaled(W.WORKLOADS["stress_1g"], 1 << 20))[0]
    assert 0.025 < np.abs(s).mean() < 0.035                 # 0.99*0.02 + 0.01*1.0
