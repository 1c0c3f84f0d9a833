"""Seeded synthetic workloads for the precision-switch search.

This module only manufactures INPUTS (tensor shapes, value distributions,
candidate grids).  It holds none of the method's arithmetic and is the one
module both the CUDA path's callers and the CPU oracle's callers may use, so
that both sides read identical bytes.

The tensors stand in for the paper's workloads (AlexNet / ResNet trained on
CIFAR, Sec. 4.1): same layer shapes, weight values drawn like a fan-in
variance-scaling initialiser (Sec. 3.1), gradients heavy-tailed with exact
zeros, activations post-ReLU.  Values are generated chunk by chunk from a
counter-based generator (Philox keyed by seed, layer and chunk), so any chunk
of any layer can be regenerated on its own and the result does not depend on
the number of worker threads.
"""
from __future__ import annotations

import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

CHUNK = 1 << 22  # elements per independently seeded chunk

ROUND_RNE = 0
ROUND_STOCHASTIC = 1


@dataclass(frozen=True)
class LayerSpec:
    name: str
    shape: Tuple[int, ...]
    dist: str            # "normal" | "laplace" | "relu_normal" | "laplace_outliers" | "uniform" |
                         # "fixed_point"
    scale: float         # std (normal, fixed_point), b (laplace), std before ReLU (relu_normal),
                         # half width (uniform)
    zero_frac: float = 0.0      # share of positions forced to exactly 0
    outlier_frac: float = 0.0   # share of positions multiplied by outlier_gain
    outlier_gain: float = 1.0
    word: Tuple[int, int] = (0, 0)   # "fixed_point": the <WL,FL> whose representable values the
                                     # tensor is drawn from (a layer as a float32 simulation of
                                     # fixed-point training holds it, Sec. 4.1)

    @property
    def numel(self) -> int:
        return int(np.prod(self.shape)) if len(self.shape) else 1


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    layers: Tuple[LayerSpec, ...]
    wl_values: Tuple[int, ...]   # candidate word lengths; FL runs 0..WL-1 for each
    n_bins: int
    round_mode: int
    description: str = ""

    @property
    def numel(self) -> int:
        return sum(l.numel for l in self.layers)

    def grid(self):
        return candidate_grid(self.wl_values)


def candidate_grid(wl_values: Sequence[int]):
    """All <WL,FL> with FL in 0..WL-1, ordered by WL then FL. Returns (wl[], fl[]) int32."""
    wl, fl = [], []
    for w in sorted(wl_values):
        for f in range(w):
            wl.append(w)
            fl.append(f)
    return np.asarray(wl, dtype=np.int32), np.asarray(fl, dtype=np.int32)


def _kaiming(name: str, shape: Tuple[int, ...]) -> LayerSpec:
    fan_in = int(np.prod(shape[1:]))
    return LayerSpec(name, shape, "normal", math.sqrt(2.0 / fan_in))


def _alexnet_cifar_weights() -> List[LayerSpec]:
    shapes = [("conv1", (64, 3, 3, 3)), ("conv2", (192, 64, 3, 3)), ("conv3", (384, 192, 3, 3)),
              ("conv4", (256, 384, 3, 3)), ("conv5", (256, 256, 3, 3)),
              ("fc1", (4096, 1024)), ("fc2", (4096, 4096)), ("fc3", (10, 4096))]
    return [_kaiming(n, s) for n, s in shapes]


def _resnet20_shapes() -> List[Tuple[str, Tuple[int, ...]]]:
    shapes = [("conv1", (16, 3, 3, 3))]
    c_in = 16
    for stage, c in enumerate((16, 32, 64)):
        for blk in range(3):
            shapes.append((f"s{stage}b{blk}c1", (c, c_in, 3, 3)))
            shapes.append((f"s{stage}b{blk}c2", (c, c, 3, 3)))
            c_in = c
    shapes.append(("fc", (10, 64)))
    return shapes


def _resnet18_cifar_weights() -> List[LayerSpec]:
    shapes = [("conv1", (64, 3, 3, 3))]
    c_in = 64
    for stage, c in enumerate((64, 128, 256, 512)):
        for blk in range(2):
            shapes.append((f"l{stage}b{blk}c1", (c, c_in, 3, 3)))
            shapes.append((f"l{stage}b{blk}c2", (c, c, 3, 3)))
            if blk == 0 and c_in != c:
                shapes.append((f"l{stage}b{blk}ds", (c, c_in, 1, 1)))
            c_in = c
    shapes.append(("fc", (10, 512)))
    return [_kaiming(n, s) for n, s in shapes]


def _build_workloads():
    full = tuple(range(2, 33))
    w = {}
    w["single4k"] = Workload(
        "single4k", 0, (LayerSpec("t", (4096,), "normal", 0.05),), (4, 8, 12, 16), 64, ROUND_RNE,
        "one 4096-element N(0, sigma=0.05) tensor, 40 candidates, 64 bins")
    w["alexnet_weights"] = Workload(
        "alexnet_weights", 1, tuple(_alexnet_cifar_weights()), full, 256, ROUND_RNE,
        "AlexNet-for-CIFAR weight set, 8 tensors, fan-in normal init, 527 candidates, 256 bins")
    r20 = _resnet20_shapes()
    r20_w = [_kaiming("w_" + n, s) for n, s in r20]
    r20_g = [LayerSpec("g_" + n, s, "laplace", 1e-4, zero_frac=0.05) for n, s in r20]
    w["resnet20_weights_grads"] = Workload(
        "resnet20_weights_grads", 7, tuple(r20_w + r20_g), tuple(range(2, 17)), 128,
        ROUND_STOCHASTIC,
        "ResNet-20 weights + Laplace(0,1e-4) weight gradients with 5% exact zeros, "
        "stochastic rounding, 135 candidates, 128 bins")
    acts = [LayerSpec("act1", (128, 64, 32, 32), "relu_normal", 1.0),
            LayerSpec("act2", (128, 128, 16, 16), "relu_normal", 1.0),
            LayerSpec("act3", (128, 256, 8, 8), "relu_normal", 1.0),
            LayerSpec("act4", (128, 512, 4, 4), "relu_normal", 1.0)]
    w["resnet18_weights_acts"] = Workload(
        "resnet18_weights_acts", 4, tuple(_resnet18_cifar_weights() + acts), full, 512, ROUND_RNE,
        "ResNet-18 (CIFAR) weights + post-ReLU activations at batch 128, 527 candidates, 512 bins")
    w["stress_1g"] = Workload(
        "stress_1g", 3,
        (LayerSpec("t", (1 << 30,), "laplace_outliers", 0.02, outlier_frac=0.01, outlier_gain=50.0),),
        full, 2048, ROUND_RNE,
        "2^30 elements Laplace(0,0.02) with 1% outliers at 50x, 527 candidates, 2048 bins")
    return w


WORKLOADS = _build_workloads()
WORKLOAD_ORDER = ("single4k", "alexnet_weights", "resnet20_weights_grads",
                  "resnet18_weights_acts", "stress_1g")


def distribution_sweep(numel: int) -> List[Tuple[str, LayerSpec]]:
    """Single-layer tensors of other value classes than the stress workload's, for the bench's
    sweep of the fused kernel: smooth wide distributions, post-ReLU activations, a mostly-zero
    tensor, and tensors that already lie on a fixed-point grid."""
    n = (int(numel),)
    return [("normal", LayerSpec("t", n, "normal", 1.0)),
            ("uniform", LayerSpec("t", n, "uniform", 1.0)),
            ("half_zero_relu", LayerSpec("t", n, "relu_normal", 1.0)),
            ("zeros_90pct", LayerSpec("t", n, "normal", 1.0, zero_frac=0.9)),
            ("on_grid_8_4", LayerSpec("t", n, "fixed_point", 1.0, word=(8, 4))),
            ("on_grid_16_12", LayerSpec("t", n, "fixed_point", 1.0, word=(16, 12)))]


def scaled(workload: Workload, numel: int, name: Optional[str] = None) -> Workload:
    """A copy of a single-layer workload with a different element count (same
    distribution, grid, bins); for multi-tile parity cases and size sweeps."""
    assert len(workload.layers) == 1
    l = workload.layers[0]
    nl = LayerSpec(l.name, (int(numel),), l.dist, l.scale, l.zero_frac, l.outlier_frac,
                   l.outlier_gain)
    return Workload(name or f"{workload.name}_n{numel}", workload.seed, (nl,),
                    workload.wl_values, workload.n_bins, workload.round_mode, workload.description)


def _rng(seed: int, layer: int, chunk: int) -> np.random.Generator:
    key = np.array([seed & 0xFFFFFFFFFFFFFFFF, ((layer & 0xFFFFFFFF) << 32) | (chunk & 0xFFFFFFFF)],
                   dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _laplace(g: np.random.Generator, n: int, b: float) -> np.ndarray:
    u = g.random(n, dtype=np.float64) - 0.5          # [-0.5, 0.5)
    tail = np.maximum(1.0 - 2.0 * np.abs(u), 2.0 ** -60)
    return (-b * np.sign(u) * np.log(tail)).astype(np.float32)


def _fill_chunk(spec: LayerSpec, seed: int, layer: int, chunk: int, out: np.ndarray) -> None:
    n = out.size
    g = _rng(seed, layer, chunk)
    if spec.dist == "normal":
        v = g.standard_normal(n, dtype=np.float32) * np.float32(spec.scale)
    elif spec.dist == "relu_normal":
        v = np.maximum(g.standard_normal(n, dtype=np.float32) * np.float32(spec.scale),
                       np.float32(0.0))
    elif spec.dist in ("laplace", "laplace_outliers"):
        v = _laplace(g, n, spec.scale)
    elif spec.dist == "uniform":
        v = ((g.random(n, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)) *
             np.float32(spec.scale))
    elif spec.dist == "fixed_point":
        # integer words with a normal spread, kept inside the word, times the word's unit
        wl, fl = spec.word
        k = np.rint(g.standard_normal(n, dtype=np.float32) * np.float32(spec.scale * 2.0 ** fl))
        k = np.clip(k, -(2.0 ** (wl - 1)), 2.0 ** (wl - 1) - 1.0)
        v = (k * np.float32(2.0 ** -fl)).astype(np.float32)
    else:
        raise ValueError(spec.dist)
    if spec.outlier_frac > 0.0:
        m = g.random(n, dtype=np.float32) < np.float32(spec.outlier_frac)
        v = np.where(m, v * np.float32(spec.outlier_gain), v)
    if spec.zero_frac > 0.0:
        m = g.random(n, dtype=np.float32) < np.float32(spec.zero_frac)
        v = np.where(m, np.float32(0.0), v)
    out[:] = v


def default_threads() -> int:
    return max(1, min(32, (os.cpu_count() or 1)))


def generate_layer(spec: LayerSpec, seed: int, layer: int, out: Optional[np.ndarray] = None,
                   threads: Optional[int] = None, chunks: Optional[Sequence[int]] = None
                   ) -> np.ndarray:
    """Fill (or allocate) the flat fp32 values of one layer.  ``chunks`` restricts the
    work to the listed chunk indices (the rest of ``out`` is left untouched)."""
    n = spec.numel
    if out is None:
        out = np.empty(n, dtype=np.float32)
    assert out.dtype == np.float32 and out.size == n
    flat = out.reshape(-1)
    n_chunks = (n + CHUNK - 1) // CHUNK
    todo = list(range(n_chunks)) if chunks is None else list(chunks)

    def work(c):
        _fill_chunk(spec, seed, layer, c, flat[c * CHUNK:min(n, (c + 1) * CHUNK)])

    threads = threads or default_threads()
    if threads <= 1 or len(todo) <= 1:
        for c in todo:
            work(c)
    else:
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(work, todo))
    return out


def generate(workload: Workload, threads: Optional[int] = None) -> List[np.ndarray]:
    """All layers of a workload as flat fp32 numpy arrays (layer index = position)."""
    return [generate_layer(spec, workload.seed, l, threads=threads)
            for l, spec in enumerate(workload.layers)]
