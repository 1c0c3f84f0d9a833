"""numpy/ctypes front end of the CPU oracle (``adapt_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline legs, never by the product package.  It compiles the
oracle with g++ on first use (``-O2 -ffp-contract=off -fno-fast-math``) and
marshals numpy arrays; every number is computed in the C++ file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "adapt_oracle.cpp")
_SO = os.path.join(_HERE, "libadapt_oracle.so")

ROUND_RNE = 0
ROUND_STOCHASTIC = 1
FMT_FIXED = 0   # <WL, FL>
FMT_BFP = 1     # block floating point: word length, scale derived from the layer
FMT_FLOAT = 2   # <exponent bits, mantissa bits>

_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle shared object next to its source; returns its path."""
    stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _SO + ".tmp%d" % os.getpid()
        cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", "-o", tmp, _SRC]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _SO)
    return _SO


def _f32p(a):
    return a.ctypes.data_as(C.POINTER(C.c_float))


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            L.adapt_oracle_hash24.restype = C.c_uint32
            L.adapt_oracle_hash24.argtypes = [C.c_uint64, C.c_uint64, C.c_uint64]
            L.adapt_oracle_quantize_one.restype = C.c_int32
            L.adapt_oracle_quantize_one.argtypes = [C.c_float, C.c_int, C.c_int, C.c_int, C.c_uint32]
            L.adapt_oracle_dequantize_one.restype = C.c_float
            L.adapt_oracle_dequantize_one.argtypes = [C.c_int32, C.c_int]
            L.adapt_oracle_bin_index.restype = C.c_int
            L.adapt_oracle_bin_index.argtypes = [C.c_float, C.c_float, C.c_float, C.c_int]
            L.adapt_oracle_quantize.restype = None
            L.adapt_oracle_quantize.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_int,
                                                C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
            L.adapt_oracle_range.restype = C.c_int
            L.adapt_oracle_range.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
            L.adapt_oracle_histogram.restype = None
            L.adapt_oracle_histogram.argtypes = [C.c_void_p, C.c_int64, C.c_float, C.c_float,
                                                 C.c_int, C.c_void_p]
            L.adapt_oracle_kld.restype = C.c_double
            L.adapt_oracle_kld.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_double, C.c_double]
            L.adapt_oracle_select.restype = None
            L.adapt_oracle_select.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                              C.c_double, C.c_void_p]
            L.adapt_oracle_precision_search.restype = C.c_int
            L.adapt_oracle_precision_search.argtypes = [
                C.c_void_p, C.c_int64, C.c_uint64, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                C.c_int, C.c_uint64, C.c_double, C.c_double, C.c_double,
                C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
            L.adapt_oracle_select_descent.restype = None
            L.adapt_oracle_select_descent.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                                      C.c_double, C.c_int, C.c_int, C.c_void_p]
            L.adapt_oracle_gradient_diversity.restype = None
            L.adapt_oracle_gradient_diversity.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_void_p]
            L.adapt_oracle_pushup.restype = None
            L.adapt_oracle_pushup.argtypes = [C.c_double, C.c_int, C.c_int, C.c_int, C.c_int,
                                              C.c_void_p]
            L.adapt_oracle_normalize_gradient.restype = None
            L.adapt_oracle_normalize_gradient.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
            L.adapt_oracle_bfp_scale.restype = C.c_int
            L.adapt_oracle_bfp_scale.argtypes = [C.c_float, C.c_float, C.c_int]
            L.adapt_oracle_format_value_one.restype = C.c_float
            L.adapt_oracle_format_value_one.argtypes = [C.c_float, C.c_int, C.c_int, C.c_int,
                                                        C.c_int, C.c_uint32]
            L.adapt_oracle_format_quantize.restype = None
            L.adapt_oracle_format_quantize.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_int,
                                                       C.c_int, C.c_int, C.c_uint64, C.c_uint64,
                                                       C.c_void_p]
            L.adapt_oracle_format_search.restype = C.c_int
            L.adapt_oracle_format_search.argtypes = [
                C.c_void_p, C.c_int64, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                C.c_int, C.c_int, C.c_uint64, C.c_double, C.c_double, C.c_double,
                C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
            _lib = L
    return _lib


def _as_f32(x):
    a = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    return a


def hash24(seed: int, layer: int, index: int) -> int:
    return int(lib().adapt_oracle_hash24(seed, layer, index))


def quantize_one(x: float, wl: int, fl: int, round_mode: int = ROUND_RNE, k24: int = 0) -> int:
    return int(lib().adapt_oracle_quantize_one(np.float32(x), wl, fl, round_mode, k24))


def dequantize_one(code: int, fl: int) -> float:
    return float(lib().adapt_oracle_dequantize_one(code, fl))


def bin_index(v: float, lo: float, hi: float, n_bins: int) -> int:
    return int(lib().adapt_oracle_bin_index(np.float32(v), np.float32(lo), np.float32(hi), n_bins))


def quantize(x, wl: int, fl: int, round_mode: int = ROUND_RNE, seed: int = 0, layer: int = 0):
    """Returns (codes int32[n], xhat float32[n])."""
    a = _as_f32(x)
    codes = np.empty(a.size, dtype=np.int32)
    xhat = np.empty(a.size, dtype=np.float32)
    lib().adapt_oracle_quantize(a.ctypes.data, a.size, wl, fl, round_mode, seed, layer,
                                codes.ctypes.data, xhat.ctypes.data)
    return codes, xhat


def value_range(x):
    """Returns (lo, hi, nonfinite flag)."""
    a = _as_f32(x)
    lo = C.c_float()
    hi = C.c_float()
    bad = lib().adapt_oracle_range(a.ctypes.data, a.size, C.byref(lo), C.byref(hi))
    return np.float32(lo.value), np.float32(hi.value), int(bad)


def histogram(v, lo, hi, n_bins: int):
    a = _as_f32(v)
    h = np.empty(n_bins, dtype=np.uint64)
    lib().adapt_oracle_histogram(a.ctypes.data, a.size, np.float32(lo), np.float32(hi), n_bins,
                                 h.ctypes.data)
    return h


def kld(p_hist, q_hist, alpha: float = 0.0, log_base: float = 2.0) -> float:
    p = np.ascontiguousarray(p_hist, dtype=np.uint64)
    q = np.ascontiguousarray(q_hist, dtype=np.uint64)
    assert p.size == q.size
    return float(lib().adapt_oracle_kld(p.ctypes.data, q.ctypes.data, p.size, alpha, log_base))


def select(kld_values, wl, fl, eps: float = 0.0):
    k = np.ascontiguousarray(kld_values, dtype=np.float64)
    w = np.ascontiguousarray(wl, dtype=np.int32)
    f = np.ascontiguousarray(fl, dtype=np.int32)
    out = np.zeros(4, dtype=np.int32)
    lib().adapt_oracle_select(k.ctypes.data, w.ctypes.data, f.ctypes.data, k.size, eps,
                              out.ctypes.data)
    return out


def select_descent(kld_values, wl, fl, start_wl: int, start_fl: int, eps: float = 0.0):
    """PushDown as a descent from <start_wl, start_fl>; returns int32[4] {wl, fl, index, flags}."""
    k = np.ascontiguousarray(kld_values, dtype=np.float64)
    w = np.ascontiguousarray(wl, dtype=np.int32)
    f = np.ascontiguousarray(fl, dtype=np.int32)
    out = np.zeros(4, dtype=np.int32)
    lib().adapt_oracle_select_descent(k.ctypes.data, w.ctypes.data, f.ctypes.data, k.size, eps,
                                      start_wl, start_fl, out.ctypes.data)
    return out


def precision_search_layer(x, wl, fl, n_bins: int, round_mode: int = ROUND_RNE, seed: int = 0,
                           layer: int = 0, eps: float = 0.0, alpha: float = 0.0,
                           log_base: float = 2.0, want_hist: bool = False):
    """One layer, all candidates in sequence. Returns a dict of numpy arrays."""
    a = _as_f32(x)
    w = np.ascontiguousarray(wl, dtype=np.int32)
    f = np.ascontiguousarray(fl, dtype=np.int32)
    nc = w.size
    kl = np.zeros(nc, dtype=np.float64)
    zeros = np.zeros(nc, dtype=np.int64)
    best = np.zeros(4, dtype=np.int32)
    rng = np.zeros(2, dtype=np.float32)
    hist = np.zeros((nc + 1, n_bins), dtype=np.uint64) if want_hist else None
    bad = lib().adapt_oracle_precision_search(
        a.ctypes.data, a.size, layer, w.ctypes.data, f.ctypes.data, nc, n_bins, round_mode,
        seed, eps, alpha, log_base, kl.ctypes.data, zeros.ctypes.data, best.ctypes.data,
        hist.ctypes.data if want_hist else None, rng.ctypes.data)
    return {"kld": kl, "zeros": zeros, "best": best, "hist": hist, "range": rng,
            "nonfinite": int(bad)}


def precision_search(tensors, wl, fl, n_bins: int, round_mode: int = ROUND_RNE, seed: int = 0,
                     layer_base: int = 0, eps: float = 0.0, alpha: float = 0.0,
                     log_base: float = 2.0, want_hist: bool = False, threads: int = 1):
    """All layers. ``threads`` > 1 farms whole (layer, candidate-slice) calls of the
    single-threaded oracle over a thread pool (ctypes releases the GIL); the
    per-candidate arithmetic is untouched and the selection is redone over the
    gathered divergences by the oracle's own select()."""
    w = np.ascontiguousarray(wl, dtype=np.int32)
    f = np.ascontiguousarray(fl, dtype=np.int32)
    nc = w.size
    results = []
    if threads <= 1:
        for l, t in enumerate(tensors):
            results.append(precision_search_layer(t, w, f, n_bins, round_mode, seed,
                                                  layer_base + l, eps, alpha, log_base, want_hist))
        return results

    jobs = []
    for l, t in enumerate(tensors):
        a = _as_f32(t)
        n_slices = max(1, min(nc, threads if a.size >= (1 << 16) else 1))
        bounds = np.linspace(0, nc, n_slices + 1).astype(int)
        for s in range(n_slices):
            jobs.append((l, a, int(bounds[s]), int(bounds[s + 1])))

    def run(job):
        l, a, c0, c1 = job
        r = precision_search_layer(a, w[c0:c1], f[c0:c1], n_bins, round_mode, seed,
                                   layer_base + l, eps, alpha, log_base, want_hist)
        return l, c0, c1, r

    with ThreadPoolExecutor(max_workers=threads) as pool:
        parts = list(pool.map(run, jobs))
    for l, t in enumerate(tensors):
        kl = np.zeros(nc, dtype=np.float64)
        zeros = np.zeros(nc, dtype=np.int64)
        hist = np.zeros((nc + 1, n_bins), dtype=np.uint64) if want_hist else None
        rng = None
        bad = 0
        for (pl, c0, c1, r) in parts:
            if pl != l:
                continue
            kl[c0:c1] = r["kld"]
            zeros[c0:c1] = r["zeros"]
            rng = r["range"]
            bad |= r["nonfinite"]
            if want_hist:
                hist[0] = r["hist"][0]
                hist[c0 + 1:c1 + 1] = r["hist"][1:]
        best = select(kl, w, f, eps)
        if _as_f32(t).size == 0 or rng[0] == rng[1]:
            best[3] |= 2
        results.append({"kld": kl, "zeros": zeros, "best": best, "hist": hist, "range": rng,
                        "nonfinite": bad})
    return results


def gradient_diversity(grads):
    """grads: sequence of equally long fp32 arrays (one layer's recent gradients).
    Returns float64[4] = {sum of norms, norm of the sum, delta_s, log form}."""
    arrs = [_as_f32(g) for g in grads]
    n = arrs[0].size if arrs else 0
    assert all(a.size == n for a in arrs)
    ptrs = (C.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    out = np.zeros(4, dtype=np.float64)
    lib().adapt_oracle_gradient_diversity(ptrs, len(arrs), n, out.ctypes.data)
    return out


STRATEGY_MIN, STRATEGY_MEAN, STRATEGY_MAX = 0, 1, 2


def pushup(log_diversity: float, wl_min: int, fl_min: int, strategy: int, buff: int):
    """PushUp's scalar step for one layer. Returns int32[5] = {WL, FL, s_1, s_2, s}."""
    out = np.zeros(5, dtype=np.int32)
    lib().adapt_oracle_pushup(C.c_double(log_diversity), int(wl_min), int(fl_min), int(strategy),
                              int(buff), out.ctypes.data)
    return out


def normalize_gradient(g):
    """g / ||g||_2 as fp32 (norm and quotients in double); an all-zero gradient comes back as is."""
    a = _as_f32(g)
    out = np.empty_like(a)
    lib().adapt_oracle_normalize_gradient(a.ctypes.data, a.size, out.ctypes.data)
    return out


def bfp_scale(lo: float, hi: float, wl: int) -> int:
    """Block scale s of a layer with extremes lo <= hi at word length wl."""
    return int(lib().adapt_oracle_bfp_scale(np.float32(lo), np.float32(hi), wl))


def format_value_one(x: float, kind: int, a: int, b: int, round_mode: int = ROUND_RNE,
                     k24: int = 0) -> float:
    return float(lib().adapt_oracle_format_value_one(np.float32(x), kind, a, b, round_mode, k24))


def format_quantize(x, kind: int, a: int, b: int, round_mode: int = ROUND_RNE, seed: int = 0,
                    layer: int = 0):
    """The tensor mapped to the representable values of one format; float32[n]."""
    arr = _as_f32(x)
    out = np.empty(arr.size, dtype=np.float32)
    lib().adapt_oracle_format_quantize(arr.ctypes.data, arr.size, kind, a, b, round_mode, seed,
                                       layer, out.ctypes.data)
    return out


def format_search_layer(x, kind, a, b, n_bins: int, round_mode: int = ROUND_RNE, seed: int = 0,
                        layer: int = 0, eps: float = 0.0, alpha: float = 0.0,
                        log_base: float = 2.0):
    """One layer, every format of the list in the caller's order. Returns a dict."""
    arr = _as_f32(x)
    kk = np.ascontiguousarray(kind, dtype=np.int32)
    aa = np.ascontiguousarray(a, dtype=np.int32)
    bb = np.ascontiguousarray(b, dtype=np.int32)
    nc = kk.size
    kl = np.zeros(nc, dtype=np.float64)
    zeros = np.zeros(nc, dtype=np.int64)
    b_used = np.zeros(nc, dtype=np.int32)
    best = np.zeros(4, dtype=np.int32)
    rng = np.zeros(2, dtype=np.float32)
    bad = lib().adapt_oracle_format_search(
        arr.ctypes.data, arr.size, layer, kk.ctypes.data, aa.ctypes.data, bb.ctypes.data, nc,
        n_bins, round_mode, seed, eps, alpha, log_base, kl.ctypes.data, zeros.ctypes.data,
        b_used.ctypes.data, best.ctypes.data, rng.ctypes.data)
    return {"kld": kl, "zeros": zeros, "b": b_used, "best": best, "range": rng,
            "nonfinite": int(bad)}
