"""ctypes binding of libadapt_b200.so: the same entry points as include/adapt.h,
argument marshalling only.  Tensors are torch CUDA tensors (device memory and
streams come from torch); every computation runs in the library's kernels.

The library must have been built (``python -m paper_2107_13490_b200.build``);
there is no fallback: a missing library raises at the first call.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# ADAPT_B200_LIBRARY names another build of the same library (the bounds-checking one)
LIB_PATH = os.environ.get("ADAPT_B200_LIBRARY") or os.path.join(_HERE, "libadapt_b200.so")

ROUND_RNE = 0
ROUND_STOCHASTIC = 1
FLAG_MET_EPS, FLAG_DEGENERATE, FLAG_NONFINITE, FLAG_RANGE = 1, 2, 4, 8
OK, ERR_INVALID_ARG, ERR_NONFINITE, ERR_RANGE, ERR_CUDA, ERR_WORKSPACE = range(6)

EXPORTS = (
    "adapt_version", "adapt_status_string", "adapt_last_error", "adapt_quantize",
    "adapt_quantize_ex", "adapt_quantize_selected", "adapt_quantize_selected_batch",
    "adapt_requantize_selected_batch", "adapt_quantize_selected_batch_packed",
    "adapt_search_workspace_bytes", "adapt_gradient_diversity", "adapt_normalize_gradients",
    "adapt_precision_search", "adapt_precision_search_ex", "adapt_precision_search_host",
    "adapt_precision_switch_host", "adapt_precision_switch_host_packed",
    "adapt_quantize_host", "adapt_kernel_launch_count", "adapt_kernel_timing",
    "adapt_kernel_times", "adapt_precision_search_static", "adapt_release",
    "adapt_format_search_workspace_bytes", "adapt_format_search", "adapt_format_quantize",
    "adapt_pushup", "adapt_bounds_check_status",
)
STRATEGY_MIN, STRATEGY_MEAN, STRATEGY_MAX = 0, 1, 2
FMT_FIXED, FMT_BFP, FMT_FLOAT = 0, 1, 2
MAX_FORMATS = 1024
STATIC_MAX_LAYERS, STATIC_MAX_BINS, STATIC_MAX_CAND = 8, 512, 1024
KERNEL_KINDS = ("range", "range_finalize", "search", "kld", "select", "quantize", "plan",
                "expand", "search_direct", "diversity", "format_resolve", "format_search",
                "format_kld", "format_quantize")
ALGO_AUTO, ALGO_KEYED, ALGO_DIRECT = 0, 1, 2


class AdaptGrid(C.Structure):
    _fields_ = [("n_cand", C.c_int32), ("wl", C.POINTER(C.c_int32)), ("fl", C.POINTER(C.c_int32))]


class AdaptSearchOpts(C.Structure):
    _fields_ = [("round_mode", C.c_int32), ("layer_base", C.c_int32), ("seed", C.c_uint64),
                ("eps", C.c_double), ("pseudo_count", C.c_double), ("log_base", C.c_double),
                ("stream", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("hist_out", C.c_void_p), ("range_out", C.c_void_p), ("algorithm", C.c_int32),
                ("n_bins_per_layer", C.c_void_p), ("start_wl_fl", C.c_void_p),
                ("status_out", C.c_void_p)]


class AdaptFormat(C.Structure):
    _fields_ = [("kind", C.c_int32), ("a", C.c_int32), ("b", C.c_int32)]


class AdaptError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        L = lib()
        msg = L.adapt_status_string(status).decode()
        detail = L.adapt_last_error().decode() if status == ERR_CUDA else ""
        super().__init__(f"{where}: {msg}" + (f" ({detail})" if detail else ""))


_lib = None


def lib():
    """Loads the shared library (once). Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2107_13490_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.adapt_version.restype = C.c_char_p
        L.adapt_status_string.restype = C.c_char_p
        L.adapt_status_string.argtypes = [C.c_int]
        L.adapt_last_error.restype = C.c_char_p
        L.adapt_quantize.restype = C.c_int
        L.adapt_quantize.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_uint64,
                                     C.c_void_p]
        L.adapt_quantize_ex.restype = C.c_int
        L.adapt_quantize_ex.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_uint64,
                                        C.c_int32, C.c_int, C.c_void_p, C.c_void_p]
        L.adapt_quantize_selected.restype = C.c_int
        L.adapt_quantize_selected.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int, C.c_uint64,
                                              C.c_int32, C.c_void_p, C.c_void_p]
        L.adapt_quantize_selected_batch.restype = C.c_int
        L.adapt_quantize_selected_batch.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                                    C.c_int, C.c_uint64, C.c_int32, C.c_void_p,
                                                    C.c_void_p]
        L.adapt_quantize_selected_batch_packed.restype = C.c_int
        L.adapt_quantize_selected_batch_packed.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                                           C.c_int, C.c_uint64, C.c_int32, C.c_int,
                                                           C.c_void_p, C.c_void_p, C.c_void_p]
        L.adapt_normalize_gradients.restype = C.c_int
        L.adapt_normalize_gradients.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p,
                                                C.c_void_p]
        L.adapt_requantize_selected_batch.restype = C.c_int
        L.adapt_requantize_selected_batch.argtypes = L.adapt_quantize_selected_batch.argtypes
        L.adapt_gradient_diversity.restype = C.c_int
        L.adapt_gradient_diversity.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p,
                                               C.c_void_p]
        L.adapt_bounds_check_status.restype = C.c_int
        L.adapt_bounds_check_status.argtypes = [C.c_void_p, C.c_int]
        L.adapt_pushup.restype = C.c_int
        L.adapt_pushup.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                   C.c_void_p]
        L.adapt_search_workspace_bytes.restype = C.c_size_t
        L.adapt_search_workspace_bytes.argtypes = [C.c_void_p, C.c_int, C.POINTER(AdaptGrid), C.c_int]
        search_args = [C.c_void_p, C.c_void_p, C.c_int, C.POINTER(AdaptGrid), C.c_int, C.c_void_p,
                       C.c_void_p, C.c_void_p]
        L.adapt_precision_search.restype = C.c_int
        L.adapt_precision_search.argtypes = search_args
        L.adapt_precision_search_ex.restype = C.c_int
        L.adapt_precision_search_ex.argtypes = search_args + [C.POINTER(AdaptSearchOpts)]
        L.adapt_precision_search_host.restype = C.c_int
        L.adapt_precision_search_host.argtypes = search_args + [C.POINTER(AdaptSearchOpts)]
        L.adapt_precision_switch_host.restype = C.c_int
        L.adapt_precision_switch_host.argtypes = search_args + [C.c_void_p, C.POINTER(AdaptSearchOpts)]
        L.adapt_precision_switch_host_packed.restype = C.c_int
        L.adapt_precision_switch_host_packed.argtypes = search_args + [C.c_int, C.c_void_p, C.c_void_p,
                                                                       C.POINTER(AdaptSearchOpts)]
        L.adapt_precision_search_static.restype = C.c_int
        L.adapt_precision_search_static.argtypes = search_args + [C.c_void_p]
        L.adapt_quantize_host.restype = C.c_int
        L.adapt_quantize_host.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_int,
                                          C.c_uint64, C.c_int32, C.c_int, C.c_void_p]
        L.adapt_kernel_launch_count.restype = C.c_uint64
        L.adapt_release.restype = C.c_int
        L.adapt_kernel_timing.restype = C.c_int
        L.adapt_kernel_timing.argtypes = [C.c_int]
        L.adapt_kernel_times.restype = C.c_int
        L.adapt_kernel_times.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.adapt_format_search_workspace_bytes.restype = C.c_size_t
        L.adapt_format_search_workspace_bytes.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int,
                                                          C.c_int]
        L.adapt_format_search.restype = C.c_int
        L.adapt_format_search.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int,
                                          C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.POINTER(AdaptSearchOpts)]
        L.adapt_format_quantize.restype = C.c_int
        L.adapt_format_quantize.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_int,
                                            C.c_int, C.c_uint64, C.c_int, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != OK:
        raise AdaptError(status, where)


class Grid:
    """Host-side candidate grid: keeps the numpy arrays alive for the C struct."""

    def __init__(self, wl: Sequence[int], fl: Sequence[int]):
        self.wl = np.ascontiguousarray(wl, dtype=np.int32)
        self.fl = np.ascontiguousarray(fl, dtype=np.int32)
        assert self.wl.shape == self.fl.shape and self.wl.ndim == 1
        self.c = AdaptGrid(int(self.wl.size), self.wl.ctypes.data_as(C.POINTER(C.c_int32)),
                           self.fl.ctypes.data_as(C.POINTER(C.c_int32)))

    def __len__(self):
        return int(self.wl.size)


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        return int(torch.cuda.current_stream().cuda_stream) or None
    return int(stream.cuda_stream) or None


_CODE_DTYPES = {8: torch.int8, 16: torch.int16, 32: torch.int32}


def adapt_version() -> str:
    return lib().adapt_version().decode()


def adapt_kernel_launch_count() -> int:
    return int(lib().adapt_kernel_launch_count())


def adapt_kernel_timing(enable: bool) -> None:
    _check(lib().adapt_kernel_timing(1 if enable else 0), "adapt_kernel_timing")


def adapt_kernel_times(reset: bool = False):
    """Returns {kind: (milliseconds, launches)} accumulated while timing was on."""
    ms = np.zeros(len(KERNEL_KINDS), dtype=np.float64)
    cnt = np.zeros(len(KERNEL_KINDS), dtype=np.uint64)
    _check(lib().adapt_kernel_times(ms.ctypes.data, cnt.ctypes.data, 1 if reset else 0),
           "adapt_kernel_times")
    return {k: (float(ms[i]), int(cnt[i])) for i, k in enumerate(KERNEL_KINDS)}


def adapt_bounds_check_status(clear: bool = False):
    """adapt_bounds_check_status of adapt.h: (checking build?, uint32[4] = {events, site, index, limit})."""
    word = np.zeros(4, dtype=np.uint32)
    rc = lib().adapt_bounds_check_status(word.ctypes.data, 1 if clear else 0)
    if rc < 0:
        raise AdaptError(-rc, "adapt_bounds_check_status")
    return bool(rc), word


def adapt_release() -> None:
    _check(lib().adapt_release(), "adapt_release")


def adapt_quantize(x: torch.Tensor, wl: int, fl: int, round_mode: int = ROUND_RNE, seed: int = 0,
                   codes_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """adapt_quantize of adapt.h (int32 codes, hash layer 0, legacy default stream)."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    if codes_out is None:
        codes_out = torch.empty(x.numel(), dtype=torch.int32, device=x.device)
    assert codes_out.dtype == torch.int32 and codes_out.numel() == x.numel()
    torch.cuda.current_stream().synchronize()  # the named call runs on the legacy default stream
    _check(lib().adapt_quantize(x.data_ptr(), x.numel(), wl, fl, round_mode, seed,
                                codes_out.data_ptr()), "adapt_quantize")
    return codes_out


def adapt_quantize_ex(x: torch.Tensor, wl: int, fl: int, round_mode: int = ROUND_RNE, seed: int = 0,
                      layer: int = 0, code_bits: int = 32, codes_out: Optional[torch.Tensor] = None,
                      stream=None) -> torch.Tensor:
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    if codes_out is None:
        codes_out = torch.empty(x.numel(), dtype=_CODE_DTYPES.get(code_bits, torch.int32),
                                device=x.device)
    _check(lib().adapt_quantize_ex(x.data_ptr(), x.numel(), wl, fl, round_mode, seed, layer,
                                   code_bits, codes_out.data_ptr(), _stream_handle(stream)),
           "adapt_quantize_ex")
    return codes_out


def adapt_quantize_selected(x: torch.Tensor, selected: torch.Tensor, round_mode: int = ROUND_RNE,
                            seed: int = 0, layer: int = 0,
                            codes_out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    assert selected.is_cuda and selected.dtype == torch.int32 and selected.numel() >= 2
    if codes_out is None:
        codes_out = torch.empty(x.numel(), dtype=torch.int32, device=x.device)
    _check(lib().adapt_quantize_selected(x.data_ptr(), x.numel(), selected.data_ptr(), round_mode,
                                         seed, layer, codes_out.data_ptr(), _stream_handle(stream)),
           "adapt_quantize_selected")
    return codes_out


def adapt_quantize_selected_batch(tensors: Sequence[torch.Tensor], best: torch.Tensor,
                                  round_mode: int = ROUND_RNE, seed: int = 0, layer_base: int = 0,
                                  codes_out: Optional[Sequence[torch.Tensor]] = None, stream=None):
    """All layers at the <WL,FL> a search left in ``best`` (device int32[L][4]), one launch."""
    assert best.is_cuda and best.dtype == torch.int32 and best.numel() >= 4 * len(tensors)
    if codes_out is None:
        codes_out = [torch.empty(t.numel(), dtype=torch.int32, device=t.device) for t in tensors]
    ptrs, lens = _marshal_tensors(tensors)
    outs = np.array([c.data_ptr() for c in codes_out], dtype=np.uint64)
    assert all(c.dtype == torch.int32 and c.numel() == t.numel() for c, t in zip(codes_out, tensors))
    _check(lib().adapt_quantize_selected_batch(ptrs.ctypes.data, lens.ctypes.data, len(tensors),
                                               best.data_ptr(), round_mode, seed, layer_base,
                                               outs.ctypes.data, _stream_handle(stream)),
           "adapt_quantize_selected_batch")
    return codes_out


def adapt_quantize_selected_batch_packed(tensors: Sequence[torch.Tensor], best: torch.Tensor,
                                         code_bits: int, round_mode: int = ROUND_RNE, seed: int = 0,
                                         layer_base: int = 0,
                                         codes_out: Optional[Sequence[torch.Tensor]] = None,
                                         unfit_out: Optional[torch.Tensor] = None, stream=None):
    """adapt_quantize_selected_batch with int8 / int16 / int32 codes.  Returns (codes, unfit):
    unfit is device int32[L], the word length of every layer that did not fit ``code_bits``
    (such a layer's codes are left untouched), 0 elsewhere."""
    dt = {8: torch.int8, 16: torch.int16, 32: torch.int32}[code_bits]
    assert best.is_cuda and best.dtype == torch.int32 and best.numel() >= 4 * len(tensors)
    if codes_out is None:
        codes_out = [torch.empty(t.numel(), dtype=dt, device=t.device) for t in tensors]
    if unfit_out is None:
        unfit_out = torch.empty(len(tensors), dtype=torch.int32, device=best.device)
    assert unfit_out.is_cuda and unfit_out.dtype == torch.int32 and unfit_out.numel() >= len(tensors)
    ptrs, lens = _marshal_tensors(tensors)
    outs = np.array([c.data_ptr() for c in codes_out], dtype=np.uint64)
    assert all(c.dtype == dt and c.is_cuda and c.is_contiguous() and c.numel() == t.numel()
               for c, t in zip(codes_out, tensors))
    _check(lib().adapt_quantize_selected_batch_packed(ptrs.ctypes.data, lens.ctypes.data, len(tensors),
                                                      best.data_ptr(), round_mode, seed, layer_base,
                                                      code_bits, outs.ctypes.data, unfit_out.data_ptr(),
                                                      _stream_handle(stream)),
           "adapt_quantize_selected_batch_packed")
    return codes_out, unfit_out


def adapt_requantize_selected_batch(tensors: Sequence[torch.Tensor], best: torch.Tensor,
                                    round_mode: int = ROUND_RNE, seed: int = 0, layer_base: int = 0,
                                    values_out: Optional[Sequence[torch.Tensor]] = None, stream=None):
    """All layers replaced by their dequantized values code * 2^-FL (fp32) at the <WL,FL> a search
    left in ``best``; ``values_out`` defaults to new tensors and may be ``tensors`` (in place)."""
    assert best.is_cuda and best.dtype == torch.int32 and best.numel() >= 4 * len(tensors)
    if values_out is None:
        values_out = [torch.empty(t.numel(), dtype=torch.float32, device=t.device) for t in tensors]
    ptrs, lens = _marshal_tensors(tensors)
    outs = np.array([c.data_ptr() for c in values_out], dtype=np.uint64)
    assert all(c.dtype == torch.float32 and c.is_cuda and c.is_contiguous() and c.numel() == t.numel()
               for c, t in zip(values_out, tensors))
    _check(lib().adapt_requantize_selected_batch(ptrs.ctypes.data, lens.ctypes.data, len(tensors),
                                                 best.data_ptr(), round_mode, seed, layer_base,
                                                 outs.ctypes.data, _stream_handle(stream)),
           "adapt_requantize_selected_batch")
    return values_out


def adapt_gradient_diversity(grads: Sequence[Sequence[torch.Tensor]],
                             out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """grads[l][k] = gradient k of layer l (CUDA fp32, equal lengths within a layer).
    Returns device float64[n_layers][4] = {sum of norms, norm of the sum, delta_s, log form}."""
    n_layers, n_grads = len(grads), len(grads[0])
    ptrs = np.zeros(n_layers * n_grads, dtype=np.uint64)
    lens = np.zeros(n_layers, dtype=np.int64)
    for l, gl in enumerate(grads):
        assert len(gl) == n_grads
        lens[l] = gl[0].numel()
        for k, g in enumerate(gl):
            assert g.is_cuda and g.dtype == torch.float32 and g.is_contiguous() and g.numel() == lens[l]
            ptrs[l * n_grads + k] = g.data_ptr()
    if out is None:
        out = torch.empty((n_layers, 4), dtype=torch.float64, device=grads[0][0].device)
    _check(lib().adapt_gradient_diversity(ptrs.ctypes.data, lens.ctypes.data, n_layers, n_grads,
                                          out.data_ptr(), _stream_handle(stream)),
           "adapt_gradient_diversity")
    return out


def adapt_pushup(diversity, best, strategy: int, buff: int, want_suggestions: bool = False):
    """adapt_pushup of adapt.h.  diversity: [L][4] doubles and best: [L][4] int32, host arrays or
    tensors (device tensors are copied to the host first: the call is host arithmetic).
    Returns int32[L][2] = {WL, FL} (and int32[L][3] = {s1, s2, s} when asked for)."""
    if isinstance(diversity, torch.Tensor):
        diversity = diversity.detach().cpu().numpy()
    if isinstance(best, torch.Tensor):
        best = best.detach().cpu().numpy()
    div = np.ascontiguousarray(diversity, dtype=np.float64).reshape(-1, 4)
    bst = np.ascontiguousarray(best, dtype=np.int32).reshape(-1, 4)
    assert div.shape[0] == bst.shape[0]
    out = np.zeros((div.shape[0], 2), dtype=np.int32)
    sug = np.zeros((div.shape[0], 3), dtype=np.int32) if want_suggestions else None
    _check(lib().adapt_pushup(div.ctypes.data, bst.ctypes.data, div.shape[0], strategy, buff,
                              out.ctypes.data, sug.ctypes.data if want_suggestions else None),
           "adapt_pushup")
    return (out, sug) if want_suggestions else out


def adapt_normalize_gradients(grads: Sequence[torch.Tensor],
                              out: Optional[Sequence[torch.Tensor]] = None,
                              want_sumsq: bool = False, stream=None):
    """Every layer's gradient divided by its L2 norm (``out`` defaults to new tensors and may be
    ``grads``: in place).  Returns out, or (out, device float64[L] sums of squares)."""
    if out is None:
        out = [torch.empty_like(g) for g in grads]
    ptrs, lens = _marshal_tensors(grads)
    assert all(o.is_cuda and o.dtype == torch.float32 and o.is_contiguous() and o.numel() == g.numel()
               for o, g in zip(out, grads))
    outs = np.array([o.data_ptr() for o in out], dtype=np.uint64)
    sumsq = torch.empty(len(grads), dtype=torch.float64, device=grads[0].device) if want_sumsq else None
    _check(lib().adapt_normalize_gradients(ptrs.ctypes.data, lens.ctypes.data, len(grads),
                                           outs.ctypes.data, sumsq.data_ptr() if want_sumsq else None,
                                           _stream_handle(stream)),
           "adapt_normalize_gradients")
    return (out, sumsq) if want_sumsq else out


def adapt_search_workspace_bytes(lens: Sequence[int], grid: Grid, n_bins: int) -> int:
    ln = np.ascontiguousarray(lens, dtype=np.int64)
    return int(lib().adapt_search_workspace_bytes(ln.ctypes.data, int(ln.size), C.byref(grid.c),
                                                  n_bins))


class SearchResult:
    """Device outputs of one search call (torch tensors on the input device)."""

    def __init__(self, kld, zeros, best, hist=None, value_range=None, status=None):
        self.kld, self.zeros, self.best, self.hist, self.range = kld, zeros, best, hist, value_range
        self.status = status


def _marshal_tensors(tensors):
    ptrs = np.zeros(len(tensors), dtype=np.uint64)
    lens = np.zeros(len(tensors), dtype=np.int64)
    for i, t in enumerate(tensors):
        assert t.dtype == torch.float32 and t.is_contiguous()
        ptrs[i] = t.data_ptr()
        lens[i] = t.numel()
    return ptrs, lens


def adapt_precision_search(tensors: Sequence[torch.Tensor], grid: Grid, n_bins: int,
                           out: Optional[SearchResult] = None) -> SearchResult:
    """adapt_precision_search of adapt.h (RNE, eps 0, bits, legacy default stream)."""
    dev = tensors[0].device
    assert all(t.is_cuda for t in tensors)
    ptrs, lens = _marshal_tensors(tensors)
    L, Cn = len(tensors), len(grid)
    if out is None:
        out = SearchResult(torch.empty((L, Cn), dtype=torch.float64, device=dev),
                           torch.empty((L, Cn), dtype=torch.int64, device=dev),
                           torch.empty((L, 4), dtype=torch.int32, device=dev))
    torch.cuda.current_stream().synchronize()
    _check(lib().adapt_precision_search(ptrs.ctypes.data, lens.ctypes.data, L, C.byref(grid.c),
                                        n_bins, out.kld.data_ptr(), out.zeros.data_ptr(),
                                        out.best.data_ptr()), "adapt_precision_search")
    return out


def adapt_precision_search_static(tensors: Sequence[torch.Tensor], grid: Grid, n_bins: int,
                                  out: SearchResult, stream=None) -> SearchResult:
    """adapt_precision_search_static of adapt.h: the search with all scratch in a fixed
    array inside the library.  ``out`` must be passed in (this wrapper allocates nothing
    on the device either); sizes beyond the STATIC_MAX_* limits raise ERR_WORKSPACE."""
    assert all(t.is_cuda for t in tensors)
    ptrs, lens = _marshal_tensors(tensors)
    st = lib().adapt_precision_search_static(ptrs.ctypes.data, lens.ctypes.data, len(tensors),
                                             C.byref(grid.c), n_bins, out.kld.data_ptr(),
                                             out.zeros.data_ptr(), out.best.data_ptr(),
                                             _stream_handle(stream))
    if st == ERR_WORKSPACE:
        err = AdaptError(st, "adapt_precision_search_static")
        err.args = (err.args[0] + " (" + lib().adapt_last_error().decode() + ")",)
        raise err
    _check(st, "adapt_precision_search_static")
    return out


def adapt_precision_search_ex(tensors: Sequence[torch.Tensor], grid: Grid, n_bins: int,
                              round_mode: int = ROUND_RNE, seed: int = 0, layer_base: int = 0,
                              eps: float = 0.0, pseudo_count: float = 0.0, log_base: float = 0.0,
                              stream=None, workspace: Optional[torch.Tensor] = None,
                              want_hist: bool = False, want_range: bool = False,
                              out: Optional[SearchResult] = None,
                              algorithm: int = ALGO_AUTO,
                              n_bins_per_layer: Optional[Sequence[int]] = None,
                              start_wl_fl: Optional[Sequence[Sequence[int]]] = None,
                              want_status: bool = False) -> SearchResult:
    dev = tensors[0].device
    assert all(t.is_cuda for t in tensors)
    ptrs, lens = _marshal_tensors(tensors)
    L, Cn = len(tensors), len(grid)
    per_layer = start = None
    if n_bins_per_layer is not None:
        per_layer = np.ascontiguousarray(n_bins_per_layer, dtype=np.int32)
        assert per_layer.size == L
        n_bins = int(per_layer.max())          # stride of hist_out and of the workspace
    if start_wl_fl is not None:
        start = np.ascontiguousarray(start_wl_fl, dtype=np.int32).reshape(L, 2)
    if out is None:
        out = SearchResult(
            torch.empty((L, Cn), dtype=torch.float64, device=dev),
            torch.empty((L, Cn), dtype=torch.int64, device=dev),
            torch.empty((L, 4), dtype=torch.int32, device=dev),
            torch.zeros((L, Cn + 1, n_bins), dtype=torch.int32, device=dev) if want_hist else None,
            torch.empty((L, 2), dtype=torch.float32, device=dev) if want_range else None)
    o = AdaptSearchOpts()
    o.round_mode, o.layer_base, o.seed = round_mode, layer_base, seed
    o.eps, o.pseudo_count, o.log_base = eps, pseudo_count, log_base
    o.stream = _stream_handle(stream)
    if workspace is not None:
        o.workspace, o.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    o.hist_out = out.hist.data_ptr() if out.hist is not None else None
    o.range_out = out.range.data_ptr() if out.range is not None else None
    o.algorithm = algorithm
    o.n_bins_per_layer = per_layer.ctypes.data if per_layer is not None else None
    o.start_wl_fl = start.ctypes.data if start is not None else None
    if want_status and out.status is None:
        out.status = torch.full((L,), -1, dtype=torch.int32, device=dev)
    o.status_out = out.status.data_ptr() if want_status else None
    _check(lib().adapt_precision_search_ex(ptrs.ctypes.data, lens.ctypes.data, L, C.byref(grid.c),
                                           n_bins, out.kld.data_ptr(), out.zeros.data_ptr(),
                                           out.best.data_ptr(), C.byref(o)),
           "adapt_precision_search_ex")
    return out


def adapt_precision_search_host(tensors: Sequence[torch.Tensor], grid: Grid, n_bins: int,
                                round_mode: int = ROUND_RNE, seed: int = 0, layer_base: int = 0,
                                eps: float = 0.0, pseudo_count: float = 0.0, log_base: float = 0.0,
                                out: Optional[SearchResult] = None) -> SearchResult:
    """Host-buffer form: ``tensors`` and the outputs are CPU tensors (pinned for speed)."""
    assert all(not t.is_cuda for t in tensors)
    ptrs, lens = _marshal_tensors(tensors)
    L, Cn = len(tensors), len(grid)
    if out is None:
        out = SearchResult(torch.empty((L, Cn), dtype=torch.float64),
                           torch.empty((L, Cn), dtype=torch.int64),
                           torch.empty((L, 4), dtype=torch.int32))
    o = AdaptSearchOpts()
    o.round_mode, o.layer_base, o.seed = round_mode, layer_base, seed
    o.eps, o.pseudo_count, o.log_base = eps, pseudo_count, log_base
    o.stream = _stream_handle(None)
    _check(lib().adapt_precision_search_host(ptrs.ctypes.data, lens.ctypes.data, L,
                                             C.byref(grid.c), n_bins, out.kld.data_ptr(),
                                             out.zeros.data_ptr(), out.best.data_ptr(),
                                             C.byref(o)), "adapt_precision_search_host")
    return out


def adapt_precision_switch_host(tensors: Sequence[torch.Tensor], grid: Grid, n_bins: int,
                                round_mode: int = ROUND_RNE, seed: int = 0, layer_base: int = 0,
                                eps: float = 0.0, pseudo_count: float = 0.0, log_base: float = 0.0,
                                out: Optional[SearchResult] = None,
                                codes_out: Optional[Sequence[torch.Tensor]] = None):
    """Host-buffer search + quantization of every layer at its selected format.
    Returns (SearchResult, list of CPU int32 code tensors)."""
    assert all(not t.is_cuda for t in tensors)
    ptrs, lens = _marshal_tensors(tensors)
    L, Cn = len(tensors), len(grid)
    if out is None:
        out = SearchResult(torch.empty((L, Cn), dtype=torch.float64),
                           torch.empty((L, Cn), dtype=torch.int64),
                           torch.empty((L, 4), dtype=torch.int32))
    if codes_out is None:
        codes_out = [torch.empty(t.numel(), dtype=torch.int32) for t in tensors]
    cptr = np.array([c.data_ptr() for c in codes_out], dtype=np.uint64)
    o = AdaptSearchOpts()
    o.round_mode, o.layer_base, o.seed = round_mode, layer_base, seed
    o.eps, o.pseudo_count, o.log_base = eps, pseudo_count, log_base
    o.stream = _stream_handle(None)
    _check(lib().adapt_precision_switch_host(ptrs.ctypes.data, lens.ctypes.data, L,
                                             C.byref(grid.c), n_bins, out.kld.data_ptr(),
                                             out.zeros.data_ptr(), out.best.data_ptr(),
                                             cptr.ctypes.data, C.byref(o)),
           "adapt_precision_switch_host")
    return out, codes_out


def adapt_precision_switch_host_packed(tensors: Sequence[torch.Tensor], grid: Grid, n_bins: int,
                                       code_bits: int, round_mode: int = ROUND_RNE, seed: int = 0,
                                       layer_base: int = 0, eps: float = 0.0,
                                       out: Optional[SearchResult] = None,
                                       codes_out: Optional[Sequence[torch.Tensor]] = None):
    """adapt_precision_switch_host_packed of adapt.h.  Returns (SearchResult, list of CPU code
    tensors of code_bits width, int32[L] numpy array of the word lengths that did not fit)."""
    assert all(not t.is_cuda for t in tensors)
    ptrs, lens = _marshal_tensors(tensors)
    L, Cn = len(tensors), len(grid)
    dt = {8: torch.int8, 16: torch.int16, 32: torch.int32}[code_bits]
    if out is None:
        out = SearchResult(torch.empty((L, Cn), dtype=torch.float64),
                           torch.empty((L, Cn), dtype=torch.int64),
                           torch.empty((L, 4), dtype=torch.int32))
    if codes_out is None:
        codes_out = [torch.empty(t.numel(), dtype=dt) for t in tensors]
    assert all(c.dtype == dt for c in codes_out)
    cptr = np.array([c.data_ptr() for c in codes_out], dtype=np.uint64)
    unfit = np.zeros(L, dtype=np.int32)
    o = AdaptSearchOpts()
    o.round_mode, o.layer_base, o.seed, o.eps = round_mode, layer_base, seed, eps
    o.stream = _stream_handle(None)
    _check(lib().adapt_precision_switch_host_packed(ptrs.ctypes.data, lens.ctypes.data, L,
                                                    C.byref(grid.c), n_bins, out.kld.data_ptr(),
                                                    out.zeros.data_ptr(), out.best.data_ptr(),
                                                    code_bits, cptr.ctypes.data, unfit.ctypes.data,
                                                    C.byref(o)),
           "adapt_precision_switch_host_packed")
    return out, codes_out, unfit


def adapt_quantize_host(x: torch.Tensor, wl: int, fl: int, round_mode: int = ROUND_RNE,
                        seed: int = 0, layer: int = 0, code_bits: int = 32,
                        codes_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    assert (not x.is_cuda) and x.dtype == torch.float32 and x.is_contiguous()
    if codes_out is None:
        codes_out = torch.empty(x.numel(), dtype=_CODE_DTYPES.get(code_bits, torch.int32))
    _check(lib().adapt_quantize_host(x.data_ptr(), x.numel(), wl, fl, round_mode, seed, layer,
                                     code_bits, codes_out.data_ptr()), "adapt_quantize_host")
    return codes_out


def _marshal_formats(formats):
    """formats: sequence of (kind, a, b) triples -> ctypes array of adapt_format."""
    arr = (AdaptFormat * len(formats))()
    for i, (k, a, b) in enumerate(formats):
        arr[i].kind, arr[i].a, arr[i].b = int(k), int(a), int(b)
    return arr


def adapt_format_search_workspace_bytes(lens: Sequence[int], formats, n_bins: int) -> int:
    ln = np.ascontiguousarray(lens, dtype=np.int64)
    arr = _marshal_formats(formats)
    return int(lib().adapt_format_search_workspace_bytes(
        ln.ctypes.data, int(ln.size), C.cast(arr, C.c_void_p), len(formats), n_bins))


class FormatResult:
    """Device outputs of adapt_format_search."""

    def __init__(self, kld, zeros, b, best, value_range=None, hist=None):
        self.kld, self.zeros, self.b, self.best, self.range = kld, zeros, b, best, value_range
        self.hist = hist


def adapt_format_search(tensors: Sequence[torch.Tensor], formats, n_bins: int,
                        round_mode: int = ROUND_RNE, seed: int = 0, layer_base: int = 0,
                        eps: float = 0.0, pseudo_count: float = 0.0, log_base: float = 0.0,
                        stream=None, workspace: Optional[torch.Tensor] = None,
                        want_range: bool = False, want_hist: bool = False,
                        out: Optional[FormatResult] = None) -> FormatResult:
    """adapt_format_search of adapt.h; formats = sequence of (kind, a, b)."""
    dev = tensors[0].device
    assert all(t.is_cuda for t in tensors)
    ptrs, lens = _marshal_tensors(tensors)
    L, Cn = len(tensors), len(formats)
    arr = _marshal_formats(formats)
    if out is None:
        out = FormatResult(torch.empty((L, Cn), dtype=torch.float64, device=dev),
                           torch.empty((L, Cn), dtype=torch.int64, device=dev),
                           torch.empty((L, Cn), dtype=torch.int32, device=dev),
                           torch.empty((L, 4), dtype=torch.int32, device=dev))
    if want_range and out.range is None:
        out.range = torch.empty((L, 2), dtype=torch.float32, device=dev)
    opts = AdaptSearchOpts()
    opts.round_mode, opts.layer_base, opts.seed = round_mode, layer_base, seed
    opts.eps, opts.pseudo_count, opts.log_base = eps, pseudo_count, log_base
    opts.stream = _stream_handle(stream)
    if workspace is not None:
        opts.workspace, opts.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    opts.range_out = out.range.data_ptr() if want_range else None
    if want_hist and out.hist is None:
        out.hist = torch.zeros((L, Cn + 1, n_bins), dtype=torch.int32, device=dev)
    opts.hist_out = out.hist.data_ptr() if want_hist else None
    _check(lib().adapt_format_search(ptrs.ctypes.data, lens.ctypes.data, L, C.cast(arr, C.c_void_p),
                                     Cn, n_bins, out.kld.data_ptr(), out.zeros.data_ptr(),
                                     out.b.data_ptr(), out.best.data_ptr(), C.byref(opts)),
           "adapt_format_search")
    return out


def adapt_format_quantize(x: torch.Tensor, kind: int, a: int, b: int, round_mode: int = ROUND_RNE,
                          seed: int = 0, layer: int = 0, out: Optional[torch.Tensor] = None,
                          stream=None) -> torch.Tensor:
    """adapt_format_quantize of adapt.h: x mapped to the format's values (float32)."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    if out is None:
        out = torch.empty_like(x)
    _check(lib().adapt_format_quantize(x.data_ptr(), x.numel(), kind, a, b, round_mode, seed, layer,
                                       out.data_ptr(), _stream_handle(stream)),
           "adapt_format_quantize")
    return out
