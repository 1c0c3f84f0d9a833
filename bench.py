#!/usr/bin/env python
"""Benchmark of the precision-switch search on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole path over the workload: the batched search
(range scan, fused multi-candidate quantize / zero count / histograms,
divergence, selection) followed by the re-quantisation of every layer at its
selected <WL,FL>.  Prints one JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "precision-search element-candidates/s"
UNIT = "element-candidates/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of the search kernel from an ncu capture (bytes per element per launch),
# valid only for the library version it was taken on; see profiles/.
TRAFFIC_CAPTURE = {"version": "adapt-b200 0.9", "bytes_per_element": 4.074}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="stress_1g")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-sample", type=int, default=1 << 21,
                    help="elements of the workload the CPU baseline is timed on")
    ap.add_argument("--elements", type=int, default=0,
                    help="profiling aid: shrink a single-layer workload to this many elements")
    ap.add_argument("--path", default="search", choices=["search", "diversity", "normalize", "formats"],
                    help="search: the precision-switch search step (default); diversity: the "
                         "gradient-diversity reduction that feeds PushUp; normalize: g / ||g||_2 per "
                         "layer; formats: the search over block-floating-point and floating-point "
                         "candidates")
    ap.add_argument("--algorithm", default="auto", choices=["auto", "keyed", "direct"],
                    help="profiling aid: which form of the fused search kernel runs (auto: the "
                         "library's own choice; keyed serves round-to-nearest-even only)")
    ap.add_argument("--round-mode", default="workload", choices=["workload", "rne", "stochastic"],
                    help="profiling aid: override the workload's rounding mode")
    ap.add_argument("--dist", default="",
                    help="profiling aid: replace the (single-layer) workload's tensor by one of the "
                         "value classes of the sweep (normal, uniform, half_zero_relu, zeros_90pct, "
                         "on_grid_8_4, on_grid_16_12); use with --elements")
    ap.add_argument("--bins", type=int, default=0, help="profiling aid: override the number of bins")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the blocks on the other configs and the other value classes")
    return ap.parse_args()


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi.  It is started before the
    warm-up (nvidia-smi takes a moment to come up) and keeps only the samples whose
    timestamps fall inside the timed region."""
    Q = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        out = self.window(t0, t1)
        self.close()
        return out

    def close(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self.proc = None

    def window(self, t0: float, t1: float):
        """Summary of the samples that fall inside [t0, t1] (the sampler keeps running)."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for stamp, ln in list(self.lines):
            if not (t0 <= stamp <= t1 + 0.06):     # a sample is read up to one period late
                continue
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 10:
                continue
            try:
                sm.append(float(f[2])); mx.append(float(f[3])); power.append(float(f[4]))
            except ValueError:
                continue
            for name, val in zip(names, f[6:10]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def oracle_step(O, xs, wl, fl, w, eps=0.0):
    """One pass of the path on the CPU oracle: search, then quantize at the selection."""
    res = O.precision_search(xs, wl, fl, w.n_bins, w.round_mode, w.seed, 0, eps, threads=1)
    for l, x in enumerate(xs):
        if x.size:
            O.quantize(x, int(res[l]["best"][0]), int(res[l]["best"][1]), w.round_mode, w.seed, l)
    return res


def cpu_sample(xs, n_sample):
    """A bounded prefix sample of the workload: whole layers until the budget is used."""
    out, left = [], n_sample
    for x in xs:
        if left <= 0:
            break
        out.append(x[:left])
        left -= out[-1].size
    return out


def time_oracle(xs, wl, fl, w, n_sample):
    from oracle import oracle as O
    sample = cpu_sample(xs, n_sample)
    units = sum(s.size for s in sample) * len(wl)
    t0 = time.perf_counter()
    oracle_step(O, sample, wl, fl, w)
    dt = time.perf_counter() - t0
    return {"value": units / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"first {sum(s.size for s in sample)} elements ({len(sample)} layer(s)) of "
                      f"{w.name}, all {len(wl)} candidates, {w.n_bins} bins, one pass in {dt:.1f} s"}


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on the machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import oracle as O
    from paper_2107_13490_b200 import workloads as W
    w = W.WORKLOADS[args.workload]
    wl, fl = w.grid()
    # size each step's sample so that the whole run (warm-up + steps) stays near two minutes:
    # a short calibration pass gives the oracle's rate on this host
    first = w.layers[0]
    probe_n = min(first.numel, 1 << 14)
    probe = [W.generate_layer(W.LayerSpec(first.name, (probe_n,), first.dist, first.scale,
                                          first.zero_frac, first.outlier_frac, first.outlier_gain),
                              w.seed, 0)]
    t0 = time.perf_counter()
    oracle_step(O, probe, wl, fl, w)
    rate = probe_n / max(time.perf_counter() - t0, 1e-6)          # elements per second, all candidates
    budget_s = 120.0
    n_sample = int(rate * budget_s / max(1, args.steps + args.warmup))
    n_sample = max(1 << 12, min(n_sample, 1 << 18, w.numel))
    if first.numel > n_sample:   # generate only what the sample needs
        xs = [W.generate_layer(W.LayerSpec(first.name, (n_sample,), first.dist, first.scale,
                                           first.zero_frac, first.outlier_frac, first.outlier_gain),
                               w.seed, 0)]
    else:
        xs = cpu_sample(W.generate(w), n_sample)
    units = sum(x.size for x in xs) * len(wl)
    for _ in range(args.warmup):
        oracle_step(O, xs, wl, fl, w)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(O, xs, wl, fl, w)
    dt = time.perf_counter() - t0
    value = units * args.steps / dt
    sample = f"first {sum(x.size for x in xs)} elements of {w.name} per step, all {len(wl)} candidates"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "elements": w.numel, "candidates": len(wl),
                       "n_bins": w.n_bins, "round_mode": "rne" if w.round_mode == 0 else "stochastic",
                       "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)
    return 0


def run_normalize(args):
    """Gradient normalisation g / ||g||_2: one layer of 2^28 elements (or --elements N); one
    read for the norm, one read and one write for the scaling = 12 B per element."""
    import torch
    from paper_2107_13490_b200 import binding as B
    from paper_2107_13490_b200 import workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    B.lib()
    n = args.elements or (1 << 28)
    host = W.generate_layer(W.LayerSpec("g", (n,), "laplace", 1e-4, zero_frac=0.05), 7, 0)
    g = [torch.from_numpy(host).cuda()]
    out = [torch.empty_like(g[0])]
    for _ in range(max(args.warmup, 3)):
        B.adapt_normalize_gradients(g, out=out)
    torch.cuda.synchronize()
    n0 = B.adapt_kernel_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        B.adapt_normalize_gradients(g, out=out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    peak, kind = measured_peak_gbs()
    achieved = 12.0 * n / (ms * 1e-3) / 1e9
    line = {"metric": "gradient-normalisation elements/s", "value": n / (ms * 1e-3), "unit": "elements/s",
            "n_gpus": 1, "steps": args.steps, "ms_per_step": ms, "dtype": "f64", "data": "synthetic",
            "gpu_launches": int(B.adapt_kernel_launch_count() - n0),
            "config": {"workload": f"one layer, {n} elements, Laplace(0,1e-4) with 5% zeros",
                       "l2": "inputs exceed L2" if 4 * n > 126e6 else "inputs may sit in L2"},
            "roofline": {"bound": "hbm", "kernel": "diversity (norm) + normalize (scaling), whole call",
                         "achieved": achieved, "peak": peak, "peak_kind": kind, "unit": "GB/s",
                         "frac": achieved / peak, "traffic": None}}
    if not args.no_cpu_baseline:
        from oracle import oracle as O
        m = min(n, 1 << 24)
        t0 = time.perf_counter()
        want = O.normalize_gradient(host[:m])
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": m / dt, "unit": "elements/s", "cores": 1, "kind": "oracle",
                                "sample": f"first {m} elements"}
        if m == n:
            got = out[0].cpu().numpy()
            line["parity_max_ulp"] = int(np.abs(got.view(np.int32).astype(np.int64) -
                                                want.view(np.int32).astype(np.int64)).max())
    print(json.dumps(line), flush=True)
    return 0


def run_diversity(args):
    """Gradient-diversity reduction: one layer of 2^24 elements with 32 recent gradients
    (2 GiB read per step), or --elements N."""
    import torch
    from paper_2107_13490_b200 import binding as B
    from paper_2107_13490_b200 import workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    B.lib()
    n, k = (args.elements or (1 << 24)), 32
    spec = W.LayerSpec("g", (n,), "laplace", 1e-4, zero_frac=0.05)
    host = [W.generate_layer(spec, 7, j) for j in range(k)]
    dev = [torch.from_numpy(g).cuda() for g in host]
    out = torch.empty((1, 4), dtype=torch.float64, device="cuda")
    for _ in range(max(args.warmup, 3)):
        B.adapt_gradient_diversity([dev], out=out)
    torch.cuda.synchronize()
    B.adapt_kernel_times(reset=True)
    B.adapt_kernel_timing(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        B.adapt_gradient_diversity([dev], out=out)
    e1.record()
    torch.cuda.synchronize()
    B.adapt_kernel_timing(False)
    ms = e0.elapsed_time(e1) / args.steps
    kt = B.adapt_kernel_times(reset=True)["diversity"]
    peak, kind = measured_peak_gbs()
    achieved = 4.0 * n * k / (kt[0] / args.steps * 1e-3) / 1e9
    line = {"metric": "gradient-diversity element-gradients/s", "value": n * k / (ms * 1e-3),
            "unit": "element-gradients/s", "n_gpus": 1, "steps": args.steps, "ms_per_step": ms,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"one layer, {n} elements, {k} Laplace(0,1e-4) gradients with 5% zeros",
                       "l2": "inputs exceed L2" if 4 * n * k > 2 * 126e6 else "inputs may sit in L2"},
            "roofline": {"bound": "hbm", "kernel": "diversity", "achieved": achieved, "peak": peak,
                         "peak_kind": kind, "unit": "GB/s", "frac": achieved / peak, "traffic": None}}
    if not args.no_cpu_baseline:
        from oracle import oracle as O
        m = min(n, 1 << 22)
        t0 = time.perf_counter()
        want = O.gradient_diversity([g[:m] for g in host])
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": m * k / dt, "unit": "element-gradients/s", "cores": 1,
                                "kind": "oracle", "sample": f"first {m} elements of each gradient"}
        if m == n:
            got = out.cpu().numpy()[0]
            line["parity_rel_err"] = float(abs(got[2] - want[2]) / abs(want[2]))
    print(json.dumps(line), flush=True)
    return 0


def bench_formats():
    """Block floating point at word lengths 2..16 and twelve float formats <E,M>."""
    f = [(1, wl, 0) for wl in range(2, 17)]
    f += [(2, e, m) for e in (4, 5, 8) for m in (2, 3, 7, 10)]
    return f


def run_formats(args):
    """The search over block-floating-point and floating-point candidates (27 formats) on the
    AlexNet weight tensors (or --workload / --elements)."""
    import torch
    from paper_2107_13490_b200 import binding as B
    from paper_2107_13490_b200 import workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    B.lib()
    name = args.workload if args.workload != "stress_1g" or args.elements else "alexnet_weights"
    w = W.WORKLOADS[name]
    if args.elements:
        w = W.scaled(w, args.elements)
    formats = bench_formats()
    host = W.generate(w)
    xs = [torch.from_numpy(x).cuda() for x in host]
    lens = [x.numel() for x in xs]
    total = sum(lens)
    ws = torch.empty(B.adapt_format_search_workspace_bytes(lens, formats, w.n_bins),
                     dtype=torch.uint8, device="cuda")
    out = None
    sampler = ClockSampler(0)
    sampler.start()            # started early: the first sample takes a while to arrive
    for _ in range(max(args.warmup, 3)):
        out = B.adapt_format_search(xs, formats, w.n_bins, workspace=ws, out=out)
    torch.cuda.synchronize()
    B.adapt_kernel_times(reset=True)
    B.adapt_kernel_timing(True)
    n0 = B.adapt_kernel_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    for _ in range(args.steps):
        B.adapt_format_search(xs, formats, w.n_bins, workspace=ws, out=out)
    e1.record()
    torch.cuda.synchronize()
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    B.adapt_kernel_timing(False)
    launches = B.adapt_kernel_launch_count() - n0
    ms = e0.elapsed_time(e1) / args.steps
    kt = B.adapt_kernel_times(reset=True)
    k_ms = kt["format_search"][0] / args.steps
    # Issue-bound kernel: one (element, rounding rule) evaluation needs at least 10 lane
    # instructions (scale, round, rescale; subtract, multiply, floor, two clamps, convert;
    # one shared atomic), and an SM issues 128 lane instructions per clock.
    sm_count = torch.cuda.get_device_properties(0).multi_processor_count
    sm_mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
    n_rules = 1 + len({(k, b if k == 0 else a, b if k == 2 else 0) for k, a, b in formats})
    peak = sm_count * 128 * sm_mhz * 1e6 / 10.0 / 1e9
    achieved = total * n_rules / (k_ms * 1e-3) / 1e9
    line = {"metric": "format-search element-formats/s", "value": total * len(formats) / (ms * 1e-3),
            "unit": "element-formats/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms, "higher_is_better": True,
            "dtype": "f32", "data": "synthetic", "gpu_launches": int(launches), "clocks": clocks,
            "config": {"workload": f"{w.name}: {len(xs)} layers, {total} elements, {len(formats)} formats "
                                   f"(15 block floating point, 12 floating point), {n_rules} rounding rules, "
                                   f"{w.n_bins} bins",
                       "l2": "inputs exceed L2" if 4 * total > 126e6 else "inputs fit in L2"},
            "kernel_ms": {k: v[0] / args.steps for k, v in kt.items() if v[1]},
            "roofline": {"bound": "alu", "kernel": "format_search", "achieved": achieved, "peak": peak,
                         "peak_kind": "SMs x 128 lanes x sampled SM clock / 10 instructions per evaluation",
                         "unit": "G element-rule evaluations/s", "frac": achieved / peak,
                         "hbm_gbs": 4.0 * total / (k_ms * 1e-3) / 1e9, "traffic": None}}
    if not args.no_cpu_baseline:
        from oracle import oracle as O
        l = max(range(len(host)), key=lambda i: host[i].size)
        m = min(host[l].size, 1 << 19)
        t0 = time.perf_counter()
        O.format_search_layer(host[l][:m], [f[0] for f in formats], [f[1] for f in formats],
                              [f[2] for f in formats], w.n_bins)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": m * len(formats) / dt, "unit": "element-formats/s", "cores": 1,
                                "kind": "oracle", "sample": f"first {m} elements of the largest layer"}
    print(json.dumps(line), flush=True)
    return 0


def _timed_steps(torch, step, steps, flush):
    """Per-step CUDA-event times (ms) of `steps` calls of step(), L2 flushed before each when a
    flush buffer is given (the flush lies outside the events)."""
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(steps)]
    for a, b in evs:
        if flush is not None:
            flush.zero_()
        a.record()
        step()
        b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in evs]


def workloads_block(torch, B, W, dev, sampler, peak, names, steps=30):
    """The paper's own workload shapes, device-resident, the library's per-kernel events OFF:
    median step time over L2-flushed steps, launches per step, and the time the step's
    algorithmic HBM traffic needs at the copy rate (one 4 B/element read for the search - the
    second read can come from L2 for sets that fit it - plus 8 B/element for the quantize)."""
    out = {}
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    for name in names:
        w = W.WORKLOADS[name]
        wl, fl = w.grid()
        grid = B.Grid(wl, fl)
        xs = [torch.from_numpy(x).to(dev) for x in W.generate(w)]
        lens = [x.numel() for x in xs]
        total = sum(lens)
        codes = [torch.empty(n, dtype=torch.int32, device=dev) for n in lens]
        ws = torch.empty(B.adapt_search_workspace_bytes(lens, grid, w.n_bins), dtype=torch.uint8, device=dev)
        res = B.SearchResult(torch.empty((len(xs), len(grid)), dtype=torch.float64, device=dev),
                             torch.empty((len(xs), len(grid)), dtype=torch.int64, device=dev),
                             torch.empty((len(xs), 4), dtype=torch.int32, device=dev))

        def step():
            B.adapt_precision_search_ex(xs, grid, w.n_bins, round_mode=w.round_mode, seed=w.seed,
                                        workspace=ws, out=res)
            B.adapt_quantize_selected_batch(xs, res.best, w.round_mode, w.seed, 0, codes_out=codes)

        for _ in range(5):
            step()
        torch.cuda.synchronize()
        n0 = B.adapt_kernel_launch_count()
        t0 = time.time()
        ms = _timed_steps(torch, step, steps, flush)
        # keep the region long enough for the clock sampler to see it
        while time.time() - t0 < 0.35:
            ms += _timed_steps(torch, step, steps, flush)
        t1 = time.time()
        launches = (B.adapt_kernel_launch_count() - n0) / len(ms)
        med = statistics.median(ms)
        bound_ms = 12.0 * total / (peak * 1e9) * 1e3
        out[name] = {"ms_per_step": med, "ms_min": min(ms), "steps": len(ms),
                     "launches_per_step": launches, "elements": total, "layers": len(xs),
                     "candidates": len(grid), "n_bins": w.n_bins,
                     "round_mode": "rne" if w.round_mode == 0 else "stochastic",
                     "element_candidates_per_s": total * len(grid) / (med * 1e-3),
                     "hbm_bound_ms": bound_ms, "ratio_to_hbm_bound": med / bound_ms,
                     "clocks": sampler.window(t0, t1)}
        del xs, codes, ws, res
    del flush
    return out


def distributions_block(torch, B, W, dev, sampler, peak, log2_n=28, steps=8):
    """The fused search kernel alone (library events around its launch) on single tensors of
    2^log2_n elements of other value classes, full 527-candidate grid, round-to-nearest-even,
    at 2048 and 512 bins: GB/s over the 4 B/element it must read, and the fraction of the peak."""
    out = {}
    n = 1 << log2_n
    wl, fl = W.candidate_grid(range(2, 33))
    grid = B.Grid(wl, fl)
    res = B.SearchResult(torch.empty((1, len(grid)), dtype=torch.float64, device=dev),
                         torch.empty((1, len(grid)), dtype=torch.int64, device=dev),
                         torch.empty((1, 4), dtype=torch.int32, device=dev))
    ws = torch.empty(B.adapt_search_workspace_bytes([n], grid, 2048), dtype=torch.uint8, device=dev)
    for name, spec in W.distribution_sweep(n):
        x = torch.from_numpy(W.generate_layer(spec, 11, 0)).to(dev)
        for n_bins in (2048, 512):
            def step():
                B.adapt_precision_search_ex([x], grid, n_bins, workspace=ws, out=res)
            for _ in range(3):
                step()
            torch.cuda.synchronize()
            B.adapt_kernel_times(reset=True)
            B.adapt_kernel_timing(True)
            t0 = time.time()
            k = 0
            while k < steps or time.time() - t0 < 0.35:
                step()
                k += 1
            torch.cuda.synchronize()
            t1 = time.time()
            B.adapt_kernel_timing(False)
            kt = B.adapt_kernel_times(reset=True)
            ms_k, n_k = kt["search"]
            if not n_k:
                ms_k, n_k = kt["search_direct"]
            ms = ms_k / n_k
            gbs = 4.0 * n / (ms * 1e-3) / 1e9
            out[f"{name}/{n_bins}"] = {"search_kernel_ms": ms, "gbs": gbs, "frac": gbs / peak,
                                       "launches": n_k, "clocks": sampler.window(t0, t1)}
        del x
    return out


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.path == "diversity":
        return run_diversity(args)
    if args.path == "normalize":
        return run_normalize(args)
    if args.path == "formats":
        return run_formats(args)

    import torch
    from paper_2107_13490_b200 import binding as B
    from paper_2107_13490_b200 import sharding as S
    from paper_2107_13490_b200 import workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    B.lib()
    rank, local_rank, world = S.init("nccl")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"

    base = W.WORKLOADS[args.workload]
    if args.elements:
        base = W.scaled(base, args.elements)
    if args.dist:
        spec = dict(W.distribution_sweep(base.layers[0].numel))[args.dist]
        base = W.Workload(f"{base.name}_{args.dist}", 11, (spec,), base.wl_values, base.n_bins,
                          base.round_mode, f"{args.dist} values, {spec.numel} elements")
    if args.bins:
        base = W.Workload(base.name, base.seed, base.layers, base.wl_values, args.bins,
                          base.round_mode, base.description)
    w = S.rank_workload(base, rank)
    round_mode = {"workload": w.round_mode, "rne": 0, "stochastic": 1}[args.round_mode]
    algorithm = {"auto": 0, "keyed": 1, "direct": 2}[args.algorithm]
    wl, fl = w.grid()
    grid = B.Grid(wl, fl)
    n_cand = len(grid)

    xs_np = W.generate(w)
    pinned = [torch.from_numpy(x).pin_memory() for x in xs_np]
    xs = [p.to(dev, non_blocking=True) for p in pinned]
    codes = [torch.empty(x.numel(), dtype=torch.int32, device=dev) for x in xs]
    lens = [x.numel() for x in xs]
    total = sum(lens)
    ws = torch.empty(B.adapt_search_workspace_bytes(lens, grid, w.n_bins), dtype=torch.uint8, device=dev)
    out = B.SearchResult(torch.empty((len(xs), n_cand), dtype=torch.float64, device=dev),
                         torch.empty((len(xs), n_cand), dtype=torch.int64, device=dev),
                         torch.empty((len(xs), 4), dtype=torch.int32, device=dev))
    torch.cuda.synchronize()

    def step():
        B.adapt_precision_search_ex(xs, grid, w.n_bins, round_mode=round_mode, seed=w.seed,
                                    workspace=ws, out=out, algorithm=algorithm)
        B.adapt_quantize_selected_batch(xs, out.best, round_mode, w.seed, 0, codes_out=codes)

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    # ---- device-resident timing -------------------------------------------------
    S.barrier()
    torch.cuda.synchronize()
    B.adapt_kernel_times(reset=True)
    B.adapt_kernel_timing(True)
    launches0 = B.adapt_kernel_launch_count()
    t_region0 = time.time()
    fits_l2 = 4 * total <= 2 * 126e6
    if not fits_l2:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        secs = e0.elapsed_time(e1) * 1e-3
    else:
        # inputs could stay in L2 from one step to the next: flush it between steps,
        # outside the per-step events
        flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(args.steps)]
        for a, b in evs:
            flush.zero_()
            a.record()
            step()
            b.record()
        torch.cuda.synchronize()
        secs = sum(a.elapsed_time(b) for a, b in evs) * 1e-3
        del flush
    t_region1 = time.time()
    S.barrier()
    clocks = sampler.window(t_region0, t_region1)
    launches = B.adapt_kernel_launch_count() - launches0
    B.adapt_kernel_timing(False)
    ktimes = B.adapt_kernel_times(reset=True)
    units = float(total) * n_cand * args.steps
    value, secs_max = S.job_throughput(units, secs, dev)

    # ---- roofline of the dominant kernel (the fused search kernel) ----------------
    peak, peak_kind = measured_peak_gbs()
    ms_search, n_search = ktimes["search"]
    ms_direct, n_direct = ktimes.get("search_direct", (0.0, 0))
    algo_bytes = 4.0 * total     # one fp32 read of every element per launch
    if ms_search >= ms_direct:
        achieved = algo_bytes / (ms_search / n_search * 1e-3) / 1e9 if n_search else None
        traffic = None
        if TRAFFIC_CAPTURE["version"] == B.adapt_version() and TRAFFIC_CAPTURE["bytes_per_element"]:
            traffic = TRAFFIC_CAPTURE["bytes_per_element"] * total
        roofline = {"bound": "hbm", "kernel": "search (fused quantize/zero-count/histograms)",
                    "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                    "frac": (achieved / peak) if achieved else None, "traffic": traffic,
                    "algorithmic_bytes_per_launch": algo_bytes,
                    "avg_launch_ms": ms_search / n_search if n_search else None}
    else:
        # The direct form evaluates every fraction length per element and is issue-bound: one
        # (element, FL) evaluation needs at least 10 lane instructions (scale, round, rescale;
        # subtract, multiply, floor, two clamps, convert; one shared atomic), and an SM issues
        # 128 lane instructions per clock.
        n_fl = int(max(fl)) + 1
        sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
        sm_mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
        alu_peak = sm_count * 128 * sm_mhz * 1e6 / 10.0 / 1e9
        achieved = float(total) * n_fl / (ms_direct / args.steps * 1e-3) / 1e9
        roofline = {"bound": "alu", "kernel": "search_direct (every fraction length per element)",
                    "achieved": achieved, "peak": alu_peak,
                    "peak_kind": "SMs x 128 lanes x sampled SM clock / 10 instructions per evaluation",
                    "unit": "G element-FL evaluations/s", "frac": achieved / alu_peak,
                    "hbm_gbs": algo_bytes / (ms_direct / args.steps * 1e-3) / 1e9, "traffic": None,
                    "launches_per_step": n_direct / args.steps}
    kernels = {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps}
               for k, v in ktimes.items() if v[1]}

    # ---- end to end through the host-buffer entry points ---------------------------
    e2e = None
    if not args.no_e2e:
        host_out = B.SearchResult(torch.empty((len(xs), n_cand), dtype=torch.float64).pin_memory(),
                                  torch.empty((len(xs), n_cand), dtype=torch.int64).pin_memory(),
                                  torch.empty((len(xs), 4), dtype=torch.int32).pin_memory())
        # the narrowest code type that holds every layer's selected word length (known from the
        # device-resident steps above): the download is that many bytes per element
        wl_max = int(out.best[:, 0].max().item())
        code_bits = 8 if wl_max <= 8 else (16 if wl_max <= 16 else 32)
        code_dtype = {8: torch.int8, 16: torch.int16, 32: torch.int32}[code_bits]
        host_codes = [torch.empty(n, dtype=code_dtype).pin_memory() for n in lens]

        def e2e_step():
            _, _, unfit = B.adapt_precision_switch_host_packed(pinned, grid, w.n_bins, code_bits,
                                                               round_mode=round_mode, seed=w.seed,
                                                               out=host_out, codes_out=host_codes)
            assert not unfit.any()

        e2e_step()
        S.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            e2e_step()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        S.barrier()
        e2e_value, _ = S.job_throughput(float(total) * n_cand * args.e2e_steps, dt, dev)
        res_bytes = len(xs) * (n_cand * 16 + 16 + 4)
        e2e = {"value": e2e_value, "unit": UNIT, "steps": args.e2e_steps,
               "ms_per_step": dt / args.e2e_steps * 1e3,
               "h2d_bytes_per_step": 4 * total, "d2h_bytes_per_step": res_bytes + code_bits // 8 * total,
               "code_bits": code_bits, "largest_selected_wl": wl_max,
               "api": "adapt_precision_switch_host_packed (pinned host buffers in; results and codes of "
                      "the narrowest type that holds every selected word length out, downloaded slice "
                      "by slice behind the quantize kernel)"}
        del host_codes

    # ---- the other configs and other value classes (single GPU, default workload only) -----
    workloads = distributions = None
    if world == 1 and args.workload == "stress_1g" and not args.elements and not args.no_extra:
        del codes, ws
        workloads = workloads_block(torch, B, W, dev, sampler, peak,
                                    ("single4k", "alexnet_weights", "resnet20_weights_grads",
                                     "resnet18_weights_acts"))
        distributions = distributions_block(torch, B, W, dev, sampler, peak)
    sampler.close()

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_oracle(xs_np, wl, fl, w, args.cpu_sample)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": max(args.warmup, 3),
                "ms_per_step": secs_max / args.steps * 1e3, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": base.name, "description": base.description,
                           "elements_per_gpu": total, "layers": len(xs), "candidates": n_cand,
                           "n_bins": w.n_bins,
                           "round_mode": "rne" if round_mode == 0 else "stochastic",
                           "algorithm": args.algorithm,
                           "step": "adapt_precision_search_ex + adapt_quantize_selected_batch",
                           "l2": "inputs exceed L2" if not fits_l2 else
                                 "L2 flushed (512 MiB write) between timed steps",
                           "parallelism": f"independent layer sets x{world}, no collective"},
                "hbm_gbs_whole_step": (8.0 * total + 8.0 * total) * args.steps / secs_max / 1e9 * world,
                "roofline": roofline, "kernels": kernels, "e2e": e2e,
                "cpu_baseline": cpu_baseline, "gpu_launches": int(launches), "clocks": clocks,
                "workloads": workloads, "distributions": distributions,
                "library": B.adapt_version()}
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
