"""The bounds-checking build of the library on ragged, multi-layer and adversarial inputs.

No memory checker can be run on the kernels, so the library has a build in which every table
index formed from the data is tested against its table's size (adapt_bounds_check_status).
A child process loads that build instead of the normal one, runs searches in every kernel form
(their results are compared with the oracle as usual) and reports the device's error word,
which must stay zero."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import numpy as np, torch
from oracle import oracle as O
from paper_2107_13490_b200 import binding as B, workloads as W
from tests import gpu_util as G
B.lib()
checking, word = B.adapt_bounds_check_status(clear=True)
assert checking, "the bounds-checking build was not loaded"
rng = np.random.default_rng(99)
n = 30011
base = (rng.standard_normal(n) * 0.25).astype(np.float32)
cases = {
    "normal": base,
    "half_zero": np.maximum(base, 0),
    "far_from_zero": (1000.0 + rng.random(n) * 0.01).astype(np.float32),
    "very_wide": (rng.standard_normal(n) * 1e15).astype(np.float32),
    "tiny": (rng.standard_normal(n) * 1e-9).astype(np.float32),
    "on_grid": (rng.integers(-2000, 2000, n) * 2.0 ** -6).astype(np.float32),
    "on_grid_strays": np.where(rng.random(n) < 0.001, base, np.round(base * 64) / 64).astype(np.float32),
    "ties": (rng.integers(-4000, 4000, n) * 2.0 ** -9 + 2.0 ** -10).astype(np.float32),
    "subnormals": np.float32([1e-40, -1e-41, 3e-39, 0.0, 5e-45] * 50),
    "extremes": np.float32([-1e19, 1e19, 0.0, 1.0, -1e-30]),
}
wl, fl = W.candidate_grid(range(2, 33))
for name, x in cases.items():
    for n_bins in (37, 2048):
        for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
            G.run_and_compare(B, [x], wl, fl, n_bins, round_mode=mode, seed=5, where=name)
# many layers of ragged sizes in one call, misaligned views, empty and constant layers
buf = torch.from_numpy(np.concatenate([base] * 6)).cuda()
xs, off = [], 1
for ln in (1, 5, 4097, 0, 33000, 70001, 12289, 300):
    xs.append(buf[off:off + ln]); off += ln + 1
xs.append(torch.full((500,), 0.37, device="cuda"))
host = [t.cpu().numpy() for t in xs]
ora = O.precision_search(host, wl, fl, 150, want_hist=True, threads=G.host_threads())
for algo in G.ALGORITHMS:
    res = B.adapt_precision_search_ex(xs, B.Grid(wl, fl), 150, want_hist=True, want_range=True, algorithm=algo)
    torch.cuda.synchronize()
    G.compare_search(res, ora, len(xs), f"ragged layers algo {algo}", True, True)
# the format search's kernels
fm = [(O.FMT_BFP, w, 0) for w in (2, 8, 16)] + [(O.FMT_FLOAT, 5, 10), (O.FMT_FLOAT, 4, 3), (O.FMT_FIXED, 8, 4)]
for mode in (O.ROUND_RNE, O.ROUND_STOCHASTIC):
    B.adapt_format_search([torch.from_numpy(c).cuda() for c in (base, cases["very_wide"], cases["subnormals"])],
                          fm, 128, round_mode=mode, seed=3)
checking, word = B.adapt_bounds_check_status()
print("BOUNDS", int(checking), *[int(v) for v in word])
"""


def test_no_table_index_leaves_its_table():
    from paper_2107_13490_b200 import build
    lib = build.build(check=True)
    env = dict(os.environ, ADAPT_B200_LIBRARY=lib, PYTHONPATH=ROOT)
    out = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=env, capture_output=True, text=True,
                         timeout=1500)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    line = [ln for ln in out.stdout.splitlines() if ln.startswith("BOUNDS")][-1].split()
    assert line[1] == "1"                       # the checking build did run
    assert line[2:] == ["0", "0", "0", "0"], f"an index left its table: events, site, index, limit = {line[2:]}"
