"""The multi-rank host logic on CPU: two gloo ranks, no GPU."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, {root!r})
import numpy as np
from paper_2107_13490_b200 import sharding as S, workloads as W
rank, local, world = S.init("gloo")
assert world == 2
w = S.rank_workload(W.WORKLOADS["single4k"], rank)
x = W.generate(w)[0]
S.barrier()
value, secs = S.job_throughput(1000.0 * (rank + 1), 2.0 + rank)
assert abs(secs - 3.0) < 1e-12 and abs(value - 3000.0 / 3.0) < 1e-9, (value, secs)
sums = S.sum_over_ranks(float(x[:16].astype(np.float64).sum()))
print("RANK", rank, "seed", w.seed, "sum", repr(sums), flush=True)
"""


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_gloo_ranks_get_independent_problems_and_max_time():
    port = free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD.format(root=ROOT)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    seeds = [o.split("seed")[1].split()[0] for o in outs]
    sums = [o.split("sum")[1].split()[0] for o in outs]
    assert seeds[0] != seeds[1] and sums[0] == sums[1]


def test_split_layers_partitions_everything():
    from paper_2107_13490_b200 import sharding as S
    parts = S.split_layers(25, 4)
    assert sorted(sum(parts, [])) == list(range(25))
    assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1
