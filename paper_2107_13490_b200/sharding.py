"""Multi-GPU plumbing of the search: layers are independent problems, so ranks
never exchange data.  Each rank searches its own layer set on its own GPU; the
only communication is the barrier and the max-over-ranks of the step time used
for reporting (torch.distributed: NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import os
from dataclasses import replace
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist

from . import workloads as W


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def rank_workload(w: W.Workload, rank: int) -> W.Workload:
    """Weak scaling: every rank gets a workload of the same shapes with its own seed."""
    return replace(w, seed=w.seed + 1000003 * rank, name=w.name if rank == 0 else f"{w.name}@r{rank}")


def split_layers(n_layers: int, world: int) -> List[List[int]]:
    """Strong scaling alternative: a round-robin partition of one layer list."""
    return [list(range(r, n_layers, world)) for r in range(world)]


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device: str = "cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: str = "cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_this_rank: float, seconds_this_rank: float, device: str = "cpu") -> Tuple[float, float]:
    """Whole-job units/s = units of all ranks / slowest rank's time. Returns (value, seconds)."""
    secs = max_over_ranks(seconds_this_rank, device)
    units = sum_over_ranks(units_this_rank, device)
    return units / secs, secs
