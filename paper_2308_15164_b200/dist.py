"""Process-group plumbing for running independent replicas of the delayed synchronous step,
one process per GPU.  The step itself has no exchange between replicas (the paper's workers
are buffers inside one GPU), so the only collectives are a barrier around the timed region
and max/sum reductions of the measurements."""

from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def rank_info() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = rank_info()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier(device=None):
    if dist.is_available() and dist.is_initialized():
        if device is not None and device.type == "cuda":
            dist.barrier(device_ids=[device.index])
        else:
            dist.barrier()


def reduce_max(value: float, device=None) -> float:
    """Max over ranks of a per-rank scalar (e.g. the device-timed duration of the timed region)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def reduce_sum(value: float, device=None) -> float:
    """Sum over ranks (e.g. units of work processed)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def aggregate_throughput(units_this_rank: float, seconds_this_rank: float, device=None) -> Tuple[float, float]:
    """Whole-job throughput of independent replicas: (sum of units) / (max of durations).
    Returns (throughput, max_seconds)."""
    total = reduce_sum(units_this_rank, device)
    worst = reduce_max(seconds_this_rank, device)
    return total / worst, worst


def shutdown():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
