"""Multi-GPU plumbing for the benchmark: the layer has no exchange step, so ranks run independent
batches (data parallel over the batch, as the paper's 4-GPU runs do) and only timings and unit
counts are reduced.  Works on any torch.distributed backend (nccl on GPUs, gloo in CPU tests)."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when not launched by it."""
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


def rank_seed(base_seed: int, rank: int) -> int:
    """Each rank draws its own batch: distinct, reproducible seeds."""
    return base_seed + 7919 * rank


def max_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(local_units: float, local_ms: float, device="cpu") -> tuple:
    """(units/s over all ranks, max ms): total units divided by the slowest rank's time."""
    ms = max_over_ranks(local_ms, device)
    units = sum_over_ranks(local_units, device)
    return units / (ms * 1e-3), ms
