"""Host-side helpers for running independent replicas of the step on several GPUs (one process per GPU).

The SureLock step shards by sequence with no exchange step (lock mask, K/V cache, previous logits and active rows
are per sequence; only the weights are shared), so N GPUs run N independent replicas.  The only communication is
bookkeeping for the benchmark: the slowest rank's time and the sum of the rows every rank processed.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank_world():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1)), int(os.environ.get("LOCAL_RANK", 0))


def replica_seed(base: int, rank: int) -> int:
    """Every replica draws its own weights/prompts stream, so ranks do not run bit-identical work."""
    return int(base) + 1009 * int(rank)


def max_over_ranks(value: float, device="cpu") -> float:
    """Max of a scalar over all ranks (the job is as slow as its slowest replica)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(rows_this_rank: int, ms_this_rank: float, device="cpu"):
    """(rows per second of the whole job, ms of the slowest rank): all rows of all replicas / max time."""
    ms = max_over_ranks(ms_this_rank, device)
    rows = sum_over_ranks(rows_this_rank, device)
    return rows / (ms * 1e-3), ms
