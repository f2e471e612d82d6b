"""Rank coordination of the multi-GPU benchmark.

The GEMM itself never leaves one GPU (its output tiles are independent, so N GPUs are N replicas of
the same job with no exchange step).  What the ranks share is bookkeeping: a barrier around the timed
region, the slowest rank's time, and the job's aggregate throughput.  Works on any torch.distributed
backend (NCCL on GPUs, gloo on CPU), which is how it is tested without GPUs.
"""
from __future__ import annotations

import torch


def slowest_rank_ms(local_ms: float, dist=None, device="cpu") -> float:
    """Max over ranks of a per-rank time (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_ms)
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, world_size: int, ms: float) -> float:
    """Whole-job units per second when every rank processed `units_per_rank` in `ms` (weak scaling)."""
    return world_size * units_per_rank / (ms * 1e-3)


def barrier(dist=None) -> None:
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
