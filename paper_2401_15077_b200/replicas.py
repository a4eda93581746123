"""Multi-GPU use of the tree-verification step: independent replicas.

Work units (sequence, KV head) and trees are independent, so the step has no exchange between GPUs: with N
processes (one per GPU) every rank verifies its own batch and nothing crosses NVLink on the data path.  The only
communication is what a benchmark or a serving front end needs around it: a barrier before and after the timed
region and the maximum of the ranks' device times.  These helpers hold that host-side logic so that it can be
tested on CPU with the gloo backend.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_salt(rank: int) -> int:
    """Seed salt of a rank's synthetic batch: every rank draws a different batch of the same workload."""
    return int(rank)


def is_distributed() -> bool:
    return dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1


def barrier() -> None:
    if is_distributed():
        dist.barrier()


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of a per-rank scalar over all ranks (the job is as slow as its slowest replica)."""
    if not is_distributed():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_steps_per_s(elapsed_ms: float, steps: int, device=None) -> float:
    """Steps all ranks completed per second: world * steps / slowest rank's time (weak scaling)."""
    world = dist.get_world_size() if is_distributed() else 1
    return world * steps / (max_over_ranks(elapsed_ms, device) * 1e-3)
