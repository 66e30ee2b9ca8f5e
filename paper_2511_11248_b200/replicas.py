"""Timing plumbing for runs with one independent replica of the path per GPU.

The path does not shard: `bench.py --gpus N` runs N replicas, one process per GPU.  The only
cross-rank steps are the barrier around the timed region and the maximum of the ranks' device
times; the whole-job rate is the work of all ranks divided by that maximum.  The same helpers run
over gloo on CPU tensors (tests) and over NCCL on CUDA tensors (bench).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """Largest `value` over all ranks (the value itself when no process group is up)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier() -> None:
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def whole_job_rate(units_per_rank: float, slowest_seconds: float, world: int) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return world * units_per_rank / slowest_seconds
