"""Host-side plumbing of the multi-GPU benchmark: the RoM layer forward has no exchange step (routing is
per token, conv and scan per sequence), so N GPUs run N independent replicas of the workload.  The only
cross-rank work is timing: every rank measures on its own device, the job's time is the maximum over
ranks, and the job's throughput is the sum of what all ranks processed divided by that time.

Works with any torch.distributed backend (nccl on GPUs, gloo on CPU for tests); with no process group
(single process) every function degenerates to the identity.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch


def world_info(dist) -> tuple:
    """(rank, world_size) of the default process group, (0, 1) without one."""
    if dist is None or not dist.is_available() or not dist.is_initialized():
        return 0, 1
    return dist.get_rank(), dist.get_world_size()


def max_over_ranks(values: Sequence[float], dist=None, device="cpu") -> list:
    """Element-wise maximum over ranks of a short list of floats (device times in ms)."""
    vals = [float(v) for v in values]
    rank, world = world_info(dist)
    if world == 1:
        return vals
    t = torch.tensor(vals, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def job_throughput(units_per_rank_per_step: int, world: int, steps: int, ms_max: float) -> float:
    """Whole-job units per second: every rank processed `units_per_rank_per_step` per step."""
    return units_per_rank_per_step * world * steps / (ms_max * 1e-3)


def barrier(dist=None) -> None:
    _, world = world_info(dist)
    if world > 1:
        dist.barrier()
