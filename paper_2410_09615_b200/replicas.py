"""Timing arithmetic of the replicated benchmark (one process per GPU, no data-path collective).

The layer forward does not shard across GPUs inside this library: N GPUs run N independent
replicas of the same step.  The only cross-rank operations are a barrier around the timed
region and the maximum of the ranks' elapsed times; both work on any torch.distributed backend,
so they are tested on CPU with gloo.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def world_size() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def barrier() -> None:
    if world_size() > 1:
        dist.barrier()


def max_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """The slowest rank's figure (the job is done when the last replica is)."""
    if world_size() == 1:
        return float(value)
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_us_per_call(ms_per_step: float, calls_per_step: int, world: int) -> float:
    """Microseconds per layer call over the whole job: every replica finishes
    `calls_per_step` calls in one step, so the job finishes `calls_per_step * world`."""
    return 1e3 * ms_per_step / (calls_per_step * world)
