"""Host-side plumbing for runs with one process per GPU: every rank processes its own trace of the
same shape (weak scaling, no data-path collective); ranks only meet at a barrier and to take the
maximum of their device times. Works with any torch.distributed backend (NCCL on GPUs, gloo on CPU)."""
from __future__ import annotations

import os
from dataclasses import replace


def rank_env():
    """(rank, world_size, local_rank) from the launcher's environment (1 process if absent)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_spec(spec, rank: int):
    """The trace rank `rank` generates: same shape, its own seed."""
    return replace(spec, seed=spec.seed + 1000 * rank)


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Maximum of a per-rank scalar (device time in ms) over all ranks."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: int, world: int, ms_max: float) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return units_per_rank * world / (ms_max * 1e-3)
