"""Host-side plumbing for runs with one process per GPU: every rank processes its own trace of the
same shape (weak scaling); ranks meet at a barrier, to take the maximum of their device times, and — the
one exchange step the path has when a job's warps are spread over several GPUs — to combine their
kernel-scope tables. Works with any torch.distributed backend (NCCL on GPUs, gloo on CPU)."""
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


def combine_kernel_tables(table, world: int):
    """Combines the kernel-scope table (R cells of 72 unsigned 64-bit words, given as a uint8 or int64 tensor)
    of all ranks in place: counts, sums, flag and ambiguity counters and histogram bins add up, min_incl is the
    minimum and max_incl the maximum. Three small all-reduces (R x 576 bytes in total)."""
    if world <= 1:
        return table
    import torch
    import torch.distributed as dist
    t = table.view(torch.int64).view(-1, 72)
    sign = torch.tensor(-(1 << 63), dtype=torch.int64, device=t.device)
    # unsigned order -> signed order for the two extremum fields (the collectives compare signed integers)
    lo = (t[:, 2] ^ sign).contiguous()
    hi = (t[:, 3] ^ sign).contiguous()
    add = t.clone()
    dist.all_reduce(add, op=dist.ReduceOp.SUM)   # two's complement wrap-around = unsigned addition
    dist.all_reduce(lo, op=dist.ReduceOp.MIN)
    dist.all_reduce(hi, op=dist.ReduceOp.MAX)
    t.copy_(add)
    t[:, 2] = lo ^ sign
    t[:, 3] = hi ^ sign
    return table
