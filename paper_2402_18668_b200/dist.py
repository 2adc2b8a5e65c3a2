"""Host-side helpers for running one process per GPU.

Every (b, h) head of the mixers is independent, so ranks never exchange data on the
data path: each rank runs its own copy of the per-GPU workload (weak scaling) and only
the timing is reduced (max over ranks).  These helpers use torch.distributed only and
work with the `gloo` backend on CPU as well as `nccl`.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def world() -> tuple[int, int]:
    """(rank, world_size); (0, 1) when no process group is initialised."""
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` over all ranks (the job's time is its slowest rank's)."""
    if world()[1] == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shard_heads(total_heads: int, rank: int, world_size: int) -> range:
    """Contiguous, balanced slice of the head index space owned by `rank` (strong-scaling
    split of one batch across GPUs; the first `total % world` ranks get one more head)."""
    base, extra = divmod(total_heads, world_size)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def whole_job_rate(units_per_rank: float, ms_local: float, device="cpu") -> float:
    """Units per second of the whole job: all ranks' units over the slowest rank's time."""
    _, n = world()
    ms = max_over_ranks(ms_local, device)
    return units_per_rank * n / (ms * 1e-3)
