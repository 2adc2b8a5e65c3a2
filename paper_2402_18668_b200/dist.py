"""Host-side helpers for running one process per GPU.

Every (b, h) head of the mixers is independent, so when there are heads enough ranks never
exchange data on the data path: each rank runs its own copy of the per-GPU workload (weak
scaling) and only the timing is reduced (max over ranks).

When a batch has few heads and a long sequence, the sequence itself is cut across ranks
(rank r holds the r-th block of tokens).  The linear-attention mixer then has one exchange
step: every rank computes the recurrent state of its own block (based_prefill_state), the
block states are all-gathered, each rank sums those of the ranks before it, and runs
based_prefill from that state (BASED_STATE_CONTINUE).  The sliding-window mixer needs the last
window - 1 keys and values of the rank before (one neighbour send).  `sequence_parallel_prefill`
and `sequence_parallel_swa` do this; the compute steps are arguments, so the exchange logic is
tested on CPU (gloo) with stand-ins for the kernels.

These helpers use torch.distributed only and work with the `gloo` backend on CPU as well as `nccl`.
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


def exclusive_state_prefix(kv_block, z_block, group=None):
    """All-gathers the ranks' block states (kv [B,H,D,d_v], z [B,H,D], fp32) and returns the sum over the
    ranks before this one (zeros on rank 0): the state a rank's block starts from."""
    rank, n = world()
    if n == 1:
        return torch.zeros_like(kv_block), torch.zeros_like(z_block)
    kvs = [torch.empty_like(kv_block) for _ in range(n)]
    zs = [torch.empty_like(z_block) for _ in range(n)]
    dist.all_gather(kvs, kv_block.contiguous(), group=group)
    dist.all_gather(zs, z_block.contiguous(), group=group)
    kv_in, z_in = torch.zeros_like(kv_block), torch.zeros_like(z_block)
    for r in range(rank):
        kv_in += kvs[r]
        z_in += zs[r]
    return kv_in, z_in


def sequence_parallel_prefill(q, k, v, flags: int = 0, group=None, state_fn=None, prefill_fn=None):
    """Linear-attention prefill of a sequence cut across ranks: q, k, v are this rank's block
    ([B,H,L_r,.], blocks in rank order).  Returns (out_block, kv_state, z_state), the state being the one
    after this rank's block.  state_fn(k, v, flags) -> (kv, z) and prefill_fn(q, k, v, kv, z, flags) -> out
    (updating kv, z in place) default to the library's based_prefill_state and based_prefill."""
    from . import binding as _b
    if state_fn is None:
        state_fn = lambda k_, v_, f_: _b.based_prefill_state(k_, v_, flags=f_)
    if prefill_fn is None:
        prefill_fn = lambda q_, k_, v_, kv_, z_, f_: _b.based_prefill(q_, k_, v_, kv_state=kv_, z_state=z_, flags=f_)
    if flags & _b.BASED_STATE_CONTINUE:
        raise ValueError("the sequence-parallel prefill starts from the empty state")
    # the block's own state (it also fixes the state's shape), then the sum over the ranks before this one
    kv_block, z_block = state_fn(k, v, flags)
    kv_in, z_in = exclusive_state_prefix(kv_block, z_block, group)
    # continuing from an all-zero state (rank 0) is the same as starting from the empty one
    out = prefill_fn(q, k, v, kv_in, z_in, flags | _b.BASED_STATE_CONTINUE)
    return out, kv_in, z_in


def sequence_parallel_swa(q, k, v, window: int, group=None, swa_fn=None):
    """Sliding-window attention of a sequence cut across ranks (blocks in rank order, each at least
    window - 1 tokens long): the last window - 1 keys and values of the rank before are received and put in
    front of this rank's block; the outputs of those rows are dropped.  swa_fn(q, k, v, window) -> out
    defaults to the library's swa_forward."""
    from . import binding as _b
    if swa_fn is None:
        swa_fn = lambda q_, k_, v_, w_: _b.swa_forward(q_, k_, v_, window=w_)
    rank, n = world()
    halo = window - 1
    if n == 1 or halo == 0:
        return swa_fn(q, k, v, window)
    if k.shape[2] < halo:
        raise ValueError("every rank's block must hold at least window - 1 tokens")
    send_k, send_v = k[:, :, -halo:].contiguous(), v[:, :, -halo:].contiguous()
    recv_k, recv_v = torch.empty_like(send_k), torch.empty_like(send_v)
    ops = []
    if rank + 1 < n:
        ops += [dist.P2POp(dist.isend, send_k, rank + 1, group), dist.P2POp(dist.isend, send_v, rank + 1, group)]
    if rank > 0:
        ops += [dist.P2POp(dist.irecv, recv_k, rank - 1, group), dist.P2POp(dist.irecv, recv_v, rank - 1, group)]
    for req in dist.batch_isend_irecv(ops):
        req.wait()
    if rank == 0:
        return swa_fn(q, k, v, window)
    q_ext = torch.cat([torch.zeros_like(q[:, :, :halo]), q], dim=2)
    out = swa_fn(q_ext, torch.cat([recv_k, k], dim=2), torch.cat([recv_v, v], dim=2), window)
    return out[:, :, halo:].contiguous()

