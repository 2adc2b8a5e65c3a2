"""World-size-2 check of the multi-process host logic on CPU (gloo)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2402_18668_b200 import dist as bd
    assert bd.world() == (rank, world)
    slowest = bd.max_over_ranks(10.0 + 5.0 * rank)
    rate = bd.whole_job_rate(units_per_rank=1000.0, ms_local=10.0 + 5.0 * rank)
    heads = list(bd.shard_heads(37, rank, world))
    gathered = [None] * world
    dist.all_gather_object(gathered, heads)
    if rank == 0:
        out.put((slowest, rate, gathered))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_time_and_partition_heads():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    slowest, rate, gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert slowest == 15.0
    assert abs(rate - 2 * 1000.0 / 15e-3) < 1e-6
    flat = [h for part in gathered for h in part]
    assert flat == list(range(37)) and abs(len(gathered[0]) - len(gathered[1])) <= 1


def test_single_process_defaults():
    from paper_2402_18668_b200 import dist as bd
    assert bd.world() == (0, 1)
    assert bd.max_over_ranks(3.5) == 3.5
    assert list(bd.shard_heads(5, 0, 1)) == [0, 1, 2, 3, 4]


def _seq_worker(rank, world, port, out):
    """A sequence cut across ranks: the exchange logic with the CPU oracle standing in for the kernels."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import numpy as np
    import oracle
    from paper_2402_18668_b200 import dist as bd
    B, H, d_v, window = 1, 2, 8, 5
    lens = [7, 11, 6][:world]                       # uneven blocks, each at least window - 1 long
    L = sum(lens)
    g = torch.Generator().manual_seed(123)          # every rank draws the whole sequence, keeps its block
    q = torch.randn(B, H, L, 16, generator=g, dtype=torch.float64) * 0.5
    k = torch.randn(B, H, L, 16, generator=g, dtype=torch.float64) * 0.5
    v = torch.randn(B, H, L, d_v, generator=g, dtype=torch.float64)
    qs = torch.randn(B, H, L, 64, generator=g, dtype=torch.float64)
    ks = torch.randn(B, H, L, 64, generator=g, dtype=torch.float64)
    vs = torch.randn(B, H, L, 64, generator=g, dtype=torch.float64)
    lo = sum(lens[:rank]); hi = lo + lens[rank]
    blk = lambda t: t[:, :, lo:hi].contiguous()

    def state_fn(k_, v_, flags):
        _, S, z = oracle.linattn_recurrent(k_.numpy(), k_.numpy(), v_.numpy())
        return torch.from_numpy(S), torch.from_numpy(z)

    def prefill_fn(q_, k_, v_, kv, z, flags):
        y, S, zz = oracle.linattn_recurrent(q_.numpy(), k_.numpy(), v_.numpy(), S0=kv.numpy(), z0=z.numpy())
        kv.copy_(torch.from_numpy(S)); z.copy_(torch.from_numpy(zz))
        return torch.from_numpy(y)

    swa_fn = lambda q_, k_, v_, w_: torch.from_numpy(oracle.swa(q_.numpy(), k_.numpy(), v_.numpy(), w_))
    y, kv, z = bd.sequence_parallel_prefill(blk(q), blk(k), blk(v), state_fn=state_fn, prefill_fn=prefill_fn)
    o = bd.sequence_parallel_swa(blk(qs), blk(ks), blk(vs), window, swa_fn=swa_fn)
    # the whole sequence on one process
    y_ref, S_ref, z_ref = oracle.linattn_recurrent(q.numpy(), k.numpy(), v.numpy())
    _, S_pre, z_pre = oracle.linattn_recurrent(q[:, :, :hi].numpy(), k[:, :, :hi].numpy(), v[:, :, :hi].numpy())
    o_ref = oracle.swa(qs.numpy(), ks.numpy(), vs.numpy(), window)
    errs = (float(np.abs(y.numpy() - y_ref[:, :, lo:hi]).max()), float(np.abs(kv.numpy() - S_pre).max()),
            float(np.abs(z.numpy() - z_pre).max()), float(np.abs(o.numpy() - o_ref[:, :, lo:hi]).max()))
    gathered = [None] * world
    dist.all_gather_object(gathered, errs)
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def _run_seq(world):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_seq_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    gathered = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    return gathered


def test_sequence_cut_across_two_ranks_matches_one_process():
    for errs in _run_seq(2):
        assert max(errs) < 1e-10, errs


def test_sequence_cut_across_three_ranks_matches_one_process():
    for errs in _run_seq(3):
        assert max(errs) < 1e-10, errs

