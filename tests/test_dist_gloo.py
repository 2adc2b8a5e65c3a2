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
