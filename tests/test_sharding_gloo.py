"""World-size-2 check of the multi-GPU plumbing on CPU (gloo): unit sharding is a partition and the
job throughput is total units over the slowest rank's time."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2501_15113_b200 import sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    pairs = sharding.shard_pairs(batch=3, n_layers=5, rank=rank, world=world)
    gathered = [None] * world
    dist.all_gather_object(gathered, pairs)
    ms = 10.0 if rank == 0 else 25.0           # rank 1 is the slow one
    value, slowest = sharding.job_throughput(units_this_rank=100.0, ms_this_rank=ms)
    if rank == 0:
        out.put((gathered, value, slowest, sharding.replica_seed(7, 1)))
    dist.destroy_process_group()


def test_two_ranks_partition_and_max_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gathered, value, slowest, seed1 = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    allp = [x for part in gathered for x in part]
    assert sorted(allp) == [(b, r) for b in range(3) for r in range(5)]      # every pair exactly once
    assert abs(len(gathered[0]) - len(gathered[1])) <= 1
    assert slowest == 25.0
    assert abs(value - 200.0 * 1e3 / 25.0) < 1e-9                            # 200 units over the slowest rank
    assert seed1 == 1007


def test_single_process_throughput():
    v, t = sharding.job_throughput(50.0, 5.0)
    assert v == 10000.0 and t == 5.0
