"""World-size-2 checks of the multi-GPU plumbing on CPU (gloo): unit sharding is a partition and the job throughput
is total units over the slowest rank's time; with the KV heads of a layer split over the ranks, an all-gather of the
semantic vectors and a redundant separator give every rank the classes of the unsharded method."""
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


def _head_sharded_worker(rank, world, port, out):
    import numpy as np
    from oracle import taskkv_oracle as O
    from paper_2501_15113_b200 import workloads as W
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n_kv, G = 6, 2                                   # 6 KV heads over 2 ranks; with world 4: blocks of 1, 2, 1, 2
    wl = W.Workload(name="head_sharded", batch=1, n_layers=2, n_heads=n_kv * G, n_kv_heads=n_kv, head_dim=64,
                    seq_lens=[700], dtype="f32", sink=4, recent=32, window=16, mid_budget=[40, 40],
                    n_hetero=[[2, 1]], decode_steps=0, seed=9, variance=1.0, plant_offset=2.0)
    wl.planted = W._choose_planted(wl)
    mine = sharding.shard_heads(n_kv, rank, world)
    result = []
    for r in range(wl.n_layers):
        q, k, v = (t.double().numpy() for t in W.gen_layer(wl, 0, r, "cpu"))
        # Eq. 12-15 for this rank's heads only
        local = []
        for h in mine:
            c = O.window_scores(q[h * G:(h + 1) * G], k[h])
            local.append(O.semantic_vector(c, v[h], O.top_indices(c, wl.top_t)))
        local = torch.from_numpy(np.stack(local)).float() if len(local) else torch.zeros(0, wl.head_dim)
        # the one exchange of the head-sharded variant, then Eq. 7-8 and the separator on every rank
        sem = sharding.allgather_semantic_vectors(local, n_kv).double().numpy()
        cls = O.semantic_separator(O.center_distances(sem), wl.n_hetero[0][r], wl.promote_center)
        result.append((sem, cls))
    gathered = [None] * world
    dist.all_gather_object(gathered, [(s.tolist(), c.tolist()) for s, c in result])
    if rank == 0:
        out.put((gathered, wl.planted))
    dist.destroy_process_group()


def test_head_sharded_separator_matches_the_unsharded_oracle():
    import numpy as np
    from oracle import taskkv_oracle as O
    from paper_2501_15113_b200 import workloads as W
    ctx = mp.get_context("spawn")
    for world in (2, 4):
        out = ctx.Queue()
        port = _free_port()
        procs = [ctx.Process(target=_head_sharded_worker, args=(r, world, port, out)) for r in range(world)]
        for p in procs:
            p.start()
        gathered, planted = out.get(timeout=180)
        for p in procs:
            p.join(timeout=60)
            assert p.exitcode == 0
        # every rank holds the same vectors and the same classes
        for r in range(1, world):
            assert gathered[r] == gathered[0]
        # and they are those of the method run on all heads at once
        n_kv, G = 6, 2
        wl = W.Workload(name="head_sharded", batch=1, n_layers=2, n_heads=n_kv * G, n_kv_heads=n_kv, head_dim=64,
                        seq_lens=[700], dtype="f32", sink=4, recent=32, window=16, mid_budget=[40, 40],
                        n_hetero=[[2, 1]], decode_steps=0, seed=9, variance=1.0, plant_offset=2.0)
        wl.planted = planted
        for r in range(wl.n_layers):
            q, k, v = (t.double().numpy() for t in W.gen_layer(wl, 0, r, "cpu"))
            ref = O.compress_layer(q, k, v, n_hetero=wl.n_hetero[0][r], sink=4, recent=32, mid=40)
            sem, cls = gathered[0][r]
            assert cls == ref["cls"].tolist()
            assert sorted(np.flatnonzero(np.array(cls) == 1).tolist()) == planted[0][r]     # the planted heads
            assert np.abs(np.array(sem) - ref["sem"]).max() < 1e-6 * np.abs(ref["sem"]).max()   # fp32 on the wire


def test_head_shards_partition_the_heads_and_bound_the_pool():
    for n_kv, world in ((8, 2), (8, 3), (6, 4), (1, 2)):
        blocks = [list(sharding.shard_heads(n_kv, r, world)) for r in range(world)]
        assert [h for b in blocks for h in b] == list(range(n_kv))
        assert max(len(b) for b in blocks) - min(len(b) for b in blocks) <= 1
    # 3 of 8 heads keep all 1000 rows, the others 100: a rank with 4 heads plans for 3 full ones, one with 2 for 2
    assert sharding.shard_pool_rows_bound(1000, 4, 3, 100) == 3 * 1000 + 1 * 100
    assert sharding.shard_pool_rows_bound(1000, 2, 3, 100, max_new_tokens=5) == 2 * 1005
    # summed over the ranks the bound covers the true total and exceeds it by at most (world - 1) * h heads' difference
    total = sum(sharding.shard_pool_rows_bound(1000, len(sharding.shard_heads(8, r, 2)), 3, 100) for r in range(2))
    assert 3 * 1000 + 5 * 100 <= total <= (3 * 1000 + 5 * 100) + 3 * 900
