"""Multi-GPU plumbing: the path shards by independent units, so ranks need no data-path collective.

Every (sequence, layer) is independent of every other (the separator couples only the KV heads inside
one layer), so a job is split across ranks by whole (sequence, layer) pairs -- or, as bench.py does for
weak scaling, every rank runs its own replica of the batch.  The only exchange is the timing reduce:
throughput of the whole job = units all ranks processed / the slowest rank's time.
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def shard_pairs(batch: int, n_layers: int, rank: int, world: int) -> List[Tuple[int, int]]:
    """(sequence, layer) pairs owned by `rank`: a contiguous, balanced block of the b-major order."""
    total = batch * n_layers
    lo = total * rank // world
    hi = total * (rank + 1) // world
    return [(i // n_layers, i % n_layers) for i in range(lo, hi)]


def replica_seed(seed: int, rank: int) -> int:
    """Weak scaling: rank r works on an independent replica of the workload."""
    return seed + 1000 * rank


def job_throughput(units_this_rank: float, ms_this_rank: float, device=None) -> Tuple[float, float]:
    """(whole-job units per second, slowest rank's milliseconds).  One all-reduce of two numbers."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return units_this_rank * 1e3 / ms_this_rank, ms_this_rank
    t = torch.tensor([ms_this_rank], dtype=torch.float64, device=device)
    n = torch.tensor([units_this_rank], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(n.item()) * 1e3 / float(t.item()), float(t.item())
