"""Multi-GPU plumbing: the path shards by independent units, so ranks need no data-path collective.

Every (sequence, layer) is independent of every other (the separator couples only the KV heads inside
one layer), so a job is split across ranks by whole (sequence, layer) pairs -- or, as bench.py does for
weak scaling, every rank runs its own replica of the batch.  The only exchange is the timing reduce:
throughput of the whole job = units all ranks processed / the slowest rank's time.

Sharding by KV head (tensor-parallel style, where every rank holds some heads of every layer) does need one
exchange: the center of Eq. 8 is the mean over ALL heads of a layer, so the ranks all-gather their heads'
semantic vectors (n_kv_local x d fp32 per sequence and layer) and each runs the separator of Sec. IV-A on the full
set, redundantly; everything before (window scores, top-t, Eq. 15) and after (allocation, gather, decode) is per
head.  `shard_heads`, `allgather_semantic_vectors` and `shard_pool_rows_bound` are the host side of that variant.
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


def shard_heads(n_kv_heads: int, rank: int, world: int) -> range:
    """KV heads owned by `rank`: a contiguous, balanced block (query heads follow their KV head)."""
    lo = n_kv_heads * rank // world
    hi = n_kv_heads * (rank + 1) // world
    return range(lo, hi)


def allgather_semantic_vectors(local: torch.Tensor, n_kv_heads: int) -> torch.Tensor:
    """local: [..., n_local, d] fp32 semantic vectors (Eq. 15) of this rank's heads, in `shard_heads` order.
    Returns [..., n_kv_heads, d] with every rank's block in place, identical on all ranks.  Blocks may differ in
    size by one head, so each is padded to the largest before the collective (into local memory: the result is an
    ordinary tensor of this rank)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return local
    world = dist.get_world_size()
    sizes = [len(shard_heads(n_kv_heads, r, world)) for r in range(world)]
    pad = max(sizes)
    lead, d = local.shape[:-2], local.shape[-1]
    buf = torch.zeros(*lead, pad, d, dtype=local.dtype, device=local.device)
    buf[..., :local.shape[-2], :] = local
    parts = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf.contiguous())
    return torch.cat([parts[r][..., :sizes[r], :] for r in range(world)], dim=-2)


def shard_pool_rows_bound(seq_len: int, n_local: int, full_heads: int, kept_len: int, max_new_tokens: int = 0) -> int:
    """Pool rows a rank must reserve for one (sequence, layer) when heads are sharded: how many heads of the layer
    keep everything is fixed by Eq. 16, but which rank they land on is not, so a rank plans for as many of them as it
    has heads."""
    h = min(full_heads, n_local)
    return h * (seq_len + max_new_tokens) + (n_local - h) * (kept_len + max_new_tokens)


def compress_head_sharded(params, q_win, k, v, stream=None):
    """One rank's part of a head-sharded compression: Eq. 12-15 for its own heads, the all-gather of the semantic
    vectors, then separator, allocation and gather.  `params` is a binding.Params with shard_kv_heads > 0 and
    shard_first = shard_heads(...)[0]; the tensors hold this rank's heads.  Returns the rank's cache."""
    from . import binding as tk
    cache = tk.taskkv_compress_shard_begin(params, q_win, k, v, stream=stream)
    local = cache.semantic_vectors()
    if stream is not None:
        stream.synchronize()                     # the collective runs on the process group's own stream
    else:
        torch.cuda.current_stream().synchronize()
    sem_all = allgather_semantic_vectors(local, params.c.shard_kv_heads).contiguous()
    cache.taskkv_compress_shard_finish(sem_all, stream=stream)
    return cache
