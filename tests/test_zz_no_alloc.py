"""taskkv_decode_noalloc against taskkv_decode.

The no-allocation entry point serves callers that may not allocate device
memory (an engine that owns the whole device heap through its own pool, or a
decode loop that cannot afford cudaMalloc's device-wide synchronisation); its
split-K scratch is a fixed array inside the library.  Here it is called through
the C ABI twice in a row, with different queries and lengths, and each result is
compared with the regular decode call on the same rows.  The second call would
expose partial results left in the shared scratch by the first.
This file is collected last on purpose, so an early-exit test run has already
covered everything else.
"""
import numpy as np
import pytest
import torch

from paper_2501_15113_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = {"bf16": 2e-2, "f32": 1e-5}


def _make(dtype, n, n_kv, d, N, seed):
    wl = W.Workload(name="noalloc", batch=1, n_layers=2, n_heads=n, n_kv_heads=n_kv, head_dim=d, seq_lens=[N],
                    dtype=dtype, sink=4, recent=16, window=8, mid_budget=[8, 8], n_hetero=[[0, 0]],
                    decode_steps=0, seed=seed, variance=1.0 if dtype == "f32" else 1.0 / np.sqrt(d))
    wl.planted = W._choose_planted(wl)
    return wl


@pytest.mark.parametrize("dtype,n,n_kv,d,N", [("bf16", 8, 2, 128, 3001), ("f32", 4, 4, 64, 1777)])
def test_noalloc_matches_decode_twice(dtype, n, n_kv, d, N):
    from paper_2501_15113_b200 import binding as tk
    wl = _make(dtype, n, n_kv, d, N, seed=21)
    qs, ks, vs = W.materialize(wl, DEV)
    # every head keeps its full cache, so the cache's segments hold exactly the rows of k and v
    cache = tk.taskkv_compress_ex(tk.params_from_workload(wl, max_new_tokens=0, force_class=1), qs, ks, vs)
    U = wl.n_layers * n_kv
    assert cache.lengths().tolist() == [N] * U
    k_pool = ks[0].reshape(U * N, d)
    v_pool = vs[0].reshape(U * N, d)
    seg_off = (torch.arange(U, device=DEV, dtype=torch.int64) * N).contiguous()
    gen = torch.Generator(device="cpu").manual_seed(5)
    for call in range(2):
        q, _, _ = W.gen_decode_step(wl, call, DEV)
        if call == 0:
            lens = torch.full((U,), N, dtype=torch.int32)
        else:   # ragged prefixes, one of them a single row: splits that were full in call 0 are now empty
            lens = torch.randint(1, N + 1, (U,), generator=gen, dtype=torch.int32)
            lens[0] = 1
        lens_d = lens.to(DEV)
        want = cache.taskkv_decode(q, lengths=lens_d)
        got = tk.taskkv_decode_noalloc(q.reshape(U * (n // n_kv), d), k_pool, v_pool, seg_off, lens_d,
                                       group=n // n_kv, max_len=N)
        torch.cuda.synchronize()
        err = (got.double().reshape(-1) - want.double().reshape(-1)).abs().max().item()
        assert err < TOL[dtype], f"call {call}: max abs difference {err:.3e}"
    cache.close()


def test_noalloc_rejects_sizes_beyond_the_fixed_scratch():
    from paper_2501_15113_b200 import binding as tk
    d, G = 128, 8
    too_many = (32 << 20) // (G * (d + 2) * 4) + 1
    q = torch.zeros(8, d, device=DEV, dtype=torch.bfloat16)
    pool = torch.zeros(8, d, device=DEV, dtype=torch.bfloat16)
    off = torch.zeros(too_many, device=DEV, dtype=torch.int64)
    lens = torch.zeros(too_many, device=DEV, dtype=torch.int32)
    with pytest.raises(tk.TaskKVError) as ei:
        tk.taskkv_decode_noalloc(q, pool, pool, off, lens, group=G, max_len=16, out=q)
    assert ei.value.status == tk.EINVAL
