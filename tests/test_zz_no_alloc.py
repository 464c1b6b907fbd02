"""taskkv_decode_noalloc against the CPU oracle and against taskkv_decode.

The no-allocation entry point serves callers that may not allocate device
memory (an engine that owns the whole device heap through its own pool, or a
decode loop that cannot afford cudaMalloc's device-wide synchronisation); its
split-K scratch is a fixed array inside the library.  Here it is called through
the C ABI twice in a row, with different queries and lengths, and each result is
compared with the oracle's decode attention over the same rows and with the
regular decode call.  The second call would expose partial results left in the
shared scratch by the first.
This file is collected last on purpose, so an early-exit test run has already
covered everything else.
"""
import numpy as np
import pytest
import torch

from oracle import taskkv_oracle as O
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


def _oracle_decode(q, ks, vs, lens, n_kv, G):
    """Eq. 1 per query head over the first lens[u] rows of its KV head's K and V, in float64."""
    want = np.zeros((q.shape[0], q.shape[1]))
    U = len(lens)
    k64 = ks.double().cpu().numpy().reshape(U, -1, q.shape[1])
    v64 = vs.double().cpu().numpy().reshape(U, -1, q.shape[1])
    q64 = q.double().cpu().numpy()
    for u in range(U):
        if lens[u] == 0:
            continue                     # no row to attend over: the library writes zeros
        for g in range(G):
            want[u * G + g] = O.decode_attention(q64[u * G + g], k64[u][:lens[u]], v64[u][:lens[u]])
    return want


CASES = [(dt, G, d) for dt in ("bf16", "f32") for G in (1, 2, 4, 8) for d in (64, 128)]


@pytest.mark.parametrize("dtype,G,d", CASES, ids=[f"{dt}-G{G}-d{d}" for dt, G, d in CASES])
def test_noalloc_matches_oracle_and_decode_twice(dtype, G, d):
    from paper_2501_15113_b200 import binding as tk
    n_kv = 2
    n = n_kv * G
    N = 1777 if d == 64 else 3001
    wl = _make(dtype, n, n_kv, d, N, seed=21 + G + d)
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
        else:   # ragged prefixes, a single row and an empty unit: splits that were full in call 0 are now empty
            lens = torch.randint(1, N + 1, (U,), generator=gen, dtype=torch.int32)
            lens[0] = 1
            lens[U - 1] = 0
        lens_d = lens.to(DEV)
        q2 = q.reshape(U * G, d).contiguous()
        got = tk.taskkv_decode_noalloc(q2, k_pool, v_pool, seg_off, lens_d, group=G, max_len=N)
        torch.cuda.synchronize()
        want = _oracle_decode(q2, ks[0], vs[0], lens.tolist(), n_kv, G)
        err = np.abs(got.double().cpu().numpy() - want).max()
        assert err < TOL[dtype], f"call {call}: max abs difference from the oracle {err:.3e}"
        # and the library's regular decode call on the same rows (units with at least one row)
        live = torch.repeat_interleave(lens > 0, G).to(DEV)
        ref = cache.taskkv_decode(q, lengths=torch.clamp(lens_d, min=1)).reshape(U * G, d)
        err2 = (got.double() - ref.double())[live].abs().max().item()
        assert err2 < TOL[dtype], f"call {call}: max abs difference from taskkv_decode {err2:.3e}"
    cache.close()


def test_noalloc_clamps_lengths_to_max_len():
    """A length above max_len attends over the first max_len rows only; nothing beyond is read."""
    from paper_2501_15113_b200 import binding as tk
    d, G, U, N = 64, 2, 3, 900
    g = torch.Generator(device="cpu").manual_seed(9)
    q = torch.randn(U * G, d, generator=g).to(DEV)
    k = torch.randn(U * N, d, generator=g).to(DEV)
    v = torch.randn(U * N, d, generator=g).to(DEV)
    off = (torch.arange(U, dtype=torch.int64) * N).to(DEV)
    over = torch.tensor([N, 700, 650], dtype=torch.int32, device=DEV)
    capped = torch.tensor([600, 600, 600], dtype=torch.int32, device=DEV)
    a = tk.taskkv_decode_noalloc(q, k, v, off, over, group=G, max_len=600)
    b = tk.taskkv_decode_noalloc(q, k, v, off, capped, group=G, max_len=600)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    want = _oracle_decode(q, k, v, [600] * U, U, G)
    assert np.abs(a.double().cpu().numpy() - want).max() < TOL["f32"]


def test_noalloc_rejects_sizes_beyond_the_fixed_scratch():
    from paper_2501_15113_b200 import binding as tk
    d, G = 128, 8
    too_many = (32 << 20) // (G * (d + 2) * 4) + 1
    q = torch.zeros(too_many * G, d, device=DEV, dtype=torch.bfloat16)
    pool = torch.zeros(8, d, device=DEV, dtype=torch.bfloat16)
    off = torch.zeros(too_many, device=DEV, dtype=torch.int64)
    lens = torch.zeros(too_many, device=DEV, dtype=torch.int32)
    with pytest.raises(tk.TaskKVError) as ei:
        tk.taskkv_decode_noalloc(q, pool, pool, off, lens, group=G, max_len=16, out=q)
    assert ei.value.status == tk.EINVAL


def test_noalloc_binding_checks_shapes_and_types():
    from paper_2501_15113_b200 import binding as tk
    d, G, U = 64, 2, 2
    q = torch.zeros(U * G, d, device=DEV)
    pool = torch.zeros(16, d, device=DEV)
    off = torch.zeros(U, device=DEV, dtype=torch.int64)
    lens = torch.ones(U, device=DEV, dtype=torch.int32)
    tk.taskkv_decode_noalloc(q, pool, pool, off, lens, group=G, max_len=4)
    bad = [dict(q=q.half()), dict(q=q[:3]), dict(seg_off=off.int()), dict(lengths=lens.long()),
           dict(k_pool=pool[:, :32]), dict(k_pool=pool.cpu()), dict(q=torch.zeros(U * G, 2 * d, device=DEV)[:, :d])]
    for kw in bad:
        args = dict(q=q, k_pool=pool, v_pool=pool, seg_off=off, lengths=lens)
        args.update(kw)
        with pytest.raises(ValueError):
            tk.taskkv_decode_noalloc(args["q"], args["k_pool"], args["v_pool"], args["seg_off"], args["lengths"],
                                     group=G, max_len=4)
