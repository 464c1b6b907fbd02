"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on
the same seeded inputs, element by element."""
import numpy as np
import pytest
import torch

from oracle import taskkv_oracle as O
from paper_2501_15113_b200 import workloads as W

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _tk():
    from paper_2501_15113_b200 import binding
    return binding


def _parity():
    from tests import parity
    return parity


def run_workload(wl: W.Workload, layers=None, decode_steps=None, check_pool=True, force_class=-1,
                 check_scores=True, decode_layers=None, expect_class_ties=(), page_rows=0):
    """Compress + decode on the GPU, oracle on the chosen (b, r) pairs, compare everything.  Decode outputs are
    compared on `decode_layers` (default: every chosen pair).  Ends with the bounds every test must keep: no class
    near-tie except at the (b, r) named in `expect_class_ties`, boundary ties within one per 10,000 selections.
    With page_rows > 0 the cache is a paged one in a pool with room for exactly the pages the run takes."""
    import os
    tk, P = _tk(), _parity()
    qs, ks, vs = W.materialize(wl, DEV)
    steps = wl.decode_steps if decode_steps is None else decode_steps
    params = tk.params_from_workload(wl, max_new_tokens=steps, force_class=force_class)
    pool = None
    if page_rows:
        # exactly the pages of the compression plus those the decode steps open
        info, pages = tk.taskkv_plan_paged(params, page_rows)
        lens0 = []
        for b in range(wl.batch):
            for r in range(wl.n_layers):
                full = min(wl.n_kv_heads, wl.n_hetero[b][r] + (1 if wl.promote_center else 0))
                lens0 += [wl.seq_lens[b]] * full + [wl.kept_len(b, r)] * (wl.n_kv_heads - full)
        grow = sum(-(-(x + steps) // page_rows) - -(-x // page_rows) for x in lens0)
        assert pages == sum(-(-x // page_rows) for x in lens0)
        pool = tk.Pool(page_rows, pages + grow, wl.head_dim, wl.dtype, DEV)
        cache = tk.taskkv_compress_paged(params, qs, ks, vs, pool)
        assert pool.free_pages() == grow
    else:
        cache = tk.taskkv_compress_ex(params, qs, ks, vs)
    assert cache.status() == 0
    rep = P.Report()
    scores = cache.query(tk.Q_SCORES) if check_scores else None
    topt = cache.query(tk.Q_TOPT)
    pairs = layers if layers is not None else [(b, r) for b in range(wl.batch) for r in range(wl.n_layers)]
    dec_pairs = pairs if decode_layers is None else decode_layers
    checks = {}
    for (b, r) in pairs:
        ref = P.oracle_layer(wl, b, r, qs[b][r], ks[b][r], vs[b][r], force_class=force_class)
        checks[(b, r)] = P.compare_layer(cache, wl, b, r, ref, rep, scores=scores, topt=topt, v=vs[b][r],
                                         force_class=force_class)
        if check_pool:
            P.compare_pool_rows(cache, wl, b, r, ks[b][r], vs[b][r])
        del ref
    # totals the host planned must match what the device produced
    off = cache.query(tk.Q_OFFSETS)
    cap = cache.query(tk.Q_CAPACITY)
    assert pool is not None or off[-1] == cache.info.pool_rows == int(cap.sum())
    assert int(cache.lengths().sum()) == cache.info.retained_rows == wl.retained_rows() or force_class != -1

    # decode: append + attend, every step compared on the chosen layers
    step_inputs = [W.gen_decode_step(wl, s, DEV) for s in range(steps)]
    outs = []
    for (q, kn, vn) in step_inputs:
        cache.taskkv_append(kn, vn)
        outs.append(cache.taskkv_decode(q))
    assert cache.status() == 0
    tol = P.TOL_OUT[wl.dtype]
    G = wl.group
    for (b, r) in dec_pairs:
        chk = checks[(b, r)]
        want = P.oracle_decode_steps(wl, b, r, ks[b][r], vs[b][r], chk.idx, step_inputs)
        heads = [a for a in range(wl.n_heads) if a // G not in chk.skip_heads]    # a class near-tie leaves its heads out
        for s in range(steps):
            err = float(np.abs(P.to64(outs[s][b, r]) - want[s])[heads].max()) if heads else 0.0
            rep.max_out_abs = max(rep.max_out_abs, err)
            assert err < tol, f"decode step {s} (b={b}, r={r}): max abs err {err:.3e} >= {tol}"
    lens = cache.lengths()
    assert int(lens.sum()) == int(cache.info.retained_rows) + steps * int(cache.info.n_units) or force_class != -1
    print(f"\n[{wl.name}] {rep.summary()}")
    if pool is not None:
        assert pool.free_pages() == 0            # the run took every page, by the host's count and on the device
    cache.close()
    if pool is not None:
        assert pool.free_pages() == pool.n_pages
        pool.close()
    P.write_report(os.environ.get("PYTEST_CURRENT_TEST", wl.name).split(" ")[0], rep)
    rep.check_bounds(wl.name, expect_class_ties)
    return rep


def small(name, *, n, n_kv, d, N, L, s1, s2, k, dtype, R=1, B=1, t=256, pool=7, nh=1, steps=3, seed=11,
          variance=None, seq_lens=None, promote=True):
    lens = seq_lens if seq_lens is not None else [N] * B
    wl = W.Workload(name=name, batch=len(lens), n_layers=R, n_heads=n, n_kv_heads=n_kv, head_dim=d, seq_lens=lens,
                    dtype=dtype, sink=s1, recent=s2, window=L, mid_budget=[k] * R,
                    n_hetero=[[nh] * R for _ in lens], decode_steps=steps, top_t=t, pool_kernel=pool,
                    promote_center=promote, seed=seed,
                    variance=variance if variance is not None else (1.0 if dtype == "f32" else 1.0 / np.sqrt(d)),
                    plant_offset=1.0)
    wl.planted = W._choose_planted(wl)
    return wl


def test_toy_config_exact():
    """Config 1: MHA 8 x 64, 512 tokens, fp32, planted heads 2 and 5, 16 decode steps."""
    wl = W.toy()
    rep = run_workload(wl)
    assert rep.topt_ties == 0 and rep.mid_ties == 0


def test_toy_config_without_pooling():
    wl = W.toy()
    wl.pool_kernel = 1
    run_workload(wl)


CASES = [
    # tiles and ragged tails, both dtypes and head dims
    dict(n=4, n_kv=4, d=128, N=2341, L=32, s1=4, s2=64, k=100, dtype="bf16"),
    dict(n=4, n_kv=4, d=64, N=1500, L=16, s1=4, s2=32, k=77, dtype="bf16"),
    dict(n=4, n_kv=4, d=128, N=1283, L=16, s1=3, s2=50, k=64, dtype="f32"),
    dict(n=4, n_kv=4, d=64, N=3000, L=32, s1=0, s2=17, k=129, dtype="f32"),
    dict(n=4, n_kv=4, d=64, N=5000, L=32, s1=4, s2=64, k=300, dtype="bf16"),       # tensor-core path, d = 64
    dict(n=8, n_kv=2, d=128, N=6500, L=32, s1=4, s2=64, k=300, dtype="bf16", nh=0),  # 128 window rows, 4 chunks
    dict(n=4, n_kv=2, d=128, N=4097, L=32, s1=4, s2=64, k=300, dtype="bf16", nh=0),  # 64 window rows
    # grouped queries: G = 2, 4, 8 and a single KV head
    dict(n=8, n_kv=4, d=128, N=1100, L=32, s1=4, s2=64, k=50, dtype="bf16"),
    dict(n=16, n_kv=4, d=128, N=2100, L=32, s1=4, s2=64, k=50, dtype="bf16"),
    dict(n=16, n_kv=2, d=64, N=900, L=16, s1=4, s2=64, k=50, dtype="f32", nh=0),
    dict(n=4, n_kv=1, d=128, N=700, L=32, s1=4, s2=64, k=50, dtype="bf16", nh=0),
    # bf16 decode through warp mma: G = 8 and G = 2 at both head dims; segment lengths that end inside a 16-row block
    dict(n=16, n_kv=2, d=64, N=1303, L=16, s1=4, s2=64, k=51, dtype="bf16", nh=0),   # G = 8, d = 64, 128 window rows
    dict(n=8, n_kv=1, d=128, N=811, L=16, s1=4, s2=64, k=37, dtype="bf16", nh=0),    # G = 8, d = 128
    dict(n=8, n_kv=4, d=64, N=1000, L=16, s1=3, s2=30, k=45, dtype="bf16"),          # G = 2, d = 64
    # degenerate budgets and windows
    dict(n=4, n_kv=4, d=64, N=90, L=8, s1=40, s2=60, k=10, dtype="f32"),          # N <= sink + recent
    dict(n=4, n_kv=4, d=64, N=600, L=8, s1=4, s2=32, k=0, dtype="f32"),           # no middle activations
    dict(n=4, n_kv=4, d=64, N=600, L=8, s1=4, s2=32, k=10 ** 6, dtype="bf16"),    # budget covers the middle
    dict(n=4, n_kv=4, d=64, N=200, L=8, s1=4, s2=32, k=20, dtype="f32", t=1000),  # t >= N
    dict(n=4, n_kv=4, d=64, N=300, L=1, s1=4, s2=32, k=20, dtype="f32"),          # one-row window
    dict(n=2, n_kv=2, d=64, N=128, L=128, s1=4, s2=32, k=20, dtype="f32", nh=0),  # window = whole sequence
    dict(n=4, n_kv=4, d=64, N=1000, L=8, s1=4, s2=32, k=20, dtype="bf16", nh=4),  # every head heterogeneous
    dict(n=4, n_kv=4, d=64, N=1000, L=8, s1=4, s2=32, k=20, dtype="bf16", nh=0, promote=False),
    # several layers and a ragged batch
    dict(n=16, n_kv=4, d=128, N=0, L=32, s1=4, s2=128, k=256, dtype="bf16", R=3, seq_lens=[1500, 2049, 1024], nh=1),
    # pooling kernels other than 1 and 7 take the streaming selection: all keys collected at once / after some steps
    dict(n=4, n_kv=4, d=64, N=1900, L=16, s1=4, s2=32, k=77, dtype="bf16", pool=5),
    dict(n=4, n_kv=4, d=64, N=9000, L=16, s1=5, s2=33, k=1500, dtype="f32", pool=3),
]


@pytest.mark.parametrize("case", CASES, ids=[f"case{i}" for i in range(len(CASES))])
def test_shapes_and_edge_cases(case):
    wl = small("case", **case)
    run_workload(wl)


def test_every_head_heterogeneous_is_full_attention():
    """force_class = 1: the cache is the whole K/V and decode is textbook attention."""
    wl = small("full", n=8, n_kv=4, d=128, N=1111, L=32, s1=4, s2=64, k=50, dtype="bf16")
    tk = _tk()
    qs, ks, vs = W.materialize(wl, DEV)
    params = tk.params_from_workload(wl, max_new_tokens=0, force_class=1)
    cache = tk.taskkv_compress_ex(params, qs, ks, vs)
    assert cache.lengths().tolist() == [1111] * 4 and cache.classes().tolist() == [1] * 4
    q, _, _ = W.gen_decode_step(wl, 0, DEV)
    out = cache.taskkv_decode(q)
    ref = torch.nn.functional.scaled_dot_product_attention(
        q[0, 0].double().cpu().reshape(4, 2, 128), ks[0][0].double().cpu(), vs[0][0].double().cpu())
    err = (out[0, 0].double().cpu() - ref.reshape(8, 128)).abs().max().item()
    assert err < 2e-2


def test_decode_prefix_lengths():
    """A caller-supplied lengths array attends over a prefix of every segment."""
    tk, P = _tk(), _parity()
    wl = small("prefix", n=4, n_kv=4, d=64, N=700, L=8, s1=4, s2=32, k=20, dtype="f32")
    qs, ks, vs = W.materialize(wl, DEV)
    cache = tk.taskkv_compress_ex(tk.params_from_workload(wl, max_new_tokens=0), qs, ks, vs)
    lens = cache.lengths()
    pre = np.maximum(1, lens // 3).astype(np.int32)
    q, _, _ = W.gen_decode_step(wl, 0, DEV)
    out = cache.taskkv_decode(q, lengths=torch.from_numpy(pre).to(DEV))
    ref = P.oracle_layer(wl, 0, 0, qs[0][0], ks[0][0], vs[0][0])
    kc, vc = O.gather_cache(P.to64(ks[0][0]), P.to64(vs[0][0]), ref["idx"])
    kc = [kc[u][:pre[u]] for u in range(4)]
    vc = [vc[u][:pre[u]] for u in range(4)]
    want = O.decode_layer(P.to64(q[0, 0]), kc, vc)
    assert np.abs(P.to64(out[0, 0]) - want).max() < 1e-5


def test_append_beyond_capacity_sets_status():
    tk = _tk()
    wl = small("cap", n=4, n_kv=4, d=64, N=300, L=8, s1=4, s2=32, k=20, dtype="f32")
    qs, ks, vs = W.materialize(wl, DEV)
    cache = tk.taskkv_compress_ex(tk.params_from_workload(wl, max_new_tokens=1), qs, ks, vs)
    _, kn, vn = W.gen_decode_step(wl, 0, DEV)
    cache.taskkv_append(kn, vn)
    assert cache.status() == 0
    before = cache.lengths().copy()
    cache.taskkv_append(kn, vn)
    assert cache.status() == tk.ESTATE
    assert cache.lengths().tolist() == before.tolist()


def test_compress_is_deterministic():
    tk = _tk()
    wl = small("det", n=8, n_kv=4, d=128, N=3333, L=32, s1=4, s2=64, k=200, dtype="bf16", R=2)
    qs, ks, vs = W.materialize(wl, DEV)
    res = []
    for _ in range(2):
        cache = tk.taskkv_compress_ex(tk.params_from_workload(wl, max_new_tokens=0), qs, ks, vs)
        res.append((cache.query(tk.Q_SCORES).copy(), cache.query(tk.Q_SEMVEC).copy(),
                    cache.query(tk.Q_INDICES).copy(), cache.lengths().copy()))
        cache.close()
    for a, b in zip(res[0], res[1]):
        assert np.array_equal(a, b)


def test_flat_entry_point_and_host_buffers():
    """taskkv_compress (flat form) and the host-buffer calls give the same cache as the _ex call."""
    tk = _tk()
    wl = small("flat", n=8, n_kv=8, d=128, N=2000, L=32, s1=16, s2=256, k=100, dtype="bf16", R=2, nh=2)
    # the flat call applies Eq. 16 itself: beta .25, m 4 over 8 heads and 2 layers -> 2 then 4
    wl.n_hetero = [[tk.taskkv_hetero_count(8, 0.25, 4, 2, r) for r in range(2)]]
    qs, ks, vs = W.materialize(wl, DEV)
    ref = tk.taskkv_compress_ex(tk.params_from_workload(wl, max_new_tokens=4096), qs, ks, vs)
    flat = tk.taskkv_compress(qs[0], ks[0], vs[0], sink=16, recent=256, mid_budget=100, window=32)
    params = tk.params_from_workload(wl, max_new_tokens=4096)
    host = tk.taskkv_compress_host(params, [t.cpu().pin_memory() for t in qs], [t.cpu().pin_memory() for t in ks],
                                   [t.cpu().pin_memory() for t in vs])
    for other in (flat, host):
        assert other.lengths().tolist() == ref.lengths().tolist()
        assert other.classes().tolist() == ref.classes().tolist()
        assert np.array_equal(other.query(tk.Q_SEMVEC), ref.query(tk.Q_SEMVEC))
    q, kn, vn = W.gen_decode_step(wl, 0, DEV)
    ref.taskkv_append(kn, vn)
    want = ref.taskkv_decode(q)
    out_h = torch.empty(q.shape, dtype=q.dtype).pin_memory()
    host.taskkv_decode_host(q.cpu().pin_memory(), kn.cpu().pin_memory(), vn.cpu().pin_memory(), out_h)
    assert torch.equal(out_h, want.cpu())


# ---------------------------------------------------------------- the benchmark workloads
def test_llama2_config_full_size_every_layer():
    """Config 2 at full size (32 layers, 32 heads x 128, 32768 tokens, bf16), in the launch configuration
    bench.py times; the oracle checks every stage of every layer (1024 units), then 16 decode steps on eight
    layers spread over the stack."""
    from paper_2501_15113_b200 import configs
    wl = configs.config2_llama2()
    rep = run_workload(wl, decode_steps=16, check_pool=False,
                       decode_layers=[(0, r) for r in (0, 4, 9, 13, 18, 22, 27, 31)])
    assert rep.units == 1024


def test_llama3_config_full_size_sampled_layers():
    """Config 3 at full size (32 layers, 32 query / 8 KV heads, 131072 tokens, bf16, 40 % budget), in the launch
    configuration bench.py times: 128 window rows, cluster selection, warp-mma decode with four heads per KV
    head.  The oracle checks seven layers, on both sides of the change of budget (Eq. 16 gives 2 far heads up to
    layer 19, then 1), then four decode steps on three of them."""
    from paper_2501_15113_b200 import configs
    wl = configs.config3_llama3()
    assert wl.n_hetero[0][19] == 2 and wl.n_hetero[0][20] == 1
    rep = run_workload(wl, layers=[(0, r) for r in (0, 1, 10, 19, 20, 30, 31)], decode_steps=4, check_pool=False,
                       decode_layers=[(0, 1), (0, 19), (0, 30)])
    assert rep.units == 56


@pytest.mark.parametrize("n_hetero,mid", [(0, 64), (0, 1024), (2, 256), (8, 64), (8, 1024)])
def test_sweep_config_full_size_corner_points(n_hetero, mid):
    """Config 5 at full size (8 sequences of 65536 tokens, one layer): the four corners of planted fraction x
    middle budget and the centre point; the oracle checks two of the sequences."""
    from paper_2501_15113_b200 import configs
    wl = configs.config5_sweep(n_hetero, mid, decode_steps=2)
    run_workload(wl, layers=[(0, 0), (5, 0)], decode_steps=2, check_pool=False)


def test_mistral_config_full_size_every_sequence():
    """Config 4 at full size (16 ragged sequences of 8192-32768 tokens, 32 layers, grouped queries): the oracle
    checks every sequence at layer 17 and three more (sequence, layer) pairs, then two decode steps on four pairs."""
    from paper_2501_15113_b200 import configs
    wl = configs.config4_mistral(decode_steps=2)
    pairs = [(b, 17) for b in range(wl.batch)] + [(0, 0), (7, 5), (15, 31)]
    rep = run_workload(wl, layers=pairs, decode_steps=2, check_pool=False,
                       decode_layers=[(0, 0), (3, 17), (7, 5), (15, 31)])
    assert rep.units == 19 * 8


def test_mistral_config_full_size_paged_cache():
    """Config 4 at full size in a paged cache (256-row pages, the pool holding exactly the pages the run takes):
    the oracle checks six (sequence, layer) pairs, rows read back through the page tables included, then three
    decode steps (append + attention, units opening new pages) on three of them."""
    from paper_2501_15113_b200 import configs
    wl = configs.config4_mistral(decode_steps=3)
    pairs = [(0, 0), (3, 17), (7, 5), (9, 30), (12, 1), (15, 31)]
    rep = run_workload(wl, layers=pairs, decode_steps=3, check_pool=True, decode_layers=[(3, 17), (9, 30), (15, 31)],
                       page_rows=256)
    assert rep.units == 6 * 8


def test_llama2_config_full_size_paged_cache_small_pages():
    """Config 2 at full size in a paged cache of 64-row pages (the smallest), four layers checked by the oracle with
    the rows read back through the page tables, 70 decode steps so that every unit opens at least one page."""
    from paper_2501_15113_b200 import configs
    wl = configs.config2_llama2()
    rep = run_workload(wl, layers=[(0, r) for r in (0, 11, 20, 31)], decode_steps=70, check_pool=True,
                       decode_layers=[(0, 11), (0, 31)], page_rows=64)
    assert rep.units == 4 * 32


def test_llama3_shaped_gqa_with_budget_schedule():
    """Config 3 scaled down: GQA 32q / 8kv, Eq. 16 schedule over the KV heads, Eq. 17 budgets for a 40 %
    cache, 128 window rows on the tensor-core path."""
    from paper_2501_15113_b200 import configs
    wl = configs.config3_llama3(seq_len=12000, n_layers=3, decode_steps=3)
    assert wl.n_hetero[0] == [2, 2, 1] and len(set(wl.mid_budget)) == 2
    run_workload(wl)
    full = wl.n_layers * wl.n_kv_heads * wl.seq_lens[0]
    assert 0.39 < wl.retained_rows() / full <= 0.4


def test_long_sequence_streaming_select_path():
    """More than 32768 keys per unit with a pooling kernel other than 1 and 7: the selection streams the keys from
    L2 once per bisection step."""
    wl = small("long", n=8, n_kv=2, d=128, N=40000, L=32, s1=4, s2=256, k=1500, dtype="bf16", nh=0, steps=2, pool=5)
    run_workload(wl, check_pool=False)


CLUSTER_SELECT_CASES = [
    # 32768 < N <= 262144: a thread-block cluster of 2, 4 or 8 CTAs keeps a unit's keys in registers
    dict(n=8, n_kv=2, d=128, N=40000, L=32, s1=4, s2=256, k=1500, dtype="bf16", nh=0),                  # 2 CTAs
    dict(n=2, n_kv=2, d=64, N=70001, L=32, s1=4, s2=256, k=36000, dtype="bf16", nh=0),                  # 4, k > one CTA
    dict(n=2, n_kv=2, d=64, N=98304, L=32, s1=16, s2=300, k=700, dtype="bf16", nh=0, pool=1, t=100),    # 4, 3 of them used
    dict(n=2, n_kv=1, d=64, N=140000, L=16, s1=4, s2=256, k=5000, dtype="bf16", nh=0),                  # 8 CTAs
    # ragged batch: the cluster size follows the longest sequence, the short one leaves CTAs without a key
    dict(n=4, n_kv=4, d=64, N=0, L=32, s1=4, s2=128, k=900, dtype="bf16", R=2, seq_lens=[50000, 3000, 33000], nh=1),
    dict(n=2, n_kv=2, d=64, N=33000, L=8, s1=4, s2=64, k=200, dtype="f32", nh=1),
]


@pytest.mark.parametrize("case", CLUSTER_SELECT_CASES, ids=[f"case{i}" for i in range(len(CLUSTER_SELECT_CASES))])
def test_cluster_select(case):
    wl = small("cluster_select", **case, steps=1)
    run_workload(wl, check_pool=False)


def test_sequence_longer_than_a_cluster_holds_streams_its_keys():
    """N > 262144: more keys than the largest cluster keeps in registers; the selection streams them from L2 once per
    bisection step (select_kernel), the window scores take their two-pass path with 129 work items per unit, and the
    decode splits the full head into 517 work items."""
    wl = small("very_long", n=2, n_kv=2, d=64, N=264500, L=16, s1=4, s2=200, k=3000, dtype="bf16", nh=0, steps=2)
    run_workload(wl, check_pool=False)


def test_cluster_select_equal_scores_keep_the_lower_positions():
    """All keys of a head equal: every score before the window is the same number (on the GPU and in the oracle
    alike), so both selections are decided by position alone, and the run of equal keys that is kept crosses from one
    CTA of the cluster into the next (36000 middle positions, 32768 keys per CTA)."""
    tk = _tk()
    N, k, s1, s2 = 70000, 36000, 4, 256
    wl = small("equal", n=2, n_kv=2, d=64, N=N, L=32, s1=s1, s2=s2, k=k, dtype="bf16", nh=0, steps=0, promote=False)
    qs, ks, vs = W.materialize(wl, DEV)
    for h in range(2):
        ks[0][0][h][:] = ks[0][0][h][0:1].clone()
    cache = tk.taskkv_compress_ex(tk.params_from_workload(wl, max_new_tokens=0), qs, ks, vs)
    assert cache.status() == 0
    topt = cache.query(tk.Q_TOPT)
    idx = cache.query(tk.Q_INDICES)
    lens = cache.lengths()
    want = list(range(s1 + k)) + list(range(N - s2, N))
    for u in range(2):
        assert topt[u].tolist() == list(range(256))
        assert lens[u] == s1 + k + s2
        assert idx[u, :lens[u]].tolist() == want
    cache.close()


def test_mistral_shaped_ragged_batch():
    """Config 4 scaled down: a ragged batch with a different number of heterogeneous heads per sequence."""
    from paper_2501_15113_b200 import configs
    wl = configs.config4_mistral(batch=4, lo=1500, hi=5000, n_layers=2, decode_steps=3)
    assert len(set(wl.seq_lens)) > 1
    run_workload(wl)


@pytest.mark.parametrize("case", [
    dict(n=8, n_kv=8, d=128, N=0, L=32, s1=4, s2=64, k=120, dtype="bf16", R=4, seq_lens=[9000, 7001, 12345], nh=2),
    dict(n=8, n_kv=4, d=64, N=0, L=32, s1=4, s2=64, k=120, dtype="bf16", R=6, seq_lens=[16384, 15000], nh=1),
], ids=["32rows_ragged", "64rows_d64"])
def test_window_scores_many_items_per_cta(case):
    """Large enough for every CTA of the window-score kernel to run through several work items of several
    sequences: ragged ends, units that straddle the grid, both tensor-core row counts below 128."""
    wl = small("rounds", **case, steps=1)
    run_workload(wl, layers=[(b, r) for b in range(wl.batch) for r in (0, wl.n_layers - 1)])


SINGLE_READ_CASES = [
    # cluster sizes 2, 4, 8, 16 of the kernel that keeps a unit's scores in tensor memory; slices of unequal
    # tile counts, ragged last tiles, a last tile shorter than the window
    dict(n=4, n_kv=4, d=128, N=4000, L=32, s1=4, s2=64, k=100, dtype="bf16"),
    dict(n=4, n_kv=4, d=128, N=8200, L=32, s1=4, s2=64, k=100, dtype="bf16"),
    dict(n=4, n_kv=4, d=64, N=16397, L=32, s1=4, s2=64, k=300, dtype="bf16"),
    dict(n=2, n_kv=2, d=128, N=32768, L=32, s1=4, s2=256, k=512, dtype="bf16"),
    dict(n=2, n_kv=2, d=128, N=30001, L=32, s1=4, s2=256, k=512, dtype="bf16", nh=0),
    # two query heads per KV head with a 16-row window: 32 rows, causal limit by row % 16
    dict(n=8, n_kv=4, d=128, N=5003, L=16, s1=4, s2=64, k=100, dtype="bf16"),
    # four query heads per KV head with an 8-row window
    dict(n=8, n_kv=2, d=64, N=2500, L=8, s1=4, s2=64, k=100, dtype="bf16", nh=0),
    # a batch whose sequences need different slice sizes in one launch, more units than clusters
    dict(n=8, n_kv=8, d=128, N=0, L=32, s1=4, s2=64, k=120, dtype="bf16", R=3, seq_lens=[9000, 300, 16000, 2100], nh=2),
]


@pytest.mark.parametrize("case", SINGLE_READ_CASES, ids=[f"case{i}" for i in range(len(SINGLE_READ_CASES))])
def test_window_scores_single_read(case):
    wl = small("single_read", **case, steps=1)
    run_workload(wl, layers=[(b, r) for b in range(wl.batch) for r in (0, wl.n_layers - 1)])


def test_window_scores_single_read_batch_of_ten_sequences():
    """More sequences than one launch of the single-read kernel takes (eight), of very different lengths: the cluster
    size follows the longest, short sequences leave most CTAs of a cluster without a tile."""
    lens = [300, 9000, 1500, 4097, 129, 2048, 7000, 640, 5121, 3333]
    wl = small("ten", n=4, n_kv=4, d=128, N=0, L=32, s1=4, s2=64, k=60, dtype="bf16", seq_lens=lens, steps=1)
    run_workload(wl)


def test_window_scores_and_selection_overlapped_by_layer_chunks():
    """Enough units for the library to cut the layers into chunks and run the selection of one chunk beside the
    window scores of the next (a side stream): two ragged sequences, 16 layers x 32 heads, so 4 chunks of 4 layers.
    Layers of every chunk and both sequences are checked, the chunk borders included."""
    wl = small("chunks", n=32, n_kv=32, d=64, N=0, L=32, s1=4, s2=64, k=90, dtype="bf16", R=16,
               seq_lens=[1500, 2100], nh=3, steps=1)
    run_workload(wl, layers=[(b, r) for b in range(2) for r in (0, 3, 4, 8, 11, 12, 15)])


def test_overlapped_compression_equals_the_one_launch_order_bit_for_bit():
    """The chunked, two-stream order of window scores and selection against the plain order (one launch each over all
    layers, which the library takes while per-kernel timing is switched on): scores, top-t lists, semantic vectors,
    classes, lengths, retained positions and both pools must be the same bits, three times in a row, also when the
    caller's stream is not the default one.  A race between the two streams would show here."""
    tk = _tk()
    wl = small("chunks_bits", n=32, n_kv=32, d=128, N=0, L=32, s1=4, s2=64, k=150, dtype="bf16", R=8,
               seq_lens=[2500, 1100], nh=2, steps=0)
    qs, ks, vs = W.materialize(wl, DEV)
    what = (tk.Q_SCORES, tk.Q_TOPT, tk.Q_SEMVEC, tk.Q_CLASSES, tk.Q_LENGTHS, tk.Q_INDICES, tk.Q_KPOOL, tk.Q_VPOOL)

    def run(stream=None):
        params = tk.params_from_workload(wl, max_new_tokens=0)
        if stream is None:
            cache = tk.taskkv_compress_ex(params, qs, ks, vs)
        else:
            with torch.cuda.stream(stream):
                cache = tk.taskkv_compress_ex(params, qs, ks, vs)
            stream.synchronize()
        assert cache.status() == 0
        got = [cache.query(w).copy() for w in what]
        lens, idx = got[4], got[5]
        for u in range(idx.shape[0]):
            idx[u, min(lens[u], wl.sink + 150 + wl.recent):] = -1   # slots past sinks + middle + recent are never written
        cache.close()
        return got

    tk.taskkv_timing_enable(True)
    try:
        plain = run()
    finally:
        tk.taskkv_timing_enable(False)
        tk.taskkv_timing_collect()
    side = torch.cuda.Stream()
    for stream in (None, side, None):
        for a, b in zip(plain, run(stream)):
            assert np.array_equal(a, b)


def test_window_scores_single_read_moderate_heavy_keys():
    """A few keys per head well above the rest (scores stay within fp32 range of one another): full parity."""
    wl = small("heavy", n=4, n_kv=4, d=128, N=9000, L=32, s1=4, s2=64, k=100, dtype="bf16", steps=1)
    wl.heavy_keys, wl.heavy_scale = 5, 6.0
    run_workload(wl)


def test_window_scores_single_read_extreme_keys_fall_back_to_exact_maxima():
    """Keys hundreds of score units above the rest: a warp's running sums, taken relative to an ordinary key,
    overflow and the warp redoes its tiles with its exact row maxima.  Almost all of the softmax mass sits on a few
    keys, the rest is below fp32 range, so only the scores are compared here (absolute, against the largest)."""
    tk, P = _tk(), _parity()
    from oracle import taskkv_oracle as O
    wl = small("extreme", n=2, n_kv=2, d=128, N=9000, L=32, s1=4, s2=64, k=100, dtype="bf16", steps=0, nh=0)
    wl.heavy_keys, wl.heavy_scale = 5, 600.0
    qs, ks, vs = W.materialize(wl, DEV)
    cache = tk.taskkv_compress_ex(tk.params_from_workload(wl, max_new_tokens=0), qs, ks, vs)
    assert cache.status() == 0
    got = cache.query(tk.Q_SCORES).astype(np.float64)
    off = P.score_offsets(wl)
    spread = 0.0
    for h in range(wl.n_kv_heads):
        q64, k64 = P.to64(qs[0][0][h:h + 1]), P.to64(ks[0][0][h])
        s = (q64[0] @ k64.T) / np.sqrt(wl.head_dim)
        spread = max(spread, float(s.max() - np.median(s)))
        want = O.window_scores(q64, k64)
        c = got[off[h]:off[h] + wl.seq_lens[0]]
        assert np.isfinite(c).all()
        # scores of several hundred: the fp32 rounding of a score (relative 6e-8 per operation) is ~1e-4 absolute in
        # the exponent, hence the wider bound than for ordinary inputs
        assert np.abs(c - want).max() < 1e-3 * want.max()
        assert abs(c.sum() - 1.0) < 1e-3
    assert spread > 150.0      # beyond what exp2 in fp32 holds relative to an ordinary key: the fast path cannot apply
    cache.close()


def test_ragged_batch_of_eleven_sequences():
    """More sequences than one window-score launch takes (eight): a full group and a partial one."""
    from paper_2501_15113_b200 import configs
    wl = configs.config4_mistral(batch=11, lo=700, hi=2600, n_layers=1, decode_steps=2)
    run_workload(wl)


@pytest.mark.parametrize("n_hetero,mid", [(h, k) for h in W.SWEEP_HETERO for k in W.SWEEP_MID])
def test_budget_sweep_points(n_hetero, mid):
    """Config 5 scaled down, all 15 points: planted fraction (0, 1, 2, 4, 8 of 8 heads) x middle budget (64, 256, 1024)."""
    from paper_2501_15113_b200 import configs
    wl = configs.config5_sweep(n_hetero, mid, seq_len=5000, batch=2, decode_steps=2)
    rep = run_workload(wl)
    assert rep.units == 16


# ---------------------------------------------------------------------------
# Sec. V-G: the other two compensation methods at the same cache size
# ---------------------------------------------------------------------------
POLICY_CASES = [
    dict(n=4, n_kv=4, d=64, N=1500, L=16, s1=4, s2=32, k=37, dtype="f32"),
    dict(n=4, n_kv=4, d=128, N=2341, L=32, s1=4, s2=64, k=100, dtype="bf16"),
    dict(n=8, n_kv=2, d=128, N=3000, L=32, s1=3, s2=50, k=64, dtype="bf16", nh=0),      # grouped queries
    dict(n=4, n_kv=4, d=64, N=700, L=8, s1=4, s2=32, k=0, dtype="bf16"),                # cache size 0
    dict(n=4, n_kv=4, d=64, N=700, L=8, s1=4, s2=32, k=663, dtype="f32"),               # groups of one or two rows
    dict(n=4, n_kv=4, d=64, N=700, L=8, s1=4, s2=32, k=10 ** 6, dtype="bf16"),          # budget covers the middle
    dict(n=8, n_kv=4, d=128, N=0, L=32, s1=4, s2=128, k=200, dtype="bf16", R=2, seq_lens=[1500, 2049], nh=1),
]


@pytest.mark.parametrize("policy", [1, 2], ids=["recent", "mean"])
@pytest.mark.parametrize("case", POLICY_CASES, ids=[f"case{i}" for i in range(len(POLICY_CASES))])
def test_compensation_policies(case, policy):
    tk, P = _tk(), _parity()
    from oracle import taskkv_oracle as O
    wl = small("policy", **case)
    qs, ks, vs = W.materialize(wl, DEV)
    steps = wl.decode_steps
    params = tk.params_from_workload(wl, max_new_tokens=steps, mid_policy=policy)
    cache = tk.taskkv_compress_ex(params, qs, ks, vs)
    assert cache.status() == 0
    lens, cls, idx_tab = cache.lengths(), cache.classes(), cache.query(tk.Q_INDICES)
    step_inputs = [W.gen_decode_step(wl, s, DEV) for s in range(steps)]
    outs = []
    for (q, kn, vn) in step_inputs:
        cache.taskkv_append(kn, vn)
        outs.append(cache.taskkv_decode(q))
    assert cache.status() == 0
    ulp = 2.0 ** -7 if wl.dtype == "bf16" else 1e-6      # one unit in the last place of the stored row
    worst = 0.0
    for b in range(wl.batch):
        N = wl.seq_lens[b]
        for r in range(wl.n_layers):
            k64, v64 = P.to64(ks[b][r]), P.to64(vs[b][r])
            ref = O.compress_layer(P.to64(qs[b][r]), k64, v64, n_hetero=wl.n_hetero[b][r], sink=wl.sink,
                                   recent=wl.recent, mid=wl.mid_of(b, r), top_t=wl.top_t,
                                   pool_kernel=wl.pool_kernel, promote_center=wl.promote_center, mid_policy=policy)
            u0 = P.unit_index(wl, b, r, 0)
            assert cls[u0:u0 + wl.n_kv_heads].tolist() == ref["cls"].tolist()
            assert lens[u0:u0 + wl.n_kv_heads].tolist() == ref["len"].tolist()
            kc, vc = O.gather_cache_policy(k64, v64, ref["cls"], ref["idx"], mid_policy=policy, sink=wl.sink,
                                           recent=wl.recent, mid=wl.mid_of(b, r), dtype=wl.dtype)
            for h in range(wl.n_kv_heads):
                u = u0 + h
                if len(ref["idx"][h]) < N:      # positions (group starts for the averaged rows) are exact
                    assert idx_tab[u, :lens[u]].tolist() == ref["idx"][h].tolist()
                for name, want in (("k", kc[h]), ("v", vc[h])):
                    got = P.to64(cache.pool_rows(name, u))[:len(want)]      # rows before the appended tokens
                    exact = np.ones(len(want), dtype=bool)
                    if policy == 2 and ref["cls"][h] == 0 and len(want) < N:
                        exact[wl.sink:len(want) - wl.recent] = False
                    np.testing.assert_array_equal(got[exact], want[exact])
                    if (~exact).any():
                        err = np.abs(got[~exact] - want[~exact])
                        # fp32 sums in position order against the oracle's fp64 ones, then one rounding to storage
                        assert np.all(err <= ulp * np.abs(want[~exact]) + 1e-5), f"unit {u} {name}: averaged rows"
                        if wl.dtype == "bf16":
                            assert np.mean(err > 0) < 0.01, "more than 1 % of the averaged values differ in the last place"
            for (q, kn, vn), out in zip(step_inputs, outs):
                O.append_layer(kc, vc, P.to64(kn[b, r]), P.to64(vn[b, r]))
                want = O.decode_layer(P.to64(q[b, r]), kc, vc)
                worst = max(worst, float(np.abs(P.to64(out[b, r]) - want).max()))
    assert worst < P.TOL_OUT[wl.dtype], f"decode max abs err {worst:.3e}"
    cache.close()


# ---------------------------------------------------------------------------
# Layer-range append / decode: what a model's decode loop calls, layer after layer
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("case", [
    dict(n=8, n_kv=4, d=128, N=0, L=32, s1=4, s2=64, k=100, dtype="bf16", R=4, seq_lens=[1500, 2049, 777], nh=1),
    dict(n=4, n_kv=4, d=64, N=900, L=16, s1=4, s2=32, k=50, dtype="f32", R=3),
], ids=["bf16_gqa_ragged", "f32"])
def test_layer_by_layer_decode_equals_all_layer_decode(case):
    tk = _tk()
    wl = small("layers", **case, steps=3)
    qs, ks, vs = W.materialize(wl, DEV)
    steps = wl.decode_steps
    params = tk.params_from_workload(wl, max_new_tokens=steps)
    whole = tk.taskkv_compress_ex(params, qs, ks, vs)
    split = tk.taskkv_compress_ex(params, qs, ks, vs)
    R = wl.n_layers
    for s in range(steps):
        q, kn, vn = W.gen_decode_step(wl, s, DEV)             # [B][R][heads][d]
        whole.taskkv_append(kn, vn)
        want = whole.taskkv_decode(q)
        got = torch.empty_like(want)
        # one layer at a time, then a range of two layers starting at 1 must reproduce the same slices
        for r in range(R):
            split.taskkv_append_ex(kn[:, r:r + 1].contiguous(), vn[:, r:r + 1].contiguous(), r, 1)
            got[:, r:r + 1] = split.taskkv_decode_ex(q[:, r:r + 1].contiguous(), r, 1)
        assert torch.equal(got.view(torch.uint8), want.view(torch.uint8)), f"step {s}: per-layer outputs differ"
        pair = split.taskkv_decode_ex(q[:, 1:3].contiguous(), 1, 2)
        assert torch.equal(pair.view(torch.uint8), want[:, 1:3].contiguous().view(torch.uint8))
    assert whole.status() == 0 and split.status() == 0
    assert np.array_equal(whole.lengths(), split.lengths())
    # a prefix-length override is indexed like q: [B][layers in the call][n_kv]
    lens = torch.from_numpy(split.lengths().reshape(wl.batch, R, wl.n_kv_heads)).to(DEV)
    half = (lens[:, 2:3] // 2).to(torch.int32).contiguous()
    full_half = lens.clone().to(torch.int32)
    full_half[:, 2:3] = half
    q, _, _ = W.gen_decode_step(wl, 0, DEV)
    a = split.taskkv_decode_ex(q[:, 2:3].contiguous(), 2, 1, lengths=half)
    b = whole.taskkv_decode(q, lengths=full_half.contiguous())[:, 2:3].contiguous()
    assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
    # out-of-range layers are refused before anything is launched
    with pytest.raises(tk.TaskKVError):
        split.taskkv_decode_ex(q[:, 0:1].contiguous(), R, 1)
    with pytest.raises(tk.TaskKVError):
        split.taskkv_append_ex(q[:, 0:1].contiguous(), q[:, 0:1].contiguous(), R - 1, 2)
    whole.close()
    split.close()


def test_layer_decode_equals_all_layer_decode_with_many_work_items():
    """Layer-range calls against the all-layer call on a cache with 640 split-K work items per layer (every head keeps
    40447 rows): a layer's grid is sized by its own items, the all-layer grid by all 2560, so blocks walk the items in
    different orders; the outputs must be the same bits, for plain decode, for prefix lengths and for the fused step,
    whose appended rows sit in the last item of every unit."""
    tk = _tk()
    wl = small("by_warp", n=16, n_kv=8, d=128, N=40447, L=32, s1=4, s2=64, k=100, dtype="bf16", R=4, nh=0, steps=3)
    qs, ks, vs = W.materialize(wl, DEV)
    params = tk.params_from_workload(wl, max_new_tokens=3, force_class=1)      # every head keeps all 40447 rows
    whole = tk.taskkv_compress_ex(params, qs, ks, vs)
    split = tk.taskkv_compress_ex(params, qs, ks, vs)
    assert int(whole.info.max_decode_items) == 4 * 8 * 80          # (40447 + 3 reserved rows) / 512, rounded up
    R = wl.n_layers
    q, kn, vn = W.gen_decode_step(wl, 0, DEV)
    want = whole.taskkv_decode(q)
    for r in range(R):
        got = split.taskkv_decode_ex(q[:, r:r + 1].contiguous(), r, 1)
        assert torch.equal(got.view(torch.uint8), want[:, r:r + 1].contiguous().view(torch.uint8)), f"layer {r}"
    lens = torch.from_numpy(whole.lengths().reshape(1, R, 8)).to(DEV).to(torch.int32)
    part = (lens * 2 // 3).contiguous()
    want = whole.taskkv_decode(q, lengths=part)
    got = split.taskkv_decode_ex(q[:, 2:3].contiguous(), 2, 1, lengths=part[:, 2:3].contiguous())
    assert torch.equal(got.view(torch.uint8), want[:, 2:3].contiguous().view(torch.uint8))
    for s_ in range(3):
        q, kn, vn = W.gen_decode_step(wl, s_, DEV)
        want = whole.taskkv_decode_step(q, kn, vn)
        for r in range(R):
            got = split.taskkv_decode_step_ex(q[:, r:r + 1].contiguous(), kn[:, r:r + 1].contiguous(),
                                              vn[:, r:r + 1].contiguous(), r, 1)
            assert torch.equal(got.view(torch.uint8), want[:, r:r + 1].contiguous().view(torch.uint8)), f"step {s_} layer {r}"
        assert np.array_equal(whole.lengths(), split.lengths())
    for u in (0, 13, 31):
        for which in ("k", "v"):
            assert torch.equal(whole.pool_rows(which, u)[-4:].view(torch.uint8), split.pool_rows(which, u)[-4:].view(torch.uint8))
    assert whole.status() == 0 and split.status() == 0
    whole.close()
    split.close()


def test_one_layer_problems_equal_the_all_layer_compression():
    """Compressing layer r alone as a problem of its own (Params.layer: that layer's head count and budget) gives the same
    classes, lengths, positions, cache rows and decode outputs as the all-layer call gives for layer r."""
    tk = _tk()
    wl = small("stream", n=8, n_kv=4, d=128, N=0, L=32, s1=4, s2=64, k=90, dtype="bf16", R=3,
               seq_lens=[1400, 2100], nh=1, steps=2)
    wl.mid_budget = [90, 40, 130]
    wl.n_hetero = [[2, 1, 0], [1, 1, 2]]
    wl.planted = W._choose_planted(wl)
    qs, ks, vs = W.materialize(wl, DEV)
    params = tk.params_from_workload(wl, max_new_tokens=wl.decode_steps)
    whole = tk.taskkv_compress_ex(params, qs, ks, vs)
    q, kn, vn = W.gen_decode_step(wl, 0, DEV)
    whole.taskkv_append(kn, vn)
    want_out = whole.taskkv_decode(q)
    nkv = wl.n_kv_heads
    for r in range(wl.n_layers):
        one = tk.taskkv_compress_ex(params.layer(r), [x[r:r + 1].contiguous() for x in qs],
                                    [x[r:r + 1].contiguous() for x in ks], [x[r:r + 1].contiguous() for x in vs])
        assert one.status() == 0
        for b in range(wl.batch):
            for h in range(nkv):
                u_all = (b * wl.n_layers + r) * nkv + h
                u_one = b * nkv + h
                assert int(one.classes()[u_one]) == int(whole.classes()[u_all])
                n_all = int(whole.lengths()[u_all]) - 1          # the all-layer cache already holds one appended row
                assert int(one.lengths()[u_one]) == n_all
                for which in ("k", "v"):
                    assert torch.equal(one.pool_rows(which, u_one).view(torch.uint8),
                                       whole.pool_rows(which, u_all)[:n_all].contiguous().view(torch.uint8))
        one.taskkv_append(kn[:, r:r + 1].contiguous(), vn[:, r:r + 1].contiguous())
        got = one.taskkv_decode(q[:, r:r + 1].contiguous())
        assert torch.equal(got.view(torch.uint8), want_out[:, r:r + 1].contiguous().view(torch.uint8))
        one.close()
    whole.close()


WHAT_CACHE_HOLDS = ("Q_SEMVEC", "Q_DIST", "Q_CLASSES", "Q_LENGTHS", "Q_CAPACITY", "Q_OFFSETS", "Q_KPOOL", "Q_VPOOL")


def _cache_state(tk, cache, wl):
    """Everything a cache holds after compression, as arrays that can be compared bit for bit."""
    got = {w: cache.query(getattr(tk, w)).copy() for w in WHAT_CACHE_HOLDS}
    lens = got["Q_LENGTHS"]
    idx = cache.query(tk.Q_INDICES).copy()
    for u in range(idx.shape[0]):          # slots past a unit's retained positions are never written
        b, r = u // (wl.n_layers * wl.n_kv_heads), (u // wl.n_kv_heads) % wl.n_layers
        idx[u, min(int(lens[u]), wl.kept_len(b, r)) if lens[u] < wl.seq_lens[b] else 0:] = -1
    got["Q_INDICES"] = idx
    # of the pools only the rows a unit holds (the reserve for appended tokens is not written by compression)
    off = got["Q_OFFSETS"]
    row = wl.head_dim * wl.elem_size
    for name in ("Q_KPOOL", "Q_VPOOL"):
        raw = got[name]
        got[name] = np.concatenate([raw[int(off[u]) * row:(int(off[u]) + int(lens[u])) * row] for u in range(len(lens))])
    return got


STREAM_CASES = [
    # grouped queries, 128 window rows (two-pass tensor-core window kernel), ragged batch, layer schedules
    dict(n=8, n_kv=2, d=128, N=0, L=32, s1=4, s2=64, k=90, dtype="bf16", R=4, seq_lens=[1400, 2100, 900], nh=1),
    # one query head per KV head, 32 window rows (single-read window kernel)
    dict(n=8, n_kv=8, d=128, N=0, L=32, s1=4, s2=64, k=120, dtype="bf16", R=3, seq_lens=[3000, 4500], nh=2),
    # fp32 on the CUDA cores
    dict(n=4, n_kv=4, d=64, N=0, L=16, s1=4, s2=32, k=50, dtype="f32", R=3, seq_lens=[900, 700], nh=1),
    # 64 window rows, enough units for every CTA of the all-layer window-score launch to work through several items
    # whose tile counts are odd (9 and 19 tiles), while the per-layer launches give every CTA one item: the partial
    # row statistics must not depend on what a CTA worked on before
    dict(n=16, n_kv=8, d=64, N=0, L=32, s1=4, s2=64, k=70, dtype="bf16", R=8, seq_lens=[2400, 1150, 3300], nh=1),
]


@pytest.mark.parametrize("case", STREAM_CASES, ids=["bf16_gqa_ragged", "bf16_mha", "f32", "bf16_64rows_many_items"])
def test_layers_streamed_into_one_cache_equal_the_all_layer_call(case):
    """taskkv_cache_create + one taskkv_compress_layer per layer, in a scrambled order and with every layer's
    tensors in allocations of their own, against taskkv_compress_ex over all layers: semantic vectors, distances,
    classes, lengths, capacities, segment offsets, retained positions and both pools are the same bits; so are the
    outputs of decode steps over all layers and layer by layer.  One layer is also checked against the oracle, and
    a layer-range decode runs before the last layer is in."""
    tk, P = _tk(), _parity()
    wl = small("stream_one_cache", **case, steps=2)
    R = wl.n_layers
    wl.mid_budget = [case["k"] + 13 * r for r in range(R)]
    wl.n_hetero = [[(b + r) % (wl.n_kv_heads - 1) for r in range(R)] for b in range(wl.batch)]
    wl.planted = W._choose_planted(wl)
    qs, ks, vs = W.materialize(wl, DEV)
    params = tk.params_from_workload(wl, max_new_tokens=wl.decode_steps)
    whole = tk.taskkv_compress_ex(params, qs, ks, vs)
    want = _cache_state(tk, whole, wl)

    streamed = tk.taskkv_cache_create(params, DEV)
    assert streamed.lengths().tolist() == [0] * (wl.batch * R * wl.n_kv_heads)
    order = list(range(R))[::-1] if R != 4 else [2, 0, 3, 1]
    layer_inputs = {r: ([x[r].clone() for x in qs], [x[r].clone() for x in ks], [x[r].clone() for x in vs])
                    for r in range(R)}
    q0, kn0, vn0 = W.gen_decode_step(wl, 0, DEV)
    for i, r in enumerate(order):
        ql, kl, vl = layer_inputs.pop(r)
        streamed.taskkv_compress_layer(r, ql, kl, vl)
        torch.cuda.current_stream().synchronize()
        del ql, kl, vl                      # the caller may free a layer's K and V once the stream has passed
        if i == 0:
            # a layer that is in can be decoded while the others are still missing
            early = streamed.taskkv_decode_ex(q0[:, r:r + 1].contiguous(), r, 1)
            ref = whole.taskkv_decode_ex(q0[:, r:r + 1].contiguous(), r, 1)
            assert torch.equal(early.view(torch.uint8), ref.view(torch.uint8))
    with pytest.raises(tk.TaskKVError) as ei:
        streamed.taskkv_compress_layer(order[0], [x[order[0]].contiguous() for x in qs],
                                       [x[order[0]].contiguous() for x in ks], [x[order[0]].contiguous() for x in vs])
    assert ei.value.status == tk.ESTATE                 # a layer goes in once
    with pytest.raises(tk.TaskKVError):
        streamed.taskkv_compress_layer(R, [x[0].contiguous() for x in qs], [x[0].contiguous() for x in ks],
                                       [x[0].contiguous() for x in vs])
    assert streamed.status() == 0
    got = _cache_state(tk, streamed, wl)
    for name in want:
        assert np.array_equal(want[name], got[name]), f"{name} differs between the streamed and the all-layer cache"
    # the oracle on one (sequence, layer) of the streamed cache
    rep = P.Report()
    b, r = wl.batch - 1, order[0]
    ref = P.oracle_layer(wl, b, r, qs[b][r], ks[b][r], vs[b][r])
    P.compare_layer(streamed, wl, b, r, ref, rep, v=vs[b][r])
    rep.check_bounds(wl.name)
    # decode over the streamed cache: all layers at once, then layer by layer
    for s_ in range(wl.decode_steps):
        q, kn, vn = W.gen_decode_step(wl, s_, DEV)
        a = whole.taskkv_decode_step(q, kn, vn)
        if s_ == 0:
            bb = streamed.taskkv_decode_step(q, kn, vn)
        else:
            bb = torch.empty_like(a)
            for r in range(R):
                bb[:, r:r + 1] = streamed.taskkv_decode_step_ex(q[:, r:r + 1].contiguous(), kn[:, r:r + 1].contiguous(),
                                                                vn[:, r:r + 1].contiguous(), r, 1)
        assert torch.equal(a.view(torch.uint8), bb.view(torch.uint8)), f"decode step {s_}"
    assert np.array_equal(whole.lengths(), streamed.lengths())
    assert whole.status() == 0 and streamed.status() == 0
    whole.close()
    streamed.close()


def test_layers_streamed_on_several_streams_equal_the_all_layer_call():
    """Calls for different layers touch disjoint parts of the cache and of the workspace, so a prefill loop may issue
    them on different streams: six layers go round-robin to three streams, which are then joined; the cache must be
    the all-layer one bit for bit, three times in a row (a race between two layers' kernels would show)."""
    tk = _tk()
    wl = small("stream_streams", n=16, n_kv=4, d=128, N=0, L=32, s1=4, s2=64, k=110, dtype="bf16", R=6,
               seq_lens=[2300, 1500], nh=1, steps=1)
    wl.mid_budget = [110 + 9 * r for r in range(6)]
    qs, ks, vs = W.materialize(wl, DEV)
    params = tk.params_from_workload(wl, max_new_tokens=1)
    whole = tk.taskkv_compress_ex(params, qs, ks, vs)
    want = _cache_state(tk, whole, wl)
    ins = [([x[r].contiguous() for x in qs], [x[r].contiguous() for x in ks], [x[r].contiguous() for x in vs])
           for r in range(6)]
    streams = [torch.cuda.Stream() for _ in range(3)]
    main = torch.cuda.current_stream()
    for _ in range(3):
        cache = tk.taskkv_cache_create(params, DEV)
        created = torch.cuda.Event()
        created.record(main)
        for st in streams:
            st.wait_event(created)
        for r in range(6):
            cache.taskkv_compress_layer(r, *ins[r], stream=streams[r % 3])
        for st in streams:
            done = torch.cuda.Event()
            done.record(st)
            main.wait_event(done)
        assert cache.status() == 0
        got = _cache_state(tk, cache, wl)
        for name in want:
            assert np.array_equal(want[name], got[name]), name
        q, kn, vn = W.gen_decode_step(wl, 0, DEV)
        a = cache.taskkv_decode_step(q, kn, vn)
        cache.close()
    b = whole.taskkv_decode_step(q, kn, vn)
    assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
    whole.close()


def test_gather_overlapped_compression_equals_the_plain_order_bit_for_bit():
    """Grouped queries with enough layers for the library to cut them into chunks and gather one chunk beside the
    window scores and the selection of the next (two streams): against the plain order (one launch of every step
    over all layers, which the library takes while per-kernel timing is switched on) everything a cache holds must
    be the same bits, three times in a row, also when the caller's stream is not the default one."""
    tk = _tk()
    wl = small("gather_chunks", n=32, n_kv=8, d=128, N=0, L=32, s1=4, s2=64, k=150, dtype="bf16", R=8,
               seq_lens=[2500, 1100], nh=2, steps=0)
    wl.mid_budget = [150 + 7 * r for r in range(8)]
    qs, ks, vs = W.materialize(wl, DEV)

    def run(stream=None):
        params = tk.params_from_workload(wl, max_new_tokens=2)
        if stream is None:
            cache = tk.taskkv_compress_ex(params, qs, ks, vs)
        else:
            with torch.cuda.stream(stream):
                cache = tk.taskkv_compress_ex(params, qs, ks, vs)
            stream.synchronize()
        assert cache.status() == 0
        got = _cache_state(tk, cache, wl)
        got["scores"] = cache.query(tk.Q_SCORES).copy()
        got["topt"] = cache.query(tk.Q_TOPT).copy()
        cache.close()
        return got

    tk.taskkv_timing_enable(True)
    try:
        plain = run()
    finally:
        tk.taskkv_timing_enable(False)
        tk.taskkv_timing_collect()
    side = torch.cuda.Stream()
    for stream in (None, side, None):
        got = run(stream)
        for name in plain:
            assert np.array_equal(plain[name], got[name]), name
    # and the oracle on layers of different chunks
    run_workload(wl, layers=[(0, 0), (1, 3), (0, 4), (1, 7)], decode_steps=1)


def test_budget_given_as_a_fraction_of_the_full_cache():
    """budget_frac: the middle budget of every (sequence, layer) follows Eq. 17 from 40 % of the full cache, computed
    by the library (on the device, and by the same formula on the host for the pool sizes).  A ragged batch, so the
    budgets differ by sequence as well as by layer; the oracle is given the budgets of its own Eq. 17."""
    tk = _tk()
    wl = small("budget_frac", n=16, n_kv=8, d=128, N=0, L=32, s1=4, s2=64, k=0, dtype="bf16", R=3,
               seq_lens=[3000, 5200, 1700], nh=1, steps=2)
    wl.n_hetero = [[2, 1, 0], [1, 3, 2], [0, 0, 7]]
    wl.planted = W._choose_planted(wl)
    frac = 0.4
    wl.mid_by_seq = [[O.mid_budget(frac * 8 * wl.seq_lens[b], wl.seq_lens[b], wl.full_heads(b, r), 8, wl.sink, wl.recent)
                      for r in range(3)] for b in range(3)]
    assert len({m for row in wl.mid_by_seq for m in row}) >= 6
    wl.budget_frac = frac
    rep = run_workload(wl)
    assert rep.units == 72
    # the cache holds at most 40 % of the rows of every (sequence, layer), and misses it by less than one row per head
    for b in range(3):
        for r in range(3):
            h = wl.full_heads(b, r)
            rows = h * wl.seq_lens[b] + (8 - h) * wl.kept_len(b, r)
            if wl.mid_of(b, r) > 0:
                assert 0 <= frac * 8 * wl.seq_lens[b] - rows < 8 - h


@pytest.mark.parametrize("case", [
    dict(n=8, n_kv=2, d=128, N=0, L=32, s1=4, s2=64, k=100, dtype="bf16", R=2, seq_lens=[1500, 1023], nh=1),
    dict(n=4, n_kv=4, d=128, N=2047, L=32, s1=4, s2=64, k=60, dtype="bf16", R=2),     # appended rows cross a 512-row item
    dict(n=4, n_kv=4, d=64, N=900, L=16, s1=4, s2=32, k=50, dtype="f32", R=3),
], ids=["bf16_gqa_ragged", "bf16_item_boundary", "f32"])
def test_fused_decode_step_equals_append_then_decode(case):
    tk = _tk()
    wl = small("step", **case, steps=4)
    qs, ks, vs = W.materialize(wl, DEV)
    params = tk.params_from_workload(wl, max_new_tokens=3)          # the 4th token does not fit
    two = tk.taskkv_compress_ex(params, qs, ks, vs)
    one = tk.taskkv_compress_ex(params, qs, ks, vs)
    for s in range(3):
        q, kn, vn = W.gen_decode_step(wl, s, DEV)
        two.taskkv_append(kn, vn)
        want = two.taskkv_decode(q)
        if s == 1:      # layer by layer
            got = torch.empty_like(want)
            for r in range(wl.n_layers):
                got[:, r:r + 1] = one.taskkv_decode_step_ex(q[:, r:r + 1].contiguous(), kn[:, r:r + 1].contiguous(),
                                                            vn[:, r:r + 1].contiguous(), r, 1)
        else:
            got = one.taskkv_decode_step(q, kn, vn)
        assert torch.equal(got.view(torch.uint8), want.view(torch.uint8)), f"step {s}"
        assert np.array_equal(one.lengths(), two.lengths())
    assert one.status() == 0
    for u in (0, int(one.info.n_units) - 1):
        for which in ("k", "v"):
            assert torch.equal(one.pool_rows(which, u).view(torch.uint8), two.pool_rows(which, u).view(torch.uint8))
    # at capacity: the step attends over the rows it has, keeps the lengths and raises the sticky status
    q, kn, vn = W.gen_decode_step(wl, 3, DEV)
    before = one.lengths().copy()
    got = one.taskkv_decode_step(q, kn, vn)
    want = two.taskkv_decode(q)
    assert torch.equal(got.view(torch.uint8), want.view(torch.uint8))
    assert np.array_equal(one.lengths(), before)
    assert one.status() == tk.ESTATE
    one.close()
    two.close()


def _random_case(seed: int) -> dict:
    r = np.random.default_rng(seed)
    n_kv = int(r.choice([1, 2, 4, 8]))
    G = int(r.choice([1, 2, 4, 8]))
    L = int(r.choice([l for l in (1, 8, 16, 32) if G * l <= 128]))
    d = int(r.choice([64, 128]))
    s1, s2 = int(r.integers(0, 9)), int(r.integers(1, 81))
    B = int(r.integers(1, 4))
    lens = [int(r.integers(max(L, s1 + s2 + 2, 40), 4000)) for _ in range(B)]
    return dict(n=n_kv * G, n_kv=n_kv, d=d, N=0, L=L, s1=s1, s2=s2, k=int(r.integers(0, 300)),
                dtype=str(r.choice(["bf16", "f32"])), R=int(r.integers(1, 3)), seq_lens=lens,
                pool=int(r.choice([1, 3, 5, 7])), nh=int(r.integers(0, n_kv + 1)), seed=100 + seed)


@pytest.mark.parametrize("seed", list(range(16)))
def test_random_shapes(seed):
    """Seeded random problem shapes (head counts, group sizes, window, pooling kernel, ragged batch, budgets)."""
    case = _random_case(seed)
    wl = small(f"random{seed}", **case, steps=2)
    run_workload(wl)


@pytest.mark.parametrize("case", [
    dict(n=4, n_kv=4, d=128, N=2341, L=32, s1=4, s2=64, k=100, dtype="bf16"),            # tensor-core path, 32 rows
    dict(n=8, n_kv=2, d=128, N=0, L=32, s1=4, s2=64, k=150, dtype="bf16", R=2, seq_lens=[3000, 1777], nh=1),  # 128 rows
    dict(n=4, n_kv=4, d=64, N=1500, L=16, s1=4, s2=32, k=77, dtype="f32"),               # CUDA-core path
], ids=["tc32", "tc128_ragged", "f32"])
def test_compress_with_supplied_window_lse(case):
    """With the window rows' log-sum-exp handed in (here: the oracle's, rounded to fp32) pass 1 is skipped; scores,
    selections, classes, rows and decode outputs must match the oracle exactly as in the full computation."""
    tk, P = _tk(), _parity()
    from oracle import taskkv_oracle as O
    wl = small("lse", **case)
    qs, ks, vs = W.materialize(wl, DEV)
    G = wl.group
    lse = []
    for b in range(wl.batch):
        per_layer = []
        for r in range(wl.n_layers):
            q64, k64 = P.to64(qs[b][r]), P.to64(ks[b][r])
            per_layer.append(np.stack([O.window_lse(q64[a], k64[a // G]) for a in range(wl.n_heads)]))
        lse.append(torch.from_numpy(np.stack(per_layer)).float().to(DEV).contiguous())
    steps = wl.decode_steps
    params = tk.params_from_workload(wl, max_new_tokens=steps)
    cache = tk.taskkv_compress_ex(params, qs, ks, vs, window_lse=lse)
    assert cache.status() == 0
    rep = P.Report()
    scores, topt = cache.query(tk.Q_SCORES), cache.query(tk.Q_TOPT)
    refs = {}
    for b in range(wl.batch):
        for r in range(wl.n_layers):
            ref = P.oracle_layer(wl, b, r, qs[b][r], ks[b][r], vs[b][r])
            refs[(b, r)] = P.compare_layer(cache, wl, b, r, ref, rep, scores=scores, topt=topt, v=vs[b][r])
            P.compare_pool_rows(cache, wl, b, r, ks[b][r], vs[b][r])
    step_inputs = [W.gen_decode_step(wl, s, DEV) for s in range(steps)]
    outs = [cache.taskkv_decode_step(q, kn, vn) for (q, kn, vn) in step_inputs]
    rep.check_bounds(wl.name)
    for (b, r), chk in refs.items():
        want = P.oracle_decode_steps(wl, b, r, ks[b][r], vs[b][r], chk.idx, step_inputs)
        for s in range(steps):
            assert float(np.abs(P.to64(outs[s][b, r]) - want[s]).max()) < P.TOL_OUT[wl.dtype]
    cache.close()


EXACT_CASES = [
    dict(R=1, n=2, n_kv=2, d=128, N=700),      # a ragged last block of query rows
    dict(R=2, n=4, n_kv=2, d=64, N=1000),      # two query heads per KV head, d = 64
    dict(R=1, n=2, n_kv=1, d=128, N=128),      # exactly one block
    dict(R=1, n=1, n_kv=1, d=128, N=100),      # shorter than a block
    dict(R=1, n=2, n_kv=2, d=128, N=4500),     # several work items per prefix window, 36 blocks
]


@pytest.mark.parametrize("case", EXACT_CASES, ids=[f"case{i}" for i in range(len(EXACT_CASES))])
def test_exact_semantic_vector(case):
    """Eq. 1-2 on the GPU (prefix windows on the tensor cores) against the oracle's full causal attention."""
    tk, P = _tk(), _parity()
    from oracle import taskkv_oracle as O
    R, n, n_kv, d, N = (case[x] for x in ("R", "n", "n_kv", "d", "N"))
    G = n // n_kv
    g = torch.Generator(device="cpu").manual_seed(1234 + N)
    std = float(d) ** -0.25
    q = (torch.randn(R, n, N, d, generator=g) * std).to(torch.bfloat16).to(DEV)
    k = (torch.randn(R, n_kv, N, d, generator=g) * std).to(torch.bfloat16).to(DEV)
    v = (torch.randn(R, n_kv, N, d, generator=g) * std).to(torch.bfloat16).to(DEV)
    k[:, :, N // 3, :] *= 6.0                          # one heavy key per head
    sem, c = tk.taskkv_exact_semantic(q, k, v)
    sem_only, none = tk.taskkv_exact_semantic(q, k, v, want_scores=False)
    assert none is None and torch.equal(sem, sem_only)
    for r in range(R):
        for h in range(n_kv):
            q64 = P.to64(q[r, h * G:(h + 1) * G])
            k64, v64 = P.to64(k[r, h]), P.to64(v[r, h])
            want_c = O.window_scores(q64, k64)           # the window is the whole sequence: L = N
            got_c = P.to64(c[r, h])
            assert np.abs(got_c - want_c).max() < P.TOL_SCORE_REL * want_c.max()
            assert abs(got_c.sum() - 1.0) < 1e-5
            want_v = want_c @ v64
            if G == 1:
                np.testing.assert_allclose(want_v, O.exact_semantic_vector(q64[0], k64, v64), rtol=0, atol=1e-13)
            bound = P.TOL_SCORE_REL * (want_c[:, None] * np.abs(v64)).sum(axis=0).max()
            assert np.abs(P.to64(sem[r, h]) - want_v).max() < bound


# ---------------------------------------------------------------------------
# Error reporting across the boundary
# ---------------------------------------------------------------------------
def test_bounded_device_wait_runs_out_and_reports_timeout():
    """The waits inside the tensor-core kernels have an iteration limit.  The library's self-test runs that wait in a
    one-block kernel on a barrier nothing completes (no copy or MMA in flight): the wait gives up after the limit,
    the block's later waits return at once, the kernel exits normally and leaves ETIMEOUT in its status word.  The
    context stays usable: a regular compression runs right after it."""
    tk = _tk()
    st, polls = tk.taskkv_selftest_bounded_wait(2000)
    assert st == tk.ETIMEOUT
    assert 2000 <= polls <= 2002
    st, polls = tk.taskkv_selftest_bounded_wait(1)
    assert st == tk.ETIMEOUT and polls <= 3
    wl = small("after_timeout", n=4, n_kv=4, d=128, N=1500, L=32, s1=4, s2=64, k=50, dtype="bf16", steps=1)
    run_workload(wl)


def test_host_buffer_calls_return_the_sticky_device_status():
    """taskkv_decode_host synchronises, so it can and does return what the kernels left in the cache's status word:
    a step beyond a unit's capacity is reported as ESTATE by the call itself (the attention over the rows the unit
    holds is still delivered), and stays reported until the cache is destroyed."""
    tk = _tk()
    wl = small("host_status", n=4, n_kv=4, d=64, N=300, L=8, s1=4, s2=32, k=20, dtype="f32")
    qs, ks, vs = W.materialize(wl, "cpu")
    params = tk.params_from_workload(wl, max_new_tokens=1)
    cache = tk.taskkv_compress_host(params, [t.pin_memory() for t in qs], [t.pin_memory() for t in ks],
                                    [t.pin_memory() for t in vs])
    q, kn, vn = (t.pin_memory() for t in W.gen_decode_step(wl, 0, "cpu"))
    out = torch.empty_like(q).pin_memory()
    cache.taskkv_decode_host(q, kn, vn, out)                     # fits: one reserved row per unit
    assert cache.status() == 0
    first = out.clone()
    with pytest.raises(tk.TaskKVError) as ei:
        cache.taskkv_decode_host(q, kn, vn, out)                 # no room left
    assert ei.value.status == tk.ESTATE
    assert torch.equal(out, first)                               # same rows attended, nothing appended
    with pytest.raises(tk.TaskKVError) as ei:
        cache.taskkv_decode_host(q, None, None, out)             # sticky
    assert ei.value.status == tk.ESTATE
    cache.close()


# ---------------------------------------------------------------------------
# Head sharding: the KV heads of every layer split over ranks (here: over caches on one GPU, one after the other)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("case", [
    dict(G=2, splits=[(0, 3), (3, 8)], dtype="bf16", frac=0.0),          # uneven shards, 64 window rows
    dict(G=4, splits=[(0, 2), (2, 4), (4, 8)], dtype="bf16", frac=0.35),  # three shards, 128 rows, budget as a fraction
    dict(G=1, splits=[(0, 4), (4, 8)], dtype="f32", frac=0.0),            # CUDA-core path
], ids=["g2_uneven", "g4_three_budget_frac", "f32"])
def test_head_sharded_compression_equals_the_unsharded_call(case):
    """Every shard runs Eq. 12-15 for its own heads (taskkv_compress_shard_begin), the semantic vectors of all shards
    are put side by side in head order (what the ranks' all-gather produces), and every shard finishes with the
    separator over all of them.  Vectors, distances, classes, lengths, retained positions, cache rows and decode
    outputs of every head must be those of the unsharded call, bit for bit; so must the layer's heterogeneous heads,
    wherever they land (one shard gets none of them in some layers, all of them in others)."""
    tk, P = _tk(), _parity()
    G, n_kv = case["G"], 8
    wl = small("sharded", n=n_kv * G, n_kv=n_kv, d=128 if case["dtype"] == "bf16" else 64, N=0, L=32 if G < 4 else 32,
               s1=4, s2=64, k=140, dtype=case["dtype"], R=3, seq_lens=[2100, 1300], nh=2, steps=2)
    wl.mid_budget = [140, 60, 200]
    wl.n_hetero = [[2, 0, 5], [1, 3, 7]]
    wl.planted = W._choose_planted(wl)
    if case["frac"] > 0:
        wl.budget_frac = case["frac"]
        wl.mid_by_seq = [[O.mid_budget(case["frac"] * n_kv * wl.seq_lens[b], wl.seq_lens[b], wl.full_heads(b, r), n_kv,
                                       wl.sink, wl.recent) for r in range(3)] for b in range(2)]
    qs, ks, vs = W.materialize(wl, DEV)
    whole = tk.taskkv_compress_ex(tk.params_from_workload(wl, max_new_tokens=wl.decode_steps), qs, ks, vs)
    assert whole.status() == 0
    w_cls, w_len, w_dist = whole.classes(), whole.lengths(), whole.query(tk.Q_DIST)
    w_sem, w_idx = whole.query(tk.Q_SEMVEC), whole.query(tk.Q_INDICES)

    shards = []
    for (h0, h1) in case["splits"]:
        params = tk.params_from_workload(wl, max_new_tokens=wl.decode_steps, n_heads=(h1 - h0) * G, n_kv_heads=h1 - h0,
                                         shard_kv_heads=n_kv, shard_first=h0)
        ql = [x[:, h0 * G:h1 * G].contiguous() for x in qs]
        kl = [x[:, h0:h1].contiguous() for x in ks]
        vl = [x[:, h0:h1].contiguous() for x in vs]
        shards.append((h0, h1, tk.taskkv_compress_shard_begin(params, ql, kl, vl), (ql, kl, vl)))
    # what an all-gather of the shards' vectors gives every rank
    sem_all = torch.cat([c.semantic_vectors() for (_, _, c, _) in shards], dim=1).contiguous()
    assert np.array_equal(sem_all.cpu().numpy().reshape(-1, sem_all.shape[-1]), w_sem)
    for (_, _, c, _) in shards:
        with pytest.raises(tk.TaskKVError):
            tk.taskkv_compress_ex(c.params, *shards[0][3])           # a shard cannot be compressed in one call
        c.taskkv_compress_shard_finish(sem_all)
        assert c.status() == 0
    with pytest.raises(tk.TaskKVError) as ei:
        shards[0][2].taskkv_compress_shard_finish(sem_all)
    assert ei.value.status == tk.ESTATE

    R = wl.n_layers
    full_seen = set()
    for (h0, h1, c, _) in shards:
        nl = h1 - h0
        cls, lens, dist, idx = c.classes(), c.lengths(), c.query(tk.Q_DIST), c.query(tk.Q_INDICES)
        assert int(lens.sum()) <= int(c.info.retained_rows)          # the plan is an upper bound for a shard
        for b in range(wl.batch):
            for r in range(R):
                full_seen.add(int((cls[(b * R + r) * nl:(b * R + r + 1) * nl] != 0).sum()))
                for h in range(h0, h1):
                    u, us = (b * R + r) * n_kv + h, (b * R + r) * nl + h - h0
                    assert int(cls[us]) == int(w_cls[u]) and int(lens[us]) == int(w_len[u])
                    assert dist[us] == w_dist[u]
                    if lens[us] < wl.seq_lens[b]:
                        assert np.array_equal(idx[us, :lens[us]], w_idx[u, :lens[us]])
                    for which in ("k", "v"):
                        assert torch.equal(c.pool_rows(which, us).view(torch.uint8),
                                           whole.pool_rows(which, u).view(torch.uint8))
    assert 0 in full_seen and max(full_seen) >= 3                    # shards without and with many full heads
    # and the unsharded result is the oracle's
    rep = P.Report()
    ref = P.oracle_layer(wl, 1, 2, qs[1][2], ks[1][2], vs[1][2])
    P.compare_layer(whole, wl, 1, 2, ref, rep, v=vs[1][2])
    rep.check_bounds(wl.name)
    # decode: a shard's outputs are the unsharded outputs of its query heads
    for s_ in range(wl.decode_steps):
        q, kn, vn = W.gen_decode_step(wl, s_, DEV)
        want = whole.taskkv_decode_step(q, kn, vn)
        for (h0, h1, c, _) in shards:
            got = c.taskkv_decode_step(q[:, :, h0 * G:h1 * G].contiguous(), kn[:, :, h0:h1].contiguous(),
                                       vn[:, :, h0:h1].contiguous())
            assert torch.equal(got.view(torch.uint8), want[:, :, h0 * G:h1 * G].contiguous().view(torch.uint8))
            assert c.status() == 0
    whole.close()
    for (_, _, c, _) in shards:
        c.close()


# ---------------------------------------------------------------------------
# Paged cache: rows in pages of a pool shared by several caches, block tables per unit
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("case", [
    dict(n=16, n_kv=4, d=128, N=0, L=32, s1=4, s2=64, k=120, dtype="bf16", R=3, seq_lens=[2100, 1300], nh=1, P=64),
    dict(n=8, n_kv=8, d=128, N=0, L=32, s1=4, s2=64, k=150, dtype="bf16", R=2, seq_lens=[5000], nh=2, P=256),
    dict(n=4, n_kv=4, d=64, N=0, L=16, s1=4, s2=32, k=60, dtype="f32", R=2, seq_lens=[900, 700], nh=1, P=128),
], ids=["bf16_gqa_p64", "bf16_mha_p256", "f32_p128"])
def test_paged_cache_equals_the_contiguous_cache(case):
    """The same compression with the rows in pages: classes, lengths and retained positions are the contiguous
    cache's, every unit's rows read back through its page table are the same bytes, and so are the decode outputs of
    many steps (fused and append + decode), during which units run off the end of their last page and take new pages
    from the pool; the host's count of free pages follows exactly, and destroying the cache returns every page."""
    tk, Pm = _tk(), _parity()
    P = case.pop("P")
    steps = 70 if P == 64 else 40
    wl = small("paged", **case, steps=steps)
    wl.mid_budget = [case["k"] + 17 * r for r in range(wl.n_layers)]
    qs, ks, vs = W.materialize(wl, DEV)
    params = tk.params_from_workload(wl, max_new_tokens=steps)
    flat = tk.taskkv_compress_ex(params, qs, ks, vs)
    info, pages = tk.taskkv_plan_paged(params, P)
    assert int(info.cache_bytes) < int(flat.info.cache_bytes) // 4          # tables only
    pool = tk.Pool(P, pages + 2 * int(info.n_units) + 3, wl.head_dim, wl.dtype, DEV)
    total = pool.free_pages()
    paged = tk.taskkv_compress_paged(params, qs, ks, vs, pool)
    assert paged.status() == 0 and pool.free_pages() == total - pages
    lens = flat.lengths()
    assert np.array_equal(paged.lengths(), lens) and np.array_equal(paged.classes(), flat.classes())
    assert np.array_equal(paged.query(tk.Q_INDICES), flat.query(tk.Q_INDICES))
    tab = paged.query(tk.Q_PAGETAB)
    used = np.concatenate([tab[u, :(lens[u] + P - 1) // P] for u in range(len(lens))])
    assert len(set(used.tolist())) == len(used) == pages and used.min() >= 0 and used.max() < pool.n_pages
    for u in range(len(lens)):
        for which in ("k", "v"):
            assert torch.equal(paged.pool_rows(which, u).view(torch.uint8), flat.pool_rows(which, u).view(torch.uint8))
    # one layer against the oracle, straight from the paged cache
    rep = Pm.Report()
    ref = Pm.oracle_layer(wl, 0, 1, qs[0][1], ks[0][1], vs[0][1])
    Pm.compare_layer(paged, wl, 0, 1, ref, rep, v=vs[0][1])
    rep.check_bounds(wl.name)
    # decode: units cross page ends at different steps (lengths differ by unit)
    R = wl.n_layers
    for s_ in range(steps):
        q, kn, vn = W.gen_decode_step(wl, s_, DEV)
        if s_ % 3 == 0:
            flat.taskkv_append(kn, vn)
            paged.taskkv_append(kn, vn)
            a, b = flat.taskkv_decode(q), paged.taskkv_decode(q)
        elif s_ % 3 == 1:
            a, b = flat.taskkv_decode_step(q, kn, vn), paged.taskkv_decode_step(q, kn, vn)
        else:
            a, b = flat.taskkv_decode_step(q, kn, vn), torch.empty_like(q)
            for r in range(R):
                b[:, r:r + 1] = paged.taskkv_decode_step_ex(q[:, r:r + 1].contiguous(), kn[:, r:r + 1].contiguous(),
                                                            vn[:, r:r + 1].contiguous(), r, 1)
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), f"step {s_}"
    assert paged.status() == 0 and flat.status() == 0
    lens2 = paged.lengths()
    assert np.array_equal(lens2, lens + steps)
    held = int(sum((int(x) + P - 1) // P for x in lens2))
    assert held > pages and pool.free_pages() == total - held          # the host's count, page for page
    for u in (0, len(lens) - 1):
        assert torch.equal(paged.pool_rows("k", u).view(torch.uint8), flat.pool_rows("k", u).view(torch.uint8))
    # the decode attention of the paged cache against the oracle on its own rows
    q, _, _ = W.gen_decode_step(wl, 999, DEV)
    out = paged.taskkv_decode(q)
    G = wl.group
    for u in (1, len(lens) - 2):
        b_, r_, h_ = u // (R * wl.n_kv_heads), (u // wl.n_kv_heads) % R, u % wl.n_kv_heads
        kc, vc = Pm.to64(paged.pool_rows("k", u)), Pm.to64(paged.pool_rows("v", u))
        for g in range(G):
            want = O.decode_attention(Pm.to64(q[b_, r_, h_ * G + g]), kc, vc)
            assert np.abs(Pm.to64(out[b_, r_, h_ * G + g]) - want).max() < Pm.TOL_OUT[wl.dtype]
    paged.close()
    assert pool.free_pages() == total
    flat.close()
    pool.close()


def test_paged_caches_share_a_pool_and_reuse_freed_pages():
    """Two caches in one pool; the pool is sized so that a third fits only after the first is destroyed.  A
    compression that would not fit is refused (EALLOC) before anything is launched and leaves the count untouched;
    after the destruction the third cache gets the freed pages and is as correct as the others; an append that
    needs more pages than are left is refused as well."""
    tk = _tk()
    P = 64
    wls = [small(f"pool{i}", n=8, n_kv=4, d=128, N=0, L=32, s1=4, s2=64, k=100, dtype="bf16", R=2,
                 seq_lens=[(1500, 1800, 1500)[i]], nh=1, steps=4, seed=50 + i) for i in range(3)]
    need = [tk.taskkv_plan_paged(tk.params_from_workload(w, max_new_tokens=200), P)[1] for w in wls]
    assert need[2] == need[0]                   # Eq. 16 fixes the number of full heads: pages depend on the lengths only
    pool = tk.Pool(P, need[0] + need[1] + 9, 128, "bf16", DEV)
    data = [W.materialize(w, DEV) for w in wls]
    params = [tk.params_from_workload(w, max_new_tokens=200) for w in wls]
    caches = [tk.taskkv_compress_paged(params[i], *data[i], pool) for i in range(2)]
    assert pool.free_pages() == 9
    with pytest.raises(tk.TaskKVError) as ei:
        tk.taskkv_compress_paged(params[2], *data[2], pool)
    assert ei.value.status == tk.EALLOC and pool.free_pages() == 9
    flats = [tk.taskkv_compress_ex(params[i], *data[i]) for i in range(3)]

    def step(i, s_):
        q, kn, vn = W.gen_decode_step(wls[i], s_, DEV)
        a = flats[i].taskkv_decode_step(q, kn, vn)
        b = caches[i].taskkv_decode_step(q, kn, vn)
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))

    step(0, 0)
    step(1, 0)
    caches[0].close()
    assert pool.free_pages() >= need[0] + 9 - 8                      # cache 1 may have opened up to 8 pages
    caches[0] = None
    third = tk.taskkv_compress_paged(params[2], *data[2], pool)         # takes the pages cache 0 gave back
    caches.append(third)
    assert third.status() == 0
    assert np.array_equal(third.lengths(), flats[2].lengths())
    for u in range(8):
        assert torch.equal(third.pool_rows("v", u).view(torch.uint8), flats[2].pool_rows("v", u).view(torch.uint8))
    step(1, 1)
    step(2, 0)
    # run the pool dry: appends are refused once a step needs more pages than are left, and nothing is corrupted
    refused = False
    for s_ in range(1, 200):
        q, kn, vn = W.gen_decode_step(wls[2], s_, DEV)
        try:
            b = third.taskkv_decode_step(q, kn, vn)
        except tk.TaskKVError as exc:
            assert exc.status == tk.EALLOC
            refused = True
            break
        a = flats[2].taskkv_decode_step(q, kn, vn)
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
    assert refused and third.status() == 0 and caches[1].status() == 0
    step(1, 2) if pool.free_pages() >= 8 else None
    for c in caches:
        if c is not None:
            c.close()
    assert pool.free_pages() == pool.n_pages
    for f in flats:
        f.close()
    pool.close()


def test_paged_cache_in_a_pool_the_library_allocates():
    """taskkv_pool_create with no caller memory: the library allocates the pool; compression and decode steps equal
    the contiguous cache's, the count of free pages follows, the pool is freed by taskkv_pool_destroy."""
    tk = _tk()
    wl = small("ownpool", n=8, n_kv=4, d=128, N=0, L=32, s1=4, s2=64, k=90, dtype="bf16", R=2, seq_lens=[1700, 900],
               nh=1, steps=5)
    qs, ks, vs = W.materialize(wl, DEV)
    params = tk.params_from_workload(wl, max_new_tokens=5)
    _, pages = tk.taskkv_plan_paged(params, 128)
    pool = tk.Pool(128, pages + 16, 128, "bf16", DEV, library_memory=True)
    paged = tk.taskkv_compress_paged(params, qs, ks, vs, pool)
    flat = tk.taskkv_compress_ex(params, qs, ks, vs)
    assert pool.free_pages() == 16 and np.array_equal(paged.lengths(), flat.lengths())
    assert np.array_equal(paged.query(tk.Q_INDICES), flat.query(tk.Q_INDICES))
    for u in (0, 5, 15):
        assert torch.equal(paged.pool_rows("k", u).view(torch.uint8), flat.pool_rows("k", u).view(torch.uint8))
        assert torch.equal(paged.pool_rows("v", u).view(torch.uint8), flat.pool_rows("v", u).view(torch.uint8))
    for s_ in range(5):
        q, kn, vn = W.gen_decode_step(wl, s_, DEV)
        assert torch.equal(paged.taskkv_decode_step(q, kn, vn).view(torch.uint8),
                           flat.taskkv_decode_step(q, kn, vn).view(torch.uint8))
    assert paged.status() == 0
    paged.close()
    assert pool.free_pages() == pool.n_pages
    flat.close()
    pool.close()


def test_pool_destroyed_before_its_cache_is_released_by_the_cache():
    """taskkv_pool_destroy while a cache still lives in the pool only marks the pool; the cache keeps working and
    its destruction releases the pool."""
    tk = _tk()
    wl = small("orphan", n=4, n_kv=4, d=128, N=1200, L=32, s1=4, s2=64, k=80, dtype="bf16", R=1, nh=1, steps=3)
    qs, ks, vs = W.materialize(wl, DEV)
    params = tk.params_from_workload(wl, max_new_tokens=3)
    _, pages = tk.taskkv_plan_paged(params, 64)
    pool = tk.Pool(64, pages + 8, 128, "bf16", DEV, library_memory=True)
    paged = tk.taskkv_compress_paged(params, qs, ks, vs, pool)
    flat = tk.taskkv_compress_ex(params, qs, ks, vs)
    pool.close()                                        # the pool's handle is gone; its memory is not
    for s_ in range(3):
        q, kn, vn = W.gen_decode_step(wl, s_, DEV)
        assert torch.equal(paged.taskkv_decode_step(q, kn, vn).view(torch.uint8),
                           flat.taskkv_decode_step(q, kn, vn).view(torch.uint8))
    assert paged.status() == 0
    paged.close()                                       # releases the pool
    flat.close()


def test_unit_data_read_early_never_changes_a_result():
    """A per-layer decode call whose predecessor in the stream cannot write its lengths reads them before its
    dependency wait.  One cache takes a sequence of per-layer fused steps on one stream (the case that qualifies), with
    the same layer twice in a row, a CUDA graph of two layers replayed three times and direct calls right after it; a
    second cache takes the same steps with every call on a stream other than the one before (never qualifies) and a
    synchronisation in between.  Outputs, lengths and rows must agree bit for bit."""
    tk = _tk()
    wl = small("early", n=8, n_kv=4, d=128, N=0, L=32, s1=4, s2=64, k=100, dtype="bf16", R=3, seq_lens=[1500, 900],
               nh=1, steps=1)
    qs, ks, vs = W.materialize(wl, DEV)
    params = tk.params_from_workload(wl, max_new_tokens=64)
    a = tk.taskkv_compress_ex(params, qs, ks, vs)
    b = tk.taskkv_compress_ex(params, qs, ks, vs)
    torch.cuda.synchronize()
    seq = [0, 1, 2, 2, 0, 0, 1, 2, 1, 1, 0, 2]                     # layers, in call order
    inputs = {}

    def layer_inputs(i, r):
        if (i, r) not in inputs:
            q, kn, vn = W.gen_decode_step(wl, 100 + i, DEV)
            inputs[(i, r)] = tuple(x[:, r:r + 1].contiguous() for x in (q, kn, vn))
        return inputs[(i, r)]

    other = [torch.cuda.Stream(), torch.cuda.Stream()]

    calls = [0]

    def ref_call(r, q, kn, vn):                                    # never two calls in a row on one stream
        st = other[calls[0] % 2]
        calls[0] += 1
        with torch.cuda.stream(st):
            out = b.taskkv_decode_step_ex(q, kn, vn, r, 1, stream=st)
        torch.cuda.synchronize()
        return out

    outs_a, outs_b = [], []
    for i, r in enumerate(seq):
        q, kn, vn = layer_inputs(i, r)
        outs_a.append(a.taskkv_decode_step_ex(q, kn, vn, r, 1))
        outs_b.append(ref_call(r, q, kn, vn))
    # a graph of two per-layer steps, replayed, then direct calls on the layers it touched
    gi = len(seq)
    g_in = [layer_inputs(gi, 0), layer_inputs(gi, 1)]
    g_out = [torch.empty_like(g_in[0][0]), torch.empty_like(g_in[1][0])]
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):                                  # (capture launches nothing)
        a.taskkv_decode_step_ex(*g_in[0], 0, 1, out=g_out[0])
        a.taskkv_decode_step_ex(*g_in[1], 1, 1, out=g_out[1])
    for rep in range(3):
        graph.replay()
        torch.cuda.synchronize()
        outs_a += [x.clone() for x in g_out]
        outs_b += [ref_call(0, *g_in[0]), ref_call(1, *g_in[1])]
    for i, r in enumerate([1, 0, 1, 2], start=gi + 1):
        q, kn, vn = layer_inputs(i, r)
        outs_a.append(a.taskkv_decode_step_ex(q, kn, vn, r, 1))
        outs_b.append(ref_call(r, q, kn, vn))
    torch.cuda.synchronize()
    assert a.status() == 0 and b.status() == 0
    assert np.array_equal(a.lengths(), b.lengths())
    for i, (x, y) in enumerate(zip(outs_a, outs_b)):
        assert torch.equal(x.view(torch.uint8), y.view(torch.uint8)), f"call {i}"
    for u in range(len(a.lengths())):
        assert torch.equal(a.pool_rows("k", u).view(torch.uint8), b.pool_rows("k", u).view(torch.uint8))
    a.close()
    b.close()


def test_direct_call_after_a_graph_replay_sees_the_replayed_lengths():
    """The rule for reading unit data early takes a graph launch to be a unit in stream order: a kernel launched
    directly after a replay starts once the whole graph has finished, whatever its last kernel triggered.  Here the
    host's record points at another layer (a direct step on layer 1), a graph holding a fused step on layer 0 is
    replayed, and a direct fused step on layer 0 follows at once and reads its lengths early: 150 rounds against a
    cache that takes the same steps with nothing read early."""
    tk = _tk()
    rounds = 150
    wl = small("replay", n=8, n_kv=4, d=128, N=0, L=32, s1=4, s2=64, k=100, dtype="bf16", R=2, seq_lens=[1400, 800],
               nh=1, steps=1)
    qs, ks, vs = W.materialize(wl, DEV)
    params = tk.params_from_workload(wl, max_new_tokens=2 * rounds + 4)
    a = tk.taskkv_compress_ex(params, qs, ks, vs)
    b = tk.taskkv_compress_ex(params, qs, ks, vs)
    q, kn, vn = W.gen_decode_step(wl, 7, DEV)
    l0 = tuple(x[:, 0:1].contiguous() for x in (q, kn, vn))
    l1 = tuple(x[:, 1:2].contiguous() for x in (q, kn, vn))
    g_out = torch.empty_like(l0[0])
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        a.taskkv_decode_step_ex(*l0, 0, 1, out=g_out)
    other = [torch.cuda.Stream(), torch.cuda.Stream()]
    n_ref = [0]

    def ref(r, x):
        st = other[n_ref[0] % 2]
        n_ref[0] += 1
        out = b.taskkv_decode_step_ex(*x, r, 1, stream=st)
        torch.cuda.synchronize()
        return out

    for i in range(rounds):
        a.taskkv_decode_step_ex(*l1, 1, 1)              # the host's record now names layer 1
        graph.replay()                                  # raises the lengths of layer 0 ...
        got = a.taskkv_decode_step_ex(*l0, 0, 1)        # ... which this call reads before its dependency wait
        torch.cuda.synchronize()
        ref(1, l1)
        ref(0, l0)
        want = ref(0, l0)
        assert torch.equal(got.view(torch.uint8), want.view(torch.uint8)), f"round {i}"
    assert np.array_equal(a.lengths(), b.lengths()) and a.status() == 0 and b.status() == 0
    a.close()
    b.close()
