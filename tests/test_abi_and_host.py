"""CPU-side checks: the C-ABI library loads and exports every declared symbol,
and its host-only logic (argument validation, planning, Eq. 16 / Eq. 17 helpers)
agrees with the oracle and with closed forms.  No kernel is launched here."""
import ctypes as C
import os
import re

import pytest

from oracle import taskkv_oracle as O
from paper_2501_15113_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tk():
    import __graft_entry__ as g
    g.build()
    from paper_2501_15113_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "taskkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(taskkv_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(tk):
    names = declared_functions()
    assert len(names) >= 18
    for n in names:
        assert hasattr(tk.lib, n), f"{n} is declared in taskkv.h but not exported"


def test_params_struct_layout_matches_header(tk):
    p = tk.taskkv_params()
    tk.lib.taskkv_params_default(C.byref(p))
    assert (p.top_t, p.pool_kernel, p.sink, p.recent, p.window) == (256, 7, 16, 256, 32)
    assert abs(p.beta - 0.25) < 1e-7 and p.m_top == 4 and p.promote_center == 1 and p.force_class == -1
    assert p.dtype == tk.BF16


def test_hetero_count_matches_oracle(tk):
    for n in (8, 32, 40):
        for beta in (0.2, 0.25, 0.3, 0.35, 0.4):
            for m in (0, 1, 4, 6):
                for R in (1, 2, 5, 32):
                    for r in range(R):
                        assert tk.taskkv_hetero_count(n, beta, m, R, r) == \
                            O.hetero_count(n, float(C.c_float(beta).value), m, R, r)


def test_mid_budget_matches_oracle(tk):
    for N in (512, 30000, 131072):
        for n, h in ((8, 0), (8, 2), (8, 3), (32, 5), (8, 8)):
            for frac in (0.1, 0.4, 0.6, 1.0):
                B = frac * n * N
                assert tk.taskkv_mid_budget(B, N, h, n, 4, 256) == O.mid_budget(B, N, h, n, 4, 256)


def test_mid_budget_from_far_head_count_and_literal_reading(tk):
    """Eq. 17 from f(r): the default counts the promoted head among the full caches (the layer total stays within
    the budget); literal = 1 is Eq. 17 exactly as printed, h = f(r)."""
    for N in (512, 30000, 131072):
        for n in (8, 32):
            for f in (0, 1, 2, n - 1, n):
                for frac in (0.1, 0.4, 0.6, 1.0):
                    B = frac * n * N
                    assert tk.taskkv_mid_budget_ex(B, N, f, n, 4, 256, literal=True) == O.mid_budget(B, N, f, n, 4, 256)
                    h = min(n, f + 1)
                    assert tk.taskkv_mid_budget_ex(B, N, f, n, 4, 256) == O.mid_budget(B, N, h, n, 4, 256)
                    assert tk.taskkv_mid_budget_ex(B, N, f, n, 4, 256, promote_center=False) == \
                        O.mid_budget(B, N, f, n, 4, 256)
    # the printed form overshoots the budget once the promoted head is stored in full; the default does not
    N, n, f = 131072, 8, 2
    B = 0.4 * n * N
    k_lit = tk.taskkv_mid_budget_ex(B, N, f, n, 4, 256, literal=True)
    k_def = tk.taskkv_mid_budget_ex(B, N, f, n, 4, 256)
    assert (f + 1) * N + (n - f - 1) * (k_lit + 260) > B >= (f + 1) * N + (n - f - 1) * (k_def + 260)


def test_plan_matches_closed_forms(tk):
    from paper_2501_15113_b200 import configs
    for wl in (configs.config1_toy(), configs.config2_llama2(), configs.config3_llama3(),
               configs.config4_mistral(), configs.config5_sweep(2, 256)):
        info = tk.taskkv_plan(tk.params_from_workload(wl))
        U = wl.batch * wl.n_layers * wl.n_kv_heads
        assert info.n_units == U
        assert info.retained_rows == wl.retained_rows()
        assert info.pool_rows == wl.retained_rows() + U * wl.decode_steps
        es = wl.elem_size
        assert info.cache_bytes >= 2 * info.pool_rows * wl.head_dim * es
    # config 3 keeps 40 % of the full cache (Sec. V-E budget), never more
    wl = configs.config3_llama3()
    full = wl.n_layers * wl.n_kv_heads * wl.seq_lens[0]
    assert 0.399 < wl.retained_rows() / full <= 0.4


def test_invalid_arguments_are_rejected_before_any_launch(tk):
    wl = W.toy()
    good = dict(n_layers=1, n_heads=8, n_kv_heads=8, head_dim=64, seq_lens=[512], sink=4, recent=32,
                mid_budget=32, window=16, dtype="f32")
    tk.taskkv_plan(tk.Params(**good))
    bad = [dict(head_dim=96), dict(n_kv_heads=3), dict(window=0), dict(window=1024), dict(seq_lens=[8]),
           dict(top_t=5000), dict(pool_kernel=4), dict(sink=-1), dict(n_heads=8 * 16, n_kv_heads=8),
           dict(mid_budget=-2), dict(force_class=7), dict(seq_lens=[0]), dict(mid_policy=3), dict(mid_policy=-1)]
    for override in bad:
        kw = dict(good)
        kw.update(override)
        with pytest.raises(tk.TaskKVError) as ei:
            tk.taskkv_plan(tk.Params(**kw))
        assert ei.value.status == tk.EINVAL, override
    # null pointers never reach the device
    h = C.c_void_p()
    assert tk.lib.taskkv_compress_ex(None, None, None, None, None, 0, None, 0, None, C.byref(h)) == tk.EINVAL
    assert tk.lib.taskkv_decode(None, None, None, None, None) == tk.EINVAL
    assert tk.lib.taskkv_append(None, None, None, None) == tk.EINVAL
    assert tk.lib.taskkv_append_ex(None, None, None, 0, 1, None) == tk.EINVAL
    assert tk.lib.taskkv_decode_ex(None, None, None, None, 0, 1, None) == tk.EINVAL
    assert tk.lib.taskkv_decode_step(None, None, None, None, None, None) == tk.EINVAL
    assert tk.lib.taskkv_decode_step_ex(None, None, None, None, None, 0, 1, None) == tk.EINVAL
    assert tk.lib.taskkv_cache_query(None, 0, None, 0) == tk.EINVAL
    assert tk.lib.taskkv_cache_create(None, None, 0, None, 0, None, C.byref(h)) == tk.EINVAL
    assert tk.lib.taskkv_compress_layer(None, 0, None, None, None, None, None) == tk.EINVAL
    assert tk.lib.taskkv_compress_shard_begin(None, None, None, None, None, None, 0, None, 0, None, C.byref(h)) == tk.EINVAL
    assert tk.lib.taskkv_compress_shard_finish(None, None, None) == tk.EINVAL
    assert tk.lib.taskkv_cache_semantic(None, None, None) == tk.EINVAL
    assert tk.lib.taskkv_compress_paged(None, None, None, None, None, None, 0, None, 0, None, C.byref(h)) == tk.EINVAL
    assert tk.lib.taskkv_pool_create(32, 8, 128, tk.BF16, None, 0, None, C.byref(h)) == tk.EINVAL
    assert tk.lib.taskkv_pool_create(64, 8, 128, tk.BF16, None, 0, None, None) == tk.EINVAL
    assert tk.lib.taskkv_pool_create(64, 8, 128, tk.BF16, 256, 16, None, C.byref(h)) == tk.EALLOC   # buffer too small
    assert tk.lib.taskkv_plan_paged(None, 64, None, None) == tk.EINVAL
    assert tk.lib.taskkv_pool_free_pages(None) == -1
    tk.lib.taskkv_pool_destroy(None)
    assert tk.lib.taskkv_exact_semantic(None, None, None, 1, 8, 8, 128, 512, None, None, None, 0, None) == tk.EINVAL
    # argument checks come before any device work: a head dimension or a head grouping the kernels do not take
    assert tk.lib.taskkv_exact_semantic(16, 16, 16, 1, 8, 8, 96, 512, 16, None, None, 0, None) == tk.EINVAL
    assert tk.lib.taskkv_exact_semantic(16, 16, 16, 1, 8, 3, 128, 512, 16, None, None, 0, None) == tk.EINVAL
    assert tk.lib.taskkv_exact_semantic(16, 16, 16, 1, 8, 8, 128, 0, 16, None, None, 0, None) == tk.EINVAL
    assert tk.lib.taskkv_exact_semantic_bytes(1, 8, 8, 96, 512) == 0
    # one round over all 64 query heads: the blocks' scores (64 b (b + 1) floats per head for b = 4 blocks) dominate
    assert tk.lib.taskkv_exact_semantic_bytes(2, 32, 8, 128, 512) >= 64 * 64 * 4 * 5 * 4
    # a scratch too small for even one KV group is refused before any device work
    assert tk.lib.taskkv_exact_semantic(256, 256, 256, 1, 8, 8, 128, 4096, 256, None, 256, 1024, None) == tk.EALLOC
    assert tk.lib.taskkv_status_str(tk.ESTATE) == b"cache in wrong state"
    assert wl.retained_rows() == 3 * 512 + 5 * 68


def test_plan_of_a_head_shard_is_the_upper_bound(tk):
    """A shard cannot know how many of a layer's full-cache heads it will hold: its pools are planned for
    min(full heads of the layer, its own heads) per (sequence, layer), Eq. 16 and Eq. 17 counting over the model's heads."""
    from paper_2501_15113_b200 import sharding
    n_model, R, lens, s1, s2, k, mn = 8, 4, [3000, 1700], 4, 64, 100, 5
    nh = [[tk.taskkv_hetero_count(n_model, 0.3, 1, R, r) for r in range(R)]] * 2       # 2, 2, 1, 1 far heads of 8
    for (h0, h1) in ((0, 3), (3, 8), (0, 1)):
        nl = h1 - h0
        p = tk.Params(n_layers=R, n_heads=2 * nl, n_kv_heads=nl, head_dim=128, seq_lens=lens, sink=s1, recent=s2,
                      mid_budget=k, window=32, dtype="bf16", beta=0.3, m_top=1, max_new_tokens=mn,
                      shard_kv_heads=n_model, shard_first=h0)
        info = tk.taskkv_plan(p)
        want = sum(sharding.shard_pool_rows_bound(N, nl, nh[0][r] + 1, s1 + s2 + k, mn) for N in lens for r in range(R))
        assert info.pool_rows == want and info.n_units == 2 * R * nl
    # out-of-range shards are refused
    for bad in (dict(shard_kv_heads=8, shard_first=6), dict(shard_kv_heads=2, shard_first=0), dict(shard_kv_heads=-1)):
        kw = dict(n_layers=R, n_heads=6, n_kv_heads=3, head_dim=128, seq_lens=lens, sink=s1, recent=s2, mid_budget=k,
                  window=32, dtype="bf16")
        kw.update(bad)
        with pytest.raises(tk.TaskKVError):
            tk.taskkv_plan(tk.Params(**kw))
    # budgets from a fraction count the model's heads too
    p = tk.Params(n_layers=1, n_heads=4, n_kv_heads=2, head_dim=128, seq_lens=[4000], sink=s1, recent=s2, mid_budget=0,
                  window=32, dtype="bf16", n_hetero=[[2]], budget_frac=0.5, shard_kv_heads=8, shard_first=2)
    kmid = O.mid_budget(0.5 * 8 * 4000, 4000, 3, 8, s1, s2)
    assert tk.taskkv_plan(p).pool_rows == 2 * 4000            # both of its heads may be full ones
    p0 = tk.Params(n_layers=1, n_heads=4, n_kv_heads=2, head_dim=128, seq_lens=[4000], sink=s1, recent=s2, mid_budget=0,
                   window=32, dtype="bf16", n_hetero=[[0]], promote_center=False, budget_frac=0.5, shard_kv_heads=8,
                   shard_first=2)
    assert tk.taskkv_plan(p0).pool_rows == 2 * (s1 + s2 + O.mid_budget(0.5 * 8 * 4000, 4000, 0, 8, s1, s2)) and kmid > 0


def test_plan_of_a_paged_cache_counts_pages_per_unit(tk):
    """Pages a compression takes = sum over units of ceil(retained rows / page rows), the full heads per (sequence,
    layer) from Eq. 16; the pool holds K and V pages plus the free-page stack; page sizes that are not a multiple of
    the gather's 64-row items, and paged caches of a head shard, are refused."""
    R, n, lens, s1, s2, k, mn = 3, 8, [3000, 1700, 260], 4, 64, 100, 7
    nh = [[tk.taskkv_hetero_count(n, 0.25, 4, R, r) for r in range(R)] for _ in lens]
    kw = dict(n_layers=R, n_heads=n, n_kv_heads=n, head_dim=128, seq_lens=lens, sink=s1, recent=s2, mid_budget=k,
              window=32, dtype="bf16", max_new_tokens=mn)
    p = tk.Params(**kw)
    flat = tk.taskkv_plan(p)
    for P in (64, 128, 1024):
        info, pages = tk.taskkv_plan_paged(p, P)
        want = 0
        for b, N in enumerate(lens):
            for r in range(R):
                full = min(n, nh[b][r] + 1)
                kept = min(N, s1 + s2 + k)
                want += full * -(-N // P) + (n - full) * -(-kept // P)
        assert pages == want and info.n_units == flat.n_units and info.retained_rows == flat.retained_rows
        assert info.cache_bytes < flat.cache_bytes
        assert tk.lib.taskkv_pool_bytes(P, pages, 128, tk.BF16) >= 2 * pages * P * 128 * 2 + 4 * pages
    for bad in (0, 32, 96, -64):
        with pytest.raises(tk.TaskKVError):
            tk.taskkv_plan_paged(p, bad)
        assert tk.lib.taskkv_pool_bytes(bad, 16, 128, tk.BF16) == 0
    assert tk.lib.taskkv_pool_bytes(64, 0, 128, tk.BF16) == 0 and tk.lib.taskkv_pool_bytes(64, 16, 96, tk.BF16) == 0
    shard = tk.Params(**dict(kw, n_heads=4, n_kv_heads=4, shard_kv_heads=8, shard_first=0))
    with pytest.raises(tk.TaskKVError):
        tk.taskkv_plan_paged(shard, 64)
