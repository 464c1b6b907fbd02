"""Pins for the CPU oracle: each check ties an oracle function to something
other than itself -- a closed form, an invariant, a textbook/library routine,
brute force on tiny inputs, or a value the paper fixes."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import taskkv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- brute force helpers
def loop_causal_weights(q, k):
    """Full N x N causal softmax weights by explicit loops (Eq. 1)."""
    N, d = q.shape
    A = np.zeros((N, N))
    for i in range(N):
        s = [sum(q[i, x] * k[j, x] for x in range(d)) / math.sqrt(d) for j in range(i + 1)]
        mx = max(s)
        e = [math.exp(x - mx) for x in s]
        z = sum(e)
        for j in range(i + 1):
            A[i, j] = e[j] / z
    return A


# ---------------------------------------------------------------- Eq. 12 / 13
def test_window_rows_are_last_rows_of_full_causal_attention():
    r = rng(1)
    N, d, L = 23, 5, 6
    q, k = r.normal(size=(N, d)), r.normal(size=(N, d))
    A_full = loop_causal_weights(q, k)
    A_win = O.window_attention(q[-L:], k)
    np.testing.assert_allclose(A_win, A_full[-L:], rtol=0, atol=1e-14)


def test_window_attention_matches_library_sdpa():
    r = rng(2)
    N, d, L = 40, 8, 40
    q, k, v = (r.normal(size=(N, d)) for _ in range(3))
    A = O.window_attention(q[-L:], k)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(k)[None], torch.from_numpy(v)[None], is_causal=True)[0]
    np.testing.assert_allclose(A @ v, ref.numpy(), rtol=0, atol=1e-12)


def test_equal_keys_closed_form_and_unit_mass():
    # all keys equal: row i spreads 1/(p_i+1) over its visible keys, so
    # C[j] = (1/L) * sum over window rows with p_i >= j of 1/(p_i+1).
    r = rng(3)
    N, d, L = 37, 4, 9
    q = r.normal(size=(L, d))
    k = np.tile(r.normal(size=(1, d)), (N, 1))
    C = O.column_mean(O.window_attention(q, k))
    expect = np.zeros(N)
    for j in range(N):
        expect[j] = sum(1.0 / (N - L + i + 1) for i in range(L) if N - L + i >= j) / L
    np.testing.assert_allclose(C, expect, rtol=0, atol=1e-15)
    assert abs(C.sum() - 1.0) < 1e-12


def test_column_mean_unit_mass_random_and_grouped_rule():
    r = rng(4)
    N, d, L, G = 50, 6, 7, 4
    qg = r.normal(size=(G, L, d))
    k = r.normal(size=(N, d))
    C = O.window_scores(qg, k)
    assert abs(C.sum() - 1.0) < 1e-12
    per_head = np.stack([O.column_mean(O.window_attention(qg[g], k)) for g in range(G)])
    np.testing.assert_allclose(C, per_head.mean(axis=0), rtol=0, atol=1e-15)


# ---------------------------------------------------------------- Eq. 14
@pytest.mark.parametrize("seed", range(20))
def test_top_indices_equals_brute_force_sort(seed):
    r = rng(100 + seed)
    n = int(r.integers(1, 30))
    count = int(r.integers(0, n + 3))
    score = r.integers(0, 6, size=n).astype(float)     # many exact ties
    got = O.top_indices(score, count)
    pairs = sorted(((-score[j], j) for j in range(n)))  # score descending, then position ascending
    want = sorted(j for _, j in pairs[:min(count, n)])
    assert got.tolist() == want
    if 0 < len(want) < n:
        rest = sorted(set(range(n)) - set(want))
        assert min(score[j] for j in want) >= max(score[j] for j in rest)


def test_top_indices_exhaustive_small():
    for vals in itertools.product([0.0, 1.0, 2.0], repeat=4):
        for count in range(5):
            got = O.top_indices(np.array(vals), count).tolist()
            order = sorted(range(4), key=lambda j: (-vals[j], j))[:count]
            assert got == sorted(order)


# ---------------------------------------------------------------- Eq. 15 / Eq. 2
def test_window_equals_exact_semantic_vector_when_window_and_t_cover_everything():
    r = rng(5)
    N, d = 17, 4
    q, k, v = (r.normal(size=(N, d)) for _ in range(3))
    A = loop_causal_weights(q, k)
    v_exact = np.zeros(d)
    for i in range(N):
        for j in range(N):
            v_exact += A[i, j] * v[j] / N
    C = O.column_mean(O.window_attention(q, k))
    got = O.semantic_vector(C, v, O.top_indices(C, N))
    np.testing.assert_allclose(got, v_exact, rtol=0, atol=1e-14)
    np.testing.assert_allclose(O.exact_semantic_vector(q, k, v), v_exact, rtol=0, atol=1e-14)


def test_constant_value_rows_give_selected_mass_times_constant():
    r = rng(6)
    N, d, L, t = 64, 5, 8, 10
    q, k = r.normal(size=(L, d)), r.normal(size=(N, d))
    c = r.normal(size=d)
    v = np.tile(c, (N, 1))
    C = O.column_mean(O.window_attention(q, k))
    I = O.top_indices(C, t)
    top_mass = np.sort(C)[::-1][:t].sum()
    np.testing.assert_allclose(O.semantic_vector(C, v, I), c * top_mass, rtol=0, atol=1e-15)
    assert top_mass < 1.0          # so a renormalised weighting would have failed the line above
    np.testing.assert_allclose(O.semantic_vector(C, v, O.top_indices(C, N)), c, rtol=0, atol=1e-14)


# ---------------------------------------------------------------- Eq. 7 / 8, separator
def test_center_and_distance_closed_forms():
    a = np.array([3.0, -4.0, 0.0])
    vec = np.stack([a, -a])
    np.testing.assert_allclose(O.semantic_center(vec), 0.0, atol=0)
    np.testing.assert_allclose(O.center_distances(vec), [5.0, 5.0], atol=1e-15)
    # three collinear points 0, 1, 5 on an axis: center 2, distances 2, 1, 3
    vec = np.array([[0.0, 0], [1.0, 0], [5.0, 0]])
    np.testing.assert_allclose(O.center_distances(vec), [2.0, 1.0, 3.0], atol=1e-15)
    shift = rng(7).normal(size=2)
    np.testing.assert_allclose(O.center_distances(vec + shift), [2.0, 1.0, 3.0], atol=1e-14)


def test_separator_small_known_answer_and_ties():
    dist = np.array([0.5, 3.0, 0.1, 2.0, 0.1, 0.7])
    cls = O.semantic_separator(dist, 2, True)
    assert cls.tolist() == [0, 1, 2, 1, 0, 0]          # far: 1, 3; closest of the rest: index 2 (tie -> lower)
    assert O.semantic_separator(dist, 2, False).tolist() == [0, 1, 0, 1, 0, 0]
    assert O.semantic_separator(dist, 0, True).tolist() == [0, 0, 2, 0, 0, 0]
    assert O.semantic_separator(dist, 6, True).tolist() == [1] * 6
    assert O.semantic_separator(np.array([1.0, 1.0, 1.0]), 1, True).tolist() == [1, 2, 0]


def test_separator_permutation_equivariance():
    r = rng(8)
    n, d = 12, 6
    sem = r.normal(size=(n, d))
    cls = O.semantic_separator(O.center_distances(sem), 3, True)
    perm = r.permutation(n)
    cls_p = O.semantic_separator(O.center_distances(sem[perm]), 3, True)
    assert cls_p.tolist() == cls[perm].tolist()


def _toy_layer(seed=0, n=8, N=192, d=16, L=8, planted=(2, 5)):
    r = rng(seed)
    q = r.normal(size=(n, L, d))
    k = r.normal(size=(n, N, d))
    v = r.normal(size=(n, N, d))
    k[:, 0, :] *= 8.0
    for h in planted:
        v[h] += 3.0
    return q, k, v


def test_planted_heads_are_recovered_and_center_head_is_nearest():
    q, k, v = _toy_layer()
    out = O.compress_layer(q, k, v, n_hetero=2, sink=4, recent=16, mid=8, top_t=64)
    assert np.flatnonzero(out["cls"] == 1).tolist() == [2, 5]
    rest = np.flatnonzero(out["cls"] != 1)
    promoted = np.flatnonzero(out["cls"] == 2)
    assert len(promoted) == 1
    assert out["dist"][promoted[0]] == out["dist"][rest].min()


def test_whole_layer_head_permutation_equivariance():
    q, k, v = _toy_layer(seed=3)
    perm = rng(9).permutation(8)
    a = O.compress_layer(q, k, v, n_hetero=2, sink=4, recent=16, mid=8, top_t=64)
    b = O.compress_layer(q[perm], k[perm], v[perm], n_hetero=2, sink=4, recent=16, mid=8, top_t=64)
    assert b["cls"].tolist() == a["cls"][perm].tolist()
    assert b["len"].tolist() == a["len"][perm].tolist()
    for i, p in enumerate(perm):
        assert b["idx"][i].tolist() == a["idx"][p].tolist()


# ---------------------------------------------------------------- pooling, retention
def test_average_pool_matches_library_and_impulse():
    r = rng(10)
    c = r.random(40)
    for w in (1, 3, 7):
        ref = torch.nn.functional.avg_pool1d(torch.from_numpy(c)[None, None], w, stride=1,
                                             padding=(w - 1) // 2, count_include_pad=True)[0, 0].numpy()
        np.testing.assert_allclose(O.average_pool(c, w), ref, rtol=0, atol=1e-15)
    imp = np.zeros(20)
    imp[1] = 7.0
    got = O.average_pool(imp, 7)
    expect = np.zeros(20)
    expect[0:5] = 1.0                       # positions within 3 of the impulse, zero padded at the edge
    np.testing.assert_allclose(got, expect, atol=1e-15)


def test_retained_indices_structure_and_brute_force():
    r = rng(11)
    N, s1, s2, kmid, w = 90, 3, 11, 9, 7
    c = r.random(N)
    idx = O.retained_indices(0, c, s1, s2, kmid, w)
    assert idx.tolist() == sorted(set(idx.tolist())) and len(idx) == s1 + s2 + kmid
    assert idx[:s1].tolist() == list(range(s1)) and idx[-s2:].tolist() == list(range(N - s2, N))
    pooled = [sum(c[j + o] for o in range(-3, 4) if 0 <= j + o < N) / w for j in range(N)]
    cand = sorted(range(s1, N - s2), key=lambda j: (-pooled[j], j))[:kmid]
    assert idx[s1:-s2].tolist() == sorted(cand)
    # budget larger than the middle range keeps everything; short inputs keep everything
    assert O.retained_indices(0, c, s1, s2, 10 ** 6, w).tolist() == list(range(N))
    assert O.retained_indices(0, c[:10], 4, 8, 5, w).tolist() == list(range(10))
    assert O.retained_indices(1, c, s1, s2, kmid, w).tolist() == list(range(N))
    assert O.retained_indices(2, c, s1, s2, kmid, w).tolist() == list(range(N))
    assert len(O.retained_indices(0, c, s1, s2, 0, w)) == s1 + s2


def test_lengths_closed_form():
    q, k, v = _toy_layer(seed=5)
    N = k.shape[1]
    for f, promote in ((0, True), (2, True), (3, False), (8, True)):
        out = O.compress_layer(q, k, v, n_hetero=f, sink=4, recent=16, mid=8, top_t=64, promote_center=promote)
        h = min(8, f + (1 if promote and f < 8 else 0))
        assert sorted(out["len"].tolist()) == sorted([N] * h + [4 + 16 + 8] * (8 - h))


# ---------------------------------------------------------------- Eq. 16 / Eq. 17
def test_hetero_schedule_golden_endpoints_and_monotone():
    with open(os.path.join(GOLDEN, "hetero_schedule.txt")) as fh:
        rows = [ln.split() for ln in fh if ln.strip() and not ln.startswith("#")]
    assert rows
    for n, beta, m, R, r, want in rows:
        assert O.hetero_count(int(n), float(beta), int(m), int(R), int(r)) == int(want)
    sched = [O.hetero_count(32, 0.25, 4, 32, r) for r in range(32)]
    assert all(a >= b for a, b in zip(sched, sched[1:]))
    assert O.hetero_count(32, 0.25, 4, 1, 0) == 8
    # exact linear values at layers where Eq. 16 is an integer: R-1 = 4 steps from 8 to 4
    assert [O.hetero_count(32, 0.25, 4, 5, r) for r in range(5)] == [8, 7, 6, 5, 4]


def test_mid_budget_conserves_layer_budget():
    for N, n, h, frac in ((131072, 8, 3, 0.4), (131072, 8, 2, 0.4), (30000, 32, 5, 0.4), (4096, 8, 1, 0.6)):
        s1, s2 = 4, 256
        B = frac * n * N
        k = O.mid_budget(B, N, h, n, s1, s2)
        used = h * N + (n - h) * (k + s1 + s2)
        assert used <= B < used + (n - h)
    assert O.mid_budget(0.1 * 8 * 1000, 1000, 3, 8, 4, 16) == 0        # budget already spent on full heads
    assert O.mid_budget(8 * 1000, 1000, 8, 8, 4, 16) == 0


# ---------------------------------------------------------------- Eq. 1: decode
def test_all_heads_heterogeneous_equals_full_attention():
    q, k, v = _toy_layer(seed=6)
    out = O.compress_layer(q, k, v, n_hetero=0, sink=4, recent=16, mid=8, top_t=64, force_class=1)
    kc, vc = O.gather_cache(k, v, out["idx"])
    qd = rng(12).normal(size=(8, k.shape[2]))
    got = O.decode_layer(qd, kc, vc)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(qd)[:, None, :], torch.from_numpy(k), torch.from_numpy(v))[:, 0, :]
    np.testing.assert_allclose(got, ref.numpy(), rtol=0, atol=1e-12)


def test_sink_and_recent_only_equals_masked_attention():
    q, k, v = _toy_layer(seed=7)
    N, d = k.shape[1], k.shape[2]
    s1, s2 = 4, 16
    out = O.compress_layer(q, k, v, n_hetero=0, sink=s1, recent=s2, mid=0, top_t=64, promote_center=False)
    assert (out["cls"] == 0).all()
    kc, vc = O.gather_cache(k, v, out["idx"])
    qd = rng(13).normal(size=(8, d))
    got = O.decode_layer(qd, kc, vc)
    keep = np.zeros(N, dtype=bool)
    keep[:s1] = True
    keep[N - s2:] = True
    for a in range(8):
        s = np.array([qd[a] @ k[a, j] / math.sqrt(d) if keep[j] else -np.inf for j in range(N)])
        p = np.exp(s - s[keep].max())
        p /= p.sum()
        np.testing.assert_allclose(got[a], p @ v[a], rtol=0, atol=1e-13)


def test_grouped_decode_and_append():
    r = rng(14)
    n, n_kv, N, d = 8, 2, 30, 4
    k = r.normal(size=(n_kv, N, d))
    v = r.normal(size=(n_kv, N, d))
    kc = [k[u].copy() for u in range(n_kv)]
    vc = [v[u].copy() for u in range(n_kv)]
    kn, vn = r.normal(size=(n_kv, d)), r.normal(size=(n_kv, d))
    O.append_layer(kc, vc, kn, vn)
    assert kc[0].shape == (N + 1, d)
    qd = r.normal(size=(n, d))
    got = O.decode_layer(qd, kc, vc)
    k_all = np.concatenate([k, kn[:, None, :]], axis=1)
    v_all = np.concatenate([v, vn[:, None, :]], axis=1)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(qd).reshape(n_kv, n // n_kv, d), torch.from_numpy(k_all), torch.from_numpy(v_all))
    np.testing.assert_allclose(got, ref.reshape(n, d).numpy(), rtol=0, atol=1e-13)


# ---------------------------------------------------------------------------
# Sec. V-G: the "No Cache" and "Compressed Cache" compensation methods
# ---------------------------------------------------------------------------
def test_recent_only_equals_masked_attention_with_a_longer_recent_window():
    # "No Cache" at cache size c: the c extra positions join the recent window
    q, k, v = _toy_layer(seed=21)
    N, d = k.shape[1], k.shape[2]
    s1, s2, c = 4, 16, 9
    out = O.compress_layer(q, k, v, n_hetero=0, sink=s1, recent=s2, mid=c, top_t=64, promote_center=False,
                           mid_policy=O.MID_RECENT)
    for u in range(k.shape[0]):
        assert out["idx"][u].tolist() == list(range(s1)) + list(range(N - s2 - c, N))
    kc, vc = O.gather_cache(k, v, out["idx"])
    qd = rng(22).normal(size=(8, d))
    got = O.decode_layer(qd, kc, vc)
    keep = np.zeros(N, dtype=bool)
    keep[:s1] = True
    keep[N - s2 - c:] = True
    for a in range(8):
        s = np.array([qd[a] @ k[a, j] / math.sqrt(d) if keep[j] else -np.inf for j in range(N)])
        p = np.exp(s - s[keep].max())
        p /= p.sum()
        np.testing.assert_allclose(got[a], p @ v[a], rtol=0, atol=1e-13)


@pytest.mark.parametrize("N,s1,s2,c", [(100, 4, 10, 7), (64, 0, 8, 56), (33, 3, 5, 1), (50, 4, 6, 40), (40, 4, 6, 1000)])
def test_mean_groups_partition_the_middle(N, s1, s2, c):
    b = O.mean_groups(N, s1, s2, c)
    M = N - s1 - s2
    cc = min(c, M)
    assert len(b) == cc + 1 and b[0] == s1 and b[-1] == N - s2
    sizes = np.diff(b)
    assert sizes.sum() == M and sizes.min() >= M // cc and sizes.max() <= -(-M // cc)   # contiguous, near-equal
    assert np.all(sizes > 0)


def test_compensation_rows_by_hand_loops():
    # every compensation row is the plain average of its group's rows (python loops, tiny case)
    r = rng(23)
    N, d, s1, s2, c = 23, 3, 2, 4, 5
    k, v = r.normal(size=(N, d)), r.normal(size=(N, d))
    kc, vc = O.compensated_cache(k, v, s1, s2, c, "f32")
    assert kc.shape == (s1 + c + s2, d)
    b = O.mean_groups(N, s1, s2, c)
    for x, xc in ((k, kc), (v, vc)):
        for g in range(c):
            for e in range(d):
                tot = 0.0
                for j in range(int(b[g]), int(b[g + 1])):
                    tot += x[j, e]
                assert abs(xc[s1 + g, e] - np.float32(tot / (b[g + 1] - b[g]))) <= 1e-7 * abs(tot) + 1e-12
        np.testing.assert_array_equal(xc[:s1], x[:s1])
        np.testing.assert_array_equal(xc[s1 + c:], x[N - s2:])


def test_compensation_special_cases():
    r = rng(24)
    N, d, s1, s2 = 40, 4, 3, 5
    k, v = r.normal(size=(N, d)), r.normal(size=(N, d))
    # one group per intermediate position (or more): nothing is averaged, the head keeps every row
    for c in (N - s1 - s2, 1000):
        kc, vc = O.compensated_cache(k, v, s1, s2, c, "f32")
        np.testing.assert_array_equal(kc, k)
        np.testing.assert_array_equal(vc, v)
    # constant rows: every compensation row is that constant
    kk = np.tile(np.array([[0.5, -1.25, 2.0, 3.0]]), (N, 1))
    kc, _ = O.compensated_cache(kk, v, s1, s2, 6, "bf16")
    np.testing.assert_array_equal(kc, np.tile(kk[:1], (s1 + 6 + s2, 1)))
    # conservation: sizes x means add up to the sum of the intermediate rows
    kc, _ = O.compensated_cache(k, v, s1, s2, 7, "f32")
    sizes = np.diff(O.mean_groups(N, s1, s2, 7))
    np.testing.assert_allclose((kc[s1:s1 + 7] * sizes[:, None]).sum(axis=0), k[s1:N - s2].sum(axis=0), rtol=1e-6)
    # c = 0: sinks and recent window only
    kc, _ = O.compensated_cache(k, v, s1, s2, 0, "f32")
    np.testing.assert_array_equal(kc, np.concatenate([k[:s1], k[N - s2:]]))


def test_round_to_storage_matches_library_casts():
    x = rng(25).normal(size=4096) * np.exp(rng(26).normal(size=4096) * 3)
    np.testing.assert_array_equal(O.round_to_storage(x, "bf16"),
                                  torch.from_numpy(x).to(torch.bfloat16).double().numpy())
    np.testing.assert_array_equal(O.round_to_storage(x, "f32"), torch.from_numpy(x).float().double().numpy())
    # a tie goes to the even mantissa
    assert O.round_to_storage(np.array([1.0 + 2.0 ** -8]), "bf16")[0] == 1.0
    assert O.round_to_storage(np.array([1.0 + 3 * 2.0 ** -8]), "bf16")[0] == 1.0 + 2.0 ** -6


def test_policy_pipeline_lengths_and_classes_do_not_depend_on_the_policy():
    q, k, v = _toy_layer(seed=27)
    base = O.compress_layer(q, k, v, n_hetero=2, sink=4, recent=16, mid=12, top_t=64)
    for pol in (O.MID_RECENT, O.MID_MEAN):
        out = O.compress_layer(q, k, v, n_hetero=2, sink=4, recent=16, mid=12, top_t=64, mid_policy=pol)
        assert out["cls"].tolist() == base["cls"].tolist()
        assert out["len"].tolist() == base["len"].tolist()
        kc, vc = O.gather_cache_policy(k, v, out["cls"], out["idx"], mid_policy=pol, sink=4, recent=16, mid=12,
                                       dtype="f32")
        assert [len(x) for x in kc] == base["len"].tolist()
        for u in range(k.shape[0]):
            if out["cls"][u] != 0:
                np.testing.assert_array_equal(kc[u], k[u])


def test_window_lse_is_the_normaliser_of_eq12():
    r = rng(31)
    L, N, d = 6, 40, 8
    q, k = r.normal(size=(L, d)) * 2, r.normal(size=(N, d)) * 2
    lse = O.window_lse(q, k)
    a = O.window_attention(q, k)
    s = (q @ k.T) / math.sqrt(d)
    for i in range(L):
        p_i = N - L + i
        # library cross-check on the visible keys of row i, and A' = exp(s - lse) entry by entry
        ref = torch.logsumexp(torch.from_numpy(s[i, :p_i + 1]), dim=0).item()
        assert abs(lse[i] - ref) < 1e-12
        np.testing.assert_allclose(np.exp(s[i, :p_i + 1] - lse[i]), a[i, :p_i + 1], rtol=1e-12, atol=0)
        assert np.all(a[i, p_i + 1:] == 0)


def test_exact_semantic_vector_closed_forms():
    """Eq. 1-2 with all keys equal: row i of the causal softmax is uniform over its i + 1 keys, so the column mean is
    C[j] = (1/N) sum_{i >= j} 1/(i + 1); with all value rows equal to c the semantic vector is c itself."""
    rng = np.random.default_rng(5)
    N, d = 37, 8
    q = rng.normal(size=(N, d))
    k = np.tile(rng.normal(size=(1, d)), (N, 1))
    v = rng.normal(size=(N, d))
    c_closed = np.array([sum(1.0 / (i + 1) for i in range(j, N)) / N for j in range(N)])
    np.testing.assert_allclose(O.window_scores(q[None], k), c_closed, rtol=0, atol=1e-14)
    np.testing.assert_allclose(O.exact_semantic_vector(q, k, v), c_closed @ v, rtol=0, atol=1e-14)
    const = np.tile(rng.normal(size=(1, d)), (N, 1))
    np.testing.assert_allclose(O.exact_semantic_vector(q, rng.normal(size=(N, d)), const), const[0], rtol=0, atol=1e-14)
