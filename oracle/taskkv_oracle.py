"""CPU oracle for the Task-KV hot path (arXiv 2501.15113): test infrastructure only.

This module is the slow, plain definition that the CUDA library is checked
against.  It is NOT part of the product: only the tests, the smoke check and
the benchmark's CPU-baseline leg may import it, and it imports nothing from
the CUDA package.  All floating point is numpy float64; inputs arrive as the
exact fp32 / bf16 values the GPU sees, widened to float64.

The method is a heuristic pipeline, so the oracle takes the algorithm's steps
in the paper's order and notation:

    Eq. 12   A' = Softmax(Q[-L:,:] K^T / sqrt(d) + M')        window_attention
    Eq. 13   C  = sum_i A'[i,:] / L                           column_mean
    Eq. 14   I  = Top_k(C, t)                                 top_indices
    Eq. 15   v' = C[I] . V[I,:]                               semantic_vector
    Eq. 8    center = mean of the layer's semantic vectors    semantic_center
    Eq. 7    offset delta_j = v_j - center, L2 norm           center_distances
    Sec. IV-A  rank far -> near, f(r) far heads, + nearest    semantic_separator
    Eq. 16   f(r) = n*beta - (n*beta - m)/(R-1) * r           hetero_count
    Sec. IV-B  sinks + recent + k middle activations          retained_indices
    Sec. V-D   average pooling (kernel 7) of the scores       average_pool
    Eq. 17   k = (B - N f(r))/(n - f(r)) - s1 - s2            mid_budget
    Eq. 1    decode row: softmax(q K^T / sqrt(d)) V           decode_attention
    Eq. 1-2  exact semantic vector from the N x N weights     exact_semantic_vector
    Sec. V-G   the two other compensation methods compared    recent_only_indices,
               with the middle activations                    mean_groups, compensated_cache

Readings where the paper is silent or garbled are stated in each docstring.

Pins (tests/test_oracle_pins.py) fix every function except the ones listed
here as "parity unpinned": the grouped-query rule of column_mean (mean over
the group's G*L softmax rows), the zero-padded divisor-w pooling convention,
round-half-up in hetero_count, floor in mid_budget and lowest-index tie-breaks
are readings of this build, not statements of the paper; the paper prints no
worked numeric example of C, v' or a distance.  Of the Sec. V-G variants the
paper gives only a figure caption: the contiguous near-equal groups of
mean_groups and the rounding of a compensation row to the cache's storage
type are readings too.
"""
from __future__ import annotations

import math

import numpy as np

F64 = np.float64

CLASS_NON_HETERO = 0
CLASS_HETERO = 1
CLASS_CENTER = 2


# --------------------------------------------------------------------------
# Eq. 12 / Eq. 13: observation-window weights and their column mean
# --------------------------------------------------------------------------
def window_attention(q_win: np.ndarray, k: np.ndarray) -> np.ndarray:
    """Eq. 12 (Sec. IV-A): local weight matrix A' in R^{L x N}.

    q_win is Q[-L:, :] (L x d), k is K (N x d).  Window row i is the query of
    absolute position N-L+i.  The paper gives the mask M' as L x L while A' is
    L x N; reading: the causal mask acts on the last L columns only (row i may
    not see keys after its own position), the first N-L columns are visible to
    every window row.
    """
    q_win = np.asarray(q_win, dtype=F64)
    k = np.asarray(k, dtype=F64)
    L, d = q_win.shape
    N = k.shape[0]
    if not (1 <= L <= N):
        raise ValueError("window must satisfy 1 <= L <= N")
    s = (q_win @ k.T) / math.sqrt(d)
    pos = N - L + np.arange(L)
    hidden = np.arange(N)[None, :] > pos[:, None]
    s = np.where(hidden, -np.inf, s)
    s = s - s.max(axis=1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=1, keepdims=True)


def window_lse(q_win: np.ndarray, k: np.ndarray) -> np.ndarray:
    """Natural-log normaliser of every row of Eq. 12: lse_i = log sum_j exp(s_ij) over the keys row i may see, so
    that A'[i, j] = exp(s_ij - lse_i).  This is what an attention kernel run over the prompt returns as its
    log-sum-exp for the last L query rows; a caller that has it can hand it over instead of having it recomputed."""
    q_win = np.asarray(q_win, dtype=F64)
    k = np.asarray(k, dtype=F64)
    L, d = q_win.shape
    N = k.shape[0]
    s = (q_win @ k.T) / math.sqrt(d)
    pos = N - L + np.arange(L)
    s = np.where(np.arange(N)[None, :] > pos[:, None], -np.inf, s)
    m = s.max(axis=1)
    return m + np.log(np.exp(s - m[:, None]).sum(axis=1))


def column_mean(a_rows: np.ndarray) -> np.ndarray:
    """Eq. 13: C = sum_i A'[i,:] / L, a vector of length N.

    For grouped-query attention the paper does not say how the G query heads
    that share one K/V pair are combined; reading: stack the G windows and
    take the mean over all G*L normalised rows, so one C per KV head (G = 1 is
    exactly Eq. 13).
    """
    a_rows = np.asarray(a_rows, dtype=F64)
    return a_rows.sum(axis=0) / a_rows.shape[0]


def window_scores(q_group: np.ndarray, k: np.ndarray) -> np.ndarray:
    """Eq. 12 then Eq. 13 for one KV head: q_group is (G, L, d), k is (N, d)."""
    q_group = np.asarray(q_group, dtype=F64)
    rows = [window_attention(q_group[g], k) for g in range(q_group.shape[0])]
    return column_mean(np.concatenate(rows, axis=0))


# --------------------------------------------------------------------------
# Eq. 14: top-k selection with the lowest index winning ties
# --------------------------------------------------------------------------
def top_indices(score: np.ndarray, count: int) -> np.ndarray:
    """Eq. 14: positions of the `count` largest scores, returned ascending.

    count is clamped to len(score).  Ties are not discussed in the paper;
    reading: of equal scores the smaller position is taken first.
    """
    score = np.asarray(score, dtype=F64)
    count = max(0, min(int(count), score.shape[0]))
    if count == 0:
        return np.zeros(0, dtype=np.int64)
    # stable sort of the negated scores: equal scores keep ascending position
    order = np.argsort(-score, kind="stable")
    return np.sort(order[:count]).astype(np.int64)


# --------------------------------------------------------------------------
# Eq. 15: semantic vector
# --------------------------------------------------------------------------
def semantic_vector(c: np.ndarray, v: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """Eq. 15: v' = sum_{j in I} C[j] V[j,:]  (1 x d).

    The printed "C[I,:]" indexes a vector; reading: the weights are the
    selected entries of C, not renormalised (with I = all positions this is
    exactly the Eq. 2 product).
    """
    c = np.asarray(c, dtype=F64)
    v = np.asarray(v, dtype=F64)
    idx = np.asarray(idx, dtype=np.int64)
    return c[idx] @ v[idx, :]


def exact_semantic_vector(q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
    """Eq. 1-2 (Sec. III-A): v = (sum_i A[i,:] / N) V with the full causal A."""
    q = np.asarray(q, dtype=F64)
    a = window_attention(q, k)          # L = N: every row, causal mask N x N
    return column_mean(a) @ np.asarray(v, dtype=F64)


# --------------------------------------------------------------------------
# Eq. 7-8 and Sec. IV-A: center, distance, separator
# --------------------------------------------------------------------------
def semantic_center(vectors: np.ndarray) -> np.ndarray:
    """Eq. 8: the mean vector of the layer's n semantic vectors (n x d -> d)."""
    vectors = np.asarray(vectors, dtype=F64)
    return vectors.sum(axis=0) / vectors.shape[0]


def center_distances(vectors: np.ndarray) -> np.ndarray:
    """Eq. 7 with the L2 norm of Sec. III-C: ||v_j - center||_2 per head."""
    vectors = np.asarray(vectors, dtype=F64)
    delta = vectors - semantic_center(vectors)[None, :]
    return np.sqrt((delta * delta).sum(axis=1))


def hetero_count(n: int, beta: float, m: int, R: int, r: int) -> int:
    """Eq. 16: f(r) = n*beta - (n*beta - m)/(R-1) * r, r = 0..R-1.

    f(r) is generally fractional; reading: round half up, clamp to [0, n].
    With a single layer the interpolation term is absent and f(0) = n*beta.
    """
    top = n * float(beta)
    val = top if R <= 1 else top - (top - m) / (R - 1) * r
    return int(min(n, max(0, math.floor(val + 0.5))))


def semantic_separator(dist: np.ndarray, f: int, promote_center: bool = True) -> np.ndarray:
    """Sec. IV-A: heads ranked far -> near; the f farthest are heterogeneous;
    of the remaining heads the one closest to the center joins them.

    Returns one class per head: 1 heterogeneous, 2 the promoted closest head,
    0 otherwise.  Reading: f counts the far heads only (the paper tests m = 0,
    which would be impossible if the promoted head were counted in f); equal
    distances rank the smaller head index first.
    """
    dist = np.asarray(dist, dtype=F64)
    n = dist.shape[0]
    f = max(0, min(int(f), n))
    cls = np.zeros(n, dtype=np.uint8)
    far_first = np.argsort(-dist, kind="stable")
    cls[far_first[:f]] = CLASS_HETERO
    if promote_center and f < n:
        rest = np.flatnonzero(cls == CLASS_NON_HETERO)
        near_first = rest[np.argsort(dist[rest], kind="stable")]
        cls[near_first[0]] = CLASS_CENTER
    return cls


# --------------------------------------------------------------------------
# Sec. IV-B and Sec. V-D: what a non-heterogeneous head keeps
# --------------------------------------------------------------------------
def average_pool(c: np.ndarray, w: int) -> np.ndarray:
    """Sec. V-D: average pooling of the scores with kernel w (7 in the paper).

    Reading: stride 1, centred, zeros outside [0, N), divisor always w; w = 1
    leaves the scores unchanged.
    """
    c = np.asarray(c, dtype=F64)
    if w <= 1:
        return c.copy()
    if w % 2 == 0:
        raise ValueError("pooling kernel must be odd")
    h = (w - 1) // 2
    padded = np.concatenate([np.zeros(h), c, np.zeros(h)])
    out = np.zeros_like(c)
    for off in range(w):
        out += padded[off:off + c.shape[0]]
    return out / w


def retained_indices(cls: int, c: np.ndarray, sink: int, recent: int,
                     mid_budget: int, pool_kernel: int) -> np.ndarray:
    """Sec. IV-B: the positions one head keeps, ascending.

    Heterogeneous heads (and the promoted closest head) keep every position.
    Other heads keep the first `sink` positions, the last `recent` positions
    and the `mid_budget` positions of highest pooled score among the
    intermediate positions [sink, N - recent).  If N <= sink + recent the head
    keeps everything.
    """
    c = np.asarray(c, dtype=F64)
    N = c.shape[0]
    if cls != CLASS_NON_HETERO or N <= sink + recent:
        return np.arange(N, dtype=np.int64)
    pooled = average_pool(c, pool_kernel)
    mid = sink + top_indices(pooled[sink:N - recent], mid_budget)
    return np.concatenate([np.arange(sink, dtype=np.int64), mid,
                           np.arange(N - recent, N, dtype=np.int64)])


def mid_budget(B_tokens: float, N: int, h_full: int, n: int, sink: int, recent: int) -> int:
    """Eq. 17: k = (B - N*h)/(n - h) - s1 - s2.

    B is the layer's budget in token*head units.  Reading: h is the number of
    heads that really keep the full cache in that layer (f(r) plus the promoted
    head), the quotient is floored so the layer total never exceeds B, and k is
    clamped to [0, N - s1 - s2].  With every head full k is unused (0).
    """
    if n <= h_full:
        return 0
    k = math.floor((B_tokens - N * h_full) / (n - h_full)) - sink - recent
    return int(max(0, min(k, max(0, N - sink - recent))))


# --------------------------------------------------------------------------
# Eq. 1: one decode row over a head's retained cache
# --------------------------------------------------------------------------
def decode_attention(q: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray) -> np.ndarray:
    """Eq. 1 for a single new query: softmax(q K^T / sqrt(d)) V over all cached
    rows (every cached position precedes the query, so no mask applies)."""
    q = np.asarray(q, dtype=F64)
    k_cache = np.asarray(k_cache, dtype=F64)
    v_cache = np.asarray(v_cache, dtype=F64)
    s = (k_cache @ q) / math.sqrt(q.shape[0])
    s = s - s.max()
    e = np.exp(s)
    return (e / e.sum()) @ v_cache


# --------------------------------------------------------------------------
# Sec. V-G: the two other information-compensation methods the paper compares
# the middle activations with, at the same cache size
# --------------------------------------------------------------------------
MID_SELECT = 0   # middle activations (the method itself, Sec. IV-B)
MID_RECENT = 1   # "No Cache": the budget is added to the recent window
MID_MEAN = 2     # "Compressed Cache": one averaged compensation row per group


def recent_only_indices(N: int, sink: int, recent: int, mid_budget: int) -> np.ndarray:
    """"No Cache" of Sec. V-G: a non-heterogeneous head keeps the sinks and the
    last recent + mid_budget positions, nothing from the middle."""
    if N <= sink + recent:
        return np.arange(N, dtype=np.int64)
    extra = min(mid_budget, N - sink - recent)
    return np.concatenate([np.arange(sink, dtype=np.int64),
                           np.arange(N - recent - extra, N, dtype=np.int64)])


def mean_groups(N: int, sink: int, recent: int, count: int) -> np.ndarray:
    """"Compressed Cache" of Sec. V-G: the intermediate positions [sink, N - recent)
    are divided into `count` groups.  Reading: contiguous groups in position
    order whose sizes differ by at most one, group g starting at
    sink + floor(g * M / count), M = N - sink - recent.  Returns the count + 1
    boundaries (the last one is N - recent)."""
    M = N - sink - recent
    count = min(count, M)
    return np.array([sink + (g * M) // count for g in range(count)] + [N - recent], dtype=np.int64)


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """A float64 array rounded once, to nearest even, to the cache's element type
    ("f32" or "bf16": 8 significant bits), returned as float64."""
    x = np.asarray(x, dtype=F64)
    if dtype == "f32":
        return x.astype(np.float32).astype(F64)
    m, e = np.frexp(x)
    return np.ldexp(np.round(m * 256.0) / 256.0, e)


def compensated_cache(k_u: np.ndarray, v_u: np.ndarray, sink: int, recent: int,
                      count: int, dtype: str) -> tuple:
    """"Compressed Cache" of Sec. V-G for one head: sinks, then one compensation
    row per group (the arithmetic mean of the group's K rows resp. V rows, stored
    in the cache's element type), then the recent window."""
    k_u = np.asarray(k_u, dtype=F64)
    v_u = np.asarray(v_u, dtype=F64)
    N = k_u.shape[0]
    if N <= sink + recent or count >= N - sink - recent:
        return k_u.copy(), v_u.copy()
    b = mean_groups(N, sink, recent, count)
    out = []
    for x in (k_u, v_u):
        means = np.stack([x[b[g]:b[g + 1]].sum(axis=0) / (b[g + 1] - b[g]) for g in range(len(b) - 1)]) \
            if count > 0 else np.zeros((0, x.shape[1]))
        out.append(np.concatenate([x[:sink], round_to_storage(means, dtype), x[N - recent:]]))
    return out[0], out[1]


# --------------------------------------------------------------------------
# The pipeline for one layer of one sequence, in the paper's order
# --------------------------------------------------------------------------
def compress_layer(q_win: np.ndarray, k: np.ndarray, v: np.ndarray, *,
                   n_hetero: int, sink: int, recent: int, mid: int,
                   top_t: int = 256, pool_kernel: int = 7,
                   promote_center: bool = True, force_class: int = -1,
                   mid_policy: int = MID_SELECT) -> dict:
    """Prefill-side compression of one layer (Sec. IV-A then IV-B).

    q_win: (n_heads, L, d) observation-window queries; k, v: (n_kv, N, d).
    Heads are classified per KV head (n = n_kv in Eq. 16/17) because V, and so
    the semantic vector of Eq. 15, exists once per KV head.
    force_class: -1 run the separator; 1 every head heterogeneous; 0 none.
    mid_policy: what a non-heterogeneous head keeps besides sinks and recent
    window (Sec. V-G): the middle activations, more recent positions, or
    compensation rows (then "idx" lists the first position of each group).
    Returns C, top-t indices, semantic vectors, center, distances, classes,
    retained indices and lengths per KV head.
    """
    q_win = np.asarray(q_win, dtype=F64)
    k = np.asarray(k, dtype=F64)
    v = np.asarray(v, dtype=F64)
    n_heads, L, d = q_win.shape
    n_kv, N, _ = k.shape
    G = n_heads // n_kv
    C = np.stack([window_scores(q_win[u * G:(u + 1) * G], k[u]) for u in range(n_kv)])
    top = [top_indices(C[u], top_t) for u in range(n_kv)]
    sem = np.stack([semantic_vector(C[u], v[u], top[u]) for u in range(n_kv)])
    dist = center_distances(sem)
    if force_class == 1:
        cls = np.full(n_kv, CLASS_HETERO, dtype=np.uint8)
    elif force_class == 0:
        cls = np.zeros(n_kv, dtype=np.uint8)
    else:
        cls = semantic_separator(dist, n_hetero, promote_center)
    def keep(u: int) -> np.ndarray:
        if cls[u] != CLASS_NON_HETERO or mid_policy == MID_SELECT or N <= sink + recent:
            return retained_indices(int(cls[u]), C[u], sink, recent, mid, pool_kernel)
        if mid_policy == MID_RECENT:
            return recent_only_indices(N, sink, recent, mid)
        if mid >= N - sink - recent:
            return np.arange(N, dtype=np.int64)
        return np.concatenate([np.arange(sink, dtype=np.int64), mean_groups(N, sink, recent, mid)[:-1],
                               np.arange(N - recent, N, dtype=np.int64)])
    idx = [keep(u) for u in range(n_kv)]
    return {
        "C": C, "top": top, "sem": sem, "center": semantic_center(sem), "dist": dist,
        "cls": cls, "idx": idx, "len": np.array([len(i) for i in idx], dtype=np.int64),
    }


def gather_cache(k: np.ndarray, v: np.ndarray, idx: list) -> tuple:
    """Sec. IV-B: the per-head compacted cache, rows in ascending position."""
    return ([np.asarray(k[u], dtype=F64)[idx[u]] for u in range(len(idx))],
            [np.asarray(v[u], dtype=F64)[idx[u]] for u in range(len(idx))])


def gather_cache_policy(k: np.ndarray, v: np.ndarray, cls: np.ndarray, idx: list, *, mid_policy: int,
                        sink: int, recent: int, mid: int, dtype: str) -> tuple:
    """The per-head cache under a Sec. V-G policy: as gather_cache, except that
    with MID_MEAN a non-heterogeneous head holds compensation rows."""
    if mid_policy != MID_MEAN:
        return gather_cache(k, v, idx)
    kc, vc = [], []
    for u in range(len(idx)):
        if cls[u] == CLASS_NON_HETERO:
            a, b = compensated_cache(k[u], v[u], sink, recent, mid, dtype)
        else:
            a, b = np.asarray(k[u], dtype=F64).copy(), np.asarray(v[u], dtype=F64).copy()
        kc.append(a)
        vc.append(b)
    return kc, vc


def decode_layer(q: np.ndarray, k_cache: list, v_cache: list) -> np.ndarray:
    """One decode step of one layer: q is (n_heads, d); query head a reads the
    cache of KV head a // G.  Returns (n_heads, d) in float64."""
    q = np.asarray(q, dtype=F64)
    n_heads = q.shape[0]
    G = n_heads // len(k_cache)
    return np.stack([decode_attention(q[a], k_cache[a // G], v_cache[a // G])
                     for a in range(n_heads)])


def append_layer(k_cache: list, v_cache: list, k_new: np.ndarray, v_new: np.ndarray) -> None:
    """Decode-time growth: the new token's k, v join every head's cache (the
    paper does not evict again while generating)."""
    for u in range(len(k_cache)):
        k_cache[u] = np.concatenate([k_cache[u], np.asarray(k_new[u], dtype=F64)[None, :]])
        v_cache[u] = np.concatenate([v_cache[u], np.asarray(v_new[u], dtype=F64)[None, :]])
