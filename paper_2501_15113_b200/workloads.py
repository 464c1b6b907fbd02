"""Seeded synthetic inputs shaped like the paper's long-context workloads.

This module only draws random tensors and fills in workload parameters; it
holds none of the method's arithmetic (layer schedules and budgets are passed
in by the caller), so both the CUDA library's tests and the CPU oracle's tests can be fed from it
without sharing method code.

Value recipe (Sec. V-C/V-E shapes: Llama-2-7B is MHA 32 x 128, Mistral-7B is
GQA 32 q / 8 kv x 128; inputs of up to ~30K tokens; 40 % budgets):
  * Q, K, V elements ~ Normal(0, var) * u_head with one u_head ~ U[0.5, 2]
    per (layer, head) and per tensor; var = 1 for the toy case and
    1/sqrt(head_dim) otherwise (read as a variance, so q.k/sqrt(d) has
    standard deviation u_q*u_k/sqrt(d)).
  * "planted" heads get a constant offset added to every row of V, which moves
    their semantic vector away from the layer's center: the separator then has
    a known answer.
  * the toy case scales the key at position 0 by 8 (an attention sink).
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import torch


@dataclasses.dataclass
class Workload:
    name: str
    batch: int
    n_layers: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    seq_lens: List[int]
    dtype: str                      # "f32" | "bf16"
    sink: int
    recent: int
    window: int
    mid_budget: List[int]           # per layer
    n_hetero: List[List[int]]       # [batch][layer] far heads (the promoted closest head is extra)
    decode_steps: int
    top_t: int = 256
    pool_kernel: int = 7
    promote_center: bool = True
    seed: int = 0
    variance: float = 1.0
    plant_offset: float = 1.0
    plant_signed: bool = True       # random sign per (head, dim); False: +offset on every dim
    planted: Optional[List[List[List[int]]]] = None  # [batch][layer] -> kv heads
    sink_key_scale: float = 1.0
    heavy_keys: int = 0             # keys per head, at seeded positions, scaled by heavy_scale ("heavy hitters")
    heavy_scale: float = 1.0
    note: str = ""
    mid_by_seq: Optional[List[List[int]]] = None   # [batch][layer]: overrides mid_budget where budgets differ by sequence
    budget_frac: float = 0.0        # > 0: the library derives the budgets itself (Eq. 17) from this fraction

    @property
    def group(self) -> int:
        return self.n_heads // self.n_kv_heads

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_size(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def full_heads(self, b: int, r: int) -> int:
        f = self.n_hetero[b][r]
        return min(self.n_kv_heads, f + (1 if self.promote_center and f < self.n_kv_heads else 0))

    def mid_of(self, b: int, r: int) -> int:
        """Middle budget of (sequence, layer)."""
        return self.mid_by_seq[b][r] if self.mid_by_seq is not None else self.mid_budget[r]

    def kept_len(self, b: int, r: int) -> int:
        """Rows a non-full head keeps after compression (before any append)."""
        N = self.seq_lens[b]
        if N <= self.sink + self.recent:
            return N
        return self.sink + self.recent + min(self.mid_of(b, r), N - self.sink - self.recent)

    def retained_rows(self) -> int:
        tot = 0
        for b in range(self.batch):
            for r in range(self.n_layers):
                h = self.full_heads(b, r)
                tot += h * self.seq_lens[b] + (self.n_kv_heads - h) * self.kept_len(b, r)
        return tot

    def describe(self) -> dict:
        return {
            "workload": self.name, "batch": self.batch, "n_layers": self.n_layers,
            "n_heads": self.n_heads, "n_kv_heads": self.n_kv_heads, "head_dim": self.head_dim,
            "seq_len": self.seq_lens[0] if self.batch == 1 else self.seq_lens,
            "sink": self.sink, "recent": self.recent, "window": self.window,
            "mid_budget": self.mid_budget[0] if len(set(self.mid_budget)) == 1 else self.mid_budget,
            "top_t": self.top_t, "pool_kernel": self.pool_kernel, "decode_steps": self.decode_steps,
            "seed": self.seed,
        }


def _cpu_gen(*keys: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    s = 0x9E3779B97F4A7C15
    for kx in keys:
        s = (s * 6364136223846793005 + 1442695040888963407 + int(kx)) % (1 << 63)
    g.manual_seed(s)
    return g


def _dev_gen(device, *keys: int) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x2545F4914F6CDD1D
    for kx in keys:
        s = (s * 6364136223846793005 + 1442695040888963407 + int(kx)) % (1 << 63)
    g.manual_seed(s)
    return g


def _choose_planted(wl: Workload) -> List[List[List[int]]]:
    out = []
    for b in range(wl.batch):
        per_layer = []
        for r in range(wl.n_layers):
            g = _cpu_gen(wl.seed, 101, b, r)
            perm = torch.randperm(wl.n_kv_heads, generator=g).tolist()
            per_layer.append(sorted(perm[:wl.n_hetero[b][r]]))
        out.append(per_layer)
    return out


def head_scales(wl: Workload, b: int, r: int):
    """u_head ~ U[0.5, 2] for Q (n_heads) and K, V (n_kv_heads) of one layer."""
    g = _cpu_gen(wl.seed, 202, b, r)
    if wl.name.startswith("toy"):
        return (torch.ones(wl.n_heads), torch.ones(wl.n_kv_heads), torch.ones(wl.n_kv_heads))
    uq = 0.5 + 1.5 * torch.rand(wl.n_heads, generator=g)
    uk = 0.5 + 1.5 * torch.rand(wl.n_kv_heads, generator=g)
    uv = 0.5 + 1.5 * torch.rand(wl.n_kv_heads, generator=g)
    return uq, uk, uv


def gen_layer(wl: Workload, b: int, r: int, device="cpu"):
    """(q_win [n, L, d], k [n_kv, N, d], v [n_kv, N, d]) of one layer, in wl's dtype."""
    N, d, L = wl.seq_lens[b], wl.head_dim, wl.window
    std = math.sqrt(wl.variance)
    uq, uk, uv = head_scales(wl, b, r)
    g = _dev_gen(device, wl.seed, 303, b, r)
    q = torch.randn(wl.n_heads, L, d, generator=g, device=device, dtype=torch.float32)
    k = torch.randn(wl.n_kv_heads, N, d, generator=g, device=device, dtype=torch.float32)
    v = torch.randn(wl.n_kv_heads, N, d, generator=g, device=device, dtype=torch.float32)
    q *= (std * uq).to(device)[:, None, None]
    k *= (std * uk).to(device)[:, None, None]
    v *= (std * uv).to(device)[:, None, None]
    if wl.sink_key_scale != 1.0:
        k[:, 0, :] *= wl.sink_key_scale
    if wl.heavy_keys > 0:
        gh = _cpu_gen(wl.seed, 606, b, r)
        for h in range(wl.n_kv_heads):
            pos = torch.randint(0, N, (wl.heavy_keys,), generator=gh).to(device)
            k[h, pos, :] *= wl.heavy_scale
    planted = wl.planted[b][r] if wl.planted is not None else []
    for h in planted:
        if wl.plant_signed:
            gs = _cpu_gen(wl.seed, 404, b, r, h)
            sign = (torch.randint(0, 2, (d,), generator=gs).float() * 2 - 1).to(device)
            v[h] += wl.plant_offset * sign[None, :]
        else:
            v[h] += wl.plant_offset
    dt = wl.torch_dtype
    return q.to(dt), k.to(dt), v.to(dt)


def gen_decode_step(wl: Workload, step: int, device="cpu"):
    """(q [B, R, n, d], k_new [B, R, n_kv, d], v_new [B, R, n_kv, d]) of one decode step."""
    std = math.sqrt(wl.variance)
    g = _dev_gen(device, wl.seed, 505, step)
    shp_q = (wl.batch, wl.n_layers, wl.n_heads, wl.head_dim)
    shp_kv = (wl.batch, wl.n_layers, wl.n_kv_heads, wl.head_dim)
    q = torch.randn(shp_q, generator=g, device=device, dtype=torch.float32) * std
    k = torch.randn(shp_kv, generator=g, device=device, dtype=torch.float32) * std
    v = torch.randn(shp_kv, generator=g, device=device, dtype=torch.float32) * std
    dt = wl.torch_dtype
    return q.to(dt), k.to(dt), v.to(dt)


def materialize(wl: Workload, device="cpu"):
    """Whole-model inputs: per sequence q_win [R, n, L, d], k, v [R, n_kv, N_b, d]."""
    qs, ks, vs = [], [], []
    dt = wl.torch_dtype
    for b in range(wl.batch):
        N = wl.seq_lens[b]
        q = torch.empty(wl.n_layers, wl.n_heads, wl.window, wl.head_dim, device=device, dtype=dt)
        k = torch.empty(wl.n_layers, wl.n_kv_heads, N, wl.head_dim, device=device, dtype=dt)
        v = torch.empty_like(k)
        for r in range(wl.n_layers):
            q[r], k[r], v[r] = gen_layer(wl, b, r, device)
        qs.append(q)
        ks.append(k)
        vs.append(v)
    return qs, ks, vs


# ---------------------------------------------------------------------------
# configuration tables
# ---------------------------------------------------------------------------
def _round_half_up(x: float) -> int:
    return int(math.floor(x + 0.5))


def _finish(wl: Workload) -> Workload:
    if wl.planted is None:
        wl.planted = _choose_planted(wl)
    return wl


def toy(seed: int = 0) -> Workload:
    """Single layer, MHA 8 heads x 64, 512 tokens, fp32; heads 2 and 5 carry a
    +3.0 offset on V; key 0 scaled by 8."""
    wl = Workload(name="toy_mha8_d64_n512_f32", batch=1, n_layers=1, n_heads=8, n_kv_heads=8,
                  head_dim=64, seq_lens=[512], dtype="f32", sink=4, recent=32, window=16,
                  mid_budget=[32], n_hetero=[[2]], decode_steps=16, seed=seed, variance=1.0,
                  plant_offset=3.0, plant_signed=False, planted=[[[2, 5]]], sink_key_scale=8.0)
    return wl


def llama2_7b(seq_len: int = 32768, n_layers: int = 32, decode_steps: int = 256, seed: int = 1) -> Workload:
    n = 32
    wl = Workload(name=f"llama2_7b_mha32_d128_n{seq_len}_bf16", batch=1, n_layers=n_layers, n_heads=n,
                  n_kv_heads=n, head_dim=128, seq_lens=[seq_len], dtype="bf16", sink=4, recent=256,
                  window=32, mid_budget=[512] * n_layers, n_hetero=[[4] * n_layers],
                  decode_steps=decode_steps, seed=seed, variance=1.0 / math.sqrt(128))
    return _finish(wl)


def llama3_8b(n_hetero: List[int], mid_budget: List[int], seq_len: int = 131072,
              decode_steps: int = 128, seed: int = 2) -> Workload:
    """n_hetero and mid_budget (one entry per layer) come from the caller: the
    layer schedule and the budget formula are method arithmetic and live with
    the library (and, separately, with the oracle), not here."""
    n, n_kv, s1, s2 = 32, 8, 4, 256
    n_layers = len(n_hetero)
    f, mids = list(n_hetero), list(mid_budget)
    wl = Workload(name=f"llama3_8b_gqa32x8_d128_n{seq_len}_bf16", batch=1, n_layers=n_layers, n_heads=n,
                  n_kv_heads=n_kv, head_dim=128, seq_lens=[seq_len], dtype="bf16", sink=s1, recent=s2,
                  window=32, mid_budget=mids, n_hetero=[f], decode_steps=decode_steps, seed=seed,
                  variance=1.0 / math.sqrt(128))
    return _finish(wl)


def mistral_batch(batch: int = 16, lo: int = 8192, hi: int = 32768, n_layers: int = 32,
                  decode_steps: int = 512, seed: int = 3) -> Workload:
    n, n_kv = 32, 8
    g = _cpu_gen(seed, 606)
    lens = torch.randint(lo, hi + 1, (batch,), generator=g).tolist()
    frac = (0.10 + 0.30 * torch.rand(batch, generator=g)).tolist()
    nh = [[max(0, min(n_kv, _round_half_up(n_kv * frac[b])))] * n_layers for b in range(batch)]
    wl = Workload(name=f"mistral_7b_gqa32x8_d128_b{batch}_n{lo}-{hi}_bf16", batch=batch, n_layers=n_layers,
                  n_heads=n, n_kv_heads=n_kv, head_dim=128, seq_lens=lens, dtype="bf16", sink=4,
                  recent=128, window=32, mid_budget=[256] * n_layers, n_hetero=nh,
                  decode_steps=decode_steps, seed=seed, variance=1.0 / math.sqrt(128))
    return _finish(wl)


def budget_sweep_point(n_hetero: int, mid: int, seq_len: int = 65536, batch: int = 8,
                       decode_steps: int = 64, seed: int = 4) -> Workload:
    n, n_kv = 32, 8
    wl = Workload(name=f"sweep_gqa32x8_d128_b{batch}_n{seq_len}_h{n_hetero}_k{mid}_bf16", batch=batch,
                  n_layers=1, n_heads=n, n_kv_heads=n_kv, head_dim=128, seq_lens=[seq_len] * batch,
                  dtype="bf16", sink=4, recent=256, window=32, mid_budget=[mid],
                  n_hetero=[[n_hetero]] * batch, decode_steps=decode_steps, seed=seed,
                  variance=1.0 / math.sqrt(128))
    return _finish(wl)


SWEEP_HETERO = (0, 1, 2, 4, 8)
SWEEP_MID = (64, 256, 1024)
