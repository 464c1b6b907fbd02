"""The five benchmark workloads.  Layer schedules (Eq. 16) and budgets (Eq. 17) are method arithmetic: by default
they come from the library's own host helpers; a caller that must not load the library (the CPU oracle's timing
run) passes its own pair of functions as `helpers = (hetero_count, mid_budget)`."""
from __future__ import annotations

from . import workloads as W


def _library_helpers():
    from .binding import taskkv_hetero_count, taskkv_mid_budget
    return taskkv_hetero_count, taskkv_mid_budget


def config1_toy() -> W.Workload:
    return W.toy()


def config2_llama2(seq_len: int = 32768, n_layers: int = 32, decode_steps: int = 256) -> W.Workload:
    return W.llama2_7b(seq_len=seq_len, n_layers=n_layers, decode_steps=decode_steps)


def config3_llama3(seq_len: int = 131072, n_layers: int = 32, decode_steps: int = 128,
                   budget_frac: float = 0.4, helpers=None) -> W.Workload:
    """GQA 32q/8kv; beta 0.3, m 1 counted over the 8 KV heads; the retained cache is
    budget_frac of the full one, which fixes the middle budget of every layer."""
    hetero_count, mid_budget = helpers or _library_helpers()
    n_kv, s1, s2 = 8, 4, 256
    f = [hetero_count(n_kv, 0.3, 1, n_layers, r) for r in range(n_layers)]
    mids = [mid_budget(budget_frac * n_kv * seq_len, seq_len, min(n_kv, f[r] + 1), n_kv, s1, s2)
            for r in range(n_layers)]
    return W.llama3_8b(f, mids, seq_len=seq_len, decode_steps=decode_steps)


def config4_mistral(batch: int = 16, lo: int = 8192, hi: int = 32768, n_layers: int = 32,
                    decode_steps: int = 512) -> W.Workload:
    return W.mistral_batch(batch=batch, lo=lo, hi=hi, n_layers=n_layers, decode_steps=decode_steps)


def config5_sweep(n_hetero: int, mid: int, seq_len: int = 65536, batch: int = 8,
                  decode_steps: int = 64) -> W.Workload:
    return W.budget_sweep_point(n_hetero, mid, seq_len=seq_len, batch=batch, decode_steps=decode_steps)
