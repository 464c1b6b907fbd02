#!/usr/bin/env python
"""Benchmark of the Task-KV hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic input:
prefill-side compression of every layer (window scores, top-t + semantic
vectors, separator, middle top-k, gather) followed by the workload's decode
steps (append + ragged attention each).  Default workload: the Llama-2-7B-shaped
stack (32 layers, MHA 32 x 128, 32768 tokens, bf16, 256 decode steps).

Prints ONE JSON line.  `value` is decode attention steps per second (all layers
per step), measured on the device with inputs resident in HBM; compression
tokens per second is reported beside it, and `e2e` repeats the measurement
through the host-buffer entry points with the copies inside the timed region.
On one GPU the line also carries, under `workloads`, the same device-timed
measurement of the other single-GPU workloads: the Llama-3-8B-shaped
grouped-query stack, the Mistral-7B-shaped ragged batch and the 15 points of
the budget sweep (`--no-extra` skips them).
`--impl reference` times the CPU oracle on a bounded sample instead; that arm
never builds or loads the CUDA library.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def get_workload(name: str, args, helpers=None):
    """helpers: (hetero_count, mid_budget) for Eq. 16 / Eq. 17; None takes the library's own host helpers."""
    from paper_2501_15113_b200 import configs
    if name == "llama2":
        return configs.config2_llama2(seq_len=args.seq_len or 32768, n_layers=args.layers or 32,
                                      decode_steps=args.decode_steps or 256)
    if name == "llama3":
        return configs.config3_llama3(seq_len=args.seq_len or 131072, n_layers=args.layers or 32,
                                      decode_steps=args.decode_steps or 128, helpers=helpers)
    if name == "mistral":
        return configs.config4_mistral(n_layers=args.layers or 32, decode_steps=args.decode_steps or 512)
    if name == "toy":
        return configs.config1_toy()
    if name.startswith("sweep"):
        _, h, k = name.split(":")
        return configs.config5_sweep(int(h), int(k), decode_steps=args.decode_steps or 64)
    raise SystemExit(f"unknown workload {name}")


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in out.splitlines():
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


POLICIES = {"select": 0, "recent": 1, "mean": 2}


def algorithmic_bytes(wl, info, policy="select"):
    """Bytes the method itself must move: K once, Q_win, C written once and read about twice, the top-t V rows, and
    the retained K/V rows read and written by the gather; per decode step every retained K/V row once.  With averaged
    compensation rows every intermediate K and V row of a non-heterogeneous head is read once more."""
    es, d = wl.elem_size, wl.head_dim
    G = wl.group
    comp = 0
    for b in range(wl.batch):
        N = wl.seq_lens[b]
        for r in range(wl.n_layers):
            h = wl.full_heads(b, r)
            kept = wl.kept_len(b, r)
            per_unit = N * d * es + G * wl.window * d * es + 12 * N + min(wl.top_t, N) * d * es
            comp += wl.n_kv_heads * per_unit + 4 * d * es * (h * N + (wl.n_kv_heads - h) * kept)
            if policy == "mean" and kept < N:
                comp += (wl.n_kv_heads - h) * 2 * d * es * (N - wl.sink - wl.recent)
    return comp


def measure_workload(tk, W, wl, dev, steps, warmup, policy, peak, peak_kind, sampler_gpu, world=1):
    """Device-timed measurement of one workload: `warmup` untimed and `steps` timed passes (compress every layer, then
    the workload's decode steps as fused append + attention calls), then one more pass with every kernel launch
    bracketed by events.  Returns (result dict, live objects the caller may keep using)."""
    from paper_2501_15113_b200 import sharding
    S = wl.decode_steps
    qs, ks, vs = W.materialize(wl, dev)
    steps_in = [W.gen_decode_step(wl, s, dev) for s in range(S)]
    params = tk.params_from_workload(wl, max_new_tokens=S, mid_policy=POLICIES[policy])
    info = tk.taskkv_plan(params)
    cache_mem = torch.empty(int(info.cache_bytes), dtype=torch.uint8, device=dev)
    work_mem = torch.empty(int(info.workspace_bytes), dtype=torch.uint8, device=dev)
    out = torch.empty_like(steps_in[0][0])
    stream = torch.cuda.current_stream()

    def one_pass(ev=None):
        if ev:
            ev[0].record(stream)
        cache = tk.taskkv_compress_ex(params, qs, ks, vs, cache_mem=cache_mem, workspace_mem=work_mem)
        if ev:
            ev[1].record(stream)
        for (q, kn, vn) in steps_in:
            cache.taskkv_decode_step(q, kn, vn, out=out)        # append + attention, fused
        if ev:
            ev[2].record(stream)
        return cache

    for _ in range(warmup):
        one_pass().close()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(sampler_gpu)
    launches0 = tk.taskkv_launch_count()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    barrier()
    sampler.start()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    caches = []
    for i in range(steps):
        caches.append(one_pass(evs[i]))
    t1.record(stream)
    barrier()
    clocks = sampler.stop()
    launches = tk.taskkv_launch_count() - launches0
    status = caches[-1].status()
    for c in caches:
        c.close()
    total_ms = t0.elapsed_time(t1)
    comp_each = [e[0].elapsed_time(e[1]) for e in evs]
    dec_each = [e[1].elapsed_time(e[2]) / S for e in evs]       # per decode step, one value per timed pass
    comp_ms = sum(comp_each)
    dec_ms = sum(e[1].elapsed_time(e[2]) for e in evs)
    K = steps
    # whole-job rates: units of all ranks over the slowest rank's time (one small all-reduce when N > 1)
    value, dec_ms = sharding.job_throughput(K * S, dec_ms, device=dev)
    comp_tps, comp_ms = sharding.job_throughput(K * sum(wl.seq_lens), comp_ms, device=dev)
    _, total_ms = sharding.job_throughput(K, total_ms, device=dev)

    # per-kernel durations: one more identical pass with every launch bracketed by events on its stream
    tk.taskkv_timing_enable(True)
    one_pass().close()
    recs = tk.taskkv_timing_collect()
    tk.taskkv_timing_enable(False)
    per = {}
    for name, ms in recs:
        a = per.setdefault(name, [0, 0.0])
        a[0] += 1
        a[1] += ms

    es, d = wl.elem_size, wl.head_dim
    comp_bytes = algorithmic_bytes(wl, info, policy)
    U = int(info.n_units)
    # decode step s (1-based) reads K and V rows of every segment once: retained rows + s appended per unit
    dec_bytes_avg = 2 * d * es * (int(info.retained_rows) + U * (S + 1) / 2.0)
    dec_step_ms = dec_ms / (K * S)
    comp_pass_ms = comp_ms / K

    kern = {}
    for name, (n, ms) in per.items():
        kern[name] = {"launches": n, "avg_ms": ms / n, "total_ms": ms}
    attn = kern.get("decode_attn", {"avg_ms": float("nan")})
    attn_gbs = dec_bytes_avg / (attn["avg_ms"] * 1e-3) / 1e9
    comp_kernel_ms = sum(v["total_ms"] for k, v in kern.items() if not k.startswith(("decode", "append")))
    dec_gbs = dec_bytes_avg / (dec_step_ms * 1e-3) / 1e9
    comp_gbs = comp_bytes / (comp_pass_ms * 1e-3) / 1e9
    traffic, traffic_src = ncu_traffic(wl, int(info.retained_rows))
    res = {
        "value": value, "ms_per_step": total_ms / K,
        "decode_ms_per_step": dec_step_ms, "compress_ms": comp_pass_ms, "compress_tokens_per_s": comp_tps,
        "per_pass": {"compress_ms_median": statistics.median(comp_each), "compress_ms_min": min(comp_each),
                     "decode_ms_per_step_median": statistics.median(dec_each),
                     "decode_ms_per_step_min": min(dec_each), "passes": len(evs)},
        "hbm": {
            "peak_gbs": peak, "peak_kind": peak_kind, "nominal_gbs": NOMINAL_HBM_GBS,
            "decode_gbs": dec_gbs, "decode_frac": dec_gbs / peak, "decode_frac_of_nominal": dec_gbs / NOMINAL_HBM_GBS,
            "compress_gbs": comp_gbs, "compress_frac": comp_gbs / peak,
            "compress_frac_of_nominal": comp_gbs / NOMINAL_HBM_GBS,
            "decode_bytes_per_step": dec_bytes_avg, "compress_bytes": comp_bytes,
        },
        "roofline": {"bound": "hbm", "kernel": "decode_attn", "achieved": attn_gbs, "peak": peak, "unit": "GB/s",
                     "frac": attn_gbs / peak, "frac_of_nominal": attn_gbs / NOMINAL_HBM_GBS, "peak_kind": peak_kind,
                     "traffic": traffic, "traffic_unit": "bytes per launch", "traffic_source": traffic_src,
                     "algorithmic_bytes": dec_bytes_avg, "avg_launch_ms": attn["avg_ms"]},
        "kernels": kern, "compress_kernel_ms": comp_kernel_ms,
        "gpu_launches": launches, "device_status": status, "clocks": clocks,
    }
    live = {"qs": qs, "ks": ks, "vs": vs, "steps_in": steps_in, "params": params, "comp_bytes": comp_bytes}
    return res, live


EXTRA_WORKLOADS = ["llama3", "mistral"] + [f"sweep:{h}:{k}" for h in (0, 1, 2, 4, 8) for k in (64, 256, 1024)]


def run_extra_workloads(tk, W, args, dev, peak, peak_kind, gpu):
    """The other single-GPU workloads, each measured like the headline one (3 warm-up and 3 timed passes, per-kernel
    pass, clocks sampled): the grouped-query stack, the ragged serving batch, and the 15 budget-sweep points."""
    out = {}
    for name in EXTRA_WORKLOADS:
        if name == args.workload:
            continue
        wl = get_workload(name, args)
        wl.planted = W._choose_planted(wl)
        try:
            res, live = measure_workload(tk, W, wl, dev, steps=3, warmup=3, policy=args.policy, peak=peak,
                                         peak_kind=peak_kind, sampler_gpu=gpu)
        except Exception as exc:            # one workload failing must not lose the headline line
            out[name] = {"workload": wl.name, "error": f"{type(exc).__name__}: {str(exc)[:200]}"}
            torch.cuda.empty_cache()
            continue
        del live
        torch.cuda.empty_cache()
        k = res["kernels"]
        out[name] = {
            "workload": wl.name, "decode_steps": wl.decode_steps, "passes": 3,
            "compress_ms": res["compress_ms"], "compress_tokens_per_s": res["compress_tokens_per_s"],
            "decode_ms_per_step": res["decode_ms_per_step"], "decode_steps_per_s": res["value"],
            "hbm": {x: res["hbm"][x] for x in ("compress_frac", "decode_frac", "compress_frac_of_nominal",
                                               "decode_frac_of_nominal", "compress_gbs", "decode_gbs",
                                               "compress_bytes", "decode_bytes_per_step")},
            "decode_attn": {x: res["roofline"][x] for x in ("achieved", "frac", "traffic", "avg_launch_ms")},
            "kernel_ms": {n: round(v["total_ms"], 4) for n, v in k.items() if not n.startswith(("decode", "append"))},
            "kernel_ms_per_decode_launch": {n: round(v["avg_ms"], 4) for n, v in k.items()
                                            if n.startswith(("decode", "append"))},
            "gpu_launches": res["gpu_launches"], "device_status": res["device_status"], "clocks": res["clocks"],
        }
    return out


def run_ours(args):
    import __graft_entry__ as ge
    ge.build()
    from paper_2501_15113_b200 import binding as tk
    from paper_2501_15113_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    peak, peak_kind = load_peaks()

    wl = get_workload(args.workload, args)
    from paper_2501_15113_b200 import sharding
    wl.seed = sharding.replica_seed(wl.seed, rank)   # weak scaling: every rank owns an independent replica
    wl.planted = W._choose_planted(wl)
    res, live = measure_workload(tk, W, wl, dev, steps=args.steps, warmup=args.warmup, policy=args.policy, peak=peak,
                                 peak_kind=peak_kind, sampler_gpu=local, world=world)
    qs, ks, vs, steps_in, params = (live[x] for x in ("qs", "ks", "vs", "steps_in", "params"))
    comp_bytes = live["comp_bytes"]

    line = {
        "metric": "decode attn steps/s (compress tokens/s beside it)",
        "value": res["value"], "unit": "steps/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": wl.dtype, "data": "synthetic",
        "config": dict(wl.describe(), mid_policy=args.policy, l2="inputs (>=8 GB of K, >=3 GB retained cache) exceed the 126 MB L2",
                       step="compress all layers + decode_steps x (append + attention, one fused call)"),
    }
    line.update({k: v for k, v in res.items() if k not in ("value", "ms_per_step")})

    if rank == 0 and not args.no_latency:
        line["latency_mode"] = run_latency_mode(tk, wl, qs, ks, vs, steps_in, args)
        line["layer_streamed_compress"] = run_layer_streamed(tk, wl, qs, ks, vs, args, steps_in)
        line["compress_with_window_lse"] = run_with_window_lse(tk, wl, qs, ks, vs, args, comp_bytes, peak)
        line["paged_cache"] = run_paged(tk, wl, qs, ks, vs, steps_in, args, comp_bytes, res["hbm"]["decode_bytes_per_step"], peak)
        if wl.seq_lens[0] <= 32768:
            line["exact_semantic"] = run_exact_semantic(tk, wl, qs, ks, vs)
    if rank == 0 and not args.no_e2e:
        line["e2e"] = run_e2e(tk, wl, params, qs, ks, vs, steps_in, world)
    if rank == 0 and world == 1 and not args.no_cpu and args.policy != "select":
        line["cpu_baseline"] = None      # the oracle is timed on the method's own policy only
    elif rank == 0 and world == 1 and not args.no_cpu:
        line["cpu_baseline"] = cpu_baseline(wl, qs, ks, vs, steps_in)
    del qs, ks, vs, steps_in, params, live
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_extra:
        line["workloads"] = run_extra_workloads(tk, W, args, dev, peak, peak_kind, local)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


def run_latency_mode(tk, wl, qs, ks, vs, steps_in, args, n_steps=16):
    """Decode as a model runs it: one append + attention call per layer (layer r's query depends on layer r-1),
    n_steps tokens; first as plain launches, then with one token's 2 x n_layers launches replayed from a CUDA graph."""
    import torch
    R = wl.n_layers
    params = tk.params_from_workload(wl, max_new_tokens=3 * n_steps + 4, mid_policy=POLICIES[args.policy])
    cache = tk.taskkv_compress_ex(params, qs, ks, vs)
    q, kn, vn = steps_in[0]
    ql = [q[:, r:r + 1].contiguous() for r in range(R)]
    kl = [kn[:, r:r + 1].contiguous() for r in range(R)]
    vl = [vn[:, r:r + 1].contiguous() for r in range(R)]
    ol = [torch.empty_like(x) for x in ql]
    stream = torch.cuda.current_stream()

    def token():
        for r in range(R):
            cache.taskkv_decode_step_ex(ql[r], kl[r], vl[r], r, 1, out=ol[r])

    def timed(fn, n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    for _ in range(3):
        token()
    eager_ms = timed(token, n_steps)
    out = {"layers_per_token": R, "launches_per_token": 2 * R, "tokens_timed": n_steps,
           "eager_ms_per_token": eager_ms, "graph_ms_per_token": None}
    try:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            token()
        g.replay()
        out["graph_ms_per_token"] = timed(g.replay, n_steps)
    except Exception as exc:      # capture is an optimisation of the launch path only
        out["graph_error"] = str(exc)[:200]
    out["device_status"] = cache.status()
    cache.close()
    return out


def run_paged(tk, wl, qs, ks, vs, steps_in, args, comp_bytes, decode_bytes, peak):
    """The same compression and decode steps with the rows in pages of a shared pool (block tables), as a serving
    engine would hold them: compression time, time of a fused decode step, both against the same algorithmic bytes
    as the contiguous cache."""
    import torch
    n_dec = len(steps_in)
    params = tk.params_from_workload(wl, max_new_tokens=n_dec, mid_policy=POLICIES[args.policy])
    P = args.page_rows
    info, pages = tk.taskkv_plan_paged(params, P)
    pool = tk.Pool(P, pages + (n_dec // P + 2) * int(info.n_units), wl.head_dim, wl.dtype, qs[0].device)
    cmem = torch.empty(int(info.cache_bytes), dtype=torch.uint8, device=qs[0].device)
    wmem = torch.empty(int(info.workspace_bytes), dtype=torch.uint8, device=qs[0].device)
    stream = torch.cuda.current_stream()

    def timed(fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        r = fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1), r

    comp, dec = [], []
    status = 0
    for it in range(4):
        ms, cache = timed(lambda: tk.taskkv_compress_paged(params, qs, ks, vs, pool, cache_mem=cmem, workspace_mem=wmem))
        out = torch.empty_like(steps_in[0][0])

        def steps():
            for (q, kn, vn) in steps_in:
                cache.taskkv_decode_step(q, kn, vn, out=out)

        msd, _ = timed(steps)
        if it:
            comp.append(ms)
            dec.append(msd / n_dec)
        status = max(status, cache.status())
        cache.close()
    # per-kernel durations of one more pass, every launch bracketed by events
    tk.taskkv_timing_enable(True)
    cache = tk.taskkv_compress_paged(params, qs, ks, vs, pool, cache_mem=cmem, workspace_mem=wmem)
    for (q, kn, vn) in steps_in:
        cache.taskkv_decode_step(q, kn, vn, out=out)
    torch.cuda.synchronize()
    recs = tk.taskkv_timing_collect()
    tk.taskkv_timing_enable(False)
    cache.close()
    per = {}
    for name, ms in recs:
        a = per.setdefault(name, [0, 0.0])
        a[0] += 1
        a[1] += ms
    free_after = pool.free_pages()
    n_pages = pool.n_pages
    pool.close()
    cms, dms = statistics.median(comp), statistics.median(dec)
    return {"page_rows": P, "pages": pages, "pool_pages": n_pages, "all_pages_returned": free_after == n_pages,
            "compress_ms": cms, "compress_frac_of_peak": comp_bytes / (cms * 1e-3) / 1e9 / peak,
            "decode_ms_per_step": dms, "decode_frac_of_peak": decode_bytes / (dms * 1e-3) / 1e9 / peak,
            "kernel_avg_ms": {k: v[1] / v[0] for k, v in per.items()}, "device_status": status}


def run_layer_streamed(tk, wl, qs, ks, vs, args, steps_in):
    """Compression as a prefill loop would issue it: the cache for the whole model is created first, then one
    taskkv_compress_layer call per layer, each as soon as that layer's K and V exist (here: back to back on one
    stream), all into that one cache; a decode step over all layers follows to show the cache is the usual one."""
    import torch
    params = tk.params_from_workload(wl, max_new_tokens=4, mid_policy=POLICIES[args.policy])
    R = wl.n_layers
    info = tk.taskkv_plan(params)
    dev = qs[0].device
    cmem = torch.empty(int(info.cache_bytes), dtype=torch.uint8, device=dev)
    wmem = torch.empty(int(info.workspace_bytes), dtype=torch.uint8, device=dev)
    ins = [([x[r] for x in qs], [x[r] for x in ks], [x[r] for x in vs]) for r in range(R)]
    stream = torch.cuda.current_stream()

    def all_layers():
        cache = tk.taskkv_cache_create(params, dev, cache_mem=cmem, workspace_mem=wmem)
        for r in range(R):
            cache.taskkv_compress_layer(r, *ins[r])
        return cache

    all_layers().close()
    times = []
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        cache = all_layers()
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
        if len(times) < 3:
            cache.close()
    q, kn, vn = steps_in[0]
    cache.taskkv_decode_step(q, kn, vn)
    torch.cuda.synchronize()
    status = cache.status()
    rows = int(cache.lengths().sum())
    cache.close()
    ms = statistics.median(times)

    # the same calls round-robin on four streams: a layer's latency-bound selection, planning and short grids then
    # overlap the next layers' window scores, as they would overlap the prefill's own kernels
    side = [torch.cuda.Stream() for _ in range(4)]

    def all_layers_side():
        cache = tk.taskkv_cache_create(params, dev, cache_mem=cmem, workspace_mem=wmem)
        start = torch.cuda.Event()
        start.record(stream)
        for st in side:
            st.wait_event(start)
        for r in range(R):
            cache.taskkv_compress_layer(r, *ins[r], stream=side[r % 4])
        for st in side:
            done = torch.cuda.Event()
            done.record(st)
            stream.wait_event(done)
        return cache

    all_layers_side().close()
    times4 = []
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        cache = all_layers_side()
        e1.record(stream)
        torch.cuda.synchronize()
        times4.append(e0.elapsed_time(e1))
        status = max(status, cache.status())
        cache.close()
    return {"calls": R, "total_ms": ms, "ms_per_layer": ms / R, "four_streams_total_ms": statistics.median(times4),
            "device_status": status,
            "rows_after_one_step": rows, "expected_rows": int(info.retained_rows) + int(info.n_units),
            "note": "one cache for all layers (taskkv_cache_create), one taskkv_compress_layer call per layer on one "
                    "stream; the all-layer call of the headline overlaps steps of different layers, these calls "
                    "cannot"}


def run_exact_semantic(tk, wl, qs, ks, vs):
    """The exact semantic vector of Eq. 1-2 (full causal attention, quadratic in N) for layer 0 of sequence 0, beside
    the window approximation of Eq. 12-15 that compression uses.  The query rows before the window are seeded random
    rows with the workload's scale; the last L rows are the workload's own window."""
    import numpy as np
    import torch
    N, d, n, L = wl.seq_lens[0], wl.head_dim, wl.n_heads, wl.window
    g = torch.Generator(device=qs[0].device).manual_seed(wl.seed * 7919 + 17)
    q = torch.randn(1, n, N, d, generator=g, device=qs[0].device, dtype=torch.float32) * (wl.variance ** 0.5)
    q = q.to(torch.bfloat16)
    q[0, :, N - L:, :] = qs[0][0]
    k, v = ks[0][0:1].contiguous(), vs[0][0:1].contiguous()
    stream = torch.cuda.current_stream()
    ws = torch.empty(int(tk.lib.taskkv_exact_semantic_bytes(1, n, wl.n_kv_heads, d, N)), dtype=torch.uint8,
                     device=qs[0].device)
    times = []
    for i in range(1 + 3):
        tk.taskkv_timing_enable(i == 3)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        sem, _ = tk.taskkv_exact_semantic(q, k, v, want_scores=False, workspace_mem=ws)
        e1.record(stream)
        torch.cuda.synchronize()
        if i >= 1:
            times.append(e0.elapsed_time(e1))
    kern = {}
    for name, t in tk.taskkv_timing_collect():
        kern[name] = round(kern.get(name, 0.0) + t, 3)
    tk.taskkv_timing_enable(False)
    ms = statistics.median(times)
    nb = (N + 127) // 128
    scores = n * 128 * 128 * nb * (nb + 1) // 2            # per pass: the causal half in 128 x 128 tiles
    tflops = 2 * scores * 2 * d / (ms * 1e-3) / 1e12
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            tpeak, kind = float(json.load(fh)["bf16_tflops"]), "measured"
    except Exception:
        tpeak, kind = 1590.0, "fallback"
    out = {"layers": 1, "query_heads": n, "seq_len": N, "ms": ms, "tflops": tflops, "tensor_peak_tflops": tpeak,
           "tensor_frac": tflops / tpeak, "peak_kind": kind, "exp_per_s": 2 * scores / (ms * 1e-3), "kernel_ms": kern,
           "note": "two passes (row normalisers, column sums) over the causal half of Q K^T; one exponential per "
                   "score and pass bounds it before the tensor pipe does"}
    # the share of the exact column means held by the t largest of them (the premise of Eq. 14), median over heads
    _, c_exact = tk.taskkv_exact_semantic(q, k, v, want_scores=True, workspace_mem=ws)
    top = torch.sort(c_exact[0], dim=1, descending=True).values.cumsum(dim=1)
    out["top_t_mass"] = {str(t): float(top[:, min(t, N) - 1].median()) for t in (64, 256, 1024, 4096)}
    del c_exact, top
    # how far the window's v' is from v, and whether the two pick the same far heads (one layer, one sequence)
    if wl.batch == 1:
        one = tk.params_from_workload(wl, max_new_tokens=0).layer(0)
        c = tk.taskkv_compress_ex(one, [qs[0][0:1].contiguous()], [k], [v])
        approx = c.query(tk.Q_SEMVEC).reshape(wl.n_kv_heads, d).astype(np.float64)
        c.close()
        exact = sem[0].double().cpu().numpy()
        rel = np.linalg.norm(approx - exact, axis=1) / np.linalg.norm(exact, axis=1)
        f = wl.n_hetero[0][0]
        far = lambda x: set(np.argsort(-np.linalg.norm(x - x.mean(0), axis=1), kind="stable")[:f].tolist())
        out.update({"window_vs_exact_rel_dist_median": float(np.median(rel)),
                    "far_heads_agree": len(far(approx) & far(exact)), "far_heads": f})
    return out


def run_with_window_lse(tk, wl, qs, ks, vs, args, comp_bytes, peak):
    """Compression when the prompt's attention has already produced the log-sum-exp of the window rows (flash
    attention returns it): pass 1 of the window scores is skipped.  The normalisers are prepared here with torch,
    outside the timed region, standing in for that by-product of prefill."""
    import torch
    G, L = wl.group, wl.window
    lse = []
    for b in range(wl.batch):
        N = wl.seq_lens[b]
        pos = (N - L + torch.arange(L, device=qs[b].device))[:, None]
        hidden = torch.arange(N, device=qs[b].device)[None, :] > pos
        per_layer = []
        for r in range(wl.n_layers):
            q = qs[b][r].float()                                          # [n, L, d]
            k = ks[b][r].float().repeat_interleave(G, dim=0)              # [n, N, d]
            sc = torch.matmul(q, k.transpose(1, 2)) / (wl.head_dim ** 0.5)
            sc.masked_fill_(hidden[None], float("-inf"))
            per_layer.append(torch.logsumexp(sc, dim=2))
            del sc, k
        lse.append(torch.stack(per_layer).contiguous())
    params = tk.params_from_workload(wl, max_new_tokens=4, mid_policy=POLICIES[args.policy])
    info = tk.taskkv_plan(params)
    cm = torch.empty(int(info.cache_bytes), dtype=torch.uint8, device=qs[0].device)
    wm = torch.empty(int(info.workspace_bytes), dtype=torch.uint8, device=qs[0].device)
    stream = torch.cuda.current_stream()
    times = []
    for i in range(3 + 5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        c = tk.taskkv_compress_ex(params, qs, ks, vs, cache_mem=cm, workspace_mem=wm, window_lse=lse)
        e1.record(stream)
        torch.cuda.synchronize()
        status = c.status()
        c.close()
        if i >= 3:
            times.append(e0.elapsed_time(e1))
    ms = statistics.median(times)
    return {"compress_ms": ms, "compress_tokens_per_s": sum(wl.seq_lens) / (ms * 1e-3),
            "compress_frac": comp_bytes / (ms * 1e-3) / 1e9 / peak, "device_status": status,
            "note": "window-row log-sum-exp supplied by the caller (a by-product of prefill attention); not the headline"}


def ncu_traffic(wl, retained_rows):
    """DRAM bytes per decode_attn launch, from the committed ncu captures of the kernel as it is now, scaled by the
    rows a launch reads (traffic grows in proportion to them; a full-size launch holds too much on the device for a
    multi-pass capture).  Returns (bytes or None, the capture it comes from)."""
    if wl.dtype != "bf16" or wl.head_dim != 128:
        return None, None
    if wl.n_heads == wl.n_kv_heads:
        # 378.42 MB read + 4.25 MB written for 739,056 retained rows of 256 bytes, K and V
        return 382.67e6 / 739056 * retained_rows, "profiles/decode_attn_llama2_4layers.md (one query head per KV head)"
    if wl.group == 4:
        # 859.09 MB read + 9.02 MB written for a launch whose K and V rows are 859.03 MB
        return 868.11e6 / (859.03e6 / 512.0) * retained_rows, "profiles/decode_attn_llama2_4layers.md (four query heads per KV head)"
    return None, None


def run_e2e(tk, wl, params, qs, ks, vs, steps_in, world):
    """Same metric through the host-buffer entry points: pinned host inputs, copies inside the timed region."""
    hq = [t.cpu().pin_memory() for t in qs]
    hk = [t.cpu().pin_memory() for t in ks]
    hv = [t.cpu().pin_memory() for t in vs]
    hsteps = [tuple(t.cpu().pin_memory() for t in s) for s in steps_in]
    hout = torch.empty(steps_in[0][0].shape, dtype=steps_in[0][0].dtype).pin_memory()
    torch.cuda.synchronize()
    cache = tk.taskkv_compress_host(params, hq, hk, hv)      # warm-up (allocations, page mapping)
    for s in range(min(3, len(hsteps))):
        cache.taskkv_decode_host(hsteps[s][0], None, None, hout)
    cache.close()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    cache = tk.taskkv_compress_host(params, hq, hk, hv)
    t1 = time.perf_counter()
    for (q, kn, vn) in hsteps:
        cache.taskkv_decode_host(q, kn, vn, hout)
    t2 = time.perf_counter()
    cache.close()
    S = len(hsteps)
    h2d = sum(t.numel() * t.element_size() for t in hq + hk + hv) + \
        sum(t.numel() * t.element_size() for s in hsteps for t in s)
    d2h = S * hout.numel() * hout.element_size()
    return {"value": world * S / (t2 - t1), "unit": "steps/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "compress_tokens_per_s": sum(wl.seq_lens) / (t1 - t0), "compress_s": t1 - t0,
            "decode_ms_per_step": (t2 - t1) * 1e3 / S, "timing": "host wall clock around synchronous calls"}


def oracle_sample(wl, qs, ks, vs, steps_in, n_units: int, n_steps: int, budget_s: float = 0.0):
    """Times the oracle on the first n_units KV heads of sequence 0, layer after layer until budget_s seconds
    of compression are spent (at least layer 0), then on decode steps of those layers (at most n_steps per
    layer, same time budget).  Returns seconds (compress, decode), keys scanned and rows read."""
    from oracle import taskkv_oracle as O
    G = wl.group
    n_units = min(n_units, wl.n_kv_heads)
    caches, keys = [], 0
    t0 = time.perf_counter()
    for r in range(wl.n_layers):
        q = qs[0][r][:n_units * G].double().cpu().numpy()
        k = ks[0][r][:n_units].double().cpu().numpy()
        v = vs[0][r][:n_units].double().cpu().numpy()
        ref = O.compress_layer(q, k, v, n_hetero=min(wl.n_hetero[0][r], n_units), sink=wl.sink, recent=wl.recent,
                               mid=wl.mid_budget[r], top_t=wl.top_t, pool_kernel=wl.pool_kernel,
                               promote_center=wl.promote_center)
        caches.append((r, *O.gather_cache(k, v, ref["idx"])))
        keys += n_units * wl.seq_lens[0]
        if time.perf_counter() - t0 >= budget_s:
            break
    t1 = time.perf_counter()
    rows = 0
    for (r, kc, vc) in caches:
        for s in range(n_steps):
            qd, kn, vn = steps_in[s]
            O.append_layer(kc, vc, kn[0, r, :n_units].double().cpu().numpy(), vn[0, r, :n_units].double().cpu().numpy())
            O.decode_layer(qd[0, r, :n_units * G].double().cpu().numpy(), kc, vc)
            rows += int(sum(len(x) for x in kc))
        if time.perf_counter() - t1 >= budget_s:
            break
    t2 = time.perf_counter()
    return (t1 - t0), (t2 - t1), keys, rows, len(caches)


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(wl, qs, ks, vs, steps_in):
    n_steps = min(4, len(steps_in))
    comp_s, dec_s, keys, rows, layers = oracle_sample(wl, qs, ks, vs, steps_in, wl.n_kv_heads, n_steps, budget_s=8.0)
    tokens_units = sum(wl.seq_lens[b] * wl.n_layers * wl.n_kv_heads for b in range(wl.batch))
    # compress cost scales with keys scanned; decode cost with rows read
    comp_full = comp_s * tokens_units / keys
    dec_full = dec_s * wl.retained_rows() / rows
    return {"value": 1.0 / dec_full, "unit": "steps/s", "cores": cpu_threads(), "kind": "oracle",
            "threads": "single-process numpy float64; only its BLAS matrix products run on `cores` threads",
            "compress_tokens_per_s": sum(wl.seq_lens) / comp_full,
            "sample": f"all KV heads of {layers} layer(s) of sequence 0: compress {comp_s:.1f} s ({keys} keys), "
                      f"decode steps {dec_s:.1f} s ({rows} rows read); scaled by keys scanned ({tokens_units}) and "
                      f"by rows read per step ({wl.retained_rows()})"}


def run_reference(args):
    """The oracle, as it stands, on the host cores: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import taskkv_oracle as O
    from paper_2501_15113_b200 import workloads as W
    wl = get_workload(args.workload, args, helpers=(O.hetero_count, O.mid_budget))   # no CUDA library on this arm
    n_units = 4
    sub = W.Workload(**{**wl.__dict__})
    qs, ks, vs = [], [], []
    q, k, v = W.gen_layer(wl, 0, 0, "cpu")
    qs.append(q[None])
    ks.append(k[None])
    vs.append(v[None])
    steps_in = [W.gen_decode_step(wl, s, "cpu") for s in range(2)]
    times = []
    for i in range(args.warmup + args.steps):
        c, d, keys, rows, _ = oracle_sample(sub, qs, ks, vs, steps_in, n_units, 2)
        if i >= args.warmup:
            times.append((c, d, keys, rows))
    comp_s = statistics.mean(t[0] for t in times)
    dec_s = statistics.mean(t[1] for t in times)
    keys, rows = times[0][2], times[0][3]
    tokens_units = sum(wl.seq_lens[b] * wl.n_layers * wl.n_kv_heads for b in range(wl.batch))
    comp_full = comp_s * tokens_units / keys
    dec_full = dec_s * wl.retained_rows() / rows
    dec_s /= 2
    value = 1.0 / dec_full
    sample = (f"{n_units} KV heads of layer 0 per step: oracle compress {comp_s:.2f} s + 2 decode steps; scaled to the "
              f"whole workload by keys scanned and rows read")
    line = {"impl": "reference", "metric": "decode attn steps/s (compress tokens/s beside it)", "value": value,
            "unit": "steps/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": (comp_s + 2 * dec_s) * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": wl.describe(),
            "compress_tokens_per_s": sum(wl.seq_lens) / comp_full,
            "cpu_baseline": {"value": value, "unit": "steps/s", "cores": cpu_threads(), "kind": "oracle",
                             "threads": "single-process numpy float64; only its BLAS matrix products run on `cores` "
                                        "threads", "sample": sample},
            "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2")
    ap.add_argument("--seq-len", type=int, default=0)
    ap.add_argument("--layers", type=int, default=0)
    ap.add_argument("--decode-steps", type=int, default=0)
    ap.add_argument("--policy", default="select", choices=sorted(POLICIES),
                    help="what a non-heterogeneous head keeps beside sinks and recent window (Sec. V-G)")
    ap.add_argument("--no-latency", action="store_true", help="skip the layer-by-layer decode measurement")
    ap.add_argument("--page-rows", type=int, default=256, help="page size of the paged-cache measurement")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the other workloads (grouped-query, batch, sweep)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
