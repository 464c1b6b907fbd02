"""ctypes binding of libtaskkv.so: argument marshalling only.

Every step of the Task-KV hot path runs inside the CUDA library; this module
turns torch tensors into pointers, keeps buffers alive, and reads results
back.  There is no fallback: if the library is missing, importing this module
raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtaskkv.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2501_15113_b200.build` "
        "(the Task-KV path has no non-CUDA implementation)")

lib = C.CDLL(LIB_PATH)

OK, EINVAL, EALLOC, ECUDA, ETIMEOUT, ESTATE = 0, -1, -2, -3, -4, -5
F32, BF16 = 0, 1
(Q_LENGTHS, Q_CLASSES, Q_DIST, Q_SEMVEC, Q_OFFSETS, Q_INDICES, Q_SCORES, Q_TOPT, Q_STATUS, Q_KPOOL,
 Q_VPOOL, Q_CAPACITY, Q_PAGETAB) = range(13)


class taskkv_params(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("batch", C.c_int32), ("sink", C.c_int32), ("recent", C.c_int32), ("mid_budget", C.c_int32),
        ("window", C.c_int32), ("top_t", C.c_int32), ("pool_kernel", C.c_int32), ("m_top", C.c_int32),
        ("beta", C.c_float), ("promote_center", C.c_int32), ("force_class", C.c_int32), ("dtype", C.c_int32),
        ("max_new_tokens", C.c_int32), ("mid_policy", C.c_int32),
        ("seq_lens", C.POINTER(C.c_int32)), ("mid_budget_per_layer", C.POINTER(C.c_int32)),
        ("n_hetero", C.POINTER(C.c_int32)), ("budget_frac", C.c_float),
        ("shard_kv_heads", C.c_int32), ("shard_first", C.c_int32),
    ]


class taskkv_plan_info(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "n_units", "pool_rows", "retained_rows", "cache_bytes", "workspace_bytes", "max_decode_items",
        "gather_items", "index_stride")]


_vp = C.c_void_p
_pp = C.POINTER(C.c_void_p)
lib.taskkv_params_default.argtypes = [C.POINTER(taskkv_params)]
lib.taskkv_params_default.restype = None
lib.taskkv_plan.argtypes = [C.POINTER(taskkv_params), C.POINTER(taskkv_plan_info)]
lib.taskkv_plan.restype = C.c_int32
lib.taskkv_compress_ex.argtypes = [C.POINTER(taskkv_params), _pp, _pp, _pp, _vp, C.c_size_t, _vp, C.c_size_t,
                                   _vp, C.POINTER(_vp)]
lib.taskkv_compress_ex.restype = C.c_int32
lib.taskkv_cache_create.argtypes = [C.POINTER(taskkv_params), _vp, C.c_size_t, _vp, C.c_size_t, _vp, C.POINTER(_vp)]
lib.taskkv_cache_create.restype = C.c_int32
lib.taskkv_compress_layer.argtypes = [_vp, C.c_int32, _pp, _pp, _pp, _pp, _vp]
lib.taskkv_compress_layer.restype = C.c_int32
lib.taskkv_compress_shard_begin.argtypes = [C.POINTER(taskkv_params), _pp, _pp, _pp, _pp, _vp, C.c_size_t, _vp, C.c_size_t,
                                            _vp, C.POINTER(_vp)]
lib.taskkv_compress_shard_begin.restype = C.c_int32
lib.taskkv_cache_semantic.argtypes = [_vp, C.POINTER(_vp), C.POINTER(C.c_int64)]
lib.taskkv_cache_semantic.restype = C.c_int32
lib.taskkv_compress_shard_finish.argtypes = [_vp, _vp, _vp]
lib.taskkv_compress_shard_finish.restype = C.c_int32
lib.taskkv_pool_bytes.argtypes = [C.c_int32] * 4
lib.taskkv_pool_bytes.restype = C.c_size_t
lib.taskkv_pool_create.argtypes = [C.c_int32] * 4 + [_vp, C.c_size_t, _vp, C.POINTER(_vp)]
lib.taskkv_pool_create.restype = C.c_int32
lib.taskkv_pool_free_pages.argtypes = [_vp]
lib.taskkv_pool_free_pages.restype = C.c_int32
lib.taskkv_pool_destroy.argtypes = [_vp]
lib.taskkv_pool_destroy.restype = None
lib.taskkv_plan_paged.argtypes = [C.POINTER(taskkv_params), C.c_int32, C.POINTER(taskkv_plan_info), C.POINTER(C.c_int64)]
lib.taskkv_plan_paged.restype = C.c_int32
lib.taskkv_compress_paged.argtypes = [C.POINTER(taskkv_params), _pp, _pp, _pp, _vp, _vp, C.c_size_t, _vp, C.c_size_t,
                                      _vp, C.POINTER(_vp)]
lib.taskkv_compress_paged.restype = C.c_int32
lib.taskkv_compress_lse.argtypes = [C.POINTER(taskkv_params), _pp, _pp, _pp, _pp, _vp, C.c_size_t, _vp, C.c_size_t,
                                    _vp, C.POINTER(_vp)]
lib.taskkv_compress_lse.restype = C.c_int32
lib.taskkv_exact_semantic.argtypes = [_vp, _vp, _vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _vp, _vp, _vp,
                                      C.c_size_t, _vp]
lib.taskkv_exact_semantic.restype = C.c_int32
lib.taskkv_exact_semantic_bytes.argtypes = [C.c_int32] * 5
lib.taskkv_exact_semantic_bytes.restype = C.c_size_t
lib.taskkv_compress.argtypes = [_vp, _vp, _vp] + [C.c_int32] * 9 + [_vp, C.POINTER(_vp)]
lib.taskkv_compress.restype = C.c_int32
lib.taskkv_compress_host.argtypes = [C.POINTER(taskkv_params), _pp, _pp, _pp, _vp, C.POINTER(_vp)]
lib.taskkv_compress_host.restype = C.c_int32
lib.taskkv_append.argtypes = [_vp, _vp, _vp, _vp]
lib.taskkv_append.restype = C.c_int32
lib.taskkv_decode.argtypes = [_vp, _vp, _vp, _vp, _vp]
lib.taskkv_decode.restype = C.c_int32
lib.taskkv_append_ex.argtypes = [_vp, _vp, _vp, C.c_int32, C.c_int32, _vp]
lib.taskkv_append_ex.restype = C.c_int32
lib.taskkv_decode_ex.argtypes = [_vp, _vp, _vp, _vp, C.c_int32, C.c_int32, _vp]
lib.taskkv_decode_ex.restype = C.c_int32
lib.taskkv_decode_step_ex.argtypes = [_vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int32, _vp]
lib.taskkv_decode_step_ex.restype = C.c_int32
lib.taskkv_decode_step.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp]
lib.taskkv_decode_step.restype = C.c_int32
lib.taskkv_decode_host.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp]
lib.taskkv_decode_host.restype = C.c_int32
lib.taskkv_decode_noalloc.argtypes = [_vp, _vp, _vp, _vp, _vp] + [C.c_int32] * 5 + [_vp, _vp]
lib.taskkv_decode_noalloc.restype = C.c_int32
lib.taskkv_cache_query_bytes.argtypes = [_vp, C.c_int32]
lib.taskkv_cache_query_bytes.restype = C.c_int64
lib.taskkv_cache_query.argtypes = [_vp, C.c_int32, _vp, C.c_size_t]
lib.taskkv_cache_query.restype = C.c_int32
lib.taskkv_cache_plan.argtypes = [_vp, C.POINTER(taskkv_plan_info)]
lib.taskkv_cache_plan.restype = C.c_int32
lib.taskkv_cache_destroy.argtypes = [_vp]
lib.taskkv_cache_destroy.restype = None
lib.taskkv_status_str.argtypes = [C.c_int32]
lib.taskkv_status_str.restype = C.c_char_p
lib.taskkv_hetero_count.argtypes = [C.c_int32, C.c_float, C.c_int32, C.c_int32, C.c_int32]
lib.taskkv_hetero_count.restype = C.c_int32
lib.taskkv_mid_budget.argtypes = [C.c_double] + [C.c_int32] * 5
lib.taskkv_mid_budget.restype = C.c_int32
lib.taskkv_mid_budget_ex.argtypes = [C.c_double] + [C.c_int32] * 7
lib.taskkv_mid_budget_ex.restype = C.c_int32
lib.taskkv_selftest_bounded_wait.argtypes = [C.c_int32, C.POINTER(C.c_int32), _vp]
lib.taskkv_selftest_bounded_wait.restype = C.c_int32
lib.taskkv_launch_count.argtypes = []
lib.taskkv_launch_count.restype = C.c_int64
lib.taskkv_timing_enable.argtypes = [C.c_int32]
lib.taskkv_timing_enable.restype = None
lib.taskkv_timing_collect.argtypes = [C.POINTER(C.c_int32), C.POINTER(C.c_float), C.c_int32]
lib.taskkv_timing_collect.restype = C.c_int32
lib.taskkv_timing_name.argtypes = [C.c_int32]
lib.taskkv_timing_name.restype = C.c_char_p


class TaskKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.taskkv_status_str(status).decode()} ({status})")


def _check(status: int, where: str) -> None:
    if status != OK:
        raise TaskKVError(status, where)


def taskkv_hetero_count(n: int, beta: float, m: int, R: int, r: int) -> int:
    return int(lib.taskkv_hetero_count(n, beta, m, R, r))


def taskkv_mid_budget(budget_tokens: float, N: int, h_full: int, n: int, sink: int, recent: int) -> int:
    return int(lib.taskkv_mid_budget(budget_tokens, N, h_full, n, sink, recent))


def taskkv_mid_budget_ex(budget_tokens: float, N: int, f: int, n: int, sink: int, recent: int,
                         promote_center: bool = True, literal: bool = False) -> int:
    return int(lib.taskkv_mid_budget_ex(budget_tokens, N, f, n, sink, recent, 1 if promote_center else 0,
                                        1 if literal else 0))


def taskkv_selftest_bounded_wait(max_polls: int = 2000, stream=None):
    """(status, polls): status is ETIMEOUT when the bounded wait gave up as designed."""
    polls = C.c_int32(0)
    st = int(lib.taskkv_selftest_bounded_wait(max_polls, C.byref(polls), _stream_handle(stream)))
    return st, int(polls.value)


def taskkv_launch_count() -> int:
    return int(lib.taskkv_launch_count())


def taskkv_timing_enable(on: bool) -> None:
    lib.taskkv_timing_enable(1 if on else 0)


def taskkv_timing_collect(max_records: int = 1 << 16) -> List[tuple]:
    ids = (C.c_int32 * max_records)()
    ms = (C.c_float * max_records)()
    n = lib.taskkv_timing_collect(ids, ms, max_records)
    return [(lib.taskkv_timing_name(ids[i]).decode(), float(ms[i])) for i in range(n)]


def _stream_handle(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


class Params:
    """Owns a taskkv_params struct and the host arrays it points to."""

    def __init__(self, *, n_layers, n_heads, n_kv_heads, head_dim, seq_lens: Sequence[int], sink, recent,
                 mid_budget, window, dtype, top_t=256, pool_kernel=7, beta=0.25, m_top=4,
                 n_hetero: Optional[Sequence[Sequence[int]]] = None, promote_center=True, force_class=-1,
                 max_new_tokens=0, mid_policy=0, budget_frac=0.0, shard_kv_heads=0, shard_first=0):
        self.kw = dict(n_layers=n_layers, n_heads=n_heads, n_kv_heads=n_kv_heads, head_dim=head_dim,
                       seq_lens=list(seq_lens), sink=sink, recent=recent, mid_budget=mid_budget, window=window,
                       dtype=dtype, top_t=top_t, pool_kernel=pool_kernel, beta=beta, m_top=m_top, n_hetero=n_hetero,
                       promote_center=promote_center, force_class=force_class, max_new_tokens=max_new_tokens,
                       mid_policy=mid_policy, budget_frac=budget_frac, shard_kv_heads=shard_kv_heads,
                       shard_first=shard_first)
        p = taskkv_params()
        lib.taskkv_params_default(C.byref(p))
        p.n_layers, p.n_heads, p.n_kv_heads, p.head_dim = n_layers, n_heads, n_kv_heads, head_dim
        p.batch = len(seq_lens)
        self._seq = (C.c_int32 * len(seq_lens))(*[int(x) for x in seq_lens])
        p.seq_lens = C.cast(self._seq, C.POINTER(C.c_int32))
        p.sink, p.recent, p.window = sink, recent, window
        if isinstance(mid_budget, (list, tuple)):
            self._mid = (C.c_int32 * len(mid_budget))(*[int(x) for x in mid_budget])
            p.mid_budget_per_layer = C.cast(self._mid, C.POINTER(C.c_int32))
            p.mid_budget = int(mid_budget[0])
        else:
            self._mid = None
            p.mid_budget = int(mid_budget)
        p.top_t, p.pool_kernel, p.beta, p.m_top = top_t, pool_kernel, beta, m_top
        if n_hetero is not None:
            flat = [int(x) for row in n_hetero for x in row]
            self._nh = (C.c_int32 * len(flat))(*flat)
            p.n_hetero = C.cast(self._nh, C.POINTER(C.c_int32))
        else:
            self._nh = None
        p.promote_center = 1 if promote_center else 0
        p.force_class = force_class
        p.dtype = BF16 if dtype in (BF16, "bf16", torch.bfloat16) else F32
        p.max_new_tokens = max_new_tokens
        p.mid_policy = int(mid_policy)
        p.budget_frac = float(budget_frac)
        p.shard_kv_heads, p.shard_first = int(shard_kv_heads), int(shard_first)
        self.c = p

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.c.dtype == BF16 else torch.float32

    def layer(self, r: int) -> "Params":
        """The same problem restricted to layer r, as a one-layer problem of its own: Eq. 16's head count and the
        layer's middle budget are fixed here, so that compressing layer r alone (as soon as its K and V exist,
        while later layers are still being computed) gives exactly the cache rows the all-layer call gives."""
        kw = dict(self.kw)
        R = kw["n_layers"]
        if not 0 <= r < R:
            raise ValueError("layer out of range")
        mid = kw["mid_budget"]
        kw["mid_budget"] = int(mid[r]) if isinstance(mid, (list, tuple)) else int(mid)
        if kw["n_hetero"] is not None:
            kw["n_hetero"] = [[int(row[r])] for row in kw["n_hetero"]]
        else:
            f = int(lib.taskkv_hetero_count(kw["n_kv_heads"], kw["beta"], kw["m_top"], R, r))
            kw["n_hetero"] = [[f] for _ in kw["seq_lens"]]
        kw["n_layers"] = 1
        return Params(**kw)


def taskkv_plan(params: Params) -> taskkv_plan_info:
    info = taskkv_plan_info()
    _check(lib.taskkv_plan(C.byref(params.c), C.byref(info)), "taskkv_plan")
    return info


def _ptr_array(tensors: Sequence[torch.Tensor]):
    arr = (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])
    return arr


class Cache:
    """Handle of a compacted cache (taskkv_cache*) plus the torch buffers backing it."""

    def __init__(self, handle: int, params: Params, keep):
        self._h = C.c_void_p(handle)
        self.params = params
        self._keep = keep
        info = taskkv_plan_info()
        _check(lib.taskkv_cache_plan(self._h, C.byref(info)), "taskkv_cache_plan")
        self.info = info

    def release_workspace(self):
        """Drops the compress-time workspace (scores and top-t queries stop working)."""
        self._keep.pop("workspace", None)

    def close(self):
        if self._h:
            lib.taskkv_cache_destroy(self._h)
            self._h = None
            self._keep = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def taskkv_compress_layer(self, layer: int, q_win: Sequence[torch.Tensor], k: Sequence[torch.Tensor],
                              v: Sequence[torch.Tensor], window_lse: Optional[Sequence[torch.Tensor]] = None,
                              stream=None) -> None:
        """Steps a1-a5 for one layer of every sequence of a cache made by taskkv_cache_create.
        q_win[b]: [n, L, d]; k[b], v[b]: [n_kv, N_b, d] of that layer, contiguous CUDA tensors."""
        for t in list(q_win) + list(k) + list(v):
            if not t.is_contiguous() or not t.is_cuda:
                raise ValueError("inputs must be contiguous CUDA tensors")
        la = None
        if window_lse is not None:
            for t in window_lse:
                if not t.is_contiguous() or not t.is_cuda or t.dtype != torch.float32:
                    raise ValueError("window_lse must be contiguous fp32 CUDA tensors")
            la = _ptr_array(window_lse)
        _check(lib.taskkv_compress_layer(self._h, layer, _ptr_array(q_win), _ptr_array(k), _ptr_array(v), la,
                                         _stream_handle(stream)), "taskkv_compress_layer")

    def semantic_vectors(self) -> torch.Tensor:
        """The cache's semantic vectors (Eq. 15) as a view of its device memory: fp32 [batch * n_layers, n_kv, d]."""
        ptr, n = C.c_void_p(), C.c_int64()
        _check(lib.taskkv_cache_semantic(self._h, C.byref(ptr), C.byref(n)), "taskkv_cache_semantic")
        mem = self._keep["cache"]
        off = ptr.value - mem.data_ptr()
        d = self.params.c.head_dim
        return mem[off:off + 4 * n.value].view(torch.float32).view(-1, self.params.c.n_kv_heads, d)

    def taskkv_compress_shard_finish(self, sem_all: torch.Tensor, stream=None) -> None:
        """sem_all: fp32 [batch * n_layers, shard_kv_heads, d], every shard's vectors in head order."""
        if sem_all.dtype != torch.float32 or not sem_all.is_cuda or not sem_all.is_contiguous():
            raise ValueError("sem_all must be a contiguous fp32 CUDA tensor")
        p = self.params.c
        if sem_all.numel() != p.batch * p.n_layers * p.shard_kv_heads * p.head_dim:
            raise ValueError("sem_all must hold batch * n_layers * shard_kv_heads * d floats")
        _check(lib.taskkv_compress_shard_finish(self._h, sem_all.data_ptr(), _stream_handle(stream)),
               "taskkv_compress_shard_finish")

    # -- the decode-side calls
    def taskkv_append(self, k_new: torch.Tensor, v_new: torch.Tensor, stream=None) -> None:
        _check(lib.taskkv_append(self._h, k_new.data_ptr(), v_new.data_ptr(), _stream_handle(stream)),
               "taskkv_append")

    def taskkv_decode(self, q: torch.Tensor, out: Optional[torch.Tensor] = None,
                      lengths: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        if out is None:
            out = torch.empty_like(q)
        lp = lengths.data_ptr() if lengths is not None else None
        _check(lib.taskkv_decode(q.data_ptr(), self._h, lp, out.data_ptr(), _stream_handle(stream)),
               "taskkv_decode")
        return out

    def taskkv_append_ex(self, k_new: torch.Tensor, v_new: torch.Tensor, layer_begin: int, layer_count: int,
                         stream=None) -> None:
        _check(lib.taskkv_append_ex(self._h, k_new.data_ptr(), v_new.data_ptr(), layer_begin, layer_count,
                                    _stream_handle(stream)), "taskkv_append_ex")

    def taskkv_decode_ex(self, q: torch.Tensor, layer_begin: int, layer_count: int,
                         out: Optional[torch.Tensor] = None, lengths: Optional[torch.Tensor] = None,
                         stream=None) -> torch.Tensor:
        if out is None:
            out = torch.empty_like(q)
        lp = lengths.data_ptr() if lengths is not None else None
        _check(lib.taskkv_decode_ex(q.data_ptr(), self._h, lp, out.data_ptr(), layer_begin, layer_count,
                                    _stream_handle(stream)), "taskkv_decode_ex")
        return out

    def taskkv_decode_step(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                           out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        if out is None:
            out = torch.empty_like(q)
        _check(lib.taskkv_decode_step(q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), self._h, out.data_ptr(),
                                      _stream_handle(stream)), "taskkv_decode_step")
        return out

    def taskkv_decode_step_ex(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, layer_begin: int,
                              layer_count: int, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        if out is None:
            out = torch.empty_like(q)
        _check(lib.taskkv_decode_step_ex(q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), self._h, out.data_ptr(),
                                         layer_begin, layer_count, _stream_handle(stream)), "taskkv_decode_step_ex")
        return out

    def taskkv_decode_host(self, q: torch.Tensor, k_new: Optional[torch.Tensor], v_new: Optional[torch.Tensor],
                           out: torch.Tensor, stream=None) -> torch.Tensor:
        kp = k_new.data_ptr() if k_new is not None else None
        vp = v_new.data_ptr() if v_new is not None else None
        _check(lib.taskkv_decode_host(q.data_ptr(), kp, vp, self._h, out.data_ptr(), _stream_handle(stream)),
               "taskkv_decode_host")
        return out

    # -- synchronising reads
    def query(self, what: int) -> np.ndarray:
        nbytes = lib.taskkv_cache_query_bytes(self._h, what)
        if nbytes < 0:
            raise TaskKVError(EINVAL, "taskkv_cache_query_bytes")
        buf = np.empty(max(int(nbytes), 1), dtype=np.uint8)
        _check(lib.taskkv_cache_query(self._h, what, buf.ctypes.data, int(nbytes)), "taskkv_cache_query")
        buf = buf[:nbytes]
        U = int(self.info.n_units)
        if what in (Q_LENGTHS, Q_CLASSES, Q_CAPACITY, Q_STATUS):
            return buf.view(np.int32)
        if what == Q_PAGETAB:
            return buf.view(np.int32).reshape(U, -1)
        if what == Q_DIST:
            return buf.view(np.float32)
        if what == Q_SEMVEC:
            return buf.view(np.float32).reshape(U, -1)
        if what == Q_OFFSETS:
            return buf.view(np.int64)
        if what == Q_INDICES:
            return buf.view(np.int32).reshape(U, -1)
        if what == Q_SCORES:
            return buf.view(np.float32)
        if what == Q_TOPT:
            return buf.view(np.int32).reshape(U, -1)
        return buf

    def lengths(self):
        return self.query(Q_LENGTHS)

    def classes(self):
        return self.query(Q_CLASSES)

    def status(self) -> int:
        return int(self.query(Q_STATUS)[0])

    def pool_rows(self, which: str, u: int) -> torch.Tensor:
        """Rows of unit u's K ('k') or V ('v') segment as a CPU tensor [len_u, d] (for a paged cache: gathered from
        the unit's pages in order)."""
        ln = int(self.query(Q_LENGTHS)[u])
        d = self.params.c.head_dim
        es = 2 if self.params.c.dtype == BF16 else 4
        if self._keep is not None and "pool" in self._keep:
            pool = self._keep["pool"]
            P = pool.page_rows
            n = (ln + P - 1) // P
            tab = self.query(Q_PAGETAB)[u, :n].astype(np.int64)
            if pool.k_pages is None:
                # a pool the library allocated: its pages come back through the query (the whole pool: tests only)
                raw = self.query(Q_KPOOL if which == "k" else Q_VPOOL)
                pb = P * d * es
                seg = np.concatenate([raw[int(t) * pb:(int(t) + 1) * pb] for t in tab]) if n else raw[:0]
                return torch.from_numpy(seg[:ln * d * es].copy()).view(self.params.torch_dtype).reshape(ln, d)
            pages = (pool.k_pages if which == "k" else pool.v_pages)[torch.from_numpy(tab).to(pool.mem.device)]   # [n, P, d]
            return pages.reshape(n * P, d)[:ln].cpu().contiguous()
        raw = self.query(Q_KPOOL if which == "k" else Q_VPOOL)
        off = self.query(Q_OFFSETS)
        seg = raw[int(off[u]) * d * es:(int(off[u]) + ln) * d * es]
        t = torch.from_numpy(seg.copy())
        return t.view(self.params.torch_dtype).reshape(ln, d)

    def retained_indices(self, u: int, N: int) -> np.ndarray:
        ln = int(self.query(Q_LENGTHS)[u])
        if ln >= N:
            return np.arange(N, dtype=np.int64)
        return self.query(Q_INDICES)[u, :ln].astype(np.int64)


def taskkv_compress_ex(params: Params, q_win: Sequence[torch.Tensor], k: Sequence[torch.Tensor],
                       v: Sequence[torch.Tensor], stream=None, cache_mem: Optional[torch.Tensor] = None,
                       workspace_mem: Optional[torch.Tensor] = None,
                       window_lse: Optional[Sequence[torch.Tensor]] = None) -> Cache:
    """q_win[b]: [R, n, L, d]; k[b], v[b]: [R, n_kv, N_b, d] contiguous CUDA tensors.
    Cache and workspace memory are torch allocations unless supplied.  window_lse[b] (fp32 [R, n, L], optional):
    the log-sum-exp of the window rows from the prompt's attention; then taskkv_compress_lse is called."""
    info = taskkv_plan(params)
    dev = k[0].device
    if cache_mem is None:
        cache_mem = torch.empty(int(info.cache_bytes), dtype=torch.uint8, device=dev)
    if workspace_mem is None:
        workspace_mem = torch.empty(int(info.workspace_bytes), dtype=torch.uint8, device=dev)
    for t in list(q_win) + list(k) + list(v):
        if not t.is_contiguous() or not t.is_cuda:
            raise ValueError("inputs must be contiguous CUDA tensors")
    qa, ka, va = _ptr_array(q_win), _ptr_array(k), _ptr_array(v)
    h = C.c_void_p()
    if window_lse is not None:
        for t in window_lse:
            if not t.is_contiguous() or not t.is_cuda or t.dtype != torch.float32:
                raise ValueError("window_lse must be contiguous fp32 CUDA tensors")
        la = _ptr_array(window_lse)
        _check(lib.taskkv_compress_lse(C.byref(params.c), qa, ka, va, la, cache_mem.data_ptr(), cache_mem.numel(),
                                       workspace_mem.data_ptr(), workspace_mem.numel(), _stream_handle(stream),
                                       C.byref(h)), "taskkv_compress_lse")
        return Cache(h.value, params, {"cache": cache_mem, "workspace": workspace_mem, "lse": list(window_lse)})
    _check(lib.taskkv_compress_ex(C.byref(params.c), qa, ka, va, cache_mem.data_ptr(), cache_mem.numel(),
                                  workspace_mem.data_ptr(), workspace_mem.numel(), _stream_handle(stream),
                                  C.byref(h)), "taskkv_compress_ex")
    return Cache(h.value, params, {"cache": cache_mem, "workspace": workspace_mem})


def taskkv_cache_create(params: Params, device, stream=None, cache_mem: Optional[torch.Tensor] = None,
                        workspace_mem: Optional[torch.Tensor] = None) -> Cache:
    """An empty cache for the whole problem (every layer of every sequence); layers are then compressed one at a
    time with Cache.taskkv_compress_layer.  Cache and workspace memory are torch allocations unless supplied."""
    info = taskkv_plan(params)
    if cache_mem is None:
        cache_mem = torch.empty(int(info.cache_bytes), dtype=torch.uint8, device=device)
    if workspace_mem is None:
        workspace_mem = torch.empty(int(info.workspace_bytes), dtype=torch.uint8, device=device)
    h = C.c_void_p()
    with torch.cuda.device(cache_mem.device):
        _check(lib.taskkv_cache_create(C.byref(params.c), cache_mem.data_ptr(), cache_mem.numel(),
                                       workspace_mem.data_ptr(), workspace_mem.numel(), _stream_handle(stream),
                                       C.byref(h)), "taskkv_cache_create")
    return Cache(h.value, params, {"cache": cache_mem, "workspace": workspace_mem})


def taskkv_compress_shard_begin(params: Params, q_win: Sequence[torch.Tensor], k: Sequence[torch.Tensor],
                                v: Sequence[torch.Tensor], stream=None) -> Cache:
    """Steps a1-a2 for the KV heads of one shard (params.shard_kv_heads > 0).  The tensors hold the shard's own heads:
    q_win[b]: [R, n_local * G, L, d]; k[b], v[b]: [R, n_local, N_b, d]."""
    info = taskkv_plan(params)
    dev = k[0].device
    cache_mem = torch.empty(int(info.cache_bytes), dtype=torch.uint8, device=dev)
    workspace_mem = torch.empty(int(info.workspace_bytes), dtype=torch.uint8, device=dev)
    for t in list(q_win) + list(k) + list(v):
        if not t.is_contiguous() or not t.is_cuda:
            raise ValueError("inputs must be contiguous CUDA tensors")
    h = C.c_void_p()
    _check(lib.taskkv_compress_shard_begin(C.byref(params.c), _ptr_array(q_win), _ptr_array(k), _ptr_array(v), None,
                                           cache_mem.data_ptr(), cache_mem.numel(), workspace_mem.data_ptr(),
                                           workspace_mem.numel(), _stream_handle(stream), C.byref(h)),
           "taskkv_compress_shard_begin")
    return Cache(h.value, params, {"cache": cache_mem, "workspace": workspace_mem})


class Pool:
    """A page pool for paged caches (taskkv_pool*) plus the torch buffer backing it."""

    def __init__(self, page_rows: int, n_pages: int, head_dim: int, dtype, device, stream=None,
                 library_memory: bool = False):
        dt = BF16 if dtype in (BF16, "bf16", torch.bfloat16) else F32
        nbytes = int(lib.taskkv_pool_bytes(page_rows, n_pages, head_dim, dt))
        if nbytes == 0:
            raise TaskKVError(EINVAL, "taskkv_pool_bytes")
        self.page_rows, self.n_pages = page_rows, n_pages
        if library_memory:
            # the library allocates (and frees) the pool; its pages cannot be viewed from here
            self.mem = self.k_pages = self.v_pages = None
            h = C.c_void_p()
            with torch.cuda.device(torch.device(device)):
                _check(lib.taskkv_pool_create(page_rows, n_pages, head_dim, dt, None, 0, _stream_handle(stream),
                                              C.byref(h)), "taskkv_pool_create")
            self._h = h
            return
        self.mem = torch.empty(nbytes, dtype=torch.uint8, device=device)
        # layout of the pool memory (taskkv.h): K pages, then V pages from the next multiple of 256 bytes
        tdt = torch.bfloat16 if dt == BF16 else torch.float32
        page_bytes = page_rows * head_dim * (2 if dt == BF16 else 4)
        v_off = (n_pages * page_bytes + 255) // 256 * 256
        self.k_pages = self.mem[:n_pages * page_bytes].view(tdt).view(n_pages, page_rows, head_dim)
        self.v_pages = self.mem[v_off:v_off + n_pages * page_bytes].view(tdt).view(n_pages, page_rows, head_dim)
        h = C.c_void_p()
        with torch.cuda.device(self.mem.device):
            _check(lib.taskkv_pool_create(page_rows, n_pages, head_dim, dt, self.mem.data_ptr(), nbytes,
                                          _stream_handle(stream), C.byref(h)), "taskkv_pool_create")
        self._h = h

    def free_pages(self) -> int:
        return int(lib.taskkv_pool_free_pages(self._h))

    def close(self):
        if self._h:
            lib.taskkv_pool_destroy(self._h)
            self._h = None
            self.mem = None


def taskkv_plan_paged(params: Params, page_rows: int):
    """(plan info, pages the compression takes) for a paged cache."""
    info = taskkv_plan_info()
    pages = C.c_int64()
    _check(lib.taskkv_plan_paged(C.byref(params.c), page_rows, C.byref(info), C.byref(pages)), "taskkv_plan_paged")
    return info, int(pages.value)


def taskkv_compress_paged(params: Params, q_win: Sequence[torch.Tensor], k: Sequence[torch.Tensor],
                          v: Sequence[torch.Tensor], pool: Pool, stream=None,
                          cache_mem: Optional[torch.Tensor] = None,
                          workspace_mem: Optional[torch.Tensor] = None) -> Cache:
    """As taskkv_compress_ex, the compacted rows going to pages of `pool`."""
    dev = k[0].device
    if cache_mem is None or workspace_mem is None:
        info, _ = taskkv_plan_paged(params, pool.page_rows)
        if cache_mem is None:
            cache_mem = torch.empty(int(info.cache_bytes), dtype=torch.uint8, device=dev)
        if workspace_mem is None:
            workspace_mem = torch.empty(int(info.workspace_bytes), dtype=torch.uint8, device=dev)
    for t in list(q_win) + list(k) + list(v):
        if not t.is_contiguous() or not t.is_cuda:
            raise ValueError("inputs must be contiguous CUDA tensors")
    h = C.c_void_p()
    _check(lib.taskkv_compress_paged(C.byref(params.c), _ptr_array(q_win), _ptr_array(k), _ptr_array(v), pool._h,
                                     cache_mem.data_ptr(), cache_mem.numel(), workspace_mem.data_ptr(),
                                     workspace_mem.numel(), _stream_handle(stream), C.byref(h)),
           "taskkv_compress_paged")
    return Cache(h.value, params, {"cache": cache_mem, "workspace": workspace_mem, "pool": pool})


def taskkv_compress_host(params: Params, q_win: Sequence[torch.Tensor], k: Sequence[torch.Tensor],
                         v: Sequence[torch.Tensor], stream=None) -> Cache:
    """Same call with HOST tensors (pinned for asynchronous copies)."""
    qa, ka, va = _ptr_array(q_win), _ptr_array(k), _ptr_array(v)
    h = C.c_void_p()
    _check(lib.taskkv_compress_host(C.byref(params.c), qa, ka, va, _stream_handle(stream), C.byref(h)),
           "taskkv_compress_host")
    return Cache(h.value, params, {})


def taskkv_exact_semantic(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, want_scores: bool = True, stream=None,
                          workspace_mem: Optional[torch.Tensor] = None):
    """Eq. 1-2 for one sequence.  q: [R, n, N, d], k, v: [R, n_kv, N, d], contiguous bf16 CUDA tensors.
    Returns (sem [R, n_kv, d] fp32, C [R, n_kv, N] fp32 or None).  The scratch is a torch allocation unless supplied."""
    for t in (q, k, v):
        if not t.is_contiguous() or not t.is_cuda or t.dtype != torch.bfloat16:
            raise ValueError("inputs must be contiguous bf16 CUDA tensors")
    R, n, N, d = q.shape
    n_kv = k.shape[1]
    if k.shape != (R, n_kv, N, d) or v.shape != k.shape:
        raise ValueError("k and v must be [R, n_kv, N, d] with q's R, N and d")
    sem = torch.empty(R, n_kv, d, dtype=torch.float32, device=q.device)
    c = torch.empty(R, n_kv, N, dtype=torch.float32, device=q.device) if want_scores else None
    if workspace_mem is None:
        workspace_mem = torch.empty(int(lib.taskkv_exact_semantic_bytes(R, n, n_kv, d, N)), dtype=torch.uint8,
                                    device=q.device)
    _check(lib.taskkv_exact_semantic(q.data_ptr(), k.data_ptr(), v.data_ptr(), R, n, n_kv, d, N, sem.data_ptr(),
                                     c.data_ptr() if c is not None else None, workspace_mem.data_ptr(),
                                     workspace_mem.numel(), _stream_handle(stream)), "taskkv_exact_semantic")
    return sem, c


def taskkv_compress(q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor, *, sink: int, recent: int,
                    mid_budget: int, window: int, stream=None) -> Cache:
    """The flat form: one bf16 sequence, Sec. V-D defaults, library-owned memory."""
    R, n, L, d = q_win.shape
    _, n_kv, N, _ = k.shape
    h = C.c_void_p()
    _check(lib.taskkv_compress(q_win.data_ptr(), k.data_ptr(), v.data_ptr(), R, n, n_kv, d, N, sink, recent,
                               mid_budget, window, _stream_handle(stream), C.byref(h)), "taskkv_compress")
    beta, m = (0.25, 4) if n == n_kv else (0.3, 1)
    params = Params(n_layers=R, n_heads=n, n_kv_heads=n_kv, head_dim=d, seq_lens=[N], sink=sink, recent=recent,
                    mid_budget=mid_budget, window=window, dtype=BF16, beta=beta, m_top=m, max_new_tokens=4096)
    return Cache(h.value, params, {})


def taskkv_decode_noalloc(q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, seg_off: torch.Tensor,
                          lengths: torch.Tensor, *, group: int, max_len: int,
                          out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Decode attention over caller-held pools with the library's fixed scratch: no
    allocation happens inside the call (`out` is allocated here, by torch, only if
    the caller passes none).  q: [n_units * group, d]; pools: [rows, d];
    seg_off int64 [n_units]; lengths int32 [n_units]; a length above max_len is
    clamped to max_len.  The C side sees only pointers, so shapes, types and
    devices are checked here."""
    if q.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("q must be bf16 or fp32")
    if out is None:
        out = torch.empty_like(q)
    n_units = lengths.numel()
    if q.dim() != 2 or q.shape[0] != n_units * group:
        raise ValueError("q must be [n_units * group, head_dim]")
    d = q.shape[1]
    if out.shape != q.shape or out.dtype != q.dtype:
        raise ValueError("out must match q")
    for name, t in (("k_pool", k_pool), ("v_pool", v_pool)):
        if t.dim() != 2 or t.shape[1] != d or t.dtype != q.dtype:
            raise ValueError(f"{name} must be [rows, head_dim] in q's dtype")
    if k_pool.shape != v_pool.shape:
        raise ValueError("k_pool and v_pool must have the same shape")
    if seg_off.dtype != torch.int64 or seg_off.numel() != n_units:
        raise ValueError("seg_off must be int64 [n_units]")
    if lengths.dtype != torch.int32:
        raise ValueError("lengths must be int32 [n_units]")
    for name, t in (("q", q), ("out", out), ("k_pool", k_pool), ("v_pool", v_pool), ("seg_off", seg_off),
                    ("lengths", lengths)):
        if not t.is_cuda or t.device != q.device or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous CUDA tensor on q's device")
    dtype = BF16 if q.dtype == torch.bfloat16 else F32
    _check(lib.taskkv_decode_noalloc(q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(), seg_off.data_ptr(),
                                     lengths.data_ptr(), n_units, group, d, dtype, int(max_len), out.data_ptr(),
                                     _stream_handle(stream)), "taskkv_decode_noalloc")
    return out


def params_from_workload(wl, max_new_tokens: Optional[int] = None, **overrides) -> Params:
    kw = dict(n_layers=wl.n_layers, n_heads=wl.n_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
              seq_lens=wl.seq_lens, sink=wl.sink, recent=wl.recent, mid_budget=list(wl.mid_budget),
              window=wl.window, dtype=wl.dtype, top_t=wl.top_t, pool_kernel=wl.pool_kernel,
              n_hetero=wl.n_hetero, promote_center=wl.promote_center,
              budget_frac=getattr(wl, "budget_frac", 0.0),
              max_new_tokens=wl.decode_steps if max_new_tokens is None else max_new_tokens)
    kw.update(overrides)
    return Params(**kw)
