"""TEST INFRASTRUCTURE ONLY: ctypes front end of the fp64 CPU oracle.

Only the tests, the smoke check and the bench's cpu_baseline / reference leg
may import this package.  It compiles ``reform_oracle.cpp`` with g++ on first
use (or through :func:`build`) and exposes one Python function per oracle
operation, taking and returning torch CPU tensors.  It never touches the CUDA
library and shares no code with it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "reform_oracle.cpp")
_LIB = os.path.join(_HERE, "libreform_oracle.so")
_lock = threading.Lock()
_lib = None

F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle shared library next to its source; returns its path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-o", tmp, _SRC]
            )
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_set_threads.restype = ctypes.c_int
        _lib.oracle_get_threads.restype = ctypes.c_int
    return _lib


def set_threads(n: int) -> int:
    return _load().oracle_set_threads(ctypes.c_int(n))


def get_threads() -> int:
    return _load().oracle_get_threads()


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"oracle takes float32 or bfloat16 inputs, got {t.dtype}")


def _p(t):
    if t is None:
        return ctypes.c_void_p(0)
    assert t.device.type == "cpu" and t.is_contiguous()
    return ctypes.c_void_p(t.data_ptr())


def attention(q, k, v, n_cache, scale=None, causal=True, rows=None):
    """O and LSE (fp64) for chunk rows ``rows`` (default: all).

    q [B,Hq,Lc,d]; k, v [B,Hkv,cap,d] holding cache rows then chunk rows.
    Returns (out [B,Hq,n_rows,d], lse [B,Hq,n_rows]).
    """
    B, Hq, Lc, d = q.shape
    _, Hkv, cap, _ = k.shape
    scale = float(scale) if scale else d ** -0.5
    if rows is not None:
        rows_t = torch.as_tensor(rows, dtype=torch.int32).contiguous()
        n_rows = rows_t.numel()
    else:
        rows_t, n_rows = None, Lc
    out = torch.empty(B, Hq, n_rows, d, dtype=torch.float64)
    lse = torch.empty(B, Hq, n_rows, dtype=torch.float64)
    rc = _load().oracle_attention(
        _dt(q), B, Hq, Hkv, d, Lc, int(n_cache), cap, ctypes.c_double(scale), int(bool(causal)),
        _p(q), _p(k), _p(v), _p(rows_t), n_rows, _p(out), _p(lse))
    if rc != 0:
        raise ValueError("oracle_attention: bad arguments")
    return out, lse


def key_scores(q, k, n_cache, window, scale=None, causal=True, score_in=None, accumulate=False):
    """Attention mass per key, fp64 [B,Hkv,cap]; entries past n_cache+Lc are 0."""
    B, Hq, Lc, d = q.shape
    _, Hkv, cap, _ = k.shape
    scale = float(scale) if scale else d ** -0.5
    out = torch.zeros(B, Hkv, cap, dtype=torch.float64)
    if score_in is not None:
        score_in = score_in.to(torch.float64).contiguous()
    rc = _load().oracle_key_scores(
        _dt(q), B, Hq, Hkv, d, Lc, int(n_cache), cap, int(window), ctypes.c_double(scale),
        int(bool(causal)), int(bool(accumulate)), _p(q), _p(k), _p(score_in), _p(out))
    if rc != 0:
        raise ValueError("oracle_key_scores: bad arguments")
    return out


def evict_topk(k_src, v_src, score_src, n_keys, budget, n_sink, n_recent, cap_dst=None, pos_src=None):
    """Returns dict(k, v, score, pos, kept_idx, n_kept) after compression."""
    B, Hkv, cap_src, d = k_src.shape
    cap_dst = cap_dst or cap_src
    row_bytes = d * k_src.element_size()
    k_dst = torch.zeros(B, Hkv, cap_dst, d, dtype=k_src.dtype)
    v_dst = torch.zeros(B, Hkv, cap_dst, d, dtype=v_src.dtype)
    score64 = score_src.to(torch.float64).contiguous()
    score_dst = torch.zeros(B, Hkv, cap_dst, dtype=torch.float64)
    kept = torch.full((B, Hkv, budget), -1, dtype=torch.int32)
    pos_dst = torch.zeros(B, Hkv, cap_dst, dtype=torch.int32) if pos_src is not None else None
    _load().oracle_evict_topk.restype = ctypes.c_int
    rc = _load().oracle_evict_topk(
        B, Hkv, int(n_keys), cap_src, cap_dst, int(budget), int(n_sink), int(n_recent),
        ctypes.c_longlong(row_bytes), _p(k_src), _p(v_src), _p(score64), _p(pos_src),
        _p(k_dst), _p(v_dst), _p(score_dst), _p(pos_dst), _p(kept))
    if rc < 0:
        raise ValueError("oracle_evict_topk: bad arguments")
    return dict(k=k_dst, v=v_dst, score=score_dst, pos=pos_dst, kept_idx=kept, n_kept=rc)


def embed_append(bank, token_offset, sel, q_state=None, k_state=None, v_state=None, eps=0.0,
                 want_f64=False):
    """Writes normalised head states into ``bank`` [B,N_cap,E] in place.

    sel: list of (kind, head, slot), kind 0/1/2 = Q/K/V state.  Returns the
    unrounded fp64 bank (same shape, zeros elsewhere) when want_f64.
    """
    ref = q_state if q_state is not None else (k_state if k_state is not None else v_state)
    B, _, Lc, d = ref.shape
    Hq = q_state.shape[1] if q_state is not None else 0
    kv = k_state if k_state is not None else v_state
    Hkv = kv.shape[1] if kv is not None else 0
    _, N_cap, E = bank.shape
    sel_t = torch.tensor([list(s) for s in sel], dtype=torch.int32).contiguous()
    f64 = torch.zeros(bank.shape, dtype=torch.float64) if want_f64 else None
    rc = _load().oracle_embed_append(
        _dt(bank), B, Lc, d, Hq, Hkv, _p(q_state), _p(k_state), _p(v_state), len(sel), _p(sel_t),
        _p(bank), _p(f64), ctypes.c_longlong(N_cap), E, ctypes.c_longlong(int(token_offset)),
        ctypes.c_double(eps))
    if rc != 0:
        raise ValueError("oracle_embed_append: bad arguments")
    return f64


def retrieve_topk(bank, queries, N, k, scale=1.0, pool_window=1, n_keep_head=0, n_keep_tail=0,
                  pool_mode="max"):
    """Returns dict(idx [B,n_out] int32 ascending, ts [B,N], pooled [B,N] fp64).  pool_mode "max"
    (Sec. 3.3) or "mean" (the smoothing of the head-ranking procedure)."""
    B, N_cap, E = bank.shape
    nq = queries.shape[1]
    idx = torch.full((B, k), -1, dtype=torch.int32)
    ts = torch.empty(B, N, dtype=torch.float64)
    pooled = torch.empty(B, N, dtype=torch.float64)
    rc = _load().oracle_retrieve_topk(
        _dt(bank), B, ctypes.c_longlong(int(N)), ctypes.c_longlong(N_cap), E, _p(bank), nq,
        _p(queries), ctypes.c_double(scale), int(pool_window), int(n_keep_head), int(n_keep_tail),
        int(k), _p(idx), _p(ts), _p(pooled), {"max": 0, "mean": 1}[pool_mode])
    if rc < 0:
        raise ValueError("oracle_retrieve_topk: bad arguments")
    return dict(idx=idx[:, :rc].contiguous(), ts=ts, pooled=pooled, n_out=rc)


def rope(x, row_begin, rows, pos_begin, base=10000.0, interleaved=False):
    """Rotary embedding of rows [row_begin, row_begin+rows) of x [B,H,cap,d] at consecutive
    positions pos_begin, pos_begin+1, ...; returns a new tensor (other rows copied)."""
    B, H, cap, d = x.shape
    y = x.clone()
    rc = _load().oracle_rope(
        _dt(x), B, H, d, ctypes.c_longlong(cap), ctypes.c_longlong(int(row_begin)),
        ctypes.c_longlong(int(rows)), ctypes.c_longlong(int(pos_begin)), ctypes.c_double(base),
        int(bool(interleaved)), _p(x), _p(y))
    if rc != 0:
        raise ValueError("oracle_rope: bad arguments")
    return y


def gather(src, idx):
    """src [B,n_rows,D] (any dtype), idx [B,k] int32 -> [B,k,D]."""
    B, n_rows, D = src.shape
    k = idx.shape[1]
    dst = torch.empty(B, k, D, dtype=src.dtype)
    idx32 = idx.to(torch.int32).contiguous()
    rc = _load().oracle_gather(
        B, ctypes.c_longlong(n_rows), ctypes.c_longlong(D * src.element_size()), _p(src),
        _p(idx32), k, _p(dst))
    if rc != 0:
        raise ValueError("oracle_gather: index out of range")
    return dst
