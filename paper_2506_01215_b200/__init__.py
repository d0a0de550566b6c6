"""Python binding of the REFORM compress-and-gather C-ABI library (B200, sm_100a).

Argument marshalling only: every function here fills the matching params
struct of ``include/reform.h`` from torch tensors (device memory and streams
are torch's) and calls the ``reform_*`` entry point of ``libreform.so``.  All
arithmetic runs in the CUDA kernels of that library; there is no CPU or
PyTorch fallback -- if the library is missing or a call fails, an exception
is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libreform.so")

F32, BF16 = 0, 1
SCORE_ACCUMULATE, NO_SCORE, FORCE_SIMT, ROPE, ROPE_INTERLEAVED = 1, 2, 4, 8, 16
STATE_Q, STATE_K, STATE_V = 0, 1, 2
POOL_MAX, POOL_MEAN = 0, 1
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TOO_LARGE = 0, -1, -2, -3, -4, -5
EVICT_STATIC_MAX_SEGS, EVICT_STATIC_MAX_KEYS, EVICT_STATIC_MAX_BUDGET = 32, 65536, 16384
DEV_TIMEOUT, DEV_BAD_INDEX = 1, 2
MAX_SEL = 16

_vp, _i32, _i64, _f32, _u32, _sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float,
                                    ctypes.c_uint32, ctypes.c_size_t)


class ChunkParams(ctypes.Structure):
    _fields_ = [("struct_size", _sz), ("dtype", _i32), ("B", _i32), ("Hq", _i32), ("Hkv", _i32),
                ("d", _i32), ("Lc", _i32), ("n_cache", _i32), ("cap", _i32), ("score_window", _i32),
                ("softmax_scale", _f32), ("flags", _u32), ("rope_theta", _f32), ("q", _vp), ("k", _vp), ("v", _vp),
                ("out", _vp), ("lse", _vp), ("score", _vp), ("workspace", _vp),
                ("workspace_bytes", _sz), ("dev_status", _vp)]


class EvictParams(ctypes.Structure):
    _fields_ = [("struct_size", _sz), ("dtype", _i32), ("B", _i32), ("Hkv", _i32), ("d", _i32),
                ("n_keys", _i32), ("cap_src", _i32), ("cap_dst", _i32), ("budget", _i32),
                ("n_sink", _i32), ("n_recent", _i32), ("k_src", _vp), ("v_src", _vp),
                ("score_src", _vp), ("pos_src", _vp), ("k_dst", _vp), ("v_dst", _vp),
                ("score_dst", _vp), ("pos_dst", _vp), ("kept_idx", _vp), ("n_kept_host", _vp),
                ("workspace", _vp), ("workspace_bytes", _sz), ("dev_status", _vp)]


class HeadSel(ctypes.Structure):
    _fields_ = [("kind", _i32), ("head", _i32), ("slot", _i32)]


class EmbedParams(ctypes.Structure):
    _fields_ = [("struct_size", _sz), ("dtype", _i32), ("B", _i32), ("Lc", _i32), ("d", _i32),
                ("Hq", _i32), ("Hkv", _i32), ("n_sel", _i32), ("E", _i32), ("N_cap", _i64),
                ("token_offset", _i64), ("eps", _f32), ("sel", ctypes.POINTER(HeadSel)),
                ("q_state", _vp), ("k_state", _vp), ("v_state", _vp), ("bank", _vp),
                ("dev_status", _vp)]


class RetrieveParams(ctypes.Structure):
    _fields_ = [("struct_size", _sz), ("dtype", _i32), ("B", _i32), ("N", _i64), ("N_cap", _i64),
                ("E", _i32), ("nq", _i32), ("scale", _f32), ("pool_window", _i32),
                ("n_keep_head", _i32), ("n_keep_tail", _i32), ("k", _i32), ("pool_mode", _i32), ("bank", _vp),
                ("queries", _vp), ("idx_out", _vp), ("token_score_out", _vp),
                ("pooled_score_out", _vp), ("workspace", _vp), ("workspace_bytes", _sz),
                ("dev_status", _vp)]


class GatherParams(ctypes.Structure):
    _fields_ = [("struct_size", _sz), ("B", _i32), ("k", _i32), ("n_rows", _i64),
                ("row_bytes", _i64), ("src", _vp), ("idx", _vp), ("dst", _vp), ("dev_status", _vp)]


class RopeParams(ctypes.Structure):
    _fields_ = [("struct_size", _sz), ("dtype", _i32), ("B", _i32), ("H", _i32), ("d", _i32),
                ("interleaved", _i32), ("cap", _i64), ("row_begin", _i64), ("rows", _i64),
                ("pos_begin", _i64), ("theta_base", _f32), ("src", _vp), ("dst", _vp),
                ("dev_status", _vp)]


EXPORTS = (
    "reform_chunk_step", "reform_chunk_step_workspace_size", "reform_evict_topk",
    "reform_evict_topk_workspace_size", "reform_evict_topk_static", "reform_debug_evict_wait_expiry",
    "reform_embed_append", "reform_retrieve_topk",
    "reform_retrieve_topk_workspace_size", "reform_gather", "reform_rope", "reform_status_string",
    "reform_last_cuda_error", "reform_device_error", "reform_version", "reform_kernel_launch_count",
    "reform_debug_last_path",
)

_lib = None


class ReformError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        msg = lib().reform_status_string(status).decode()
        if status == ERR_CUDA:
            msg += f" (cudaError {lib().reform_last_cuda_error()})"
        super().__init__(f"{fn}: {msg} [{status}]")


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2506_01215_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        for name, ptype in (("reform_chunk_step", ChunkParams), ("reform_evict_topk", EvictParams),
                            ("reform_retrieve_topk", RetrieveParams)):
            getattr(L, name).argtypes = [ctypes.POINTER(ptype), _vp]
            getattr(L, name).restype = ctypes.c_int
            getattr(L, name + "_workspace_size").argtypes = [ctypes.POINTER(ptype)]
            getattr(L, name + "_workspace_size").restype = _sz
        L.reform_evict_topk_static.argtypes = [ctypes.POINTER(EvictParams), _vp]
        L.reform_evict_topk_static.restype = ctypes.c_int
        L.reform_debug_evict_wait_expiry.argtypes = [ctypes.POINTER(EvictParams), ctypes.c_longlong, _vp]
        L.reform_debug_evict_wait_expiry.restype = ctypes.c_int
        L.reform_embed_append.argtypes = [ctypes.POINTER(EmbedParams), _vp]
        L.reform_embed_append.restype = ctypes.c_int
        L.reform_gather.argtypes = [ctypes.POINTER(GatherParams), _vp]
        L.reform_gather.restype = ctypes.c_int
        L.reform_rope.argtypes = [ctypes.POINTER(RopeParams), _vp]
        L.reform_rope.restype = ctypes.c_int
        L.reform_status_string.argtypes = [ctypes.c_int]
        L.reform_status_string.restype = ctypes.c_char_p
        L.reform_last_cuda_error.restype = ctypes.c_int
        L.reform_device_error.argtypes = [ctypes.c_int]
        L.reform_device_error.restype = ctypes.c_int
        L.reform_version.restype = ctypes.c_int
        L.reform_kernel_launch_count.restype = ctypes.c_longlong
        L.reform_debug_last_path.restype = ctypes.c_int
        _lib = L
    return _lib


def device_error(clear: bool = True) -> int:
    """DEV_* bits raised by any kernel of the library on the current device since the last clear
    (synchronises the device first)."""
    torch.cuda.synchronize()
    rc = int(lib().reform_device_error(1 if clear else 0))
    if rc < 0:
        raise ReformError("reform_device_error", rc)
    return rc


def kernel_launch_count() -> int:
    return int(lib().reform_kernel_launch_count())


PATH_NONE, PATH_CLUSTER, PATH_COOPERATIVE, PATH_PER_SEGMENT, PATH_PER_PASS = 0, 1, 2, 3, 4


def debug_last_path() -> int:
    """reform_debug_last_path: the launch form (PATH_*) the calling thread's last evict_topk or
    retrieve_topk chose for its selection."""
    return int(lib().reform_debug_last_path())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"reform kernels take float32 or bfloat16 tensors, got {t.dtype}")


def _ptr(t: Optional[torch.Tensor], pinned_ok: bool = False) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda and not (pinned_ok and t.is_pinned()):
        raise ValueError("reform entry points take device tensors" +
                         (" (or, here, page-locked host memory)" if pinned_ok else ""))
    if not t.is_contiguous():
        raise ValueError("reform entry points take contiguous tensors")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    return getattr(stream, "cuda_stream", stream) or None


_ws_cache = {}


def workspace(nbytes: int, device) -> Optional[torch.Tensor]:
    """A cached per-device scratch tensor of at least nbytes (None for 0)."""
    if nbytes == 0:
        return None
    key = torch.device(device)
    w = _ws_cache.get(key)
    if w is None or w.numel() < nbytes:
        w = torch.empty(max(nbytes, 1 << 20), dtype=torch.uint8, device=device)
        _ws_cache[key] = w
    return w


def _check(fn: str, rc: int):
    if rc != OK:
        raise ReformError(fn, rc)


def chunk_step(q, k, v, out, score, n_cache: int, score_window: int, *, lse=None,
               softmax_scale: float = 0.0, flags: int = 0, rope_theta: float = 0.0, ws=None, dev_status=None,
               stream=None):
    """reform_chunk_step: q [B,Hq,Lc,d], k/v [B,Hkv,cap,d], out like q,
    score [B,Hkv,cap] fp32 (in/out), lse [B,Hq,Lc] fp32 (optional).  With ROPE in flags, q and k
    are un-rotated and the call applies the rotary embedding (base rope_theta) itself."""
    B, Hq, Lc, d = q.shape
    _, Hkv, cap, _ = k.shape
    p = ChunkParams(ctypes.sizeof(ChunkParams), _dtype_code(q), B, Hq, Hkv, d, Lc, int(n_cache), cap,
                    int(score_window), float(softmax_scale), int(flags), float(rope_theta), _ptr(q), _ptr(k), _ptr(v),
                    _ptr(out), _ptr(lse), _ptr(score), None, 0, _ptr(dev_status))
    need = lib().reform_chunk_step_workspace_size(ctypes.byref(p))
    ws = ws if ws is not None else workspace(need, q.device)
    if ws is not None:
        p.workspace, p.workspace_bytes = ws.data_ptr(), ws.numel() * ws.element_size()
    _check("reform_chunk_step", lib().reform_chunk_step(ctypes.byref(p), _stream(stream)))


def evict_topk(k_src, v_src, score_src, k_dst, v_dst, score_dst, n_keys: int, budget: int,
               n_sink: int, n_recent: int, *, pos_src=None, pos_dst=None, kept_idx=None, ws=None,
               stream=None) -> int:
    """reform_evict_topk; returns n_kept = min(n_keys, budget)."""
    B, Hkv, cap_src, d = k_src.shape
    cap_dst = k_dst.shape[2]
    n_kept = ctypes.c_int32(0)
    p = EvictParams(ctypes.sizeof(EvictParams), _dtype_code(k_src), B, Hkv, d, int(n_keys), cap_src,
                    cap_dst, int(budget), int(n_sink), int(n_recent), _ptr(k_src), _ptr(v_src),
                    _ptr(score_src), _ptr(pos_src), _ptr(k_dst), _ptr(v_dst), _ptr(score_dst),
                    _ptr(pos_dst), _ptr(kept_idx), ctypes.addressof(n_kept), None, 0, None)
    need = lib().reform_evict_topk_workspace_size(ctypes.byref(p))
    ws = ws if ws is not None else workspace(need, k_src.device)
    if ws is not None:
        p.workspace, p.workspace_bytes = ws.data_ptr(), ws.numel() * ws.element_size()
    _check("reform_evict_topk", lib().reform_evict_topk(ctypes.byref(p), _stream(stream)))
    return n_kept.value


def debug_evict_wait_expiry(k_src, v_src, score_src, k_dst, v_dst, score_dst, n_keys: int, budget: int,
                            n_sink: int, n_recent: int, wait_cycles: int, dev_status, *, stream=None):
    """reform_debug_evict_wait_expiry: the eviction's one-launch form with its hand-off waits
    limited to wait_cycles and waiting for a flag that nothing sets; REFORM_DEV_TIMEOUT lands in
    dev_status (a device int32 tensor) and in the per-device error word.  Outputs are unspecified."""
    B, Hkv, cap_src, d = k_src.shape
    p = EvictParams(ctypes.sizeof(EvictParams), _dtype_code(k_src), B, Hkv, d, int(n_keys), cap_src,
                    k_dst.shape[2], int(budget), int(n_sink), int(n_recent), _ptr(k_src), _ptr(v_src),
                    _ptr(score_src), None, _ptr(k_dst), _ptr(v_dst), _ptr(score_dst), None, None, None,
                    None, 0, _ptr(dev_status))
    need = lib().reform_evict_topk_workspace_size(ctypes.byref(p))
    ws = workspace(need, k_src.device)
    p.workspace, p.workspace_bytes = ws.data_ptr(), ws.numel() * ws.element_size()
    _check("reform_debug_evict_wait_expiry",
           lib().reform_debug_evict_wait_expiry(ctypes.byref(p), int(wait_cycles), _stream(stream)))


def evict_topk_static(k_src, v_src, score_src, k_dst, v_dst, score_dst, n_keys: int, budget: int,
                      n_sink: int, n_recent: int, *, pos_src=None, pos_dst=None, kept_idx=None,
                      stream=None) -> int:
    """reform_evict_topk_static: reform_evict_topk for callers that cannot allocate device memory
    (no workspace argument; the library's built-in scratch is used, and neither this wrapper nor the
    call allocates anything).  Raises ReformError(ERR_TOO_LARGE) beyond B*Hkv <= 32, n_keys <= 65536,
    budget <= 16384.  Calls that overlap on the GPU share the scratch and race; keep them on one
    stream.  Returns n_kept."""
    B, Hkv, cap_src, d = k_src.shape
    cap_dst = k_dst.shape[2]
    n_kept = ctypes.c_int32(0)
    p = EvictParams(ctypes.sizeof(EvictParams), _dtype_code(k_src), B, Hkv, d, int(n_keys), cap_src,
                    cap_dst, int(budget), int(n_sink), int(n_recent), _ptr(k_src), _ptr(v_src),
                    _ptr(score_src), _ptr(pos_src), _ptr(k_dst), _ptr(v_dst), _ptr(score_dst),
                    _ptr(pos_dst), _ptr(kept_idx), ctypes.addressof(n_kept), None, 0, None)
    _check("reform_evict_topk_static", lib().reform_evict_topk_static(ctypes.byref(p), _stream(stream)))
    return n_kept.value


def embed_append(bank, token_offset: int, sel: Sequence[Tuple[int, int, int]], *, q_state=None,
                 k_state=None, v_state=None, eps: float = 0.0, stream=None):
    """reform_embed_append: bank [B,N_cap,E]; sel = [(kind, head, slot), ...]."""
    ref = q_state if q_state is not None else (k_state if k_state is not None else v_state)
    B, _, Lc, d = ref.shape
    Hq = q_state.shape[1] if q_state is not None else 0
    kv = k_state if k_state is not None else v_state
    Hkv = kv.shape[1] if kv is not None else 0
    _, N_cap, E = bank.shape
    arr = (HeadSel * max(len(sel), 1))(*[HeadSel(*map(int, s)) for s in sel])
    p = EmbedParams(ctypes.sizeof(EmbedParams), _dtype_code(bank), B, Lc, d, Hq, Hkv, len(sel), E,
                    N_cap, int(token_offset), float(eps), arr, _ptr(q_state), _ptr(k_state),
                    _ptr(v_state), _ptr(bank), None)
    _check("reform_embed_append", lib().reform_embed_append(ctypes.byref(p), _stream(stream)))


def retrieve_topk(bank, queries, N: int, k: int, idx_out, *, scale: float = 1.0,
                  pool_window: int = 1, n_keep_head: int = 0, n_keep_tail: int = 0,
                  token_score_out=None, pooled_score_out=None, pool_mode: int = POOL_MAX, ws=None,
                  stream=None) -> int:
    """reform_retrieve_topk; returns n_out = min(k, N)."""
    B, N_cap, E = bank.shape
    nq = queries.shape[1]
    p = RetrieveParams(ctypes.sizeof(RetrieveParams), _dtype_code(bank), B, int(N), N_cap, E, nq,
                       float(scale), int(pool_window), int(n_keep_head), int(n_keep_tail), int(k),
                       int(pool_mode), _ptr(bank), _ptr(queries), _ptr(idx_out), _ptr(token_score_out),
                       _ptr(pooled_score_out), None, 0, None)
    need = lib().reform_retrieve_topk_workspace_size(ctypes.byref(p))
    ws = ws if ws is not None else workspace(need, bank.device)
    if ws is not None:
        p.workspace, p.workspace_bytes = ws.data_ptr(), ws.numel() * ws.element_size()
    _check("reform_retrieve_topk", lib().reform_retrieve_topk(ctypes.byref(p), _stream(stream)))
    return min(int(k), int(N))


def gather(src, idx, dst, *, dev_status=None, stream=None):
    """reform_gather: src [B,n_rows,D] (device, or pinned host memory read in place), idx [B,k]
    int32, dst [B,k,D]."""
    B, n_rows, D = src.shape
    k = idx.shape[1]
    p = GatherParams(ctypes.sizeof(GatherParams), B, k, n_rows, D * src.element_size(),
                     _ptr(src, pinned_ok=True), _ptr(idx), _ptr(dst), _ptr(dev_status))
    _check("reform_gather", lib().reform_gather(ctypes.byref(p), _stream(stream)))


def rope(src, dst, row_begin: int, rows: int, pos_begin: int, *, theta_base: float = 0.0,
         interleaved: bool = False, stream=None):
    """reform_rope: rotary embedding of rows [row_begin, row_begin+rows) of src [B,H,cap,d] at
    consecutive positions pos_begin, pos_begin+1, ... into dst (may be src)."""
    B, H, cap, d = src.shape
    p = RopeParams(ctypes.sizeof(RopeParams), _dtype_code(src), B, H, d, int(bool(interleaved)), cap,
                   int(row_begin), int(rows), int(pos_begin), float(theta_base), _ptr(src), _ptr(dst), None)
    _check("reform_rope", lib().reform_rope(ctypes.byref(p), _stream(stream)))


# the C entry points' own names, for callers that prefer them
reform_chunk_step = chunk_step
reform_evict_topk = evict_topk
reform_evict_topk_static = evict_topk_static
reform_embed_append = embed_append
reform_retrieve_topk = retrieve_topk
reform_gather = gather
reform_rope = rope
