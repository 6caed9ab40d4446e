"""Thin ctypes binding of libkvs.so: same names as the C ABI, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  PyTorch is used here for
device memory and streams.  There is no CPU fallback: if the library is missing or
the tensors are not on a CUDA device the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvs.so")

KVS_OK = 0
KVS_ERR_INVALID_ARG = -1
KVS_ERR_UNSUPPORTED = -2
KVS_ERR_ALIGNMENT = -3
KVS_ERR_WORKSPACE = -4
KVS_ERR_CUDA = -5
KVS_ERR_BAD_EVICT = -6
KVS_ERR_TIMEOUT = -7
KVS_ERR_BAD_META = -8
GRAD_BF16, GRAD_FP32 = 0, 1
CLASS_EMPTY, CLASS_PARTIAL, CLASS_FULL = 0, 1, 2
TILE = 128

_vp, _i, _f, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t

# name -> (restype, argtypes); mirrors include/kvs.h
SIGNATURES = {
    "kvs_strerror": (ctypes.c_char_p, [_i]),
    "kvs_mask_meta_bytes": (_sz, [_i, _i, _i]),
    "kvs_evict_at_from_events": (_i, [_vp, _i, _vp, _i, _i, _vp, _vp]),
    "kvs_mask_meta": (_i, [_vp, _vp, _i, _i, _i, _vp, _sz, _vp]),
    "kvs_mask_meta_keys": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _sz, _vp]),
    "kvs_reorder_keys": (_i, [_vp, _vp, _i, _i, _i, _i, _vp, _vp, _vp, _vp]),
    "kvs_permute_rows": (_i, [_vp, _vp, _vp, ctypes.c_longlong, ctypes.c_longlong, _i, _vp]),
    "kvs_mask_meta_export": (_i, [_vp, _i, _vp, _i, _i, _vp, _vp, _vp, _vp]),
    "kvs_attn_fwd": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _f, _vp, _vp, _vp]),
    "kvs_mask_meta_evicted": (_i, [_vp, _vp, _i, _i, _i, _vp, _sz, _vp]),
    "kvs_attn_fwd_dual": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _f, _vp, _vp, _vp, _vp, _vp]),
    "kvs_attn_fwd_packed": (_i, [_vp, _vp, _i, _i, _i, _i, _i, _i, _f, _vp, _vp, _vp]),
    "kvs_attn_bwd_packed": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _f, _i, _vp, _vp, _sz, _vp]),
    "kvs_rope_qk": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _f, _i, _i, _vp, _vp, _vp]),
    "kvs_attn_bwd_workspace_bytes": (_sz, [_i, _i, _i, _i, _i]),
    "kvs_attn_bwd": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _f, _i, _vp, _vp, _vp, _vp, _sz, _vp]),
    "kvs_attn_bwd_ex": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _f, _i, _vp, _vp, _vp, _vp, _sz, _vp,
                             _vp, _vp]),
    "kvs_attn_bwd_noalloc": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _f, _vp, _vp, _vp,
                                  ctypes.POINTER(ctypes.c_void_p), _vp]),
    "kvs_device_status": (_i, [_vp, _vp]),
    "kvs_selftest_bounded_wait": (_i, [_vp, _i, ctypes.c_longlong, _vp]),
    "kvs_cache_free_list_bytes": (_sz, [_i]),
    "kvs_cache_init": (_i, [_vp, _i, _vp]),
    "kvs_cache_append": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "kvs_cache_evict": (_i, [_vp, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp]),
    "kvs_cache_status": (_i, [_vp, ctypes.POINTER(ctypes.c_int), _vp]),
    "kvs_host_chunk_plan": (_i, [_vp, _i, _i, _i, _i, _vp, ctypes.POINTER(ctypes.c_int)]),
    "kvs_decode_num_splits": (_i, [_i, _i, _i]),
    "kvs_decode_workspace_bytes": (_sz, [_i, _i, _i, _i]),
    "kvs_decode_attn": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _i, _f, _i, _vp, _vp, _vp, _sz, _vp]),
    "kvs_host_arena_bytes": (_sz, [_i, _i, _i, _i, _i, _i, _i]),
    "kvs_attn_fwd_bwd_host": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _f, _i,
                                   _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
}

_lib = None


class KvsError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


def load() -> ctypes.CDLL:
    """Loads libkvs.so (built by paper_2609_35750_b200.build).  Raises if absent."""
    global _lib
    if _lib is None:
        path = LIB_PATH
        if not os.path.exists(path):
            raise FileNotFoundError(
                f"{path} not found: build it with `python -m paper_2609_35750_b200.build`; there is no fallback path")
        lib = ctypes.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def strerror(code: int) -> str:
    return load().kvs_strerror(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != KVS_OK:
        raise KvsError(code, where)


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _dev(t: torch.Tensor, name: str, dtype=None) -> int:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (there is no CPU path)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


# ------------------------------------------------------------------------------------------
# same names as the C ABI
# ------------------------------------------------------------------------------------------
def kvs_mask_meta_bytes(batch: int, total_tokens: int, max_seqlen: int) -> int:
    return int(load().kvs_mask_meta_bytes(batch, total_tokens, max_seqlen))


def kvs_evict_at_from_events(events: torch.Tensor, cu_seqlens: torch.Tensor, total_tokens: int,
                             evict_at: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """events int32 [n, 4] rows (trace, when, start, end), cu_seqlens int32 [batch+1] (device).
    Returns evict_at int32 [total_tokens]."""
    if evict_at is None:
        evict_at = torch.empty(total_tokens, dtype=torch.int32, device=cu_seqlens.device)
    n = events.shape[0] if events.numel() else 0
    _check(load().kvs_evict_at_from_events(_dev(events, "events", torch.int32) if n else None, n,
                                           _dev(cu_seqlens, "cu_seqlens", torch.int32), cu_seqlens.numel() - 1, total_tokens,
                                           _dev(evict_at, "evict_at", torch.int32), _stream(stream)), "kvs_evict_at_from_events")
    return evict_at


def kvs_mask_meta(evict_at: torch.Tensor, cu_seqlens: torch.Tensor, max_seqlen: int,
                  meta_buf: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """evict_at int32 [Ttot], cu_seqlens int32 [batch+1] (device).  Returns meta_buf (uint8)."""
    batch = cu_seqlens.numel() - 1
    total = evict_at.numel()
    need = kvs_mask_meta_bytes(batch, total, max_seqlen)
    if meta_buf is None:
        meta_buf = torch.empty(need, dtype=torch.uint8, device=evict_at.device)
    _check(load().kvs_mask_meta(_dev(evict_at, "evict_at", torch.int32), _dev(cu_seqlens, "cu_seqlens", torch.int32),
                                batch, total, max_seqlen, _dev(meta_buf, "meta_buf", torch.uint8),
                                meta_buf.numel(), _stream(stream)), "kvs_mask_meta")
    return meta_buf


def kvs_mask_meta_keys(key_first: torch.Tensor, key_evict: torch.Tensor, cu_seqlens: torch.Tensor, max_seqlen: int,
                       meta_buf: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Metadata for key slots with their own visibility interval [key_first, key_evict) (int32 [Ttot], device)."""
    batch = cu_seqlens.numel() - 1
    total = key_evict.numel()
    if meta_buf is None:
        meta_buf = torch.empty(kvs_mask_meta_bytes(batch, total, max_seqlen), dtype=torch.uint8, device=key_evict.device)
    _check(load().kvs_mask_meta_keys(_dev(key_first, "key_first", torch.int32), _dev(key_evict, "key_evict", torch.int32),
                                     _dev(cu_seqlens, "cu_seqlens", torch.int32), batch, total, max_seqlen,
                                     _dev(meta_buf, "meta_buf", torch.uint8), meta_buf.numel(), _stream(stream)), "kvs_mask_meta_keys")
    return meta_buf


def kvs_reorder_keys(evict_at: torch.Tensor, cu_seqlens: torch.Tensor, max_seqlen: int, window: int, perm=None, key_first=None,
                     key_evict=None, stream=None):
    """Returns (perm, key_first, key_evict), int32 [Ttot] each: the keys of every trace sorted by (evict_at, index)
    within windows of `window` keys."""
    total = evict_at.numel()
    mk = lambda t: t if t is not None else torch.empty(total, dtype=torch.int32, device=evict_at.device)
    perm, key_first, key_evict = mk(perm), mk(key_first), mk(key_evict)
    _check(load().kvs_reorder_keys(_dev(evict_at, "evict_at", torch.int32), _dev(cu_seqlens, "cu_seqlens", torch.int32),
                                   cu_seqlens.numel() - 1, total, max_seqlen, window, _dev(perm, "perm", torch.int32),
                                   _dev(key_first, "key_first", torch.int32), _dev(key_evict, "key_evict", torch.int32),
                                   _stream(stream)), "kvs_reorder_keys")
    return perm, key_first, key_evict


def kvs_permute_rows(src: torch.Tensor, perm: torch.Tensor, dst: Optional[torch.Tensor] = None, inverse: bool = False, stream=None):
    """dst[s] = src[perm[s]] (inverse False) or dst[perm[s]] = src[s] (inverse True) along the leading dimension."""
    if dst is None:
        dst = torch.empty_like(src)
    n = src.shape[0]
    row_bytes = (src.numel() // max(n, 1)) * src.element_size()
    if not src.is_cuda or not src.is_contiguous() or not dst.is_contiguous() or dst.shape != src.shape or dst.dtype != src.dtype:
        raise ValueError("src and dst must be contiguous CUDA tensors of the same shape and dtype")
    _check(load().kvs_permute_rows(src.data_ptr(), _dev(perm, "perm", torch.int32), dst.data_ptr(), n, row_bytes, 1 if inverse else 0,
                                   _stream(stream)), "kvs_permute_rows")
    return dst


def kvs_mask_meta_export(meta_buf: torch.Tensor, cu_seqlens_host, total_tokens: int, max_seqlen: int, stream=None):
    """Returns (tile_class uint8 [sum nb^2], kmin int32 [sum nb], kmax int32 [sum nb]) as numpy arrays."""
    import numpy as np
    cu = np.ascontiguousarray(np.asarray(cu_seqlens_host, dtype=np.int32))
    batch = cu.shape[0] - 1
    nb = (np.diff(cu).astype(np.int64) + TILE - 1) // TILE
    cls = np.zeros(int((nb * nb).sum()), dtype=np.uint8)
    kmin = np.zeros(int(nb.sum()), dtype=np.int32)
    kmax = np.zeros(int(nb.sum()), dtype=np.int32)
    _check(load().kvs_mask_meta_export(_dev(meta_buf, "meta_buf", torch.uint8), batch, cu.ctypes.data, total_tokens, max_seqlen,
                                       cls.ctypes.data, kmin.ctypes.data, kmax.ctypes.data, _stream(stream)),
           "kvs_mask_meta_export")
    return cls, kmin, kmax


def kvs_attn_fwd(q, k, v, meta_buf, batch: int, max_seqlen: int, softmax_scale: float = 0.0,
                 out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None, stream=None):
    """q [Ttot,Hq,d], k, v [Ttot,Hkv,d] bf16 (device).  Returns (out bf16 [Ttot,Hq,d], lse fp32 [Hq,Ttot])."""
    total, Hq, d = q.shape
    Hkv = k.shape[1]
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((Hq, total), dtype=torch.float32, device=q.device)
    _check(load().kvs_attn_fwd(_dev(q, "q", torch.bfloat16), _dev(k, "k", torch.bfloat16), _dev(v, "v", torch.bfloat16),
                               _dev(meta_buf, "meta_buf", torch.uint8), batch, total, max_seqlen, Hq, Hkv, d,
                               float(softmax_scale), _dev(out, "out", torch.bfloat16), _dev(lse, "lse", torch.float32),
                               _stream(stream)), "kvs_attn_fwd")
    return out, lse


def kvs_mask_meta_evicted(key_evict: torch.Tensor, cu_seqlens: torch.Tensor, max_seqlen: int,
                          meta_buf: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Metadata for the keys the eviction mask no longer shows (visible from their eviction step on)."""
    batch = cu_seqlens.numel() - 1
    total = key_evict.numel()
    if meta_buf is None:
        meta_buf = torch.empty(kvs_mask_meta_bytes(batch, total, max_seqlen), dtype=torch.uint8, device=key_evict.device)
    _check(load().kvs_mask_meta_evicted(_dev(key_evict, "key_evict", torch.int32), _dev(cu_seqlens, "cu_seqlens", torch.int32),
                                        batch, total, max_seqlen, _dev(meta_buf, "meta_buf", torch.uint8), meta_buf.numel(),
                                        _stream(stream)), "kvs_mask_meta_evicted")
    return meta_buf


def kvs_attn_fwd_dual(q, k, v, meta_student, meta_evicted, batch: int, max_seqlen: int, softmax_scale: float = 0.0,
                      out_student=None, lse_student=None, out_teacher=None, lse_teacher=None, stream=None):
    """Student (eviction mask) and teacher (every key seen or evicted: the full causal context) forward.
    Returns (out_student, lse_student, out_teacher, lse_teacher)."""
    total, Hq, d = q.shape
    Hkv = k.shape[1]
    if out_student is None:
        out_student = torch.empty_like(q)
    if out_teacher is None:
        out_teacher = torch.empty_like(q)
    if lse_student is None:
        lse_student = torch.empty((Hq, total), dtype=torch.float32, device=q.device)
    if lse_teacher is None:
        lse_teacher = torch.empty((Hq, total), dtype=torch.float32, device=q.device)
    _check(load().kvs_attn_fwd_dual(_dev(q, "q", torch.bfloat16), _dev(k, "k", torch.bfloat16), _dev(v, "v", torch.bfloat16),
                                    _dev(meta_student, "meta_student", torch.uint8), _dev(meta_evicted, "meta_evicted", torch.uint8),
                                    batch, total, max_seqlen, Hq, Hkv, d, float(softmax_scale),
                                    _dev(out_student, "out_student", torch.bfloat16), _dev(lse_student, "lse_student", torch.float32),
                                    _dev(out_teacher, "out_teacher", torch.bfloat16), _dev(lse_teacher, "lse_teacher", torch.float32),
                                    _stream(stream)), "kvs_attn_fwd_dual")
    return out_student, lse_student, out_teacher, lse_teacher


def kvs_attn_fwd_packed(qkv, meta_buf, batch: int, max_seqlen: int, Hq: int, Hkv: int, softmax_scale: float = 0.0,
                        out=None, lse=None, stream=None):
    """qkv bf16 [Ttot, Hq + 2 Hkv, d] (q heads, k heads, v heads).  Returns (out [Ttot,Hq,d], lse [Hq,Ttot])."""
    total, H, d = qkv.shape
    if H != Hq + 2 * Hkv:
        raise ValueError("qkv must have Hq + 2 Hkv heads")
    if out is None:
        out = torch.empty((total, Hq, d), dtype=torch.bfloat16, device=qkv.device)
    if lse is None:
        lse = torch.empty((Hq, total), dtype=torch.float32, device=qkv.device)
    _check(load().kvs_attn_fwd_packed(_dev(qkv, "qkv", torch.bfloat16), _dev(meta_buf, "meta_buf", torch.uint8), batch, total,
                                      max_seqlen, Hq, Hkv, d, float(softmax_scale), _dev(out, "out", torch.bfloat16),
                                      _dev(lse, "lse", torch.float32), _stream(stream)), "kvs_attn_fwd_packed")
    return out, lse


def kvs_attn_bwd_packed(dout, qkv, out, lse, meta_buf, batch: int, max_seqlen: int, Hq: int, Hkv: int, softmax_scale: float = 0.0,
                        grad_dtype: int = GRAD_FP32, dqkv=None, workspace=None, stream=None):
    """Returns dqkv [Ttot, Hq + 2 Hkv, d] (bf16 or fp32): dq, dk, dv in the head order of qkv."""
    total, H, d = qkv.shape
    gdt = torch.float32 if grad_dtype == GRAD_FP32 else torch.bfloat16
    if dqkv is None:
        dqkv = torch.empty(qkv.shape, dtype=gdt, device=qkv.device)
    if workspace is None:
        workspace = torch.empty(kvs_attn_bwd_workspace_bytes(total, Hq, Hkv, d, grad_dtype), dtype=torch.uint8, device=qkv.device)
    _check(load().kvs_attn_bwd_packed(_dev(dout, "dout", torch.bfloat16), _dev(qkv, "qkv", torch.bfloat16),
                                      _dev(out, "out", torch.bfloat16), _dev(lse, "lse", torch.float32),
                                      _dev(meta_buf, "meta_buf", torch.uint8), batch, total, max_seqlen, Hq, Hkv, d,
                                      float(softmax_scale), grad_dtype, _dev(dqkv, "dqkv", gdt),
                                      _dev(workspace, "workspace", torch.uint8), workspace.numel(), _stream(stream)),
           "kvs_attn_bwd_packed")
    return dqkv


def kvs_rope_qk(q, k, cu_seqlens=None, positions=None, theta_base: float = 10000.0, inverse: bool = False, q_out=None, k_out=None,
                stream=None):
    """Rotary embedding of q and/or k (bf16 or fp32, [Ttot, H, d]); inverse=True applies the transposed rotation (for
    gradients).  positions int32 [Ttot] or None for the trace-local index (cu_seqlens then required).  Returns (q_out, k_out)."""
    ref = q if q is not None else k
    total, _, d = ref.shape
    dt = GRAD_FP32 if ref.dtype == torch.float32 else GRAD_BF16
    if q is not None and q_out is None:
        q_out = torch.empty_like(q)
    if k is not None and k_out is None:
        k_out = torch.empty_like(k)
    ptr = lambda t, n: _dev(t, n, ref.dtype) if t is not None else None
    _check(load().kvs_rope_qk(ptr(q, "q"), ptr(k, "k"), _dev(positions, "positions", torch.int32) if positions is not None else None,
                              _dev(cu_seqlens, "cu_seqlens", torch.int32) if cu_seqlens is not None else None,
                              (cu_seqlens.numel() - 1) if cu_seqlens is not None else 0, total,
                              q.shape[1] if q is not None else 0, k.shape[1] if k is not None else 0, d, float(theta_base), dt,
                              1 if inverse else 0, ptr(q_out, "q_out"), ptr(k_out, "k_out"), _stream(stream)), "kvs_rope_qk")
    return q_out, k_out


def kvs_host_chunk_plan(cu_seqlens, max_seqlen: int, Hkv: int):
    """The trace ranges kvs_attn_fwd_bwd_host cuts a batch into: a list of (first trace, one past the last).
    cu_seqlens: int32 numpy array or CPU tensor [batch + 1].  Host only."""
    import numpy as np
    cu = np.ascontiguousarray(np.asarray(cu_seqlens), dtype=np.int32)
    batch = int(cu.shape[0]) - 1
    buf = np.zeros(max(2 * batch, 2), dtype=np.int32)
    n = ctypes.c_int(0)
    _check(load().kvs_host_chunk_plan(cu.ctypes.data, batch, int(cu[-1]) if batch >= 0 else 0, int(max_seqlen), int(Hkv), buf.ctypes.data,
                                      ctypes.byref(n)), "kvs_host_chunk_plan")
    return [(int(buf[2 * i]), int(buf[2 * i + 1])) for i in range(n.value)]


def kvs_attn_bwd_workspace_bytes(total_tokens: int, Hq: int, Hkv: int, head_dim: int, grad_dtype: int) -> int:
    return int(load().kvs_attn_bwd_workspace_bytes(total_tokens, Hq, Hkv, head_dim, grad_dtype))


def kvs_attn_bwd(dout, q, k, v, out, lse, meta_buf, batch: int, max_seqlen: int, softmax_scale: float = 0.0,
                 grad_dtype: int = GRAD_FP32, dq=None, dk=None, dv=None, workspace=None, stream=None,
                 main_events: Optional[Tuple[torch.cuda.Event, torch.cuda.Event]] = None):
    """Returns (dq, dk, dv) in bf16 or fp32 according to grad_dtype.  main_events: two timing
    events (already recorded once, so that their handles exist) to be recorded around the
    main kernel; this routes through kvs_attn_bwd_ex."""
    total, Hq, d = q.shape
    Hkv = k.shape[1]
    gdt = torch.float32 if grad_dtype == GRAD_FP32 else torch.bfloat16
    if dq is None:
        dq = torch.empty(q.shape, dtype=gdt, device=q.device)
    if dk is None:
        dk = torch.empty(k.shape, dtype=gdt, device=q.device)
    if dv is None:
        dv = torch.empty(v.shape, dtype=gdt, device=q.device)
    need = kvs_attn_bwd_workspace_bytes(total, Hq, Hkv, d, grad_dtype)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    args = (_dev(dout, "dout", torch.bfloat16), _dev(q, "q", torch.bfloat16), _dev(k, "k", torch.bfloat16),
            _dev(v, "v", torch.bfloat16), _dev(out, "out", torch.bfloat16), _dev(lse, "lse", torch.float32),
            _dev(meta_buf, "meta_buf", torch.uint8), batch, total, max_seqlen, Hq, Hkv, d,
            float(softmax_scale), grad_dtype, _dev(dq, "dq", gdt), _dev(dk, "dk", gdt), _dev(dv, "dv", gdt),
            _dev(workspace, "workspace", torch.uint8), workspace.numel(), _stream(stream))
    if main_events is None:
        _check(load().kvs_attn_bwd(*args), "kvs_attn_bwd")
    else:
        e0, e1 = (int(e.cuda_event) for e in main_events)
        if not e0 or not e1:
            raise ValueError("main_events must have been recorded once before the call")
        _check(load().kvs_attn_bwd_ex(*args, e0, e1), "kvs_attn_bwd_ex")
    return dq, dk, dv


NOALLOC_MAX_ROWS = 1 << 20


def kvs_attn_bwd_noalloc(dout, q, k, v, out, lse, meta_buf, batch: int, max_seqlen: int, softmax_scale: float = 0.0,
                         dq=None, dk=None, dv=None, stream=None):
    """Backward for callers that must not allocate device memory at call time: the scratch is a
    fixed array inside the library (fp32 gradients only, total_tokens * Hq <= NOALLOC_MAX_ROWS).
    Pass dq, dk, dv to keep this wrapper from allocating too.  Returns (dq, dk, dv, scratch_address);
    the address can be given to kvs_device_status_ptr()."""
    total, Hq, d = q.shape
    Hkv = k.shape[1]
    if dq is None:
        dq = torch.empty(q.shape, dtype=torch.float32, device=q.device)
    if dk is None:
        dk = torch.empty(k.shape, dtype=torch.float32, device=q.device)
    if dv is None:
        dv = torch.empty(v.shape, dtype=torch.float32, device=q.device)
    scratch = ctypes.c_void_p(0)
    _check(load().kvs_attn_bwd_noalloc(_dev(dout, "dout", torch.bfloat16), _dev(q, "q", torch.bfloat16),
                                       _dev(k, "k", torch.bfloat16), _dev(v, "v", torch.bfloat16),
                                       _dev(out, "out", torch.bfloat16), _dev(lse, "lse", torch.float32),
                                       _dev(meta_buf, "meta_buf", torch.uint8), batch, total, max_seqlen, Hq, Hkv, d,
                                       float(softmax_scale), _dev(dq, "dq", torch.float32), _dev(dk, "dk", torch.float32),
                                       _dev(dv, "dv", torch.float32), ctypes.byref(scratch), _stream(stream)),
           "kvs_attn_bwd_noalloc")
    return dq, dk, dv, int(scratch.value or 0)


def kvs_device_status_ptr(device_address: int, stream=None) -> int:
    """kvs_device_status on a raw device address (e.g. the scratch of kvs_attn_bwd_noalloc)."""
    return int(load().kvs_device_status(device_address, _stream(stream)))


def kvs_device_status(buf: torch.Tensor, stream=None) -> int:
    return int(load().kvs_device_status(_dev(buf, "buf", torch.uint8), _stream(stream)))


def kvs_selftest_bounded_wait(expected_arrivals: int, limit_clocks: int, stream=None) -> int:
    """Runs the bounded-wait self-test and returns the status word (KVS_OK or KVS_ERR_TIMEOUT)."""
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(load().kvs_selftest_bounded_wait(word.data_ptr(), expected_arrivals, limit_clocks, _stream(stream)),
           "kvs_selftest_bounded_wait")
    return int(word.item())


def kvs_host_arena_bytes(batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, grad_dtype) -> int:
    return int(load().kvs_host_arena_bytes(batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, grad_dtype))


def kvs_attn_fwd_bwd_host(evict_at, cu_seqlens, q, k, v, dout, max_seqlen: int, softmax_scale: float,
                          grad_dtype: int, out, lse, dq, dk, dv, arena: torch.Tensor, stream=None) -> None:
    """All tensors except `arena` are HOST tensors (pinned for asynchronous copies); results
    are written into out, lse, dq, dk, dv.  Synchronises the stream."""
    for name, t in (("evict_at", evict_at), ("cu_seqlens", cu_seqlens), ("q", q), ("k", k), ("v", v), ("dout", dout),
                    ("out", out), ("lse", lse), ("dq", dq), ("dk", dk), ("dv", dv)):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous host tensor")
    total, Hq, d = q.shape
    Hkv = k.shape[1]
    batch = cu_seqlens.numel() - 1
    _check(load().kvs_attn_fwd_bwd_host(evict_at.data_ptr(), cu_seqlens.data_ptr(), q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                        dout.data_ptr(), batch, total, max_seqlen, Hq, Hkv, d, float(softmax_scale), grad_dtype,
                                        out.data_ptr(), lse.data_ptr(), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(),
                                        _dev(arena, "arena", torch.uint8), arena.numel(), _stream(stream)),
           "kvs_attn_fwd_bwd_host")


# ------------------------------------------------------------------------------------------
# rollout side: paged KV cache with physical eviction, decode attention
# ------------------------------------------------------------------------------------------
class PagedCache:
    """Device buffers of a paged KV cache plus the calls that maintain it.  Holds no logic:
    every operation is one call into the library."""

    def __init__(self, num_pages: int, page_size: int, num_seqs: int, max_pages: int, Hkv: int, head_dim: int, device="cuda"):
        self.num_pages, self.page_size, self.num_seqs, self.max_pages = num_pages, page_size, num_seqs, max_pages
        self.Hkv, self.d = Hkv, head_dim
        self.k_cache = torch.zeros((num_pages, page_size, Hkv, head_dim), dtype=torch.bfloat16, device=device)
        self.v_cache = torch.zeros_like(self.k_cache)
        self.block_table = torch.zeros((num_seqs, max_pages), dtype=torch.int32, device=device)
        self.n_tokens = torch.zeros(num_seqs, dtype=torch.int32, device=device)
        self.free_list = torch.zeros(int(load().kvs_cache_free_list_bytes(num_pages)) // 4, dtype=torch.int32, device=device)
        _check(load().kvs_cache_init(self.free_list.data_ptr(), num_pages, _stream(None)), "kvs_cache_init")

    def append(self, k_new: torch.Tensor, v_new: torch.Tensor, active: Optional[torch.Tensor] = None, stream=None) -> None:
        _check(load().kvs_cache_append(_dev(k_new, "k_new", torch.bfloat16), _dev(v_new, "v_new", torch.bfloat16),
                                       _dev(active, "active", torch.uint8) if active is not None else None,
                                       self.num_seqs, self.Hkv, self.d, self.page_size, self.max_pages, self.num_pages,
                                       self.block_table.data_ptr(), self.n_tokens.data_ptr(), self.free_list.data_ptr(),
                                       self.k_cache.data_ptr(), self.v_cache.data_ptr(), _stream(stream)), "kvs_cache_append")

    def evict(self, ranges: torch.Tensor, stream=None) -> None:
        """ranges int32 [n, 3] rows (sequence, first_page_slot, n_pages) (device)."""
        n = ranges.shape[0] if ranges.numel() else 0
        _check(load().kvs_cache_evict(_dev(ranges, "ranges", torch.int32) if n else None, n, self.num_seqs, self.page_size,
                                      self.max_pages, self.num_pages, self.block_table.data_ptr(), self.n_tokens.data_ptr(),
                                      self.free_list.data_ptr(), _stream(stream)), "kvs_cache_evict")

    def status(self, stream=None) -> Tuple[int, int]:
        """(status code, free pages).  Synchronises."""
        free = ctypes.c_int(0)
        rc = int(load().kvs_cache_status(self.free_list.data_ptr(), ctypes.byref(free), _stream(stream)))
        return rc, int(free.value)

    def decode(self, q: torch.Tensor, softmax_scale: float = 0.0, num_splits: int = 0, out=None, lse=None, workspace=None,
               max_tokens: Optional[int] = None, stream=None):
        """q bf16 [num_seqs, Hq, d] -> (out bf16 [num_seqs, Hq, d], lse fp32 [num_seqs, Hq])."""
        S, Hq, d = q.shape
        if num_splits <= 0:
            num_splits = int(load().kvs_decode_num_splits(S, self.Hkv, max_tokens or self.max_pages * self.page_size))
        need = int(load().kvs_decode_workspace_bytes(S, Hq, d, num_splits))
        if workspace is None:
            workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
        if out is None:
            out = torch.empty_like(q)
        if lse is None:
            lse = torch.empty((S, Hq), dtype=torch.float32, device=q.device)
        _check(load().kvs_decode_attn(_dev(q, "q", torch.bfloat16), self.k_cache.data_ptr(), self.v_cache.data_ptr(),
                                      self.block_table.data_ptr(), self.n_tokens.data_ptr(), S, Hq, self.Hkv, d, self.page_size,
                                      self.max_pages, self.num_pages, float(softmax_scale), num_splits, _dev(out, "out", torch.bfloat16),
                                      _dev(lse, "lse", torch.float32), _dev(workspace, "workspace", torch.uint8),
                                      workspace.numel(), _stream(stream)), "kvs_decode_attn")
        return out, lse
