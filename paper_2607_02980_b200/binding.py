"""ctypes binding of libhils.so -- argument marshalling only.

Every step of the operator runs in the CUDA kernels of the library; this module checks tensor
types, builds the parameter struct, provides the workspace from torch's allocator and passes raw
device pointers and the current CUDA stream through the C ABI declared in include/hils.h.
There is no CPU or PyTorch fallback: if the shared library is missing, every call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhils.so")

HILS_F32, HILS_BF16 = 0, 1
IMPL_AUTO, IMPL_GENERIC, IMPL_FAST, IMPL_PACKED = 0, 1, 2, 3
_IMPL = {"auto": IMPL_AUTO, "generic": IMPL_GENERIC, "fast": IMPL_FAST, "packed": IMPL_PACKED}

EXPORTS = [
    "hils_workspace_bytes", "hils_prefill", "hils_decode", "hils_host_arena_bytes",
    "hils_prefill_host", "hils_decode_host", "hils_poll_status", "hils_last_launch_count",
    "hils_status_string", "hils_version", "hils_trace_enable", "hils_trace_read", "hils_decode_noalloc",
    "hils_landmark_summary", "hils_decode_paged", "hils_prefill_at", "hils_prefill_at_workspace_bytes",
    "hils_prefill_routed", "hils_decode_routed", "hils_chunk_overlap", "hils_prefill_backward",
    "hils_prefill_backward_workspace_bytes", "hils_decode_multi", "hils_decode_multi_workspace_bytes",
]


class HilsParams(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("Hl", ctypes.c_int32),
                ("L", ctypes.c_int32), ("T_max", ctypes.c_int32), ("C", ctypes.c_int32), ("d", ctypes.c_int32),
                ("chunk_size", ctypes.c_int32), ("top_k", ctypes.c_int32), ("window", ctypes.c_int32),
                ("scale", ctypes.c_float), ("dtype", ctypes.c_int32), ("impl", ctypes.c_int32)]


class HilsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (%d)" % (where, status_string(status), status))


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libhils.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "HiLS CUDA library not built: %s is missing. Run `python -m paper_2607_02980_b200.build` "
            "(there is no CPU fallback)." % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32p, f32p = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
    pp = ctypes.POINTER(HilsParams)
    lib.hils_workspace_bytes.restype = ctypes.c_size_t
    lib.hils_workspace_bytes.argtypes = [pp, ctypes.c_int]
    lib.hils_host_arena_bytes.restype = ctypes.c_size_t
    lib.hils_host_arena_bytes.argtypes = [pp, ctypes.c_int]
    lib.hils_prefill.restype = ctypes.c_int
    lib.hils_prefill.argtypes = [pp, vp, vp, vp, vp, f32p, vp, f32p, i32p, vp, ctypes.c_size_t, vp]
    lib.hils_decode.restype = ctypes.c_int
    lib.hils_decode.argtypes = [pp, vp, vp, vp, vp, f32p, i32p, vp, f32p, i32p, vp, ctypes.c_size_t, vp]
    lib.hils_prefill_host.restype = ctypes.c_int
    lib.hils_prefill_host.argtypes = [pp, vp, vp, vp, vp, f32p, vp, f32p, i32p, vp, ctypes.c_size_t, vp]
    lib.hils_decode_host.restype = ctypes.c_int
    lib.hils_decode_host.argtypes = [pp, vp, vp, vp, vp, f32p, i32p, vp, f32p, i32p, vp, ctypes.c_size_t, vp]
    lib.hils_decode_noalloc.restype = ctypes.c_int
    lib.hils_decode_noalloc.argtypes = [pp, vp, vp, vp, vp, f32p, i32p, vp, f32p, i32p, i32p, vp]
    lib.hils_prefill_routed.restype = ctypes.c_int
    lib.hils_prefill_routed.argtypes = [pp, vp, vp, vp, vp, vp, f32p, vp, f32p, i32p, vp, ctypes.c_size_t, vp]
    lib.hils_decode_routed.restype = ctypes.c_int
    lib.hils_decode_routed.argtypes = [pp, vp, vp, vp, vp, vp, f32p, i32p, vp, f32p, i32p, vp, ctypes.c_size_t, vp]
    lib.hils_prefill_at.restype = ctypes.c_int
    lib.hils_prefill_at.argtypes = [pp, vp, vp, vp, vp, f32p, ctypes.c_int64, vp, f32p, i32p, vp, ctypes.c_size_t, vp]
    lib.hils_prefill_at_workspace_bytes.restype = ctypes.c_size_t
    lib.hils_prefill_at_workspace_bytes.argtypes = [pp, ctypes.c_int64]
    lib.hils_decode_paged.restype = ctypes.c_int
    lib.hils_decode_paged.argtypes = [pp, vp, vp, vp, vp, f32p, i32p, ctypes.c_int32, i32p, vp, f32p, i32p, vp,
                                      ctypes.c_size_t, vp]
    lib.hils_landmark_summary.restype = ctypes.c_int
    lib.hils_landmark_summary.argtypes = [pp, vp, vp, i32p, ctypes.c_int32, ctypes.c_int32, vp, f32p, vp]
    lib.hils_prefill_backward_workspace_bytes.restype = ctypes.c_size_t
    lib.hils_prefill_backward_workspace_bytes.argtypes = [pp]
    lib.hils_prefill_backward.restype = ctypes.c_int
    lib.hils_prefill_backward.argtypes = [pp, vp, vp, vp, vp, f32p, vp, f32p, i32p, vp, f32p, f32p, f32p, f32p, f32p,
                                          vp, ctypes.c_size_t, vp]
    lib.hils_decode_multi_workspace_bytes.restype = ctypes.c_size_t
    lib.hils_decode_multi_workspace_bytes.argtypes = [pp, ctypes.c_int32]
    lib.hils_decode_multi.restype = ctypes.c_int
    lib.hils_decode_multi.argtypes = [pp, ctypes.c_int32, vp, vp, vp, vp, f32p, i32p, ctypes.c_int32, i32p, vp, f32p,
                                      i32p, vp, ctypes.c_size_t, vp]
    lib.hils_chunk_overlap.restype = ctypes.c_int
    lib.hils_chunk_overlap.argtypes = [pp, i32p, ctypes.c_int32, i32p, f32p, vp]
    lib.hils_poll_status.restype = ctypes.c_int
    lib.hils_poll_status.argtypes = [vp, vp]
    lib.hils_last_launch_count.restype = ctypes.c_int
    lib.hils_status_string.restype = ctypes.c_char_p
    lib.hils_status_string.argtypes = [ctypes.c_int]
    lib.hils_version.restype = ctypes.c_char_p
    lib.hils_trace_enable.restype = ctypes.c_int
    lib.hils_trace_enable.argtypes = [ctypes.c_int]
    lib.hils_trace_read.restype = ctypes.c_int
    lib.hils_trace_read.argtypes = [ctypes.c_char_p, ctypes.c_size_t, ctypes.POINTER(ctypes.c_float), ctypes.c_int]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().hils_status_string(int(status)).decode()


def version() -> str:
    return load_library().hils_version().decode()


def last_launch_count() -> int:
    return int(load_library().hils_last_launch_count())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return HILS_F32
    if t.dtype == torch.bfloat16:
        return HILS_BF16
    raise TypeError("HiLS supports float32 and bfloat16 tensors, got %s" % t.dtype)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _check(t: torch.Tensor, name: str, shape: Tuple[int, ...], dtype, cuda: bool):
    if tuple(t.shape) != tuple(shape):
        raise ValueError("%s has shape %s, expected %s" % (name, tuple(t.shape), tuple(shape)))
    if t.dtype != dtype:
        raise TypeError("%s has dtype %s, expected %s" % (name, t.dtype, dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    if cuda != t.is_cuda:
        raise ValueError("%s must live on %s" % (name, "a CUDA device" if cuda else "the host"))


def make_params(*, B, Hq, Hkv, Hl, L, T_max, C, d, chunk_size, top_k, window=1, scale=0.0, dtype, impl="auto"):
    return HilsParams(B, Hq, Hkv, Hl, L, T_max, C, d, chunk_size, top_k, window, float(scale), dtype, _IMPL[impl])


def workspace_bytes(params: HilsParams, is_decode: bool) -> int:
    return int(load_library().hils_workspace_bytes(ctypes.byref(params), 1 if is_decode else 0))


def host_arena_bytes(params: HilsParams, is_decode: bool) -> int:
    return int(load_library().hils_host_arena_bytes(ctypes.byref(params), 1 if is_decode else 0))


def alloc_workspace(params: HilsParams, is_decode: bool, device) -> torch.Tensor:
    n = workspace_bytes(params, is_decode)
    if n == 0:
        raise HilsError(-2, "hils_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    ws[:256].zero_()
    return ws


def _stream_ptr(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def hils_prefill(q, k, v, landmarks, chunk_size: int, top_k: int, out=None, lse=None, sel_idx=None, stream=None, *,
                 bias=None, window: int = 1, scale: float = 0.0, impl: str = "auto", workspace=None, q_route=None):
    """HiLS prefill on CUDA tensors: q [B,Hq,L,d], k,v [B,Hkv,L,d], landmarks [B,Hl,C,d].
    q_route (optional, shape of q): the routing query of Eq. (Q-Cal), used for the surrogate scores only.

    Returns (out [B,Hq,L,d], lse [B,Hq,L] fp32, sel_idx [B,Hkv,L,K] int32).  Asynchronous on the
    given (default: current) CUDA stream.
    """
    lib = load_library()
    B, Hq, L, d = q.shape
    Hkv, T = k.shape[1], k.shape[2]
    Hl, C = landmarks.shape[1], landmarks.shape[2]
    dt = q.dtype
    _check(q, "q", (B, Hq, L, d), dt, True)
    _check(k, "k", (B, Hkv, T, d), dt, True)
    _check(v, "v", (B, Hkv, T, d), dt, True)
    _check(landmarks, "landmarks", (B, Hl, C, d), dt, True)
    if bias is not None:
        _check(bias, "bias", (B, Hl, C), torch.float32, True)
    out = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Hq, L), dtype=torch.float32, device=q.device) if lse is None else lse
    sel_idx = torch.empty((B, Hkv, L, top_k), dtype=torch.int32, device=q.device) if sel_idx is None else sel_idx
    _check(out, "out", (B, Hq, L, d), dt, True)
    _check(lse, "lse", (B, Hq, L), torch.float32, True)
    _check(sel_idx, "sel_idx", (B, Hkv, L, top_k), torch.int32, True)
    p = make_params(B=B, Hq=Hq, Hkv=Hkv, Hl=Hl, L=L, T_max=T, C=C, d=d, chunk_size=chunk_size, top_k=top_k,
                    window=window, scale=scale, dtype=_dtype_code(q), impl=impl)
    ws = alloc_workspace(p, False, q.device) if workspace is None else workspace
    if q_route is not None:
        _check(q_route, "q_route", (B, Hq, L, d), dt, True)
        rc = lib.hils_prefill_routed(ctypes.byref(p), _ptr(q), _ptr(q_route), _ptr(k), _ptr(v), _ptr(landmarks),
                                     _ptr(bias), _ptr(out), _ptr(lse), _ptr(sel_idx), _ptr(ws), ws.numel(),
                                     _stream_ptr(stream))
    else:
        rc = lib.hils_prefill(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(landmarks), _ptr(bias), _ptr(out),
                              _ptr(lse), _ptr(sel_idx), _ptr(ws), ws.numel(), _stream_ptr(stream))
    if rc != 0:
        raise HilsError(rc, "hils_prefill")
    return out, lse, sel_idx


def hils_decode(q, k_cache, v_cache, landmarks, seq_lens, chunk_size: int, top_k: int, out=None, lse=None,
                sel_idx=None, stream=None, *, bias=None, window: int = 1, scale: float = 0.0, impl: str = "auto",
                workspace=None, q_route=None):
    """HiLS single-token decode: q [B,Hq,d], caches [B,Hkv,T_max,d], seq_lens [B] int32 (CUDA).

    Returns (out [B,Hq,d], lse [B,Hq], sel_idx [B,Hkv,K])."""
    lib = load_library()
    B, Hq, d = q.shape
    Hkv, T = k_cache.shape[1], k_cache.shape[2]
    Hl, C = landmarks.shape[1], landmarks.shape[2]
    dt = q.dtype
    _check(q, "q", (B, Hq, d), dt, True)
    _check(k_cache, "k_cache", (B, Hkv, T, d), dt, True)
    _check(v_cache, "v_cache", (B, Hkv, T, d), dt, True)
    _check(landmarks, "landmarks", (B, Hl, C, d), dt, True)
    _check(seq_lens, "seq_lens", (B,), torch.int32, True)
    if bias is not None:
        _check(bias, "bias", (B, Hl, C), torch.float32, True)
    out = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, Hq), dtype=torch.float32, device=q.device) if lse is None else lse
    sel_idx = torch.empty((B, Hkv, top_k), dtype=torch.int32, device=q.device) if sel_idx is None else sel_idx
    _check(out, "out", (B, Hq, d), dt, True)
    _check(lse, "lse", (B, Hq), torch.float32, True)
    _check(sel_idx, "sel_idx", (B, Hkv, top_k), torch.int32, True)
    p = make_params(B=B, Hq=Hq, Hkv=Hkv, Hl=Hl, L=0, T_max=T, C=C, d=d, chunk_size=chunk_size, top_k=top_k,
                    window=window, scale=scale, dtype=_dtype_code(q), impl=impl)
    ws = alloc_workspace(p, True, q.device) if workspace is None else workspace
    if q_route is not None:
        _check(q_route, "q_route", tuple(q.shape), q.dtype, True)
        rc = lib.hils_decode_routed(ctypes.byref(p), _ptr(q), _ptr(q_route), _ptr(k_cache), _ptr(v_cache), _ptr(landmarks),
                                    _ptr(bias), _ptr(seq_lens), _ptr(out), _ptr(lse), _ptr(sel_idx), _ptr(ws), ws.numel(),
                                    _stream_ptr(stream))
    else:
        rc = lib.hils_decode(ctypes.byref(p), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(landmarks), _ptr(bias),
                             _ptr(seq_lens), _ptr(out), _ptr(lse), _ptr(sel_idx), _ptr(ws), ws.numel(),
                             _stream_ptr(stream))
    if rc != 0:
        raise HilsError(rc, "hils_decode")
    return out, lse, sel_idx


def hils_decode_noalloc(q, k_cache, v_cache, landmarks, seq_lens, chunk_size: int, top_k: int, out, lse, sel_idx,
                        stream=None, *, bias=None, scale: float = 0.0, device_status=None):
    """hils_decode without a workspace: the library's own fixed device array holds the scratch.

    For embedders that cannot allocate device memory (all HBM already given to a KV-cache pool, no
    allocator handle, or a loop that must not call cudaMalloc).  Every output tensor has to be
    passed in; this wrapper allocates nothing either.  Calls share one scratch array, so calls whose
    kernels could overlap on the GPU must be serialised by the caller.  `device_status` is an optional
    int32 CUDA tensor of one element that receives the device status word (0 = ok).
    """
    lib = load_library()
    B, Hq, d = q.shape
    Hkv, T = k_cache.shape[1], k_cache.shape[2]
    Hl, C = landmarks.shape[1], landmarks.shape[2]
    dt = q.dtype
    _check(q, "q", (B, Hq, d), dt, True)
    _check(k_cache, "k_cache", (B, Hkv, T, d), dt, True)
    _check(v_cache, "v_cache", (B, Hkv, T, d), dt, True)
    _check(landmarks, "landmarks", (B, Hl, C, d), dt, True)
    _check(seq_lens, "seq_lens", (B,), torch.int32, True)
    if bias is not None:
        _check(bias, "bias", (B, Hl, C), torch.float32, True)
    _check(out, "out", (B, Hq, d), dt, True)
    _check(lse, "lse", (B, Hq), torch.float32, True)
    _check(sel_idx, "sel_idx", (B, Hkv, top_k), torch.int32, True)
    if device_status is not None:
        _check(device_status, "device_status", (1,), torch.int32, True)
    p = make_params(B=B, Hq=Hq, Hkv=Hkv, Hl=Hl, L=0, T_max=T, C=C, d=d, chunk_size=chunk_size, top_k=top_k,
                    window=1, scale=scale, dtype=_dtype_code(q), impl="auto")
    rc = lib.hils_decode_noalloc(ctypes.byref(p), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(landmarks),
                                 _ptr(bias), _ptr(seq_lens), _ptr(out), _ptr(lse), _ptr(sel_idx),
                                 _ptr(device_status), _stream_ptr(stream))
    if rc != 0:
        raise HilsError(rc, "hils_decode_noalloc")
    return out, lse, sel_idx


def hils_prefill_at(q, k, v, landmarks, chunk_size: int, top_k: int, pos0: int, stream=None, *, bias=None,
                    window: int = 1, scale: float = 0.0, impl: str = "auto", out=None, lse=None, sel_idx=None,
                    workspace=None):
    """hils_prefill for the L query tokens at positions pos0 .. pos0 + L - 1 of sequences whose caches k, v
    [B,Hkv,T,d] hold at least pos0 + L tokens (chunked prefill / multi-token decode).  Returns (out, lse, sel_idx)."""
    lib = load_library()
    B, Hq, L, d = q.shape
    Hkv, T = k.shape[1], k.shape[2]
    Hl, C = landmarks.shape[1], landmarks.shape[2]
    dt = q.dtype
    _check(q, "q", (B, Hq, L, d), dt, True)
    _check(k, "k", (B, Hkv, T, d), dt, True)
    _check(v, "v", (B, Hkv, T, d), dt, True)
    _check(landmarks, "landmarks", (B, Hl, C, d), dt, True)
    if bias is not None:
        _check(bias, "bias", (B, Hl, C), torch.float32, True)
    p = make_params(B=B, Hq=Hq, Hkv=Hkv, Hl=Hl, L=L, T_max=T, C=C, d=d, chunk_size=chunk_size, top_k=top_k,
                    window=window, scale=scale, dtype=_dtype_code(q), impl=impl)
    nbytes = int(lib.hils_prefill_at_workspace_bytes(ctypes.byref(p), int(pos0)))
    if nbytes == 0:
        raise HilsError(-2, "hils_prefill_at_workspace_bytes")
    if workspace is None:
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
        workspace[:256].zero_()                   # only the status block has to start at zero
    ws = workspace
    out = torch.empty((B, Hq, L, d), dtype=dt, device=q.device) if out is None else out
    lse = torch.empty((B, Hq, L), dtype=torch.float32, device=q.device) if lse is None else lse
    sel_idx = torch.empty((B, Hkv, L, top_k), dtype=torch.int32, device=q.device) if sel_idx is None else sel_idx
    rc = lib.hils_prefill_at(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(landmarks), _ptr(bias), int(pos0),
                             _ptr(out), _ptr(lse), _ptr(sel_idx), _ptr(ws), nbytes, _stream_ptr(stream))
    if rc != 0:
        raise HilsError(rc, "hils_prefill_at")
    return out, lse, sel_idx


def hils_decode_paged(q, k_pages, v_pages, landmarks, block_table, seq_lens, chunk_size: int, top_k: int, stream=None, *,
                      bias=None, window: int = 1, scale: float = 0.0, out=None, lse=None, sel_idx=None, workspace=None):
    """hils_decode over paged caches with page = chunk: k_pages, v_pages [num_pages, Hkv, S, d], block_table [B, C]
    int32 (page of every logical chunk); landmarks / bias stay logical.  Returns (out, lse, sel_idx)."""
    lib = load_library()
    B, Hq, d = q.shape
    P, Hkv, S, _ = k_pages.shape
    Hl, C = landmarks.shape[1], landmarks.shape[2]
    dt = q.dtype
    _check(q, "q", (B, Hq, d), dt, True)
    _check(k_pages, "k_pages", (P, Hkv, chunk_size, d), dt, True)
    _check(v_pages, "v_pages", (P, Hkv, chunk_size, d), dt, True)
    _check(landmarks, "landmarks", (B, Hl, C, d), dt, True)
    _check(block_table, "block_table", (B, C), torch.int32, True)
    _check(seq_lens, "seq_lens", (B,), torch.int32, True)
    if bias is not None:
        _check(bias, "bias", (B, Hl, C), torch.float32, True)
    p = make_params(B=B, Hq=Hq, Hkv=Hkv, Hl=Hl, L=0, T_max=C * chunk_size, C=C, d=d, chunk_size=chunk_size,
                    top_k=top_k, window=window, scale=scale, dtype=_dtype_code(q), impl="auto")
    ws = alloc_workspace(p, True, q.device) if workspace is None else workspace
    out = torch.empty((B, Hq, d), dtype=dt, device=q.device) if out is None else out
    lse = torch.empty((B, Hq), dtype=torch.float32, device=q.device) if lse is None else lse
    sel_idx = torch.empty((B, Hkv, top_k), dtype=torch.int32, device=q.device) if sel_idx is None else sel_idx
    rc = lib.hils_decode_paged(ctypes.byref(p), _ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(landmarks), _ptr(bias),
                               _ptr(block_table), int(P), _ptr(seq_lens), _ptr(out), _ptr(lse), _ptr(sel_idx),
                               _ptr(ws), ws.numel() * ws.element_size(), _stream_ptr(stream))
    if rc != 0:
        raise HilsError(rc, "hils_decode_paged")
    return out, lse, sel_idx


def hils_landmark_summary(landmark_queries, k, chunk_size: int, *, seq_lens=None, scale: float = 0.0,
                          chunk_begin: int = 0, chunk_count: int = 0, landmarks=None, bias=None, stream=None):
    """Chunk summaries of Proposition 3.1: landmarks k'_c = Attn(q'_c, K_c, K_c) and bias b'_c = entropy.

    landmark_queries [B,Hl,C,d] and k [B,Hkv,T,d] are CUDA tensors of one dtype; seq_lens [B] int32 or None.
    Computes the chunks [chunk_begin, chunk_begin + chunk_count) (chunk_count <= 0: up to C) into `landmarks`
    [B,Hl,C,d] / `bias` [B,Hl,C] (allocated, zero-filled, when not passed).  Returns (landmarks, bias).
    """
    lib = load_library()
    B, Hl, C, d = landmark_queries.shape
    Hkv, T = k.shape[1], k.shape[2]
    dt = landmark_queries.dtype
    _check(landmark_queries, "landmark_queries", (B, Hl, C, d), dt, True)
    _check(k, "k", (B, Hkv, T, d), dt, True)
    if seq_lens is not None:
        _check(seq_lens, "seq_lens", (B,), torch.int32, True)
    if landmarks is None:
        landmarks = torch.zeros((B, Hl, C, d), dtype=dt, device=k.device)
    if bias is None:
        bias = torch.zeros((B, Hl, C), dtype=torch.float32, device=k.device)
    _check(landmarks, "landmarks", (B, Hl, C, d), dt, True)
    _check(bias, "bias", (B, Hl, C), torch.float32, True)
    p = make_params(B=B, Hq=Hl, Hkv=Hkv, Hl=Hl, L=0, T_max=T, C=C, d=d, chunk_size=chunk_size, top_k=1,
                    window=1, scale=scale, dtype=_dtype_code(k), impl="auto")
    rc = lib.hils_landmark_summary(ctypes.byref(p), _ptr(landmark_queries), _ptr(k), _ptr(seq_lens),
                                   int(chunk_begin), int(chunk_count), _ptr(landmarks), _ptr(bias), _stream_ptr(stream))
    if rc != 0:
        raise HilsError(rc, "hils_landmark_summary")
    return landmarks, bias


def hils_prefill_backward(q, k, v, landmarks, chunk_size: int, top_k: int, out, lse, sel_idx, dout, *, bias=None,
                          window: int = 1, scale: float = 0.0, impl: str = "auto", workspace=None, stream=None):
    """Gradients of a loss through `out` of hils_prefill (selection fixed): dout [B,Hq,L,d] in q's dtype;
    out, lse, sel_idx as hils_prefill returned them.

    Returns (dq [B,Hq,L,d], dk, dv [B,Hkv,T,d], dlandmarks [B,Hl,C,d], dbias [B,Hl,C] or None), all fp32.
    """
    lib = load_library()
    B, Hq, L, d = q.shape
    Hkv, T = k.shape[1], k.shape[2]
    Hl, C = landmarks.shape[1], landmarks.shape[2]
    dt = q.dtype
    _check(q, "q", (B, Hq, L, d), dt, True)
    _check(k, "k", (B, Hkv, T, d), dt, True)
    _check(v, "v", (B, Hkv, T, d), dt, True)
    _check(landmarks, "landmarks", (B, Hl, C, d), dt, True)
    _check(out, "out", (B, Hq, L, d), dt, True)
    _check(dout, "dout", (B, Hq, L, d), dt, True)
    _check(lse, "lse", (B, Hq, L), torch.float32, True)
    _check(sel_idx, "sel_idx", (B, Hkv, L, top_k), torch.int32, True)
    if bias is not None:
        _check(bias, "bias", (B, Hl, C), torch.float32, True)
    f32 = dict(dtype=torch.float32, device=q.device)
    dq = torch.empty((B, Hq, L, d), **f32)
    dk = torch.empty((B, Hkv, T, d), **f32)
    dv = torch.empty((B, Hkv, T, d), **f32)
    dlm = torch.empty((B, Hl, C, d), **f32)
    dbias = torch.empty((B, Hl, C), **f32) if bias is not None else None
    p = make_params(B=B, Hq=Hq, Hkv=Hkv, Hl=Hl, L=L, T_max=T, C=C, d=d, chunk_size=chunk_size, top_k=top_k,
                    window=window, scale=scale, dtype=_dtype_code(q), impl=impl)
    if workspace is None:
        n = int(lib.hils_prefill_backward_workspace_bytes(ctypes.byref(p)))
        if n == 0:
            raise HilsError(-2, "hils_prefill_backward_workspace_bytes")
        workspace = torch.empty(n, dtype=torch.uint8, device=q.device)
        workspace[:256].zero_()
    rc = lib.hils_prefill_backward(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(landmarks), _ptr(bias), _ptr(out),
                                   _ptr(lse), _ptr(sel_idx), _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dlm),
                                   _ptr(dbias), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != 0:
        raise HilsError(rc, "hils_prefill_backward")
    return dq, dk, dv, dlm, dbias


class _HilsAttentionFn(torch.autograd.Function):
    """hils_prefill / hils_prefill_backward as one differentiable op (argument marshalling only: both passes run
    in the library's kernels).  The selection is a constant of the backward pass; lse and sel_idx are returned
    without gradient."""

    @staticmethod
    def forward(ctx, q, k, v, landmarks, bias, chunk_size, top_k, window, scale):
        out, lse, sel = hils_prefill(q, k, v, landmarks, chunk_size, top_k, bias=bias, window=window, scale=scale)
        ctx.save_for_backward(q, k, v, landmarks, bias if bias is not None else q.new_empty(0), out, lse, sel)
        ctx.has_bias = bias is not None
        ctx.cfg = (chunk_size, top_k, window, scale)
        ctx.mark_non_differentiable(lse, sel)
        return out, lse, sel

    @staticmethod
    def backward(ctx, dout, _dlse, _dsel):
        q, k, v, landmarks, bias, out, lse, sel = ctx.saved_tensors
        chunk_size, top_k, window, scale = ctx.cfg
        dq, dk, dv, dlm, db = hils_prefill_backward(q, k, v, landmarks, chunk_size, top_k, out, lse, sel,
                                                    dout.contiguous(), bias=bias if ctx.has_bias else None,
                                                    window=window, scale=scale)
        return (dq.to(q.dtype), dk.to(k.dtype), dv.to(v.dtype), dlm.to(landmarks.dtype),
                db if ctx.has_bias else None, None, None, None, None)


def hils_attention(q, k, v, landmarks, chunk_size: int, top_k: int, *, bias=None, window: int = 1, scale: float = 0.0):
    """Differentiable HiLS prefill for training: returns (out, lse, sel_idx); gradients flow through `out` to
    q, k, v, landmarks and bias (cast to the inputs' dtypes)."""
    return _HilsAttentionFn.apply(q, k, v, landmarks, bias, chunk_size, top_k, window, scale)


def hils_chunk_overlap(sel_idx, block_queries: int, num_chunks: int, *, stats=None, overlap=None, stream=None):
    """Chunk-id overlap of blocks of `block_queries` adjacent queries (Sec. "Chunk Overlap", Eq. Overlap).

    sel_idx [B,Hkv,L,K] int32 CUDA tensor as written by hils_prefill; num_chunks = C bounds the chunk ids.
    Returns (stats [B,Hkv,nblk,4] int32: total, union, reused, full; overlap [B,Hkv,nblk] fp32, NaN where the
    equation does not apply), nblk = ceil(L / block_queries).
    """
    lib = load_library()
    B, Hkv, L, K = sel_idx.shape
    _check(sel_idx, "sel_idx", (B, Hkv, L, K), torch.int32, True)
    nblk = (L + int(block_queries) - 1) // max(int(block_queries), 1)
    if stats is None:
        stats = torch.empty((B, Hkv, nblk, 4), dtype=torch.int32, device=sel_idx.device)
    if overlap is None:
        overlap = torch.empty((B, Hkv, nblk), dtype=torch.float32, device=sel_idx.device)
    _check(stats, "stats", (B, Hkv, nblk, 4), torch.int32, True)
    _check(overlap, "overlap", (B, Hkv, nblk), torch.float32, True)
    p = make_params(B=B, Hq=Hkv, Hkv=Hkv, Hl=Hkv, L=L, T_max=0, C=int(num_chunks), d=1, chunk_size=1, top_k=K,
                    window=1, scale=0.0, dtype=0, impl="auto")
    rc = lib.hils_chunk_overlap(ctypes.byref(p), _ptr(sel_idx), int(block_queries), _ptr(stats), _ptr(overlap),
                                _stream_ptr(stream))
    if rc != 0:
        raise HilsError(rc, "hils_chunk_overlap")
    return stats, overlap


def hils_decode_multi(q, k_cache, v_cache, landmarks, seq_lens, chunk_size: int, top_k: int, stream=None, *,
                      bias=None, window: int = 1, scale: float = 0.0, block_table=None, out=None, lse=None,
                      sel_idx=None, workspace=None):
    """Multi-token decode: q [B,M,Hq,d], the M newest tokens of every sequence (already in the caches; seq_lens [B]
    counts them).  Caches [B,Hkv,T,d], or page pools [P,Hkv,S,d] with block_table [B,C].
    Returns (out [B,M,Hq,d], lse [B,M,Hq], sel_idx [B,M,Hkv,K])."""
    lib = load_library()
    B, M, Hq, d = q.shape
    Hkv = k_cache.shape[1]
    Hl, C = landmarks.shape[1], landmarks.shape[2]
    dt = q.dtype
    _check(q, "q", (B, M, Hq, d), dt, True)
    _check(landmarks, "landmarks", (B, Hl, C, d), dt, True)
    _check(seq_lens, "seq_lens", (B,), torch.int32, True)
    num_pages = 0
    if block_table is None:
        T = k_cache.shape[2]
        _check(k_cache, "k_cache", (B, Hkv, T, d), dt, True)
        _check(v_cache, "v_cache", (B, Hkv, T, d), dt, True)
    else:
        num_pages = k_cache.shape[0]
        T = C * chunk_size
        _check(k_cache, "k_pages", (num_pages, Hkv, chunk_size, d), dt, True)
        _check(v_cache, "v_pages", (num_pages, Hkv, chunk_size, d), dt, True)
        _check(block_table, "block_table", (B, C), torch.int32, True)
    if bias is not None:
        _check(bias, "bias", (B, Hl, C), torch.float32, True)
    out = torch.empty_like(q) if out is None else out
    lse = torch.empty((B, M, Hq), dtype=torch.float32, device=q.device) if lse is None else lse
    sel_idx = torch.empty((B, M, Hkv, top_k), dtype=torch.int32, device=q.device) if sel_idx is None else sel_idx
    _check(out, "out", (B, M, Hq, d), dt, True)
    _check(lse, "lse", (B, M, Hq), torch.float32, True)
    _check(sel_idx, "sel_idx", (B, M, Hkv, top_k), torch.int32, True)
    p = make_params(B=B, Hq=Hq, Hkv=Hkv, Hl=Hl, L=0, T_max=T, C=C, d=d, chunk_size=chunk_size, top_k=top_k,
                    window=window, scale=scale, dtype=_dtype_code(q), impl="auto")
    if workspace is None:
        n = int(lib.hils_decode_multi_workspace_bytes(ctypes.byref(p), int(M)))
        if n == 0:
            raise HilsError(-2, "hils_decode_multi_workspace_bytes")
        workspace = torch.empty(n, dtype=torch.uint8, device=q.device)
        workspace[:256].zero_()
    rc = lib.hils_decode_multi(ctypes.byref(p), int(M), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(landmarks),
                               _ptr(bias), _ptr(block_table), int(num_pages), _ptr(seq_lens), _ptr(out), _ptr(lse),
                               _ptr(sel_idx), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != 0:
        raise HilsError(rc, "hils_decode_multi")
    return out, lse, sel_idx


class HostRunner:
    """End-to-end calls with HOST tensors through hils_prefill_host / hils_decode_host.

    Owns the device arena (allocated once from torch) and pinned output buffers; each `run`
    enqueues host->device copies, the kernels and device->host copies on the current stream.
    """

    def __init__(self, params: HilsParams, is_decode: bool, device="cuda"):
        self.params, self.is_decode = params, is_decode
        n = host_arena_bytes(params, is_decode)
        if n == 0:
            raise HilsError(-2, "hils_host_arena_bytes")
        self.arena = torch.empty(n + 256, dtype=torch.uint8, device=device)
        off = (-self.arena.data_ptr()) % 256
        self.arena = self.arena[off:off + n]
        self.arena[:256].zero_()
        p = params
        R = 1 if is_decode else p.L
        dt = torch.float32 if p.dtype == HILS_F32 else torch.bfloat16
        oshape = (p.B, p.Hq, p.d) if is_decode else (p.B, p.Hq, R, p.d)
        lshape = (p.B, p.Hq) if is_decode else (p.B, p.Hq, R)
        sshape = (p.B, p.Hkv, p.top_k) if is_decode else (p.B, p.Hkv, R, p.top_k)
        self.out = torch.empty(oshape, dtype=dt).pin_memory()
        self.lse = torch.empty(lshape, dtype=torch.float32).pin_memory()
        self.sel = torch.empty(sshape, dtype=torch.int32).pin_memory()

    def bytes_per_step(self, tensors: Dict[str, torch.Tensor]) -> Tuple[int, int]:
        h2d = sum(t.numel() * t.element_size() for t in tensors.values() if t is not None)
        d2h = sum(t.numel() * t.element_size() for t in (self.out, self.lse, self.sel))
        return h2d, d2h

    def run(self, q, k, v, landmarks, bias=None, seq_lens=None, stream=None):
        lib = load_library()
        for name, t in (("q", q), ("k", k), ("v", v), ("landmarks", landmarks)):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("%s must be a contiguous host tensor" % name)
        sp = _stream_ptr(stream)
        if self.is_decode:
            rc = lib.hils_decode_host(ctypes.byref(self.params), _ptr(q), _ptr(k), _ptr(v), _ptr(landmarks),
                                      _ptr(bias), _ptr(seq_lens), _ptr(self.out), _ptr(self.lse), _ptr(self.sel),
                                      _ptr(self.arena), self.arena.numel(), sp)
        else:
            rc = lib.hils_prefill_host(ctypes.byref(self.params), _ptr(q), _ptr(k), _ptr(v), _ptr(landmarks),
                                       _ptr(bias), _ptr(self.out), _ptr(self.lse), _ptr(self.sel),
                                       _ptr(self.arena), self.arena.numel(), sp)
        if rc != 0:
            raise HilsError(rc, "hils_decode_host" if self.is_decode else "hils_prefill_host")
        return self.out, self.lse, self.sel


def trace_enable(on: bool) -> None:
    rc = load_library().hils_trace_enable(1 if on else 0)
    if rc != 0:
        raise HilsError(rc, "hils_trace_enable")


def trace_read():
    """[(kernel name, device milliseconds)] of the last traced call (waits for it to finish)."""
    names = ctypes.create_string_buffer(32768)
    ms = (ctypes.c_float * 1024)()
    n = load_library().hils_trace_read(names, 32768, ms, 1024)
    if n < 0:
        raise HilsError(n, "hils_trace_read")
    parts = [x for x in names.value.decode().split(";") if x]
    return [(parts[i] if i < len(parts) else "?", float(ms[i])) for i in range(n)]


def poll_status(workspace: torch.Tensor, stream=None) -> int:
    return int(load_library().hils_poll_status(_ptr(workspace), _stream_ptr(stream)))
