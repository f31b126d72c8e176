"""CPU oracle for HiLS attention -- TEST INFRASTRUCTURE, not product code.

Thin ctypes wrapper around ``hils_oracle.c`` (plain C, fp64).  Only the tests,
the smoke check and the benchmark's CPU-baseline leg may import this package;
the CUDA library and its Python binding never do, and this package imports
nothing from them.

Parity status: the paper prints no numeric example, so every function here is
pinned by identities (see tests/test_oracle_pins.py); absolute agreement with
the authors' own implementation is unpinned.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hils_oracle.c")
_SO = os.path.join(_HERE, "libhils_oracle.so")
_lib = None


class _Params(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int), ("Hq", ctypes.c_int), ("Hkv", ctypes.c_int), ("Hl", ctypes.c_int),
                ("Lq", ctypes.c_int), ("T", ctypes.c_int), ("C", ctypes.c_int),
                ("d", ctypes.c_int), ("S", ctypes.c_int), ("K", ctypes.c_int), ("W", ctypes.c_int),
                ("scale", ctypes.c_double), ("group_mode", ctypes.c_int), ("in_bf16", ctypes.c_int)]


_CFLAGS = ["-O3", "-march=native", "-fopenmp", "-shared", "-fPIC", "-std=c11"]


def _stamp() -> str:
    """What the built object depends on: the source, the flags and (because of -march=native) this machine's CPU."""
    import hashlib
    h = hashlib.sha256()
    with open(_SRC, "rb") as f:
        h.update(f.read())
    h.update(" ".join(_CFLAGS).encode())
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags") or line.startswith("model name"):
                    h.update(line.encode())
                    if line.startswith("flags"):
                        break
    except OSError:
        pass
    return h.hexdigest()


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O3 -march=native, OpenMP) if the shared object is missing, stale or was built
    on a machine with another CPU."""
    stamp_path = _SO + ".stamp"
    want = _stamp()
    if not force and os.path.exists(_SO) and os.path.exists(stamp_path):
        with open(stamp_path) as f:
            if f.read() == want:
                return _SO
    tmp = _SO + ".tmp%d" % os.getpid()
    cmd = ["gcc"] + _CFLAGS + ["-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _SO)
    with open(stamp_path, "w") as f:
        f.write(want)
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_SO)
        _lib.hils_oracle_rows.restype = ctypes.c_int
        _lib.hils_oracle_num_threads.restype = ctypes.c_int
        _lib.hils_oracle_landmarks.restype = ctypes.c_int
        _lib.hils_oracle_rows_routed.restype = ctypes.c_int
        _lib.hils_oracle_backward.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().hils_oracle_num_threads())


def _is_bf16(a) -> bool:
    return hasattr(a, "detach") and str(a.dtype) == "torch.bfloat16"


def _f32(a) -> np.ndarray:
    """fp32 C-contiguous numpy view/copy of a numpy array or a CPU torch tensor (bf16 widens exactly)."""
    if hasattr(a, "detach"):
        a = a.detach().to("cpu").float().contiguous().numpy()
    return np.ascontiguousarray(a, dtype=np.float32)


def _raw_bf16(a) -> np.ndarray:
    """The 16-bit patterns of a CPU bf16 torch tensor as a uint16 numpy array (no copy if contiguous)."""
    import torch
    return a.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16)


def _ptr(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def hils_rows(q, k, v, landmarks, bias, *, S: int, K: int, W: int = 1, scale: float = 0.0,
              row_b, row_qi, row_pos, sel_idx=None, attend: bool = True, group_mode: int = 0,
              want_alpha: bool = False, q_route=None):
    """Run the oracle on a list of query rows.

    q [B,Hq,Lq,d]; k,v [B,Hkv,T,d]; landmarks [B,Hl,C,d]; bias [B,Hl,C] or None.
    Row r is q[row_b[r], :, row_qi[r], :] at sequence position row_pos[r].
    If ``sel_idx`` ([n,Hkv,K] int32, ascending, -1 padded) is given it is used as the
    selection instead of computing one.
    Returns dict(sel_idx, margin, out, lse[, alpha]) as numpy arrays indexed by row.
    """
    lib = _load()
    in_bf16 = int(all(_is_bf16(t) for t in (q, k, v, landmarks)))
    conv = _raw_bf16 if in_bf16 else _f32
    q = conv(q); k = conv(k); v = conv(v); landmarks = conv(landmarks)
    # routing query (Eq. Q-Cal): replaces q in the surrogate scores only; same shape and dtype as q
    qr = None if q_route is None else conv(q_route)
    if qr is not None and qr.shape != q.shape:
        raise ValueError("q_route must have the shape of q")
    bias_a = None if bias is None else _f32(bias)
    B, Hq, Lq, d = q.shape
    _, Hkv, T, _ = k.shape
    _, Hl, C, _ = landmarks.shape
    row_b = np.ascontiguousarray(row_b, dtype=np.int32)
    row_qi = np.ascontiguousarray(row_qi, dtype=np.int32)
    row_pos = np.ascontiguousarray(row_pos, dtype=np.int64)
    n = row_b.shape[0]
    p = _Params(B, Hq, Hkv, Hl, Lq, T, C, d, S, K, W, float(scale), group_mode, in_bf16)
    sel_mode = 0
    if sel_idx is None:
        sel = np.full((n, Hkv, K), -1, dtype=np.int32)
    else:
        sel = np.ascontiguousarray(sel_idx, dtype=np.int32).reshape(n, Hkv, K).copy()
        sel_mode = 1
    margin = np.full((n, Hkv), np.inf, dtype=np.float64)
    out = np.zeros((n, Hq, d), dtype=np.float64) if attend else None
    lse = np.zeros((n, Hq), dtype=np.float64) if attend else None
    alpha = np.zeros((n, Hq, K + 1), dtype=np.float64) if (attend and want_alpha) else None
    rc = lib.hils_oracle_rows_routed(
        ctypes.byref(p), ctypes.c_void_p(q.ctypes.data), ctypes.c_void_p(None if qr is None else qr.ctypes.data),
        ctypes.c_void_p(k.ctypes.data),
        ctypes.c_void_p(v.ctypes.data), ctypes.c_void_p(landmarks.ctypes.data), _ptr(bias_a, ctypes.c_float),
        ctypes.c_int64(n), _ptr(row_b, ctypes.c_int32), _ptr(row_qi, ctypes.c_int32),
        _ptr(row_pos, ctypes.c_int64), ctypes.c_int(sel_mode), ctypes.c_int(1 if attend else 0),
        _ptr(sel, ctypes.c_int32), _ptr(margin, ctypes.c_double),
        _ptr(out, ctypes.c_double), _ptr(lse, ctypes.c_double), _ptr(alpha, ctypes.c_double))
    if rc != 0:
        raise ValueError("hils_oracle_rows rejected its arguments (rc=%d)" % rc)
    res = {"sel_idx": sel, "margin": margin, "out": out, "lse": lse}
    if alpha is not None:
        res["alpha"] = alpha
    return res


def hils_prefill(q, k, v, landmarks, bias=None, *, S: int, K: int, W: int = 1, scale: float = 0.0,
                 rows=None, sel_idx=None, group_mode: int = 0, want_alpha: bool = False, q_route=None):
    """Prefill oracle: every position (or the positions in ``rows``) of every sequence.

    Returns arrays shaped [B, n_rows, ...]: sel_idx [B,n,Hkv,K], margin [B,n,Hkv],
    out [B,n,Hq,d], lse [B,n,Hq].
    """
    B, L = q.shape[0], q.shape[2]
    rows = np.arange(L, dtype=np.int64) if rows is None else np.asarray(rows, dtype=np.int64)
    n = rows.shape[0]
    row_b = np.repeat(np.arange(B, dtype=np.int32), n)
    row_pos = np.tile(rows, B)
    if sel_idx is not None:
        sel_idx = np.asarray(sel_idx).reshape(B * n, -1, K)
    res = hils_rows(q, k, v, landmarks, bias, S=S, K=K, W=W, scale=scale, row_b=row_b,
                    row_qi=row_pos.astype(np.int32), row_pos=row_pos, sel_idx=sel_idx,
                    group_mode=group_mode, want_alpha=want_alpha, q_route=q_route)
    return {key: val.reshape((B, n) + val.shape[1:]) for key, val in res.items() if val is not None}


def hils_decode(q, k_cache, v_cache, landmarks, bias, seq_lens, *, S: int, K: int, W: int = 1,
                scale: float = 0.0, sel_idx=None, group_mode: int = 0, want_alpha: bool = False, q_route=None):
    """Decode oracle: one query per sequence at position seq_lens[b]-1 (its own k,v are in the cache).

    q [B,Hq,d].  Returns sel_idx [B,Hkv,K], margin [B,Hkv], out [B,Hq,d], lse [B,Hq].
    """
    qn = q if _is_bf16(q) else _f32(q)
    B, Hq, d = qn.shape
    seq = np.asarray(seq_lens.cpu() if hasattr(seq_lens, "cpu") else seq_lens, dtype=np.int64)
    qr = None
    if q_route is not None:
        qr = (q_route if _is_bf16(q_route) else _f32(q_route)).reshape(B, Hq, 1, d)
    return hils_rows(qn.reshape(B, Hq, 1, d), k_cache, v_cache, landmarks, bias, S=S, K=K, W=W,
                     scale=scale, row_b=np.arange(B, dtype=np.int32), row_qi=np.zeros(B, dtype=np.int32),
                     row_pos=seq - 1, sel_idx=sel_idx, group_mode=group_mode, want_alpha=want_alpha, q_route=qr)


def hils_landmarks(lq, k, seq_lens=None, *, S: int, scale: float = 0.0):
    """Chunk summaries of Proposition 3.1 (Eq. prop_q_c): k'_c = Attn(q'_c, K_c, K_c), b'_c = entropy.

    lq [B,Hl,C,d] learnable chunk queries, k [B,Hkv,T,d] keys (both fp32 or both bf16), seq_lens [B] or None.
    Returns (landmarks [B,Hl,C,d], bias [B,Hl,C]) as float64 numpy arrays.
    """
    lib = _load()
    in_bf16 = int(_is_bf16(lq) and _is_bf16(k))
    conv = _raw_bf16 if in_bf16 else _f32
    lq = conv(lq); k = conv(k)
    B, Hl, C, d = lq.shape
    _, Hkv, T, _ = k.shape
    sl = None if seq_lens is None else np.ascontiguousarray(
        seq_lens.detach().cpu().numpy() if hasattr(seq_lens, "detach") else seq_lens, dtype=np.int32)
    p = _Params(B, Hl, Hkv, Hl, 0, T, C, d, S, 1, 1, float(scale), 0, in_bf16)
    lm = np.zeros((B, Hl, C, d), dtype=np.float64)
    bias = np.zeros((B, Hl, C), dtype=np.float64)
    rc = lib.hils_oracle_landmarks(ctypes.byref(p), ctypes.c_void_p(lq.ctypes.data), ctypes.c_void_p(k.ctypes.data),
                                   _ptr(sl, ctypes.c_int32), _ptr(lm, ctypes.c_double), _ptr(bias, ctypes.c_double))
    if rc != 0:
        raise ValueError("hils_oracle_landmarks rejected its arguments (rc=%d)" % rc)
    return lm, bias


def hils_backward(q, k, v, landmarks, bias, sel_idx, dout, *, S: int, K: int, W: int = 1, scale: float = 0.0,
                  pos0: int = 0):
    """Gradients of a scalar loss through `out` of the operator (chain rule on Eq. HiLS weights, selection fixed).

    q, dout [B,Hq,Lq,d]; k, v [B,Hkv,T,d]; landmarks [B,Hl,C,d]; bias [B,Hl,C] or None; sel_idx [B,Hkv,Lq,K]
    as the forward wrote it; query row r sits at position pos0 + r.  dout is taken as float64.
    Returns dict(dq, dk, dv, dlandmarks, dbias) of float64 arrays shaped like q, k, v, landmarks, bias.
    """
    lib = _load()
    in_bf16 = int(all(_is_bf16(t) for t in (q, k, v, landmarks)))
    conv = _raw_bf16 if in_bf16 else _f32
    q = conv(q); k = conv(k); v = conv(v); landmarks = conv(landmarks)
    bias_a = None if bias is None else _f32(bias)
    B, Hq, Lq, d = q.shape
    _, Hkv, T, _ = k.shape
    _, Hl, C, _ = landmarks.shape
    sel = np.ascontiguousarray(sel_idx.detach().cpu().numpy() if hasattr(sel_idx, "detach") else sel_idx,
                               dtype=np.int32)
    assert sel.shape == (B, Hkv, Lq, K)
    do = np.ascontiguousarray(dout.detach().cpu().double().numpy() if hasattr(dout, "detach") else dout,
                              dtype=np.float64)
    assert do.shape == (B, Hq, Lq, d)
    p = _Params(B, Hq, Hkv, Hl, Lq, T, C, d, S, K, W, float(scale), 0, in_bf16)
    res = {"dq": np.zeros((B, Hq, Lq, d)), "dk": np.zeros((B, Hkv, T, d)), "dv": np.zeros((B, Hkv, T, d)),
           "dlandmarks": np.zeros((B, Hl, C, d)), "dbias": np.zeros((B, Hl, C))}
    rc = lib.hils_oracle_backward(
        ctypes.byref(p), ctypes.c_void_p(q.ctypes.data), ctypes.c_void_p(k.ctypes.data),
        ctypes.c_void_p(v.ctypes.data), ctypes.c_void_p(landmarks.ctypes.data), _ptr(bias_a, ctypes.c_float),
        _ptr(sel, ctypes.c_int32), ctypes.c_int64(pos0), _ptr(do, ctypes.c_double),
        _ptr(res["dq"], ctypes.c_double), _ptr(res["dk"], ctypes.c_double), _ptr(res["dv"], ctypes.c_double),
        _ptr(res["dlandmarks"], ctypes.c_double), _ptr(res["dbias"], ctypes.c_double))
    if rc != 0:
        raise ValueError("hils_oracle_backward rejected its arguments (rc=%d)" % rc)
    return res


def chunk_overlap(sel_idx, M: int):
    """Chunk-id overlap among blocks of M adjacent queries (Sec. "Chunk Overlap", Eq. Overlap).

    sel_idx: integer array [..., L, K], the selected chunk ids of L consecutive queries (-1 = empty slot).
    Queries r*M .. r*M + M - 1 form block r; a trailing block holds the L mod M queries that are left.
    For every block, written out with Python sets:
        total   = sum over its queries m of |I_m|
        union   = | union over m of I_m |                       (the chunks a packed kernel loads once)
        reused  = | union  intersected with  the previous block's union |   (0 for block 0: inter-block reuse)
        overlap = (M K - union) / ((M - 1) K)    as the equation has it, for blocks of M queries that each hold
                  K chunks; NaN for any other block (fewer than K candidates, or the short trailing block)
    Returns a dict of arrays [..., ceil(L / M)]: int64 total / union / reused, float64 overlap.
    """
    sel = np.asarray(sel_idx)
    assert M >= 1 and sel.ndim >= 2
    lead, (L, K) = sel.shape[:-2], sel.shape[-2:]
    flat = sel.reshape((-1, L, K))
    nblk = (L + M - 1) // M
    total = np.zeros((flat.shape[0], nblk), np.int64)
    union = np.zeros_like(total)
    reused = np.zeros_like(total)
    overlap = np.full((flat.shape[0], nblk), np.nan, np.float64)
    for x in range(flat.shape[0]):
        prev = set()
        for r in range(nblk):
            sets = [set(int(c) for c in flat[x, i] if c >= 0) for i in range(r * M, min(L, r * M + M))]
            u = set().union(*sets)
            total[x, r] = sum(len(s) for s in sets)
            union[x, r] = len(u)
            reused[x, r] = len(u & prev)
            if M > 1 and len(sets) == M and all(len(s) == K for s in sets):
                overlap[x, r] = (M * K - len(u)) / ((M - 1) * K)
            prev = u
    shape = lead + (nblk,)
    return {"total": total.reshape(shape), "union": union.reshape(shape), "reused": reused.reshape(shape),
            "overlap": overlap.reshape(shape)}


def loaded_fraction(union_size, visible_chunks):
    """Share of the visible historical chunks that a block of adjacent queries loads (Sec. "Chunk Overlap", the
    percentages of Fig. chunk_overlap, left): union size / visible pool."""
    return np.asarray(union_size, dtype=np.float64) / np.asarray(visible_chunks, dtype=np.float64)
