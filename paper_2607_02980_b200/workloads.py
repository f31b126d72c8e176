"""Seeded synthetic inputs for HiLS attention (prefill and decode).

This module only draws random tensors and plants "needle" chunks. It holds none
of the operator's arithmetic (no scoring, no selection, no softmax); both the
CUDA path and the CPU oracle consume the tensors it returns unchanged.

Shapes follow the paper's long-context setting (chunk size S=64, top-K 16..64,
contexts 16K..1M; hyper-parameter table, App. D) with GQA 32/8 heads, d=128.

Layouts (last dimension contiguous):
    q          [B, Hq, L, d]   (decode: [B, Hq, d])
    k, v       [B, Hkv, T, d]
    landmarks  [B, Hkv, C, d]   C = T // S, one summary key per complete chunk
    seq_lens   [B] int32        (decode only)

Value recipe:
    fp32 config : Q, K, V ~ N(0,1)/sqrt(d)
    bf16 configs: Q, K, V ~ N(0,1) rounded to bf16
    landmarks   : fp32 mean of the (already rounded) K rows of the chunk
                  + 0.1 * N(0,1), rounded to the config dtype (mean-pooled
                  summary of Sec. 3.2 plus noise)
    needles     : for a query row and KV group, `n_needles` chunks are drawn
                  uniformly from its complete past chunks and
                  3 * k'_n / ||k'_n|| is added to every query head of the group
                  before rounding (a +3 sigma shift of the projection of an
                  N(0, I) query on the landmark direction), so that selection
                  has margin.

    structured overlap (optional, `overlap_block=M`): adjacent queries of a
                  real model retrieve largely the same chunks (Sec. "Chunk
                  Overlap": up to 80-93 % shared).  One base query per block
                  of M adjacent tokens and head, q_i = base + noise * N(0,1);
                  no needles.  The other tensors are unchanged.  With
                  `overlap_drift=rho` the base queries of consecutive blocks
                  form an AR(1) sequence (inter-block reuse, 92.8 % in the
                  paper's measurement).

Every tensor has its own generator seeded with seed*1000 + tensor_id, so a
tensor does not change when another one is added or resized.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import torch


@dataclasses.dataclass(frozen=True)
class HilsConfig:
    name: str
    mode: str            # "prefill" | "decode"
    B: int
    Hq: int
    Hkv: int
    L: int               # prefill: sequence length; decode: KV-cache length T
    d: int
    S: int
    K: int
    dtype: str           # "f32" | "bf16"
    seed: int
    n_needles: int = 0
    needle_shared: bool = False   # decode: one needle chunk per sequence shared by all groups
    window: int = 1

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def C(self) -> int:
        return self.L // self.S

    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def scaled(self, **kw) -> "HilsConfig":
        return dataclasses.replace(self, **kw)


# The five benchmark configurations (index = config number).
CONFIGS = [
    HilsConfig("cfg0_tiny_f32_prefill", "prefill", 1, 1, 1, 2048, 64, 64, 4, "f32", 0),
    HilsConfig("cfg1_gqa_bf16_prefill_16k", "prefill", 1, 32, 8, 16384, 128, 64, 16, "bf16", 1, n_needles=2),
    HilsConfig("cfg2_long_bf16_prefill_128k", "prefill", 1, 32, 8, 131072, 128, 64, 32, "bf16", 2, n_needles=2),
    HilsConfig("cfg3_batched_bf16_decode_64k", "decode", 64, 32, 8, 65536, 128, 64, 32, "bf16", 3, n_needles=2),
    HilsConfig("cfg4_ultralong_bf16_decode_1m", "decode", 4, 32, 8, 1048576, 128, 64, 64, "bf16", 4, n_needles=1,
               needle_shared=True),
]


def _gen(seed: int, tensor_id: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed * 1000 + tensor_id)
    return g


def _randn(shape, gen, device, dtype=torch.float32):
    return torch.randn(shape, generator=gen, device=device, dtype=dtype)


def _draw_kv(cfg: HilsConfig, gen, device) -> torch.Tensor:
    """K or V cache [B, Hkv, T, d] in the config dtype, drawn slab by slab."""
    out = torch.empty((cfg.B, cfg.Hkv, cfg.L, cfg.d), dtype=cfg.torch_dtype(), device=device)
    mul = 1.0 / math.sqrt(cfg.d) if cfg.dtype == "f32" else 1.0
    for b in range(cfg.B):
        for h in range(cfg.Hkv):
            slab = _randn((cfg.L, cfg.d), gen, device)
            if mul != 1.0:
                slab = slab * mul
            out[b, h].copy_(slab)
    return out


def _draw_landmarks(cfg: HilsConfig, k: torch.Tensor, gen, device) -> torch.Tensor:
    """Chunk mean of the rounded K rows plus 0.1*N(0,1) noise, in the config dtype."""
    C = cfg.C
    out = torch.empty((cfg.B, cfg.Hkv, C, cfg.d), dtype=cfg.torch_dtype(), device=device)
    for b in range(cfg.B):
        for h in range(cfg.Hkv):
            mean = k[b, h, : C * cfg.S].float().view(C, cfg.S, cfg.d).mean(dim=1)
            noise = _randn((C, cfg.d), gen, device)
            out[b, h].copy_(mean + 0.1 * noise)
    return out


def make_landmark_queries(cfg: HilsConfig, device="cpu", Hl: Optional[int] = None, C: Optional[int] = None) -> torch.Tensor:
    """Seeded learnable chunk queries q'_c [B, Hl, C, d] for the chunk-summary step (stand-ins for the query
    vectors of trained landmark tokens): N(0, 1) in the config dtype, times sqrt(d) for the fp32 config whose
    keys are N(0, 1)/sqrt(d), so that the scores inside a chunk have a standard deviation of about 1."""
    dev = torch.device(device)
    Hl = cfg.Hkv if Hl is None else Hl
    C = cfg.C if C is None else C
    gen = _gen(cfg.seed, 7, dev)
    mul = math.sqrt(cfg.d) if cfg.dtype == "f32" else 1.0
    out = torch.empty((cfg.B, Hl, C, cfg.d), dtype=cfg.torch_dtype(), device=dev)
    for b in range(cfg.B):
        for h in range(Hl):
            out[b, h].copy_(_randn((C, cfg.d), gen, dev) * mul)
    return out


def _needle_dirs(lm_bh: torch.Tensor, idx: torch.Tensor) -> torch.Tensor:
    """3 * k'_n / ||k'_n|| for the landmark rows `idx` of one (b, KV head)."""
    rows = lm_bh.float()[idx]
    return 3.0 * rows / rows.norm(dim=-1, keepdim=True).clamp_min(1e-20)


def make_prefill_inputs(cfg: HilsConfig, device="cpu", overlap_block: int = 0,
                        overlap_noise: float = 0.3, overlap_drift: float = 0.0) -> Dict[str, torch.Tensor]:
    assert cfg.mode == "prefill"
    dev = torch.device(device)
    k = _draw_kv(cfg, _gen(cfg.seed, 1, dev), dev)
    v = _draw_kv(cfg, _gen(cfg.seed, 2, dev), dev)
    landmarks = _draw_landmarks(cfg, k, _gen(cfg.seed, 3, dev), dev)
    gq = _gen(cfg.seed, 0, dev)
    gn = _gen(cfg.seed, 4, dev)
    q = torch.empty((cfg.B, cfg.Hq, cfg.L, cfg.d), dtype=cfg.torch_dtype(), device=dev)
    mul = 1.0 / math.sqrt(cfg.d) if cfg.dtype == "f32" else 1.0
    G = cfg.G
    pos = torch.arange(cfg.L, device=dev)
    ci = pos // cfg.S                         # number of complete past chunks of each row
    gb = _gen(cfg.seed, 8, dev)
    for b in range(cfg.B):
        for g in range(cfg.Hkv):
            qg = _randn((G, cfg.L, cfg.d), gq, dev) * mul
            if overlap_block > 1:
                nblk = (cfg.L + overlap_block - 1) // overlap_block
                base = _randn((G, nblk, cfg.d), gb, dev) * mul
                if overlap_drift > 0.0:
                    # slowly drifting base queries: base_r = rho * base_{r-1} + sqrt(1 - rho^2) * N(0,1), so that a
                    # block also shares most of its chunks with the block before it (the paper measures 92.8 %)
                    rho, fresh = overlap_drift, math.sqrt(1.0 - overlap_drift * overlap_drift)
                    for r in range(1, nblk):
                        base[:, r] = rho * base[:, r - 1] + fresh * base[:, r]
                qg = base.repeat_interleave(overlap_block, dim=1)[:, :cfg.L] + overlap_noise * qg
            elif cfg.n_needles > 0:
                ok = ci >= cfg.n_needles      # rows with enough past chunks to plant into
                u = torch.rand((cfg.n_needles, cfg.L), generator=gn, device=dev)
                chosen = []
                for n in range(cfg.n_needles):
                    # n-th needle: uniform over the past chunks not chosen yet
                    cand = torch.floor(u[n] * (ci - n).clamp_min(1).float()).long()
                    for prev in sorted_stack(chosen):
                        cand = cand + (cand >= prev).long()
                    cand = cand.clamp_max((ci - 1).clamp_min(0))
                    chosen.append(cand)
                    add = _needle_dirs(landmarks[b, g], cand)
                    add = add * ok.unsqueeze(-1).float()
                    qg = qg + add.unsqueeze(0)
            q[b, g * G:(g + 1) * G].copy_(qg)
    return {"q": q, "k": k, "v": v, "landmarks": landmarks}


def sorted_stack(chosen):
    """Earlier needle draws in ascending order per row (for distinct sampling)."""
    if not chosen:
        return []
    st = torch.stack(chosen, 0).sort(dim=0).values
    return [st[i] for i in range(st.shape[0])]


def make_decode_inputs(cfg: HilsConfig, device="cpu", seq_lens: Optional[torch.Tensor] = None,
                       query_set: int = 0) -> Dict[str, torch.Tensor]:
    """Decode inputs. `query_set` draws a different q (and needles) over the same cache."""
    assert cfg.mode == "decode"
    dev = torch.device(device)
    k = _draw_kv(cfg, _gen(cfg.seed, 1, dev), dev)
    v = _draw_kv(cfg, _gen(cfg.seed, 2, dev), dev)
    landmarks = _draw_landmarks(cfg, k, _gen(cfg.seed, 3, dev), dev)
    if seq_lens is None:
        seq_lens = torch.full((cfg.B,), cfg.L, dtype=torch.int32, device=dev)
    seq_lens = seq_lens.to(device=dev, dtype=torch.int32)
    q = make_decode_queries(cfg, landmarks, seq_lens, query_set)
    return {"q": q, "k": k, "v": v, "landmarks": landmarks, "seq_lens": seq_lens}


def make_decode_queries(cfg: HilsConfig, landmarks: torch.Tensor, seq_lens: torch.Tensor,
                        query_set: int = 0) -> torch.Tensor:
    dev = landmarks.device
    gq = _gen(cfg.seed, 10 + 2 * query_set, dev)
    gn = _gen(cfg.seed, 11 + 2 * query_set, dev)
    G = cfg.G
    mul = 1.0 / math.sqrt(cfg.d) if cfg.dtype == "f32" else 1.0
    qf = _randn((cfg.B, cfg.Hq, cfg.d), gq, dev) * mul
    if cfg.n_needles > 0:
        ncand = ((seq_lens.long() - 1) // cfg.S)          # complete past chunks per sequence
        ngrp = 1 if cfg.needle_shared else cfg.Hkv
        u = torch.rand((cfg.B, ngrp, cfg.n_needles), generator=gn, device=dev)
        for b in range(cfg.B):
            nc = int(ncand[b])
            if nc < cfg.n_needles:
                continue
            for g in range(cfg.Hkv):
                ug = u[b, 0 if cfg.needle_shared else g]
                chosen = []
                for n in range(cfg.n_needles):
                    c = int(math.floor(float(ug[n]) * (nc - n)))
                    for prev in sorted(chosen):
                        if c >= prev:
                            c += 1
                    c = min(c, nc - 1)
                    chosen.append(c)
                idx = torch.tensor(chosen, device=dev, dtype=torch.long)
                add = _needle_dirs(landmarks[b, g], idx).sum(0)
                qf[b, g * G:(g + 1) * G] += add
    return qf.to(cfg.torch_dtype())


def make_bias(cfg: HilsConfig, device="cpu") -> torch.Tensor:
    """Optional entropy-like bias b'_c in [0, log S] (Prop. 3.1), fp32 [B, Hkv, C]."""
    dev = torch.device(device)
    g = _gen(cfg.seed, 5, dev)
    return torch.rand((cfg.B, cfg.Hkv, cfg.C), generator=g, device=dev) * math.log(cfg.S)


def sample_rows(cfg: HilsConfig, n: int, seed: int = 12345) -> torch.Tensor:
    """Seeded sample of query positions for large-L parity, always holding the edge rows."""
    L, S, K = cfg.L, cfg.S, cfg.K
    edges = [0, S - 1, S, K * S - 1, K * S, (K + 1) * S, (K + 1) * S - 1, L - 1, L - S, L - S - 1]
    edges = sorted({e for e in edges if 0 <= e < L})
    if n >= L:
        return torch.arange(L, dtype=torch.int64)
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    perm = torch.randperm(L, generator=g)[: max(0, n - len(edges))]
    rows = torch.unique(torch.cat([torch.tensor(edges, dtype=torch.int64), perm]))
    return rows
