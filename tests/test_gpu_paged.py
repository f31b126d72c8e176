"""hils_decode_paged (KV pages of one chunk each, addressed through a block table) against the contiguous
entry point and the CPU oracle: the paging is a pure change of addressing, so the results must be identical
to hils_decode on the de-paged caches bit for bit, and match the oracle within the usual tolerances."""
import numpy as np
import pytest
import torch

import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import workloads as wl
from parity import check_decode

pytestmark = pytest.mark.gpu
DEV = "cuda"


def paginate(inp, cfg, seed, spare=7):
    """Scatter the contiguous caches [B,Hkv,T,d] into shuffled pages [P,Hkv,S,d]; unmapped pages hold NaN."""
    B, Hkv, T, d = inp["k"].shape
    S, C = cfg.S, T // cfg.S
    P = B * C + spare
    perm = torch.randperm(P, generator=torch.Generator().manual_seed(seed))
    table = perm[:B * C].reshape(B, C).to(torch.int32)
    kp = torch.full((P, Hkv, S, d), float("nan"), dtype=inp["k"].dtype)
    vp = torch.full((P, Hkv, S, d), float("nan"), dtype=inp["v"].dtype)
    for b in range(B):
        for c in range(C):
            kp[table[b, c]] = inp["k"][b, :, c * S:(c + 1) * S]
            vp[table[b, c]] = inp["v"][b, :, c * S:(c + 1) * S]
    return kp, vp, table


@pytest.mark.parametrize("W", [1, 512])
def test_paged_decode_is_identical_to_contiguous_decode_and_matches_the_oracle(W):
    cfg = wl.CONFIGS[3].scaled(B=6, L=4096, K=8, seed=81)
    seq = [4096, 4095, 1, 63, 2049, 640]
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor(seq, dtype=torch.int32))
    bias = wl.make_bias(cfg, "cpu")
    kp, vp, table = paginate(inp, cfg, 5)
    g = {n: t.to(DEV) for n, t in inp.items()}
    out_c, lse_c, sel_c = hils.hils_decode(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K,
                                           bias=bias.to(DEV), window=W)
    out_p, lse_p, sel_p = hils.hils_decode_paged(g["q"], kp.to(DEV), vp.to(DEV), g["landmarks"], table.to(DEV),
                                                 g["seq_lens"], cfg.S, cfg.K, bias=bias.to(DEV), window=W)
    torch.cuda.synchronize()
    assert hils.last_launch_count() == 3
    assert torch.equal(sel_p, sel_c)
    assert torch.equal(out_p, out_c) and torch.equal(lse_p, lse_c)
    check_decode(cfg, inp, out_p, lse_p, sel_p, bias=bias, W=W)


def test_paged_decode_many_pairs_wraps_the_ring():
    cfg = wl.CONFIGS[3].scaled(B=64, L=2048, K=16, seed=82)
    seq = [2048 - 37 * (i % 11) - (1 if i % 3 == 0 else 0) for i in range(64)]
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor(seq, dtype=torch.int32))
    kp, vp, table = paginate(inp, cfg, 6, spare=100)
    g = {n: t.to(DEV) for n, t in inp.items()}
    out_c, lse_c, sel_c = hils.hils_decode(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K)
    out_p, lse_p, sel_p = hils.hils_decode_paged(g["q"], kp.to(DEV), vp.to(DEV), g["landmarks"], table.to(DEV),
                                                 g["seq_lens"], cfg.S, cfg.K)
    torch.cuda.synchronize()
    assert torch.equal(sel_p, sel_c) and torch.equal(out_p, out_c) and torch.equal(lse_p, lse_c)


def test_out_of_range_page_sets_the_status_and_nothing_faults():
    cfg = wl.CONFIGS[3].scaled(B=2, L=1024, K=4, seed=83)
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor([1024, 512], dtype=torch.int32))
    kp, vp, table = paginate(inp, cfg, 7)
    bad = table.clone()
    bad[0, 15] = kp.shape[0] + 3                   # the query's own chunk of sequence 0
    g = {n: t.to(DEV) for n, t in inp.items()}
    p = hils.make_params(B=2, Hq=cfg.Hq, Hkv=cfg.Hkv, Hl=cfg.Hkv, L=0, T_max=cfg.L, C=cfg.C, d=cfg.d,
                         chunk_size=cfg.S, top_k=cfg.K, dtype=1, impl="auto")
    ws = hils.alloc_workspace(p, True, DEV)
    hils.hils_decode_paged(g["q"], kp.to(DEV), vp.to(DEV), g["landmarks"], bad.to(DEV), g["seq_lens"], cfg.S, cfg.K,
                           workspace=ws)
    assert hils.poll_status(ws) == -7
    ws[:256].zero_()
    hils.hils_decode_paged(g["q"], kp.to(DEV), vp.to(DEV), g["landmarks"], table.to(DEV), g["seq_lens"], cfg.S, cfg.K,
                           workspace=ws)
    assert hils.poll_status(ws) == 0


def test_unsupported_shapes_are_refused_on_the_host():
    cfg = wl.CONFIGS[0].scaled(mode="decode", B=1, L=256, K=2, seed=84)      # fp32: generic kernels only
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor([256], dtype=torch.int32))
    kp, vp, table = paginate(inp, cfg, 8)
    g = {n: t.to(DEV) for n, t in inp.items()}
    with pytest.raises(hils.HilsError):
        hils.hils_decode_paged(g["q"], kp.to(DEV), vp.to(DEV), g["landmarks"], table.to(DEV), g["seq_lens"], cfg.S, cfg.K)
