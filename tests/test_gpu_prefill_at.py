"""hils_prefill_at: the operator for a slice of query tokens at positions pos0 .. pos0 + L - 1 of a longer cache
(chunked prefill, multi-token decode).  Row r must equal position pos0 + r of the whole-sequence operator: checked
against the CPU oracle row by row, and against hils_prefill on the same sequence."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import workloads as wl
from parity import TOL_OUT, TOL_LSE

pytestmark = pytest.mark.gpu
DEV = "cuda"


def oracle_rows(cfg, inp, pos0, L, bias, W):
    rows = np.arange(L)
    res = []
    for b in range(cfg.B):
        one = {n: t[b:b + 1] for n, t in inp.items()}
        bb = None if bias is None else bias[b:b + 1]
        res.append(oracle.hils_rows(one["q"][:, :, pos0:pos0 + L], one["k"], one["v"], one["landmarks"], bb, S=cfg.S,
                                    K=cfg.K, W=W, row_b=np.zeros(L, np.int32), row_qi=rows.astype(np.int32),
                                    row_pos=(pos0 + rows).astype(np.int64)))
    return res


def compare(cfg, inp, pos0, L, got, bias, W):
    out, lse, sel = (t.float().cpu().numpy() if t.dtype != torch.int32 else t.cpu().numpy() for t in got)
    for b, r in enumerate(oracle_rows(cfg, inp, pos0, L, bias, W)):
        ok = r["margin"].min(axis=1) >= 1e-3                        # rows whose selection is unambiguous
        assert ok.mean() > 0.9
        exp_sel = r["sel_idx"]                                      # [L, Hkv, K]
        assert (sel[b].transpose(1, 0, 2)[ok] == exp_sel[ok]).all()
        err = np.abs(out[b].transpose(1, 0, 2) - r["out"])[ok].max()
        err_l = np.abs(lse[b].transpose(1, 0) - r["lse"])[ok].max()
        assert err <= TOL_OUT[cfg.dtype] and err_l <= TOL_LSE[cfg.dtype], (err, err_l)


@pytest.mark.parametrize("impl", ["generic", "fast"])
@pytest.mark.parametrize("pos0,L,W", [(3000, 1300, 1), (4097, 200, 512), (2048, 4200, 65), (4299, 1, 1)])
def test_slice_of_a_sequence_matches_the_oracle(impl, pos0, L, W):
    cfg = wl.CONFIGS[1].scaled(B=2, Hq=8, Hkv=2, L=pos0 + L + 77, K=12, seed=91)       # the cache is longer than needed
    inp = wl.make_prefill_inputs(cfg, "cpu")
    bias = wl.make_bias(cfg, "cpu")
    g = {n: t.to(DEV) for n, t in inp.items()}
    q = g["q"][:, :, pos0:pos0 + L].contiguous()
    got = hils.hils_prefill_at(q, g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, pos0, bias=bias.to(DEV), window=W,
                               impl=impl)
    torch.cuda.synchronize()
    compare(cfg, inp, pos0, L, got, bias, W)


@pytest.mark.parametrize("pos0,L,W", [(0, 3100, 200), (2049, 1500, 512), (1000, 900, 1)])
def test_more_than_32_chunks_per_query_with_window_and_offset_on_the_fast_path(pos0, L, W):
    """top_k between 33 and 64 takes the warp-MMA selection kernel: any window, any slice offset."""
    cfg = wl.CONFIGS[1].scaled(B=1, Hq=8, Hkv=2, L=pos0 + L, K=40, seed=95)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    bias = wl.make_bias(cfg, "cpu")
    g = {n: t.to(DEV) for n, t in inp.items()}
    q = g["q"][:, :, pos0:pos0 + L].contiguous()
    got = hils.hils_prefill_at(q, g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, pos0, bias=bias.to(DEV), window=W,
                               impl="fast")
    torch.cuda.synchronize()
    compare(cfg, inp, pos0, L, got, bias, W)


def test_two_slices_reproduce_the_whole_sequence_prefill_bit_for_bit():
    cfg = wl.CONFIGS[1].scaled(B=1, Hq=8, Hkv=2, L=6000, K=12, seed=92)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    g = {n: t.to(DEV) for n, t in inp.items()}
    out, lse, sel = hils.hils_prefill(g["q"], g["k"], g["v"], g["landmarks"], cfg.S, cfg.K)
    cut = 2500
    for pos0, L in ((0, cut), (cut, cfg.L - cut)):
        o, l, s = hils.hils_prefill_at(g["q"][:, :, pos0:pos0 + L].contiguous(), g["k"], g["v"], g["landmarks"],
                                       cfg.S, cfg.K, pos0)
        torch.cuda.synchronize()
        assert torch.equal(s, sel[:, :, pos0:pos0 + L])
        assert torch.equal(o, out[:, :, pos0:pos0 + L]) and torch.equal(l, lse[:, :, pos0:pos0 + L])


def test_multi_token_decode_equals_single_token_decode():
    """M = 4 new tokens at once (speculative decoding) against four single-token hils_decode calls."""
    cfg = wl.CONFIGS[3].scaled(B=2, L=4096, K=8, seed=93)
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor([4096, 4096], dtype=torch.int32))
    g = {n: t.to(DEV) for n, t in inp.items()}
    M, T = 4, 4096
    qs = torch.randn((cfg.B, cfg.Hq, M, cfg.d), generator=torch.Generator().manual_seed(1)).to(torch.bfloat16).to(DEV)
    o, l, s = hils.hils_prefill_at(qs, g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, T - M)
    for m in range(M):
        sl = torch.full((cfg.B,), T - M + m + 1, dtype=torch.int32, device=DEV)
        od, ld, sd = hils.hils_decode(qs[:, :, m].contiguous(), g["k"], g["v"], g["landmarks"], sl, cfg.S, cfg.K)
        torch.cuda.synchronize()
        assert torch.equal(sd, s[:, :, m])
        assert (od.float() - o[:, :, m].float()).abs().max() <= 1.6e-2          # two kernel sets, bf16 outputs
        assert (ld - l[:, :, m]).abs().max() <= 1e-3


def test_bad_offsets_are_refused():
    cfg = wl.CONFIGS[1].scaled(B=1, Hq=8, Hkv=2, L=1024, K=4, seed=94)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    g = {n: t.to(DEV) for n, t in inp.items()}
    with pytest.raises(hils.HilsError):
        hils.hils_prefill_at(g["q"][:, :, :600].contiguous(), g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, 500)
    with pytest.raises(hils.HilsError):
        hils.hils_prefill_at(g["q"][:, :, :10].contiguous(), g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, -1)
