"""The operators with a separate routing query q-hat (Eq. Q-Cal): q-hat replaces q in the surrogate scores
(selection and fusion weights) and nowhere else.  Both kernel sets against the oracle; q-hat = q must give the
plain entry points' results bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import workloads as wl
from parity import TOL_OUT, TOL_LSE

pytestmark = pytest.mark.gpu
DEV = "cuda"


def route_like(q, seed):
    g = torch.Generator().manual_seed(seed)
    return (q.float() + 0.8 * torch.randn(q.shape, generator=g)).to(q.dtype)


def compare(res, out, lse, sel, dtype, row_major):
    """res: oracle dict with leading [B, n] (prefill) or [B] (decode) axes."""
    o, l, s = out.float().cpu().numpy(), lse.cpu().numpy(), sel.cpu().numpy()
    if row_major:                                   # prefill: oracle [B, L, H, ...], GPU [B, H, L, ...]
        o, l, s = o.transpose(0, 2, 1, 3), l.transpose(0, 2, 1), s.transpose(0, 2, 1, 3)
    ok = res["margin"] >= 1e-3
    assert ok.mean() > 0.9
    assert (s[ok] == res["sel_idx"][ok]).all()
    rows_ok = ok.all(axis=-1)
    assert np.abs(o - res["out"])[rows_ok].max() <= TOL_OUT[dtype]
    assert np.abs(l - res["lse"])[rows_ok].max() <= TOL_LSE[dtype]


@pytest.mark.parametrize("impl", ["generic", "fast"])
@pytest.mark.parametrize("W", [1, 200])
def test_prefill_with_a_routing_query(impl, W):
    cfg = wl.CONFIGS[1].scaled(B=2, Hq=8, Hkv=2, L=4300, K=12, seed=95)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    bias = wl.make_bias(cfg, "cpu")
    qr = route_like(inp["q"], 3)
    g = {n: t.to(DEV) for n, t in inp.items()}
    out, lse, sel = hils.hils_prefill(g["q"], g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, bias=bias.to(DEV), window=W,
                                      impl=impl, q_route=qr.to(DEV))
    torch.cuda.synchronize()
    rows = wl.sample_rows(cfg, 600).numpy()
    res = oracle.hils_prefill(inp["q"], inp["k"], inp["v"], inp["landmarks"], bias, S=cfg.S, K=cfg.K, W=W, rows=rows,
                              q_route=qr)
    r = torch.as_tensor(rows)
    compare(res, out.cpu()[:, :, r], lse.cpu()[:, :, r], sel.cpu()[:, :, r], cfg.dtype, True)
    # q-hat = q: exactly the plain entry point
    a = hils.hils_prefill(g["q"], g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, bias=bias.to(DEV), window=W, impl=impl)
    b = hils.hils_prefill(g["q"], g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, bias=bias.to(DEV), window=W, impl=impl,
                          q_route=g["q"])
    torch.cuda.synchronize()
    assert torch.equal(a[2], b[2])
    assert (a[0].float() - b[0].float()).abs().max() <= 1.6e-2 and (a[1] - b[1]).abs().max() <= 1e-3


@pytest.mark.parametrize("impl", ["generic", "fast"])
def test_decode_with_a_routing_query(impl):
    cfg = wl.CONFIGS[3].scaled(B=6, L=4096, K=8, seed=96)
    seq = [4096, 4095, 1, 63, 2049, 640]
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor(seq, dtype=torch.int32))
    bias = wl.make_bias(cfg, "cpu")
    qr = route_like(inp["q"], 4)
    g = {n: t.to(DEV) for n, t in inp.items()}
    out, lse, sel = hils.hils_decode(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K,
                                     bias=bias.to(DEV), impl=impl, q_route=qr.to(DEV))
    torch.cuda.synchronize()
    res = oracle.hils_decode(inp["q"], inp["k"], inp["v"], inp["landmarks"], bias, inp["seq_lens"], S=cfg.S, K=cfg.K,
                             q_route=qr)
    compare(res, out, lse, sel, cfg.dtype, False)
    a = hils.hils_decode(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K, bias=bias.to(DEV), impl=impl)
    b = hils.hils_decode(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K, bias=bias.to(DEV), impl=impl,
                         q_route=g["q"])
    torch.cuda.synchronize()
    assert torch.equal(a[2], b[2]) and torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
