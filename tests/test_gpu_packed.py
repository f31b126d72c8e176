"""Query-major packed prefill (impl="packed": tiles of 16 adjacent tokens over the union of their chunks, pair masking,
the mix kept in registers; Sec. 4.2 and App. "Chunk Overlap") against the oracle and against the chunk-major kernels."""
import numpy as np
import pytest
import torch

import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import workloads as wl
from parity import TOL_LSE, TOL_OUT, check_prefill

pytestmark = pytest.mark.gpu
DEV = "cuda"

CASES = {
    "gqa_bf16_2k": (wl.CONFIGS[1].scaled(L=2048), {}),
    # ragged: the last tile holds 8 tokens, the last chunk 40
    "ragged_b2": (wl.CONFIGS[1].scaled(B=2, Hq=8, Hkv=2, L=1000, K=8, seed=21), {}),
    # fewer candidates than K on many rows
    "k32_short": (wl.CONFIGS[1].scaled(Hq=8, Hkv=2, L=1500, K=32, seed=22), {}),
    # adjacent queries that share most of their chunks: the regime the packed tiles are meant for
    "structured_overlap": (wl.CONFIGS[1].scaled(L=4096, seed=23), {"overlap_block": 16}),
}


def run(cfg, inp, impl, bias=None, W=1):
    g = {k: v.to(DEV) for k, v in inp.items()}
    r = hils.hils_prefill(g["q"], g["k"], g["v"], g["landmarks"], cfg.S, cfg.K,
                          bias=None if bias is None else bias.to(DEV), window=W, impl=impl)
    torch.cuda.synchronize()
    return r


@pytest.mark.parametrize("name", list(CASES))
def test_packed_matches_the_oracle_and_the_chunk_major_kernels(name):
    cfg, kw = CASES[name]
    inp = wl.make_prefill_inputs(cfg, "cpu", **kw)
    out, lse, sel = run(cfg, inp, "packed")
    stats = check_prefill(cfg, inp, out, lse, sel)
    print(name, stats)
    out_f, lse_f, sel_f = run(cfg, inp, "fast")
    assert torch.equal(sel, sel_f)          # the same selection kernel
    assert (out.float() - out_f.float()).abs().max().item() <= TOL_OUT["bf16"]
    assert (lse - lse_f).abs().max().item() <= TOL_LSE["bf16"]


@pytest.mark.parametrize("W", [64, 65, 200, 512])
def test_packed_general_window_and_bias(W):
    """Local windows of several chunks: tokens of one tile start their windows in different chunks, and a chunk can be
    local for one token and selected by another."""
    cfg = wl.CONFIGS[1].scaled(Hq=8, Hkv=2, L=1800, K=8, seed=31)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    bias = wl.make_bias(cfg, "cpu")
    out, lse, sel = run(cfg, inp, "packed", bias=bias, W=W)
    print(W, check_prefill(cfg, inp, out, lse, sel, bias=bias, W=W))


def test_packed_slice_with_an_offset():
    """Queries 1024 .. 2047 of a 2048-token cache through the slice entry point."""
    cfg = wl.CONFIGS[1].scaled(Hq=8, Hkv=2, L=2048, K=8, seed=33)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    g = {k: v.to(DEV) for k, v in inp.items()}
    full = hils.hils_prefill(g["q"], g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, impl="packed")
    part = hils.hils_prefill_at(g["q"][:, :, 1024:].contiguous(), g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, 1024,
                                impl="packed")
    torch.cuda.synchronize()
    for a, b in zip(full, part):
        assert torch.equal(a[:, :, 1024:], b)


def test_packed_is_refused_where_it_does_not_apply():
    cfg = wl.CONFIGS[1].scaled(Hq=8, Hkv=2, L=512, K=64)
    inp = wl.make_prefill_inputs(cfg, DEV)
    with pytest.raises(Exception):
        hils.hils_prefill(inp["q"], inp["k"], inp["v"], inp["landmarks"], cfg.S, cfg.K, impl="packed")
    cfg = wl.CONFIGS[0]
    inp = wl.make_prefill_inputs(cfg, DEV)
    with pytest.raises(Exception):
        hils.hils_prefill(inp["q"], inp["k"], inp["v"], inp["landmarks"], cfg.S, cfg.K, impl="packed")
