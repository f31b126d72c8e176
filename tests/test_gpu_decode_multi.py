"""hils_decode_multi (M new tokens per sequence in one call, the decode kernels over shared caches) against M
single-token hils_decode calls (same selection; outputs to one bf16 rounding: the partial sums of a query are split
over CTAs by its index in the call, so the order of the additions differs) and against the CPU oracle row by row."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import workloads as wl
from parity import TOL_OUT, TOL_LSE

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make(cfg, seq, M, seed):
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor(seq, dtype=torch.int32))
    q = torch.randn((cfg.B, M, cfg.Hq, cfg.d), generator=torch.Generator().manual_seed(seed)).to(torch.bfloat16)
    return inp, q


@pytest.mark.parametrize("M,W", [(4, 1), (3, 200), (1, 1)])
def test_multi_token_decode_equals_single_token_calls_and_the_oracle(M, W):
    cfg = wl.CONFIGS[3].scaled(B=3, L=4096, K=8, seed=301)
    seq = [4096, 2049, 1000]
    inp, q = make(cfg, seq, M, 11)
    bias = wl.make_bias(cfg, "cpu")
    g = {n: t.to(DEV) for n, t in inp.items()}
    out, lse, sel = hils.hils_decode_multi(q.to(DEV), g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K,
                                           bias=bias.to(DEV), window=W)
    torch.cuda.synchronize()
    assert hils.last_launch_count() == 3
    for m in range(M):
        sl = torch.tensor([n - M + m + 1 for n in seq], dtype=torch.int32)
        o1, l1, s1 = hils.hils_decode(q[:, m].contiguous().to(DEV), g["k"], g["v"], g["landmarks"], sl.to(DEV), cfg.S,
                                      cfg.K, bias=bias.to(DEV), window=W)
        torch.cuda.synchronize()
        assert torch.equal(s1, sel[:, m])
        assert (o1.float() - out[:, m].float()).abs().max() <= 1.6e-2 and (l1 - lse[:, m]).abs().max() <= 1e-4
        ref = oracle.hils_decode(q[:, m], inp["k"], inp["v"], inp["landmarks"], bias, sl, S=cfg.S, K=cfg.K, W=W)
        ok = ref["margin"] >= 1e-3                                   # [B, Hkv]
        assert (sel[:, m].cpu().numpy()[ok] == ref["sel_idx"][ok]).all()
        okh = np.repeat(ok, cfg.G, axis=1)                           # per query head
        assert np.abs(out[:, m].float().cpu().numpy() - ref["out"])[okh].max() <= TOL_OUT["bf16"]
        assert np.abs(lse[:, m].cpu().numpy() - ref["lse"])[okh].max() <= TOL_LSE["bf16"]


def test_multi_token_decode_over_paged_caches():
    from test_gpu_paged import paginate
    cfg = wl.CONFIGS[3].scaled(B=4, L=2048, K=8, seed=302)
    seq = [2048, 1500, 700, 65]
    M = 4
    inp, q = make(cfg, seq, M, 12)
    kp, vp, table = paginate(inp, cfg, 9)
    g = {n: t.to(DEV) for n, t in inp.items()}
    a = hils.hils_decode_multi(q.to(DEV), g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K)
    b = hils.hils_decode_multi(q.to(DEV), kp.to(DEV), vp.to(DEV), g["landmarks"], g["seq_lens"], cfg.S, cfg.K,
                               block_table=table.to(DEV))
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)                                     # same call shape: paging only changes addresses


def test_sequence_shorter_than_the_token_count_sets_the_status():
    cfg = wl.CONFIGS[3].scaled(B=2, L=1024, K=4, seed=303)
    inp, q = make(cfg, [1024, 2], 4, 13)                             # sequence 1 holds 2 tokens, 4 are asked for
    g = {n: t.to(DEV) for n, t in inp.items()}
    p = hils.make_params(B=2, Hq=cfg.Hq, Hkv=cfg.Hkv, Hl=cfg.Hkv, L=0, T_max=cfg.L, C=cfg.C, d=cfg.d,
                         chunk_size=cfg.S, top_k=cfg.K, dtype=1, impl="auto")
    n = hils.load_library().hils_decode_multi_workspace_bytes(__import__("ctypes").byref(p), 4)
    ws = torch.zeros(n, dtype=torch.uint8, device=DEV)
    out, lse, sel = hils.hils_decode_multi(q.to(DEV), g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K,
                                           workspace=ws)
    torch.cuda.synchronize()
    assert hils.poll_status(ws) == -7
    assert (out[1, :2] == 0).all() and (sel[1, :2] == -1).all()      # the two tokens at negative positions
    assert torch.isfinite(out.float()).all()


def test_generic_shapes_are_refused():
    cfg = wl.CONFIGS[0].scaled(mode="decode", B=1, L=256, K=2, seed=304)     # fp32
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor([256], dtype=torch.int32))
    g = {n: t.to(DEV) for n, t in inp.items()}
    q = torch.randn((1, 2, cfg.Hq, cfg.d), device=DEV)
    with pytest.raises(hils.HilsError):
        hils.hils_decode_multi(q, g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K)
