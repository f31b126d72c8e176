"""GPU parity of hils_landmark_summary (Proposition 3.1, Eq. prop_q_c) against the CPU oracle, element by
element on seeded inputs: every instantiation (bf16 / fp32, d = 64 / 128 / 256, chunk sizes 32 / 64 / 128, one
or several landmark heads per KV head), ragged sequence lengths, a partial and an empty chunk, chunk ranges."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"
TOL_LM = {"f32": 2e-5, "bf16": 2e-2}     # bf16: one rounding of a value of magnitude <= 4
TOL_B = 2e-5                             # fp32 accumulation of <= 128 terms and the fast exp / log

CASES = {
    # name: (config, Hl, seq_lens)
    "bf16_d128_s64": (wl.CONFIGS[3].scaled(B=3, L=1024, seed=61), None, [1024, 1000, 130]),
    "bf16_per_query_head": (wl.CONFIGS[3].scaled(B=2, Hq=8, Hkv=2, L=512, seed=62), 8, [512, 77]),
    "f32_d64_s64": (wl.CONFIGS[0].scaled(mode="decode", B=2, L=640, seed=63), None, [640, 1]),
    "f32_d128": (wl.CONFIGS[0].scaled(mode="decode", B=2, Hq=2, Hkv=2, L=512, d=128, seed=64), None, [512, 300]),
    "bf16_d64_s32": (wl.CONFIGS[3].scaled(B=2, Hq=4, Hkv=2, L=512, d=64, S=32, seed=65), None, [512, 333]),
    "bf16_d128_s128": (wl.CONFIGS[3].scaled(B=2, Hq=4, Hkv=2, L=1024, S=128, seed=66), None, [1024, 700]),
    "bf16_d256": (wl.CONFIGS[3].scaled(B=1, Hq=2, Hkv=1, L=512, d=256, seed=67), None, [500]),
}


def inputs(cfg, Hl, seq):
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor(seq, dtype=torch.int32))
    lq = wl.make_landmark_queries(cfg, "cpu", Hl=Hl)
    return inp["k"], lq, torch.tensor(seq, dtype=torch.int32)


@pytest.mark.parametrize("name", list(CASES))
def test_landmark_summary_matches_oracle(name):
    cfg, Hl, seq = CASES[name]
    k, lq, sl = inputs(cfg, Hl, seq)
    lm, b = hils.hils_landmark_summary(lq.to(DEV), k.to(DEV), cfg.S, seq_lens=sl.to(DEV))
    torch.cuda.synchronize()
    assert hils.last_launch_count() == 1
    ref_lm, ref_b = oracle.hils_landmarks(lq, k, seq_lens=sl, S=cfg.S)
    err_lm = np.abs(lm.float().cpu().numpy().astype(np.float64) - ref_lm).max()
    err_b = np.abs(b.cpu().numpy().astype(np.float64) - ref_b).max()
    print(name, "max err landmarks %.3g bias %.3g" % (err_lm, err_b))
    assert err_lm <= TOL_LM[cfg.dtype]
    assert err_b <= TOL_B
    # chunks past the end of a sequence are exactly zero
    for bi, n in enumerate(seq):
        first_empty = (n + cfg.S - 1) // cfg.S
        assert (lm[bi, :, first_empty:] == 0).all() and (b[bi, :, first_empty:] == 0).all()


def test_without_seq_lens_every_sequence_is_full_and_a_chunk_range_leaves_the_rest_untouched():
    cfg = wl.CONFIGS[3].scaled(B=2, L=1024, seed=68)
    k, lq, _ = inputs(cfg, None, [1024, 1024])
    ref_lm, ref_b = oracle.hils_landmarks(lq, k, S=cfg.S)
    lm = torch.full((cfg.B, cfg.Hkv, cfg.C, cfg.d), 7.0, dtype=torch.bfloat16, device=DEV)
    b = torch.full((cfg.B, cfg.Hkv, cfg.C), 7.0, dtype=torch.float32, device=DEV)
    hils.hils_landmark_summary(lq.to(DEV), k.to(DEV), cfg.S, chunk_begin=5, chunk_count=3, landmarks=lm, bias=b)
    torch.cuda.synchronize()
    got_lm, got_b = lm.float().cpu().numpy(), b.cpu().numpy()
    assert np.abs(got_lm[:, :, 5:8] - ref_lm[:, :, 5:8]).max() <= TOL_LM["bf16"]
    assert np.abs(got_b[:, :, 5:8] - ref_b[:, :, 5:8]).max() <= TOL_B
    assert (got_lm[:, :, :5] == 7).all() and (got_lm[:, :, 8:] == 7).all()
    assert (got_b[:, :, :5] == 7).all() and (got_b[:, :, 8:] == 7).all()
    # chunk_count <= 0: from chunk_begin to the last chunk
    hils.hils_landmark_summary(lq.to(DEV), k.to(DEV), cfg.S, chunk_begin=8, landmarks=lm, bias=b)
    torch.cuda.synchronize()
    assert np.abs(lm.float().cpu().numpy()[:, :, 8:] - ref_lm[:, :, 8:]).max() <= TOL_LM["bf16"]
    assert (lm.float().cpu().numpy()[:, :, :5] == 7).all()


def test_summaries_feed_the_operator():
    """landmarks / bias produced on the GPU, then hils_decode on them: the whole chain against the oracle chain."""
    cfg = wl.CONFIGS[3].scaled(B=2, L=2048, K=8, seed=69)
    seq = [2048, 1500]
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor(seq, dtype=torch.int32))
    lq = wl.make_landmark_queries(cfg, "cpu")
    g = {n: t.to(DEV) for n, t in inp.items()}
    lm, b = hils.hils_landmark_summary(lq.to(DEV), g["k"], cfg.S, seq_lens=g["seq_lens"])
    out, lse, sel = hils.hils_decode(g["q"], g["k"], g["v"], lm, g["seq_lens"], cfg.S, cfg.K, bias=b)
    torch.cuda.synchronize()
    # the oracle attends with the GPU's summaries (bf16 landmarks: the same inputs on both sides)
    res = oracle.hils_decode(inp["q"], inp["k"], inp["v"], lm.cpu(), b.cpu(), inp["seq_lens"], S=cfg.S, K=cfg.K)
    ok = res["margin"].min(axis=-1) >= 1e-3 if res["margin"].ndim > 1 else res["margin"] >= 1e-3
    got_sel = sel.cpu().numpy()
    for bi in range(cfg.B):
        for gk in range(cfg.Hkv):
            if res["margin"].reshape(cfg.B, cfg.Hkv)[bi, gk] >= 1e-3:
                assert (got_sel[bi, gk] == res["sel_idx"].reshape(cfg.B, cfg.Hkv, cfg.K)[bi, gk]).all()
    err = np.abs(out.float().cpu().numpy() - res["out"].reshape(out.shape)).max()
    assert err <= 2e-2


def test_argument_errors():
    cfg = wl.CONFIGS[3].scaled(B=1, L=256, seed=70)
    k, lq, _ = inputs(cfg, None, [256])
    with pytest.raises(hils.HilsError):
        hils.hils_landmark_summary(lq.to(DEV), k.to(DEV), cfg.S, chunk_begin=3, chunk_count=9)    # beyond C = 4
    with pytest.raises(hils.HilsError):
        hils.hils_landmark_summary(lq.to(DEV), k.to(DEV), 200)                                    # chunk size > 128
