"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element on
seeded inputs.  Small cases span several tiles and ragged tails; the full-size configurations are
checked on sampled rows / sequences in the launch configuration the benchmark times."""
import numpy as np
import pytest
import torch

import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import workloads as wl
from parity import check_decode, check_prefill

pytestmark = pytest.mark.gpu
DEV = "cuda"


def to_dev(d):
    return {k: v.to(DEV) for k, v in d.items()}


def run_prefill(cfg, inp, impl, bias=None, W=1):
    g = to_dev(inp)
    out, lse, sel = hils.hils_prefill(g["q"], g["k"], g["v"], g["landmarks"], cfg.S, cfg.K,
                                      bias=None if bias is None else bias.to(DEV), window=W, impl=impl)
    torch.cuda.synchronize()
    return out, lse, sel


def run_decode(cfg, inp, impl, bias=None, W=1):
    g = to_dev(inp)
    ws_out = hils.hils_decode(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K,
                              bias=None if bias is None else bias.to(DEV), window=W, impl=impl)
    torch.cuda.synchronize()
    return ws_out


def fast_or_skip(cfg, mode_decode, W=1, Hl=None):
    p = hils.make_params(B=cfg.B, Hq=cfg.Hq, Hkv=cfg.Hkv, Hl=cfg.Hkv if Hl is None else Hl,
                         L=0 if mode_decode else cfg.L, T_max=cfg.L, C=cfg.C, d=cfg.d, chunk_size=cfg.S,
                         top_k=cfg.K, window=W, dtype=0 if cfg.dtype == "f32" else 1, impl="fast")
    if hils.workspace_bytes(p, mode_decode) == 0:
        pytest.skip("no fast kernel set for this shape")


PREFILL_SMALL = {
    "cfg0_tiny_f32": wl.CONFIGS[0],
    "gqa_bf16_2k": wl.CONFIGS[1].scaled(L=2048),
    "gqa_bf16_ragged_b2": wl.CONFIGS[1].scaled(B=2, Hq=8, Hkv=2, L=1000, K=8, seed=21),
    "bf16_k_ge_chunks": wl.CONFIGS[1].scaled(Hq=8, Hkv=2, L=640, K=64, seed=22),
    "bf16_d64_g2_s32": wl.CONFIGS[1].scaled(Hq=4, Hkv=2, L=777, d=64, S=32, K=5, seed=23),
    "f32_g4_k33": wl.CONFIGS[0].scaled(Hq=4, Hkv=1, L=2500, d=128, K=33, seed=24, n_needles=2),
    # longer than one 4096-token query block of the fast path, ragged end, K between 32 and 64
    "bf16_multiblock_k40": wl.CONFIGS[1].scaled(Hq=4, Hkv=1, L=8300, K=40, seed=26),
    "bf16_multiblock_b2": wl.CONFIGS[1].scaled(B=2, Hq=8, Hkv=2, L=4200, K=12, seed=27),
}


@pytest.mark.parametrize("impl", ["generic", "fast"])
@pytest.mark.parametrize("name", list(PREFILL_SMALL))
def test_prefill_small(name, impl):
    cfg = PREFILL_SMALL[name]
    if impl == "fast":
        fast_or_skip(cfg, False)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    out, lse, sel = run_prefill(cfg, inp, impl)
    stats = check_prefill(cfg, inp, out, lse, sel)
    print(name, impl, stats)


@pytest.mark.parametrize("impl", ["generic", "fast"])
def test_prefill_window_bias_and_per_head_landmarks(impl):
    """General local window W, entropy-like bias, and one landmark per query head (App. C)."""
    cfg = wl.CONFIGS[0].scaled(Hq=4, Hkv=2, L=600, d=32, S=16, K=5, seed=31)
    if impl == "fast":
        fast_or_skip(cfg, False, W=100, Hl=cfg.Hq)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    g = torch.Generator().manual_seed(5)
    inp["landmarks"] = torch.randn((1, cfg.Hq, cfg.C, cfg.d), generator=g) * 0.5
    bias = torch.rand((1, cfg.Hq, cfg.C), generator=g) * float(np.log(cfg.S))
    out, lse, sel = run_prefill(cfg, inp, impl, bias=bias, W=100)
    check_prefill(cfg, inp, out, lse, sel, bias=bias, W=100)


@pytest.mark.parametrize("W", [2, 64, 65, 200, 512])
def test_prefill_fast_path_with_a_chunk_aligned_local_window(W):
    """The paper's operator form on the tensor-core path: local window W > 1 (Sec. 2.1; the experiments use
    W = 512), a non-null bias, several query blocks; every chunk of the window is a slot of its own."""
    cfg = wl.CONFIGS[1].scaled(B=2, Hq=8, Hkv=2, L=4300, K=12, seed=35)
    fast_or_skip(cfg, False, W=W)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    bias = wl.make_bias(cfg, "cpu")
    out, lse, sel = run_prefill(cfg, inp, "fast", bias=bias, W=W)
    check_prefill(cfg, inp, out, lse, sel, bias=bias, W=W)


@pytest.mark.parametrize("W", [1, 200])
def test_prefill_fast_path_with_one_landmark_per_query_head(W):
    """App. C on the tensor-core path: every query head scores its own landmark row and adds its own bias; the
    group score is the maximum over the heads; the fusion weight of a row uses its own head's score."""
    cfg = wl.CONFIGS[1].scaled(B=2, Hq=8, Hkv=2, L=4300, K=12, seed=36)
    fast_or_skip(cfg, False, W=W, Hl=cfg.Hq)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    g = torch.Generator().manual_seed(11)
    inp["landmarks"] = (torch.randn((cfg.B, cfg.Hq, cfg.C, cfg.d), generator=g) * 0.7).to(torch.bfloat16)
    bias = torch.rand((cfg.B, cfg.Hq, cfg.C), generator=g) * float(np.log(cfg.S))
    out, lse, sel = run_prefill(cfg, inp, "fast", bias=bias, W=W)
    check_prefill(cfg, inp, out, lse, sel, bias=bias, W=W)


@pytest.mark.parametrize("impl", ["generic", "fast"])
def test_prefill_bias_only(impl):
    cfg = wl.CONFIGS[1].scaled(L=1536, K=6, seed=32)
    if impl == "fast":
        fast_or_skip(cfg, False)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    bias = wl.make_bias(cfg, "cpu")
    out, lse, sel = run_prefill(cfg, inp, impl, bias=bias)
    check_prefill(cfg, inp, out, lse, sel, bias=bias)


def test_prefill_ties_go_to_lower_chunk_and_runs_are_deterministic():
    cfg = wl.CONFIGS[1].scaled(Hq=8, Hkv=2, L=1024, K=3, seed=33, n_needles=0)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    inp["q"].zero_()                                   # every score equals 0: ties everywhere
    for impl in ("generic", "auto"):
        out, lse, sel = run_prefill(cfg, inp, impl)
        s = sel.cpu().numpy()
        for i in (64 * 3, 64 * 7 + 5, 1023):
            assert (s[0, :, i] == np.array([0, 1, 2])).all()
        out2, lse2, sel2 = run_prefill(cfg, inp, impl)
        assert torch.equal(sel, sel2)
    inp = wl.make_prefill_inputs(cfg.scaled(n_needles=2), "cpu")
    a = run_prefill(cfg, inp, "auto")
    b = run_prefill(cfg, inp, "auto")
    assert torch.equal(a[2], b[2])
    assert (a[0].float() - b[0].float()).abs().max() <= 1e-2


@pytest.mark.parametrize("K", [8, 24])
def test_prefill_two_level_scores_cut_through_the_crowded_level(K):
    """Two-valued group scores in prefill: a few chunks on the upper level, every other chunk tied on the lower
    one, so the exact tie rule (lower chunk id) decides most of the selection, for tokens early and late in a
    long sequence (the late ones go through several compactions of the running top-K)."""
    cfg = wl.CONFIGS[1].scaled(Hq=8, Hkv=2, L=8192, K=K, seed=34, n_needles=0)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    upper = [5 + 9 * j for j in range(6)]                       # chunks 5, 14, ..., 50
    lm = torch.zeros_like(inp["landmarks"])
    lm[:, :, upper, 0] = 4.0
    q = torch.zeros_like(inp["q"])
    q[..., 0] = 4.0
    case = dict(inp, landmarks=lm, q=q)
    for impl in ("generic", "auto"):
        _, _, sel = run_prefill(cfg, case, impl)
        got = sel.cpu().numpy()
        for i in (63, 64 * 4 + 1, 64 * 30, 64 * 51 + 7, 64 * 100, 8191):
            ncand = i // cfg.S                                  # W = 1: the chunks before the token's own
            hi = [c for c in upper if c < ncand]
            lo = [c for c in range(ncand) if c not in upper]
            exp = sorted(hi[:K] + lo[:max(0, K - len(hi))])
            exp = exp + [-1] * (K - len(exp))
            for g in range(cfg.Hkv):
                assert got[0, g, i].tolist() == exp, (impl, K, i, g)


DECODE_SMALL = {
    "bf16_ragged": (wl.CONFIGS[3].scaled(B=6, L=4096, K=8, seed=41), [4096, 4095, 1, 63, 2049, 640]),
    "bf16_k_ge_chunks": (wl.CONFIGS[3].scaled(B=3, L=2048, K=64, seed=42), [2048, 1000, 65]),
    "bf16_cfg4_like": (wl.CONFIGS[4].scaled(B=2, L=32768, K=64, seed=43), [32768, 32700]),
    "f32_g1_d64": (wl.CONFIGS[0].scaled(mode="decode", B=4, L=1024, K=4, seed=44), [1024, 1, 64, 500]),
    # long candidate lists whose length is 1 / 0 / 15 past a multiple of 16
    "bf16_long_candidate_lists": (wl.CONFIGS[3].scaled(B=3, L=65536, K=8, seed=50), [65536, 64 * 640 + 5, 64 * 625 + 64]),
    # many (sequence, KV head) pairs: every persistent CTA walks several pairs and wraps its TMA ring
    "bf16_many_pairs": (wl.CONFIGS[3].scaled(B=64, L=2048, K=16, seed=49),
                        [2048 - 37 * (i % 11) - (1 if i % 3 == 0 else 0) for i in range(64)]),
}


@pytest.mark.parametrize("impl", ["generic", "fast"])
@pytest.mark.parametrize("name", list(DECODE_SMALL))
def test_decode_small(name, impl):
    cfg, seq = DECODE_SMALL[name]
    if impl == "fast":
        fast_or_skip(cfg, True)
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor(seq, dtype=torch.int32))
    out, lse, sel = run_decode(cfg, inp, impl)
    stats = check_decode(cfg, inp, out, lse, sel)
    print(name, impl, stats)


@pytest.mark.parametrize("impl", ["generic", "fast"])
def test_decode_with_bias(impl):
    cfg = wl.CONFIGS[3].scaled(B=3, L=8192, K=16, seed=45)
    if impl == "fast":
        fast_or_skip(cfg, True)
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor([8192, 8000, 4097], dtype=torch.int32))
    bias = wl.make_bias(cfg, "cpu")
    out, lse, sel = run_decode(cfg, inp, impl, bias=bias)
    check_decode(cfg, inp, out, lse, sel, bias=bias)


def test_decode_selection_reaches_the_last_candidates_of_long_lists():
    """Long candidate lists with a bias that forces the very last candidate chunk and the one 16 before it into
    the selection (the ends of the warps' slices of the list)."""
    cfg = wl.CONFIGS[3].scaled(B=2, L=65536, K=8, seed=51)
    fast_or_skip(cfg, True)
    seq = [64 * 641 + 3, 64 * 655 + 64]                 # 641 and 655 candidate chunks
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor(seq, dtype=torch.int32))
    bias = torch.zeros((cfg.B, cfg.Hkv, cfg.C), dtype=torch.float32)
    for b, n in enumerate(seq):
        ncand = (n - 1) // cfg.S
        bias[b, :, ncand - 1] = 50.0
        bias[b, :, ncand - 17] = 50.0
    out, lse, sel = run_decode(cfg, inp, "fast", bias=bias)
    got = sel.cpu().numpy()
    for b, n in enumerate(seq):
        ncand = (n - 1) // cfg.S
        assert (got[b] == ncand - 1).any(axis=-1).all() and (got[b] == ncand - 17).any(axis=-1).all()
        assert (got[b] < ncand).all()
    check_decode(cfg, inp, out, lse, sel, bias=bias)


@pytest.mark.parametrize("L", [8192, 64 * 3000, 64 * 5000])      # 127 / 2999 / 4999 candidate chunks
def test_decode_ties_and_clustered_scores_pick_the_lower_chunk_ids(L):
    """Equal and two-valued group scores: the exact tie rule decides the whole selection (Eq. surrogate
    top-k with ties to the lower chunk id); both kernel sets must return exactly the expected ids."""
    cfg = wl.CONFIGS[3].scaled(B=1, Hq=8, Hkv=2, L=L, K=24, seed=47, n_needles=0)
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor([L], dtype=torch.int32))
    ncand = (L - 1) // cfg.S
    # (a) all scores equal
    inp_a = dict(inp)
    inp_a["q"] = torch.zeros_like(inp["q"])
    # (b) two score levels: chunks with c % 5 == 2 score 16, the rest 0
    lm = torch.zeros_like(inp["landmarks"])
    lm[:, :, 2::5, 0] = 4.0
    q = torch.zeros_like(inp["q"])
    q[..., 0] = 4.0
    inp_b = dict(inp, landmarks=lm, q=q)
    hi = [c for c in range(ncand) if c % 5 == 2]
    lo = [c for c in range(ncand) if c % 5 != 2]
    exp_b = sorted(hi[:cfg.K] + lo[:max(0, cfg.K - len(hi))])
    # (c) as (b) but only 10 chunks on the upper level: the cut runs through the crowded lower level
    lm_c = torch.zeros_like(inp["landmarks"])
    top10 = [7 + 11 * j for j in range(10)]
    lm_c[:, :, top10, 0] = 4.0
    inp_c = dict(inp, landmarks=lm_c, q=q)
    rest = [c for c in range(ncand) if c not in top10]
    exp_c = sorted(top10 + rest[:cfg.K - 10])
    for impl in ("generic", "fast"):
        for case, expect in ((inp_a, list(range(cfg.K))), (inp_b, exp_b), (inp_c, exp_c)):
            _, _, sel = run_decode(cfg, case, impl)
            got = sel.cpu().numpy()
            for g in range(cfg.Hkv):
                assert got[0, g].tolist() == expect, (impl, L, g)


@pytest.mark.parametrize("W", [2, 64, 65, 200, 512])
def test_decode_fast_path_with_a_chunk_aligned_local_window(W):
    """The paper's operator form in decode: local window W > 1 (the experiments use W = 512) and a bias; the
    chunks of the window are extra slots of the persistent attend kernel, mixed by their exact masses."""
    cfg = wl.CONFIGS[3].scaled(B=6, L=4096, K=8, seed=48)
    fast_or_skip(cfg, True, W=W)
    seq = [4096, 4095, 1, 63, 2049, 640]
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor(seq, dtype=torch.int32))
    bias = wl.make_bias(cfg, "cpu")
    out, lse, sel = run_decode(cfg, inp, "fast", bias=bias, W=W)
    check_decode(cfg, inp, out, lse, sel, bias=bias, W=W)


@pytest.mark.parametrize("W", [1, 200])
def test_decode_fast_path_with_one_landmark_per_query_head(W):
    """App. C: in GQA the chunk summary has one row per query head (k'_c in R^{G x d}); every head scores its own
    landmark, the group score is still the maximum over the heads."""
    cfg = wl.CONFIGS[3].scaled(B=4, L=4096, K=8, seed=52)
    fast_or_skip(cfg, True, W=W, Hl=cfg.Hq)
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor([4096, 3000, 130, 65], dtype=torch.int32))
    g = torch.Generator().manual_seed(9)
    inp["landmarks"] = (torch.randn((cfg.B, cfg.Hq, cfg.C, cfg.d), generator=g) * 0.7).to(torch.bfloat16)
    bias = torch.rand((cfg.B, cfg.Hq, cfg.C), generator=g) * float(np.log(cfg.S))
    out, lse, sel = run_decode(cfg, inp, "fast", bias=bias, W=W)
    check_decode(cfg, inp, out, lse, sel, bias=bias, W=W)


def test_decode_invalid_seq_len_sets_status_without_fault():
    cfg = wl.CONFIGS[3].scaled(B=2, L=1024, K=4, seed=46)
    inp = wl.make_decode_inputs(cfg, "cpu", seq_lens=torch.tensor([1024, 512], dtype=torch.int32))
    g = to_dev(inp)
    g["seq_lens"] = torch.tensor([1024, 0], dtype=torch.int32, device=DEV)
    p = hils.make_params(B=2, Hq=cfg.Hq, Hkv=cfg.Hkv, Hl=cfg.Hkv, L=0, T_max=cfg.L, C=cfg.C, d=cfg.d,
                         chunk_size=cfg.S, top_k=cfg.K, dtype=1, impl="auto")
    ws = hils.alloc_workspace(p, True, DEV)
    out, lse, sel = hils.hils_decode(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K, workspace=ws)
    assert hils.poll_status(ws) == -7
    assert (sel[1] == -1).all()
    ws[:256].zero_()
    g["seq_lens"][1] = 512
    hils.hils_decode(g["q"], g["k"], g["v"], g["landmarks"], g["seq_lens"], cfg.S, cfg.K, workspace=ws)
    assert hils.poll_status(ws) == 0


def test_host_entry_points_match_device_entry_points():
    cfg = wl.CONFIGS[1].scaled(L=1024, K=4, seed=47)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    out, lse, sel = run_prefill(cfg, inp, "auto")
    p = hils.make_params(B=cfg.B, Hq=cfg.Hq, Hkv=cfg.Hkv, Hl=cfg.Hkv, L=cfg.L, T_max=cfg.L, C=cfg.C, d=cfg.d,
                         chunk_size=cfg.S, top_k=cfg.K, dtype=1, impl="auto")
    runner = hils.HostRunner(p, False, DEV)
    pinned = {k: v.pin_memory() for k, v in inp.items()}
    ho, hl, hs = runner.run(pinned["q"], pinned["k"], pinned["v"], pinned["landmarks"])
    torch.cuda.synchronize()
    assert torch.equal(hs, sel.cpu())
    assert (ho.float() - out.cpu().float()).abs().max() <= 1e-2
    dcfg = wl.CONFIGS[3].scaled(B=2, L=2048, K=4, seed=48)
    dinp = wl.make_decode_inputs(dcfg, "cpu", seq_lens=torch.tensor([2048, 777], dtype=torch.int32))
    o, l, s = run_decode(dcfg, dinp, "auto")
    dp = hils.make_params(B=2, Hq=dcfg.Hq, Hkv=dcfg.Hkv, Hl=dcfg.Hkv, L=0, T_max=dcfg.L, C=dcfg.C, d=dcfg.d,
                          chunk_size=dcfg.S, top_k=dcfg.K, dtype=1, impl="auto")
    r2 = hils.HostRunner(dp, True, DEV)
    pd = {k: v.pin_memory() for k, v in dinp.items()}
    ho, hl, hs = r2.run(pd["q"], pd["k"], pd["v"], pd["landmarks"], seq_lens=pd["seq_lens"])
    torch.cuda.synchronize()
    assert torch.equal(hs, s.cpu())
    assert (ho.float() - o.cpu().float()).abs().max() <= 1e-2


def test_pipelined_host_prefill_matches_the_device_entry_point():
    """Long sequences through hils_prefill_host are copied, computed and copied back in blocks of 4096 tokens on
    internal streams; the result must be the device entry point's, twice in a row (buffer slots are reused)."""
    cfg = wl.CONFIGS[1].scaled(B=2, Hq=8, Hkv=2, L=2 * 4096 + 808, K=12, seed=51)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    bias = wl.make_bias(cfg, "cpu")
    out, lse, sel = run_prefill(cfg, inp, "auto", bias=bias)
    p = hils.make_params(B=cfg.B, Hq=cfg.Hq, Hkv=cfg.Hkv, Hl=cfg.Hkv, L=cfg.L, T_max=cfg.L, C=cfg.C, d=cfg.d,
                         chunk_size=cfg.S, top_k=cfg.K, dtype=1, impl="auto")
    runner = hils.HostRunner(p, False, DEV)
    pinned = {k: v.pin_memory() for k, v in inp.items()}
    for _ in range(2):
        ho, hl, hs = runner.run(pinned["q"], pinned["k"], pinned["v"], pinned["landmarks"], bias=bias.pin_memory())
        torch.cuda.synchronize()
        assert torch.equal(hs, sel.cpu())
        assert torch.equal(ho, out.cpu()) and torch.equal(hl, lse.cpu())
