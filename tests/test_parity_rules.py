"""The acceptance rules of tests/parity.py, exercised on the CPU with stand-ins for the GPU's results (the oracle's
own outputs, edited): a selection that differs from the oracle's is accepted only on a row whose K-th and (K+1)-th
scores are within 1e-3 AND only if every swapped chunk lies inside that tie band."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_02980_b200 import workloads as wl
from parity import check_prefill, group_scores


def tiny(seed=5):
    cfg = wl.CONFIGS[1].scaled(L=640, K=3, n_needles=0, seed=seed, name="tie_rules")
    inp = wl.make_prefill_inputs(cfg, "cpu")
    # an exact tie: chunk 7 carries the landmark of chunk 2 (both KV heads, every sequence)
    inp["landmarks"][:, :, 7] = inp["landmarks"][:, :, 2]
    return cfg, inp


def oracle_as_gpu(cfg, inp, sel_override=None):
    """The oracle's results shaped like the library's outputs ([B,Hq,L,d], [B,Hq,L], [B,Hkv,L,K])."""
    ref = oracle.hils_prefill(inp["q"], inp["k"], inp["v"], inp["landmarks"], None, S=cfg.S, K=cfg.K, sel_idx=sel_override)
    out = torch.from_numpy(ref["out"]).permute(0, 2, 1, 3).contiguous().float()
    lse = torch.from_numpy(ref["lse"]).permute(0, 2, 1).contiguous().float()
    sel = torch.from_numpy(ref["sel_idx"]).permute(0, 2, 1, 3).contiguous().int()
    return ref, out, lse, sel


def rows_where_the_tie_decides(ref):
    """(row, group) pairs that selected chunk 2 but not its twin 7 although 7 was a candidate: the tie sits exactly at
    the K-th place."""
    sel = ref["sel_idx"][0]                                   # [L, Hkv, K]
    has2 = (sel == 2).any(-1)
    has7 = (sel == 7).any(-1)
    rows = np.arange(sel.shape[0])[:, None] >= 8 * 64
    return np.argwhere(has2 & ~has7 & rows)


def test_group_scores_match_the_oracles_margin():
    cfg, inp = tiny()
    ref, _, _, _ = oracle_as_gpu(cfg, inp)
    for r in (300, 511, 639):
        ncand = r // cfg.S
        s = group_scores(inp["q"][0, :, r].float().numpy(), inp["landmarks"][0].float().numpy(), None, ncand)
        for g in range(cfg.Hkv):
            u = np.sort(s[g * cfg.G:(g + 1) * cfg.G].max(axis=0))[::-1]
            assert abs((u[cfg.K - 1] - u[cfg.K]) - ref["margin"][0, r, g]) < 1e-9


def test_swapping_exactly_tied_chunks_is_accepted():
    cfg, inp = tiny()
    ref, _, _, _ = oracle_as_gpu(cfg, inp)
    pairs = rows_where_the_tie_decides(ref)
    assert len(pairs) > 0, "the construction must put the tie at the K-th place somewhere"
    sel = ref["sel_idx"].copy()
    for r, g in pairs:
        row = sel[0, r, g]
        row[row == 2] = 7
        sel[0, r, g] = np.sort(row)
    _, out, lse, sel_t = oracle_as_gpu(cfg, inp, sel_override=sel)
    stats = check_prefill(cfg, inp, out, lse, sel_t)
    assert stats[0]["mismatch_rows"] == len(pairs)


def test_an_arbitrary_chunk_on_an_exempt_row_is_rejected():
    cfg, inp = tiny()
    ref, _, _, _ = oracle_as_gpu(cfg, inp)
    pairs = rows_where_the_tie_decides(ref)
    r, g = pairs[-1]
    s = group_scores(inp["q"][0, :, r].float().numpy(), inp["landmarks"][0].float().numpy(), None, r // cfg.S)
    u = s[g * cfg.G:(g + 1) * cfg.G].max(axis=0)
    worst = int(np.argmin(u))                                  # far below the K-th best
    assert worst not in ref["sel_idx"][0, r, g]
    sel = ref["sel_idx"].copy()
    row = sel[0, r, g]
    row[row == 2] = worst                                      # structurally valid, but not a tie
    sel[0, r, g] = np.sort(row)
    _, out, lse, sel_t = oracle_as_gpu(cfg, inp, sel_override=sel)
    with pytest.raises(AssertionError, match="below the K-th best"):
        check_prefill(cfg, inp, out, lse, sel_t)


def test_a_mismatch_on_a_row_with_margin_is_rejected():
    cfg, inp = tiny()
    ref, _, _, _ = oracle_as_gpu(cfg, inp)
    safe = np.argwhere((ref["margin"][0] >= 1e-2) & (np.arange(cfg.L)[:, None] >= 8 * 64))
    r, g = safe[0]
    sel = ref["sel_idx"].copy()
    row = sel[0, r, g]
    spare = [c for c in range(r // cfg.S) if c not in row][0]
    row[0] = spare
    sel[0, r, g] = np.sort(row)
    _, out, lse, sel_t = oracle_as_gpu(cfg, inp, sel_override=sel)
    with pytest.raises(AssertionError, match="selection mismatch"):
        check_prefill(cfg, inp, out, lse, sel_t)
