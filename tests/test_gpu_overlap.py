"""hils_chunk_overlap (Sec. "Chunk Overlap", Eq. Overlap) against the CPU oracle: integer outputs bit for bit, the
ratio to fp32 rounding; on the selection hils_prefill writes for i.i.d. and for structured-overlap queries, and on
constructed selections (padding, short trailing block, runs of blocks split across CTAs, large chunk ids)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def check(sel, M, C):
    stats, ov = hils.hils_chunk_overlap(sel.to(DEV), M, C)
    torch.cuda.synchronize()
    assert hils.last_launch_count() == 1
    ref = oracle.chunk_overlap(sel.cpu().numpy(), M)
    st = stats.cpu().numpy()
    assert (st[..., 0] == ref["total"]).all() and (st[..., 1] == ref["union"]).all()
    assert (st[..., 2] == ref["reused"]).all()
    L, K = sel.shape[-2:]
    nq = np.minimum(M, L - M * np.arange(st.shape[-2]))           # queries per block (the last one may be short)
    assert (st[..., 3] == ((ref["total"] == M * K) & (nq == M))).all()
    full = ~np.isnan(ref["overlap"])                              # where the equation applies (needs M > 1 too)
    got = ov.cpu().numpy()
    assert np.isnan(got[~full]).all()
    if full.any():
        assert np.abs(got[full] - ref["overlap"][full]).max() <= 1e-6
    return ref


@pytest.mark.parametrize("M", [1, 2, 16, 64])
def test_overlap_of_prefill_selections(M):
    cfg = wl.CONFIGS[1].scaled(B=2, Hq=8, Hkv=2, L=3000, K=12, seed=101)
    mean = {}
    for block in (0, 16):
        inp = wl.make_prefill_inputs(cfg, DEV, overlap_block=block)
        _, _, sel = hils.hils_prefill(inp["q"], inp["k"], inp["v"], inp["landmarks"], cfg.S, cfg.K)
        ref = check(sel, M, cfg.C)
        mean[block] = np.nanmean(ref["union"][..., 20:])
    print("M=%d: mean union size, i.i.d. queries %.1f, structured queries %.1f" % (M, mean[0], mean[16]))
    if M > 1:
        assert mean[16] < mean[0]                         # the structured recipe shares chunks between neighbours


def test_constructed_selections_padding_tail_and_many_runs():
    g = torch.Generator().manual_seed(5)
    B, Hkv, L, K, C = 3, 5, 10007, 8, 300000                       # 15 pairs: runs of blocks are split across CTAs
    base = torch.randint(0, C - 64, (B, Hkv, (L + 31) // 32, 1), generator=g)
    ids = base.repeat_interleave(32, dim=2)[:, :, :L] + torch.randint(0, 24, (B, Hkv, L, K), generator=g)
    ids = ids.sort(dim=-1).values
    dup = ids[..., 1:] == ids[..., :-1]                             # selections hold distinct ids: blank duplicates
    ids[..., 1:][dup] = -1
    ids[:, :, :40, 3:] = -1                                         # early queries with fewer than K chunks
    sel = ids.to(torch.int32).contiguous()
    for M in (3, 16, 32):
        check(sel, M, C)
    check(sel[..., :7].contiguous(), 5, C)                          # K not a multiple of 4: scalar id loads


def test_argument_errors():
    sel = torch.zeros((1, 1, 64, 4), dtype=torch.int32, device=DEV)
    with pytest.raises(hils.HilsError):
        hils.hils_chunk_overlap(sel, 0, 16)
    with pytest.raises(hils.HilsError):
        hils.hils_chunk_overlap(sel, 4, (1 << 19) + 1)
