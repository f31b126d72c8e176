"""GPU-vs-oracle comparison rules shared by the GPU tests.

Acceptance:
  * sel_idx bit-exact, except rows where the oracle's K-th and (K+1)-th group scores differ by
    less than 1e-3 ("exempt" rows); a mismatch on a row with margin >= 1e-3 fails;
  * on exempt rows that differ, the GPU's selection must still be valid (ascending, distinct,
    in range, right count), it may differ from the oracle's only inside the tie band -- every chunk it took
    scores at least (K-th best - 1e-3) and every chunk it left out at most (K-th best + 1e-3), with the group
    scores recomputed here in fp64 -- and `out` is compared with the oracle attending the GPU's selection;
  * out: max-abs 1e-4 (fp32) / 2e-2 (bf16 inputs, fp32 accumulation, oracle output unrounded);
  * lse: 1e-4 (fp32) / 1e-3 (bf16).
"""
import numpy as np
import torch

import oracle

TOL_OUT = {"f32": 1e-4, "bf16": 2e-2}
TOL_LSE = {"f32": 1e-4, "bf16": 1e-3}
MARGIN = 1e-3


def _np(t):
    return t.detach().float().cpu().numpy() if isinstance(t, torch.Tensor) else np.asarray(t)


def check_selection_valid(sel_row, ncand, K):
    ids = [int(c) for c in sel_row if c >= 0]
    n = min(K, ncand)
    assert len(ids) == n, "selected %d chunks, expected %d" % (len(ids), n)
    assert all(sel_row[n:] == -1), "padding must be -1"
    assert ids == sorted(set(ids)), "ids must be ascending and distinct"
    assert all(0 <= c < ncand for c in ids), "chunk id outside the candidate range"


def group_scores(q_row, lm, bias, ncand, scale=None):
    """Per-head surrogate scores s[h, c] = scale * q^h . k'_c + b'_c (Eq. surrogate top-k) of one query row for the
    candidates c < ncand, in fp64; the group score of App. C is their maximum over a KV group's heads.
    q_row [Hq, d]; lm [Hl, C, d] with Hl = Hkv or Hq; bias [Hl, C] or None."""
    q_row = np.asarray(q_row, np.float64)
    lm = np.asarray(lm, np.float64)[:, :ncand]
    Hq, d = q_row.shape
    Hl = lm.shape[0]
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    if Hl == Hq:
        s = scale * np.einsum("hd,hcd->hc", q_row, lm)
        if bias is not None:
            s = s + np.asarray(bias, np.float64)[:, :ncand]
    else:
        G = Hq // Hl
        s = scale * np.einsum("hd,hcd->hc", q_row, np.repeat(lm, G, axis=0))
        if bias is not None:
            s = s + np.repeat(np.asarray(bias, np.float64)[:, :ncand], G, axis=0)
    return s


def check_selection_in_tie_band(sel_row, u, K):
    """sel_row: the GPU's chunk ids of one (row, KV group); u [ncand]: the group's scores.  Whatever differs from
    the exact top-K must lie within MARGIN of the K-th best score."""
    ncand = u.shape[0]
    if ncand <= K:
        return
    kth = np.sort(u)[ncand - K]
    taken = np.zeros(ncand, bool)
    taken[[int(c) for c in sel_row if c >= 0]] = True
    assert (u[taken] >= kth - MARGIN).all(), "took a chunk scoring %g below the K-th best %g" % (u[taken].min(), kth)
    assert (u[~taken] <= kth + MARGIN).all(), "left out a chunk scoring %g above the K-th best %g" % (u[~taken].max(), kth)


def compare_rows(dtype, K, S, W, ref, gpu_sel, gpu_out, gpu_lse, row_pos, rerun, scores=None):
    """ref: oracle dict indexed [n, ...]; gpu_*: numpy arrays indexed [n, Hkv|Hq, ...].

    `rerun(rows_subset_indices, sel)` must return the oracle dict attending the given selection;
    `scores(row_index, ncand)` the per-head surrogate scores [Hq, ncand] of that row (fp64).
    Returns a stats dict; raises AssertionError on a violation.
    """
    n, Hkv = gpu_sel.shape[0], gpu_sel.shape[1]
    Hq = gpu_out.shape[1]
    G = Hq // Hkv
    mism = (gpu_sel != ref["sel_idx"]).any(-1)                      # [n, Hkv]
    exempt = ref["margin"] < MARGIN
    bad = mism & ~exempt
    assert not bad.any(), "selection mismatch on %d rows with margin >= %g (first: %s)" % (
        int(bad.sum()), MARGIN, np.argwhere(bad)[0])
    ref_out, ref_lse = ref["out"].copy(), ref["lse"].copy()
    rows_m = np.where(mism.any(-1))[0]
    if len(rows_m):
        for r in rows_m:
            lo = max(0, ((int(row_pos[r]) - W + 1) // S) * S)
            sh = scores(r, lo // S) if (scores is not None and lo // S > K) else None
            for g in range(Hkv):
                check_selection_valid(gpu_sel[r, g], lo // S, K)
                if sh is not None and mism[r, g]:
                    check_selection_in_tie_band(gpu_sel[r, g], sh[g * G:(g + 1) * G].max(axis=0), K)
        alt = rerun(rows_m, gpu_sel[rows_m])
        ref_out[rows_m] = alt["out"]
        ref_lse[rows_m] = alt["lse"]
    err_out = np.abs(gpu_out - ref_out)
    err_lse = np.abs(gpu_lse - ref_lse)
    assert np.isfinite(gpu_out).all() and np.isfinite(gpu_lse).all()
    assert err_out.max() <= TOL_OUT[dtype], "out max-abs error %g > %g at %s" % (
        err_out.max(), TOL_OUT[dtype], np.unravel_index(err_out.argmax(), err_out.shape))
    assert err_lse.max() <= TOL_LSE[dtype], "lse max-abs error %g > %g" % (err_lse.max(), TOL_LSE[dtype])
    return {"rows": n, "exempt_rows": int(exempt.sum()), "mismatch_rows": int(mism.sum()),
            "max_err_out": float(err_out.max()), "max_err_lse": float(err_lse.max()), "G": G}


def check_prefill(cfg, inp_cpu, out, lse, sel, rows=None, bias=None, W=1):
    """inp_cpu: host tensors (q,k,v,landmarks); out/lse/sel: GPU results [B,...]."""
    B = inp_cpu["q"].shape[0]
    L = inp_cpu["q"].shape[2]
    rows = np.arange(L) if rows is None else np.asarray(rows)
    ref = oracle.hils_prefill(inp_cpu["q"], inp_cpu["k"], inp_cpu["v"], inp_cpu["landmarks"], bias,
                              S=cfg.S, K=cfg.K, W=W, rows=rows)
    stats = []
    go, gl, gs = _np(out), _np(lse), sel.cpu().numpy()
    for b in range(B):
        refb = {k_: v_[b] for k_, v_ in ref.items()}
        g_sel = gs[b][:, rows].transpose(1, 0, 2)                    # [n, Hkv, K]
        g_out = go[b][:, rows].transpose(1, 0, 2)                    # [n, Hq, d]
        g_lse = gl[b][:, rows].T                                     # [n, Hq]

        def rerun(idx, sel_sub, b=b):
            one = {k_: v_[b:b + 1] for k_, v_ in inp_cpu.items() if k_ in ("q", "k", "v", "landmarks")}
            bb = None if bias is None else bias[b:b + 1]
            r = oracle.hils_prefill(one["q"], one["k"], one["v"], one["landmarks"], bb, S=cfg.S, K=cfg.K, W=W,
                                    rows=rows[idx], sel_idx=sel_sub[None])
            return {k_: v_[0] for k_, v_ in r.items()}

        def scores(r, ncand, b=b):
            return group_scores(inp_cpu["q"][b, :, int(rows[r])].float().numpy(), inp_cpu["landmarks"][b].float().numpy(),
                                None if bias is None else _np(bias[b]), ncand)

        stats.append(compare_rows(cfg.dtype, cfg.K, cfg.S, W, refb, g_sel, g_out, g_lse, rows, rerun, scores))
    return stats


def check_decode(cfg, inp_cpu, out, lse, sel, bias=None, W=1):
    seq = inp_cpu["seq_lens"].cpu().numpy().astype(np.int64)
    ref = oracle.hils_decode(inp_cpu["q"], inp_cpu["k"], inp_cpu["v"], inp_cpu["landmarks"], bias, seq,
                             S=cfg.S, K=cfg.K, W=W)

    def rerun(idx, sel_sub):
        sub = {k_: inp_cpu[k_][torch.as_tensor(idx)] for k_ in ("q", "k", "v", "landmarks")}
        bb = None if bias is None else bias[torch.as_tensor(idx)]
        return oracle.hils_decode(sub["q"], sub["k"], sub["v"], sub["landmarks"], bb, seq[idx], S=cfg.S, K=cfg.K,
                                  W=W, sel_idx=sel_sub)

    def scores(r, ncand):
        return group_scores(inp_cpu["q"][r].float().numpy(), inp_cpu["landmarks"][r].float().numpy(),
                            None if bias is None else _np(bias[r]), ncand)

    return compare_rows(cfg.dtype, cfg.K, cfg.S, W, ref, sel.cpu().numpy(), _np(out), _np(lse), seq - 1, rerun, scores)
