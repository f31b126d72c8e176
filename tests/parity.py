"""GPU-vs-oracle comparison rules shared by the GPU tests.

Acceptance:
  * sel_idx bit-exact, except rows where the oracle's K-th and (K+1)-th group scores differ by
    less than 1e-3 ("exempt" rows); a mismatch on a row with margin >= 1e-3 fails;
  * on exempt rows that differ, the GPU's selection must still be valid (ascending, distinct,
    in range, right count) and `out` is compared with the oracle attending the GPU's selection;
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


def compare_rows(dtype, K, S, W, ref, gpu_sel, gpu_out, gpu_lse, row_pos, rerun):
    """ref: oracle dict indexed [n, ...]; gpu_*: numpy arrays indexed [n, Hkv|Hq, ...].

    `rerun(rows_subset_indices, sel)` must return the oracle dict attending the given selection.
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
            for g in range(Hkv):
                check_selection_valid(gpu_sel[r, g], lo // S, K)
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

        stats.append(compare_rows(cfg.dtype, cfg.K, cfg.S, W, refb, g_sel, g_out, g_lse, rows, rerun))
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

    return compare_rows(cfg.dtype, cfg.K, cfg.S, W, ref, sel.cpu().numpy(), _np(out), _np(lse), seq - 1, rerun)
