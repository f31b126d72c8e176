"""Full-size parity: the five benchmark configurations in the launch configuration bench.py times,
compared with the oracle on sampled query rows (prefill) or sampled sequences (decode)."""
import numpy as np
import pytest
import torch

import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import workloads as wl
from parity import check_decode, check_prefill

pytestmark = pytest.mark.gpu
DEV = "cuda"


def prefill_full(cfg, n_rows):
    inp = wl.make_prefill_inputs(cfg, DEV)
    out, lse, sel = hils.hils_prefill(inp["q"], inp["k"], inp["v"], inp["landmarks"], cfg.S, cfg.K)
    torch.cuda.synchronize()
    rows = wl.sample_rows(cfg, n_rows).numpy()
    cpu = {k: v.cpu() for k, v in inp.items()}
    ridx = torch.as_tensor(rows, device=DEV)
    # compare only the sampled rows: gather them on the device, then reuse the row-wise checker
    sub_out = out[:, :, ridx].contiguous()
    sub_lse = lse[:, :, ridx].contiguous()
    sub_sel = sel[:, :, ridx].contiguous()
    return cfg, cpu, sub_out, sub_lse, sub_sel, rows


def check_prefill_rows(cfg, cpu, out, lse, sel, rows):
    """check_prefill expects full-length outputs; scatter the sampled rows into sparse holders."""
    B, Hq, _, d = out.shape
    L = cfg.L
    full_out = torch.zeros((B, Hq, L, d), dtype=torch.float32)
    full_lse = torch.zeros((B, Hq, L), dtype=torch.float32)
    full_sel = torch.full((B, cfg.Hkv, L, cfg.K), -1, dtype=torch.int32)
    r = torch.as_tensor(rows)
    full_out[:, :, r] = out.float().cpu()
    full_lse[:, :, r] = lse.cpu()
    full_sel[:, :, r] = sel.cpu()
    return check_prefill(cfg, cpu, full_out, full_lse, full_sel, rows=rows)


def test_cfg1_gqa_bf16_prefill_16k_sampled_rows():
    args = prefill_full(wl.CONFIGS[1], 2048)
    report("cfg1", check_prefill_rows(*args)[0])


def test_cfg2_long_bf16_prefill_128k_sampled_rows():
    args = prefill_full(wl.CONFIGS[2], 4096)
    report("cfg2", check_prefill_rows(*args)[0])


def decode_full(cfg, per_batch):
    """Every sequence of the configuration against the oracle, `per_batch` sequences' cache slabs on the host at a time."""
    inp = wl.make_decode_inputs(cfg, DEV)
    out, lse, sel = hils.hils_decode(inp["q"], inp["k"], inp["v"], inp["landmarks"], inp["seq_lens"], cfg.S, cfg.K)
    torch.cuda.synchronize()
    sel_c = sel.cpu().numpy()
    assert (sel_c >= 0).all() and (np.diff(sel_c, axis=-1) > 0).all() and (sel_c < cfg.C - 1).all()
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
    total = {"rows": 0, "exempt_rows": 0, "mismatch_rows": 0, "max_err_out": 0.0, "max_err_lse": 0.0}
    for b0 in range(0, cfg.B, per_batch):
        s = torch.arange(b0, min(cfg.B, b0 + per_batch), device=DEV)
        cpu = {k: v[s].cpu() for k, v in inp.items()}
        st = check_decode(cfg.scaled(B=len(s)), cpu, out[s], lse[s], sel[s])
        for key in ("rows", "exempt_rows", "mismatch_rows"):
            total[key] += st[key]
        for key in ("max_err_out", "max_err_lse"):
            total[key] = max(total[key], st[key])
    assert total["rows"] == cfg.B
    return total


def report(name, stats):
    """Selections differ from the oracle's only on rows inside the 1e-3 tie band (compare_rows has already rejected any
    other mismatch and any swap outside the band); the counts go to the test log."""
    print("%s: %s" % (name, stats))
    assert stats["mismatch_rows"] <= stats["exempt_rows"]


def test_cfg3_batched_decode_every_sequence():
    report("cfg3", decode_full(wl.CONFIGS[3], 8))


def test_cfg4_ultralong_decode_every_sequence():
    report("cfg4", decode_full(wl.CONFIGS[4], 1))


def test_cfg2_shape_with_the_papers_window_and_bias_sampled_rows():
    """cfg2's shape in the paper's operator form (W = 512, bias), the configuration bench.py reports as
    extra.cfg2_window512_bias, on sampled rows."""
    cfg = wl.CONFIGS[2]
    inp = wl.make_prefill_inputs(cfg, DEV)
    bias = wl.make_bias(cfg, DEV)
    out, lse, sel = hils.hils_prefill(inp["q"], inp["k"], inp["v"], inp["landmarks"], cfg.S, cfg.K, bias=bias, window=512)
    torch.cuda.synchronize()
    rows = wl.sample_rows(cfg, 2048).numpy()
    ridx = torch.as_tensor(rows, device=DEV)
    cpu = {k: v.cpu() for k, v in inp.items()}
    B, Hq, _, d = out.shape
    full_out = torch.zeros((B, Hq, cfg.L, d), dtype=torch.float32)
    full_lse = torch.zeros((B, Hq, cfg.L), dtype=torch.float32)
    full_sel = torch.full((B, cfg.Hkv, cfg.L, cfg.K), -1, dtype=torch.int32)
    r = torch.as_tensor(rows)
    full_out[:, :, r] = out[:, :, ridx].float().cpu()
    full_lse[:, :, r] = lse[:, :, ridx].cpu()
    full_sel[:, :, r] = sel[:, :, ridx].cpu()
    report("cfg2 W=512 bias", check_prefill(cfg, cpu, full_out, full_lse, full_sel, rows=rows, bias=bias.cpu(), W=512)[0])


def test_cfg3_paged_and_windowed_decode_sampled_sequences():
    """cfg3 through hils_decode_paged (shuffled pages, as bench.py's extra.cfg3_paged) with W = 512 and bias:
    identical to the contiguous entry point on every sequence, and the oracle on sampled ones."""
    cfg = wl.CONFIGS[3]
    inp = wl.make_decode_inputs(cfg, DEV)
    bias = wl.make_bias(cfg, DEV)
    B, Hkv, T, d = inp["k"].shape
    C, S = T // cfg.S, cfg.S
    perm = torch.randperm(B * C, generator=torch.Generator(device=DEV).manual_seed(3), device=DEV)

    def pages(x):
        src = x.view(B, Hkv, C, S, d).permute(0, 2, 1, 3, 4).reshape(B * C, Hkv, S, d)
        dst = torch.empty_like(src)
        dst[perm] = src
        return dst

    table = perm.reshape(B, C).to(torch.int32)
    out_c, lse_c, sel_c = hils.hils_decode(inp["q"], inp["k"], inp["v"], inp["landmarks"], inp["seq_lens"], cfg.S, cfg.K,
                                           bias=bias, window=512)
    out_p, lse_p, sel_p = hils.hils_decode_paged(inp["q"], pages(inp["k"]), pages(inp["v"]), inp["landmarks"], table,
                                                 inp["seq_lens"], cfg.S, cfg.K, bias=bias, window=512)
    torch.cuda.synchronize()
    assert torch.equal(sel_p, sel_c) and torch.equal(out_p, out_c) and torch.equal(lse_p, lse_c)
    s = torch.as_tensor([0, 17, 63], device=DEV)
    cpu = {k: v[s].cpu() for k, v in inp.items()}
    report("cfg3 paged W=512 bias", check_decode(cfg.scaled(B=3), cpu, out_p[s], lse_p[s], sel_p[s], bias=bias[s].cpu(), W=512))


def test_landmark_summary_on_the_cfg3_key_cache_sampled_sequences():
    """The chunk-summary kernel on the full 8.6 GB key cache (the launch bench.py times); sampled sequences against
    the oracle, all of them finite and with entropies in [0, log S]."""
    import oracle
    cfg = wl.CONFIGS[3]
    inp = wl.make_decode_inputs(cfg, DEV)
    lq = wl.make_landmark_queries(cfg, DEV)
    lm, b = hils.hils_landmark_summary(lq, inp["k"], cfg.S, seq_lens=inp["seq_lens"])
    torch.cuda.synchronize()
    assert torch.isfinite(lm.float()).all() and (b >= -1e-5).all() and (b <= np.log(cfg.S) + 1e-4).all()
    for bi in (0, 31, 63):
        ref_lm, ref_b = oracle.hils_landmarks(lq[bi:bi + 1].cpu(), inp["k"][bi:bi + 1].cpu(),
                                              seq_lens=inp["seq_lens"][bi:bi + 1].cpu(), S=cfg.S)
        assert np.abs(lm[bi:bi + 1].float().cpu().numpy() - ref_lm).max() <= 2e-2
        assert np.abs(b[bi:bi + 1].cpu().numpy() - ref_b).max() <= 2e-5
