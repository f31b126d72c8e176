"""hils_prefill_backward against the CPU oracle's backward (chain rule on Eq. HiLS weights, selection fixed), element
by element on seeded inputs.  Both sides differentiate the same forward: the oracle is given the selection the GPU
forward wrote, so rows with a small selection margin need no exemption.  Tolerances are relative to the largest
entry of each gradient tensor: fp32 1e-4 (fp32 accumulation against fp64), bf16 2e-2 (the forward's `out`, which
enters through dout . out, is rounded to bf16; inputs are identical on both sides)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"
RTOL = {"f32": 1e-4, "bf16": 2e-2}

CASES = {
    # name: (config, Hl, W, with_bias)
    "f32_tiny": (wl.CONFIGS[0].scaled(L=512, seed=201), None, 1, True),
    "f32_gqa_window": (wl.CONFIGS[0].scaled(Hq=4, Hkv=2, L=448, K=3, seed=202), None, 100, True),
    "f32_per_head_landmarks": (wl.CONFIGS[0].scaled(Hq=4, Hkv=2, L=384, K=3, seed=203), 4, 1, False),
    "bf16_gqa": (wl.CONFIGS[1].scaled(B=2, Hq=8, Hkv=2, L=640, K=6, seed=204), None, 1, True),
    "bf16_window": (wl.CONFIGS[1].scaled(B=1, Hq=8, Hkv=2, L=700, K=4, seed=205), None, 130, False),
}


def run_case(cfg, Hl, W, with_bias, impl="auto"):
    inp = wl.make_prefill_inputs(cfg, "cpu")
    if Hl is not None and Hl != cfg.Hkv:
        per = Hl // cfg.Hkv
        noise = torch.randn((cfg.B, Hl, cfg.C, cfg.d), generator=torch.Generator().manual_seed(cfg.seed)) * 0.1
        inp["landmarks"] = (inp["landmarks"].float().repeat_interleave(per, dim=1) + noise).to(cfg.torch_dtype())
    bias = None
    if with_bias:
        bias = torch.randn(inp["landmarks"].shape[:3], generator=torch.Generator().manual_seed(cfg.seed + 1)) * 0.5
    dout = torch.randn(inp["q"].shape, generator=torch.Generator().manual_seed(cfg.seed + 2)).to(cfg.torch_dtype())
    g = {n: t.to(DEV) for n, t in inp.items()}
    bg = None if bias is None else bias.to(DEV)
    out, lse, sel = hils.hils_prefill(g["q"], g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, bias=bg, window=W)
    grads = hils.hils_prefill_backward(g["q"], g["k"], g["v"], g["landmarks"], cfg.S, cfg.K, out, lse, sel,
                                       dout.to(DEV), bias=bg, window=W, impl=impl)
    torch.cuda.synchronize()
    ref = oracle.hils_backward(inp["q"], inp["k"], inp["v"], inp["landmarks"], bias, sel.cpu(), dout.float(),
                               S=cfg.S, K=cfg.K, W=W)
    return grads, ref


def compare(grads, ref, dtype):
    names = ("dq", "dk", "dv", "dlandmarks", "dbias")
    for got, n in zip(grads, names):
        if got is None:
            continue
        r = ref[n]
        err = np.abs(got.cpu().numpy().astype(np.float64) - r).max()
        ref_max = np.abs(r).max()
        print("%-11s max|ref| %.3e  max err %.3e" % (n, ref_max, err))
        assert ref_max > 0
        assert err <= RTOL[dtype] * ref_max, (n, err, ref_max)


@pytest.mark.parametrize("name", list(CASES))
def test_backward_matches_oracle(name):
    cfg, Hl, W, with_bias = CASES[name]
    grads, ref = run_case(cfg, Hl, W, with_bias, impl="generic")
    compare(grads, ref, cfg.dtype)


FAST_CASES = {
    "bf16_gqa": CASES["bf16_gqa"],
    "bf16_window": CASES["bf16_window"],
    # more than one query block of 4096 tokens, ragged tiles, runs of a chunk split across CTAs
    # (K = 2 keeps the single-threaded oracle, one thread per (sequence, KV head), under a minute)
    "bf16_two_query_blocks": (wl.CONFIGS[1].scaled(B=1, Hq=4, Hkv=1, L=4400, K=2, seed=207), None, 1, True),
    "bf16_window_512": (wl.CONFIGS[1].scaled(B=1, Hq=8, Hkv=2, L=1500, K=5, seed=208), None, 512, True),
}


@pytest.mark.parametrize("name", list(FAST_CASES))
def test_tensor_core_backward_matches_oracle(name):
    cfg, Hl, W, with_bias = FAST_CASES[name]
    grads, ref = run_case(cfg, Hl, W, with_bias, impl="fast")
    assert hils.last_launch_count() >= 6          # dsum + 4 index kernels + one backward kernel per query block
    compare(grads, ref, cfg.dtype)


def test_auto_dispatch_falls_back_to_the_generic_kernel_for_per_head_landmarks():
    """One landmark per query head (App. C) is outside the tensor-core backward: `auto` must take the generic
    kernel and still match the oracle (bf16)."""
    cfg = wl.CONFIGS[1].scaled(B=1, Hq=8, Hkv=2, L=448, K=4, seed=211)
    grads, ref = run_case(cfg, 8, 1, True, impl="auto")
    assert hils.last_launch_count() == 1
    compare(grads, ref, cfg.dtype)


def test_fast_path_refuses_shapes_it_does_not_take():
    cfg = wl.CONFIGS[0].scaled(L=128, seed=209)   # fp32
    inp = {n: t.to(DEV) for n, t in wl.make_prefill_inputs(cfg, "cpu").items()}
    out, lse, sel = hils.hils_prefill(inp["q"], inp["k"], inp["v"], inp["landmarks"], cfg.S, cfg.K)
    with pytest.raises(hils.HilsError):
        hils.hils_prefill_backward(inp["q"], inp["k"], inp["v"], inp["landmarks"], cfg.S, cfg.K, out, lse, sel,
                                   torch.ones_like(inp["q"]), impl="fast")


def test_autograd_wrapper_routes_both_passes_through_the_library():
    cfg = wl.CONFIGS[1].scaled(B=1, Hq=8, Hkv=2, L=512, K=4, seed=210)
    inp = wl.make_prefill_inputs(cfg, "cpu")
    bias = torch.randn(inp["landmarks"].shape[:3], generator=torch.Generator().manual_seed(3)) * 0.5
    dout = torch.randn(inp["q"].shape, generator=torch.Generator().manual_seed(4)).to(torch.bfloat16)
    leaves = {n: t.to(DEV).requires_grad_(True) for n, t in inp.items()}
    bg = bias.to(DEV).requires_grad_(True)
    out, lse, sel = hils.hils_attention(leaves["q"], leaves["k"], leaves["v"], leaves["landmarks"], cfg.S, cfg.K, bias=bg)
    assert not lse.requires_grad and not sel.requires_grad
    (out.float() * dout.to(DEV).float()).sum().backward()
    ref = oracle.hils_backward(inp["q"], inp["k"], inp["v"], inp["landmarks"], bias, sel.cpu(), dout.float(),
                               S=cfg.S, K=cfg.K)
    got = (leaves["q"].grad, leaves["k"].grad, leaves["v"].grad, leaves["landmarks"].grad, bg.grad)
    for g, n in zip(got, ("dq", "dk", "dv", "dlandmarks", "dbias")):
        assert g is not None
        r = ref[n]
        # the wrapper rounds the gradients to the inputs' dtype (bf16) on top of the kernel's own error
        assert np.abs(g.float().cpu().numpy() - r).max() <= 2.5e-2 * np.abs(r).max(), n


def test_missing_arguments_are_refused():
    cfg = wl.CONFIGS[0].scaled(L=128, seed=206)
    inp = {n: t.to(DEV) for n, t in wl.make_prefill_inputs(cfg, "cpu").items()}
    out, lse, sel = hils.hils_prefill(inp["q"], inp["k"], inp["v"], inp["landmarks"], cfg.S, cfg.K)
    with pytest.raises((hils.HilsError, ValueError, TypeError)):
        hils.hils_prefill_backward(inp["q"], inp["k"], inp["v"], inp["landmarks"], cfg.S, cfg.K, out, lse, sel,
                                   inp["q"][:, :, :64].contiguous())
