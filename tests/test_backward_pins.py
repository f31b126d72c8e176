"""Pins of the oracle's backward pass.  The paper prints no backward equations (it only states that the
language-model loss reaches the landmarks through the forward weights, Sec. 3.2), so the derivative is pinned
against what the forward and the mathematics fix: central finite differences of the forward oracle in every input,
library autograd on the rows that reduce to causal softmax attention, library autograd on the K = 1 two-branch
mix of Eq. (HiLS weights), and linearity / zero structure."""
import numpy as np
import pytest
import torch

import oracle


def make(B=1, Hq=4, Hkv=2, Hl=None, L=40, d=8, S=8, seed=0, with_bias=True):
    rng = np.random.default_rng(seed)
    Hl = Hkv if Hl is None else Hl
    C = L // S
    t = {"q": rng.standard_normal((B, Hq, L, d)), "k": rng.standard_normal((B, Hkv, L, d)),
         "v": rng.standard_normal((B, Hkv, L, d)), "landmarks": rng.standard_normal((B, Hl, C, d)),
         "bias": rng.standard_normal((B, Hl, C)) if with_bias else None}
    t = {n: (None if a is None else a.astype(np.float32)) for n, a in t.items()}
    dout = rng.standard_normal((B, Hq, L, d))
    return t, dout


def forward_loss(t, dout, sel, S, K, W):
    """sum(out * dout) with the selection held fixed: the scalar whose gradient the backward returns."""
    res = oracle.hils_prefill(t["q"], t["k"], t["v"], t["landmarks"], t["bias"], S=S, K=K, W=W, sel_idx=sel)
    out = res["out"].transpose(0, 2, 1, 3)                       # [B, n, Hq, d] -> [B, Hq, n, d]
    return float((out * dout).sum())


@pytest.mark.parametrize("Hl_is_Hq,W,K", [(False, 1, 2), (True, 1, 3), (False, 11, 2), (False, 16, 1)])
def test_central_finite_differences_in_every_input(Hl_is_Hq, W, K):
    S = 8
    t, dout = make(Hl=4 if Hl_is_Hq else None, seed=3 + K)
    fwd = oracle.hils_prefill(t["q"], t["k"], t["v"], t["landmarks"], t["bias"], S=S, K=K, W=W)
    sel = fwd["sel_idx"]                                         # [B, n, Hkv, K]
    g = oracle.hils_backward(t["q"], t["k"], t["v"], t["landmarks"], t["bias"], sel.transpose(0, 2, 1, 3), dout,
                             S=S, K=K, W=W)
    rng = np.random.default_rng(99)
    eps = 1e-3                                                   # inputs are fp32: the step must survive the cast
    for name, gname in (("q", "dq"), ("k", "dk"), ("v", "dv"), ("landmarks", "dlandmarks"), ("bias", "dbias")):
        base = t[name]
        for _ in range(12):
            idx = tuple(rng.integers(0, n) for n in base.shape)
            hi = {**t, name: base.copy()}
            lo = {**t, name: base.copy()}
            hi[name][idx] += eps
            lo[name][idx] -= eps
            step = float(hi[name][idx]) - float(lo[name][idx])    # the step actually taken after fp32 rounding
            fd = (forward_loss(hi, dout, sel, S, K, W) - forward_loss(lo, dout, sel, S, K, W)) / step
            assert abs(fd - g[gname][idx]) <= 2e-5 + 2e-4 * abs(fd), (name, idx, fd, g[gname][idx])
    # the directional derivative along a random direction of all inputs at once (catches a systematically
    # missing term that single coordinates could miss by sampling)
    dirs = {n: rng.standard_normal(t[n].shape).astype(np.float32) for n in t}
    hi = {n: t[n] + np.float32(eps) * dirs[n] for n in t}
    lo = {n: t[n] - np.float32(eps) * dirs[n] for n in t}
    fd = (forward_loss(hi, dout, sel, S, K, W) - forward_loss(lo, dout, sel, S, K, W))
    an = sum(float((g[gn] * (hi[n].astype(np.float64) - lo[n].astype(np.float64))).sum())
             for n, gn in (("q", "dq"), ("k", "dk"), ("v", "dv"), ("landmarks", "dlandmarks"), ("bias", "dbias")))
    assert abs(fd - an) <= 1e-4 * max(1.0, abs(fd))


def test_rows_without_candidates_match_library_autograd_of_causal_attention():
    """With K = 0 nothing is retrieved and W covers the sequence: the operator is causal softmax attention
    (per KV group), whose gradient a library computes."""
    t, dout = make(B=2, Hq=4, Hkv=2, L=24, d=8, S=8, seed=5)
    sel = np.zeros((2, 2, 24, 0), np.int32)
    g = oracle.hils_backward(t["q"], t["k"], t["v"], t["landmarks"], None, sel, dout, S=8, K=0, W=64)
    q = torch.tensor(t["q"], dtype=torch.float64, requires_grad=True)
    k = torch.tensor(t["k"], dtype=torch.float64, requires_grad=True)
    v = torch.tensor(t["v"], dtype=torch.float64, requires_grad=True)
    out = torch.nn.functional.scaled_dot_product_attention(q, k.repeat_interleave(2, 1), v.repeat_interleave(2, 1),
                                                           is_causal=True)
    (out * torch.tensor(dout)).sum().backward()
    assert np.abs(g["dq"] - q.grad.numpy()).max() < 1e-12
    assert np.abs(g["dk"] - k.grad.numpy()).max() < 1e-12
    assert np.abs(g["dv"] - v.grad.numpy()).max() < 1e-12
    assert not g["dlandmarks"].any() and not g["dbias"].any()


def test_single_chunk_mix_matches_library_autograd():
    """K = 1, one past chunk: out = sigma * Attn(q, K_0, V_0) + (1 - sigma) * CausalAttn_local with
    sigma = sigmoid(s_hat - log Z_swa) (Eq. HiLS weights with two slots); autograd through library pieces."""
    S, d = 8, 8
    t, dout = make(B=1, Hq=1, Hkv=1, L=2 * S, d=d, S=S, seed=7)
    sel = np.full((1, 1, 2 * S, 1), -1, np.int32)
    sel[0, 0, S:, 0] = 0
    g = oracle.hils_backward(t["q"], t["k"], t["v"], t["landmarks"], t["bias"], sel, dout, S=S, K=1, W=1)
    T = {n: torch.tensor(a, dtype=torch.float64, requires_grad=True) for n, a in t.items()}
    scale = 1.0 / np.sqrt(d)
    loss = 0.0
    for i in range(2 * S):
        qi = T["q"][0, 0, i]
        lo = (i // S) * S
        s_loc = scale * (T["k"][0, 0, lo:i + 1] @ qi)
        o_loc = torch.softmax(s_loc, 0) @ T["v"][0, 0, lo:i + 1]
        if i < S:
            out = o_loc
        else:
            o_c = torch.softmax(scale * (T["k"][0, 0, :S] @ qi), 0) @ T["v"][0, 0, :S]
            s_hat = scale * (T["landmarks"][0, 0, 0] @ qi) + T["bias"][0, 0, 0]
            sig = torch.sigmoid(s_hat - torch.logsumexp(s_loc, 0))
            out = sig * o_c + (1 - sig) * o_loc
        loss = loss + (out * torch.tensor(dout[0, 0, i])).sum()
    loss.backward()
    for n, gn in (("q", "dq"), ("k", "dk"), ("v", "dv"), ("landmarks", "dlandmarks"), ("bias", "dbias")):
        assert np.abs(g[gn] - T[n].grad.numpy()).max() < 1e-12, n


def test_linearity_in_dout_and_untouched_entries():
    S, K = 8, 2
    t, dout = make(seed=11)
    sel = oracle.hils_prefill(t["q"], t["k"], t["v"], t["landmarks"], t["bias"], S=S, K=K)["sel_idx"].transpose(0, 2, 1, 3)
    g1 = oracle.hils_backward(t["q"], t["k"], t["v"], t["landmarks"], t["bias"], sel, dout, S=S, K=K)
    g2 = oracle.hils_backward(t["q"], t["k"], t["v"], t["landmarks"], t["bias"], sel, -2.5 * dout, S=S, K=K)
    for n in g1:
        assert np.allclose(g2[n], -2.5 * g1[n], rtol=1e-12, atol=1e-14)
    # a landmark no query selected receives no gradient; the last chunk is never a candidate
    used = np.zeros(t["landmarks"].shape[:3], bool)
    for b, gk, r, s in np.ndindex(sel.shape):
        if sel[b, gk, r, s] >= 0:
            used[b, gk, sel[b, gk, r, s]] = True
    assert not g1["dlandmarks"][~used].any() and not g1["dbias"][~used].any()
    assert not used[:, :, -1].any()
    assert np.isfinite(g1["dq"]).all()


def test_shifting_all_keys_of_a_selected_chunk_has_zero_directional_derivative():
    """The hierarchy property in derivative form: adding one vector to every key of a past chunk leaves `out`
    unchanged (its softmax is shift invariant, its mass comes from the landmark), so sum_j dk_j over that chunk
    must vanish for chunks that are only ever attended as selected chunks."""
    S, K = 8, 3
    t, dout = make(L=48, seed=13)
    sel = oracle.hils_prefill(t["q"], t["k"], t["v"], t["landmarks"], t["bias"], S=S, K=K)["sel_idx"].transpose(0, 2, 1, 3)
    # drop the queries of chunk 0 and 1 from the loss, so that those chunks are never a local span
    dout[:, :, :2 * S] = 0.0
    g = oracle.hils_backward(t["q"], t["k"], t["v"], t["landmarks"], t["bias"], sel, dout, S=S, K=K)
    for c in (0, 1):
        assert np.abs(g["dk"][:, :, c * S:(c + 1) * S]).max() > 1e-6          # the chunk does receive gradient
        assert np.abs(g["dk"][:, :, c * S:(c + 1) * S].sum(axis=2)).max() < 1e-12
