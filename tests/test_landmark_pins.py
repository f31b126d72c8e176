"""Pins of the oracle's chunk-summary function (Proposition 3.1, Eq. LogSumExp linearization and
Eq. prop_q_c) against what the paper and the mathematics fix: closed forms, the Taylor-point identity,
the tangent-plane inequality, library routines, and the end-to-end consequence for the operator."""
import numpy as np
import pytest
import torch
from scipy.special import logsumexp, softmax
from scipy.stats import entropy

import oracle


def rand(shape, seed, scale=1.0):
    return (np.random.default_rng(seed).standard_normal(shape) * scale).astype(np.float32)


def test_zero_query_gives_chunk_mean_and_log_count():
    """Uniform scores: p_j = 1/n, so k' is the mean key and b' = log n (Sec. 3: b' -> log S)."""
    S = 16
    k = rand((2, 2, 3 * S + 5, 8), 1)
    lq = np.zeros((2, 4, 4, 8), np.float32)                       # Hl = 4 landmark heads on 2 KV heads
    lm, b = oracle.hils_landmarks(lq, k, S=S)
    for c, n in ((0, S), (2, S), (3, 5)):                         # chunk 3 is partial: 5 tokens
        assert np.allclose(b[:, :, c], np.log(n), atol=1e-12)
        for hl in range(4):
            assert np.allclose(lm[:, hl, c], k[:, hl // 2, c * S:c * S + n].mean(axis=1), atol=1e-6)


def test_dominant_key_gives_that_key_and_zero_entropy():
    """One score far above the rest: p is one-hot, k' is that key, b' = 0 (Sec. 3: b' -> 0)."""
    S, d = 8, 4
    k = rand((1, 1, 2 * S, d), 2, 0.1)
    k[0, 0, S + 3] = np.array([9.0, 0, 0, 0], np.float32)
    lq = np.zeros((1, 1, 2, d), np.float32)
    lq[0, 0, 1] = np.array([40.0, 0, 0, 0], np.float32)
    lm, b = oracle.hils_landmarks(lq, k, S=S, scale=1.0)
    assert abs(b[0, 0, 1]) < 1e-12
    assert np.allclose(lm[0, 0, 1], k[0, 0, S + 3], atol=1e-9)


def test_surrogate_equals_chunk_mass_at_the_expansion_point():
    """At q = q'_c the linearization is exact: scale q'.k' + b' = log sum_j exp(scale q'.k_j) (App. B)."""
    S, d = 32, 16
    k = rand((2, 2, 4 * S, d), 3)
    lq = rand((2, 2, 4, d), 4)
    scale = 1.0 / np.sqrt(d)
    lm, b = oracle.hils_landmarks(lq, k, S=S)
    for bb in range(2):
        for h in range(2):
            for c in range(4):
                s = scale * k[bb, h, c * S:(c + 1) * S].astype(np.float64) @ lq[bb, h, c].astype(np.float64)
                assert abs(scale * lq[bb, h, c].astype(np.float64) @ lm[bb, h, c] + b[bb, h, c] - logsumexp(s)) < 1e-10


def test_surrogate_is_a_tangent_plane_below_the_chunk_mass():
    """log-sum-exp is convex in q, so its first-order expansion never exceeds it, and the gap is second order."""
    S, d = 16, 8
    k = rand((1, 1, S, d), 5)
    lq = rand((1, 1, 1, d), 6)
    lm, b = oracle.hils_landmarks(lq, k, S=S, scale=1.0)
    kk = k[0, 0].astype(np.float64)
    gaps = []
    for eps in (1.0, 0.1, 0.01):
        q = lq[0, 0, 0].astype(np.float64) + eps * rand((d,), 7).astype(np.float64)
        gap = logsumexp(kk @ q) - (q @ lm[0, 0, 0] + b[0, 0, 0])
        assert gap >= -1e-12
        gaps.append(gap)
    assert gaps[1] < gaps[0] / 30 and gaps[2] < gaps[1] / 30          # ~ eps^2


def test_against_library_softmax_and_entropy():
    S, d = 64, 32
    kt = torch.from_numpy(rand((1, 2, 3 * S, d), 8)).to(torch.bfloat16)
    qt = torch.from_numpy(rand((1, 2, 3, d), 9)).to(torch.bfloat16)
    lm, b = oracle.hils_landmarks(qt, kt, seq_lens=np.array([2 * S + 7], np.int32), S=S)
    k = kt.float().numpy().astype(np.float64)
    q = qt.float().numpy().astype(np.float64)
    for h in range(2):
        for c, n in ((0, S), (1, S), (2, 7)):
            p = softmax(k[0, h, c * S:c * S + n] @ q[0, h, c] / np.sqrt(d))
            assert np.allclose(lm[0, h, c], p @ k[0, h, c * S:c * S + n], atol=1e-12)
            assert abs(b[0, h, c] - entropy(p)) < 1e-12


def test_empty_chunk_is_zero():
    k = rand((1, 1, 64, 8), 10)
    lq = rand((1, 1, 4, 8), 11)
    lm, b = oracle.hils_landmarks(lq, k, seq_lens=np.array([20], np.int32), S=16)
    assert (lm[0, 0, 2:] == 0).all() and (b[0, 0, 2:] == 0).all()
    assert b[0, 0, 1] > 0 and abs(b[0, 0, 1] - entropy(softmax(k[0, 0, 16:20].astype(np.float64) @ lq[0, 0, 1] / np.sqrt(8)))) < 1e-12


def test_operator_with_summaries_taken_at_the_query_is_exact_full_attention():
    """If every chunk's learnable query equals the decoding query, every surrogate score equals the chunk's
    exact log mass, so HiLS over all chunks (K >= candidates) reproduces full softmax attention."""
    S, d, T = 16, 8, 16 * 5 + 9
    q = rand((1, 2, 1, d), 12)
    k = rand((1, 2, T, d), 13)
    v = rand((1, 2, T, d), 14)
    C = T // S
    lq = np.broadcast_to(q[:, :, 0][:, :, None, :], (1, 2, C, d)).copy()          # Hl = Hq = Hkv = 2 (G = 1)
    lm, b = oracle.hils_landmarks(lq, k, S=S)
    res = oracle.hils_decode(q[:, :, 0], k, v, lm.astype(np.float32), b.astype(np.float32), np.array([T], np.int32), S=S, K=C)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).double(), torch.from_numpy(k).double(), torch.from_numpy(v).double()).numpy()[:, :, 0]
    assert np.allclose(res["out"].reshape(ref.shape), ref, atol=2e-6)        # landmarks rounded to fp32 on the way in
