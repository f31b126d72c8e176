"""Independent numpy fp64 brute force of HiLS attention for tiny inputs.

Builds, for every query row, the dense weight vector w_{i,j} over all L tokens
from the three-case definition of App. C (selected distant chunk / local window /
zero) with a full argsort for the top-K, then out = w @ V.  It exponentiates raw
logits without any max subtraction, so it takes a different numerical route
from the C oracle on purpose.  Used only to pin the oracle.
"""
import numpy as np


def brute_force_prefill(q, k, v, landmarks, bias, S, K, W=1, scale=None, q_route=None, group_mode=0):
    """q [Hq,L,d], k,v [Hkv,L,d], landmarks [Hl,C,d], bias [Hl,C] or None (one sequence).

    q_route [Hq,L,d] or None: the routing query of Eq. (Q-Cal); it takes q's place in the surrogate scores only.
    group_mode 0: group score = max over the group's heads of the raw surrogate score (App. C);
    group_mode 1: each head's scores are first turned into weights over the row's candidates (a softmax over the
    candidate chunks), the group score is the largest weight any head gives the chunk (the wording of Sec. 4.1).

    Returns (out [Hq,L,d], lse [Hq,L], sel list-of-lists [Hkv][L] (ascending ids), weights [Hq,L,L]).
    """
    q = np.asarray(q, np.float64); k = np.asarray(k, np.float64); v = np.asarray(v, np.float64)
    landmarks = np.asarray(landmarks, np.float64)
    qhat = q if q_route is None else np.asarray(q_route, np.float64)
    Hq, L, d = q.shape
    Hkv = k.shape[0]
    Hl = landmarks.shape[0]
    G = Hq // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    out = np.zeros((Hq, L, d)); lse = np.zeros((Hq, L)); wts = np.zeros((Hq, L, L))
    sel = [[None] * L for _ in range(Hkv)]
    for g in range(Hkv):
        for i in range(L):
            lo = max(0, ((i - W + 1) // S) * S)          # python // floors toward -inf
            ncand = lo // S
            shat = np.zeros((G, ncand))
            for r in range(G):
                h = g * G + r
                hl = h if Hl == Hq else g
                for c in range(ncand):
                    shat[r, c] = scale * (qhat[h, i] @ landmarks[hl, c]) + (0.0 if bias is None else bias[hl, c])
            if ncand == 0:
                u = np.zeros(0)
            elif group_mode == 0:
                u = shat.max(axis=0)
            else:
                wgt = np.exp(shat)                            # raw exponentials: the inputs here are small
                wgt = wgt / wgt.sum(axis=1, keepdims=True)
                u = wgt.max(axis=0)
            order = sorted(range(ncand), key=lambda c: (-u[c], c))
            chosen = sorted(order[:K])
            sel[g][i] = chosen
            for r in range(G):
                h = g * G + r
                e = np.exp(scale * (k[g] @ q[h, i]))     # exp(s_ij) for all j
                z_swa = e[lo:i + 1].sum()
                zhat = z_swa + sum(np.exp(shat[r, c]) for c in chosen)
                w = np.zeros(L)
                for c in chosen:
                    tok = slice(c * S, (c + 1) * S)
                    w[tok] = e[tok] / e[tok].sum() * np.exp(shat[r, c]) / zhat
                w[lo:i + 1] = e[lo:i + 1] / zhat
                wts[h, i] = w
                out[h, i] = w @ v[g]
                lse[h, i] = np.log(zhat)
    return out, lse, sel, wts
