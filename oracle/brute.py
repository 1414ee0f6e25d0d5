"""Second, independently written numpy implementation for tiny inputs -- TEST INFRASTRUCTURE ONLY.

Used only to cross-check ``seka_oracle.c``.  It takes a different route on
purpose: the projector is formed as a dense d x d matrix (Eq. 2 / Section 3.3),
the whole L x L score matrix is materialised with an explicit -inf causal mask,
and the steering enters either through the edited keys (Section 2) or as the
additive low-rank logit bias B of Eq. 5.  One sequence at a time, fp64.
"""
from __future__ import annotations

import numpy as np


def dense_projector(U, h, alpha=None):
    """P = sum_m alpha_m U_m U_m^T for KV head h; U is [M, Hkv, d, r]."""
    U = np.asarray(U, dtype=np.float64)
    M = U.shape[0]
    P = np.zeros((U.shape[2], U.shape[2]))
    for m in range(M):
        a = 1.0 if alpha is None else float(np.asarray(alpha)[h, m])
        P += a * U[m, h] @ U[m, h].T
    return P


def edited_keys(K, mask, U, alpha=None, g=1.0, head_enable=None):
    """k' = k + g P k on highlighted rows of one sequence; K is [L, Hkv, d]."""
    K = np.asarray(K, dtype=np.float64)
    out = K.copy()
    hl = np.asarray(mask) != 0
    for h in range(K.shape[1]):
        if head_enable is not None and not head_enable[h]:
            continue
        P = dense_projector(U, h, alpha)
        out[hl, h, :] = K[hl, h, :] + g * (K[hl, h, :] @ P.T)
    return out


def _softmax_causal(S):
    L = S.shape[0]
    S = np.where(np.tril(np.ones((L, L), dtype=bool)), S, -np.inf)
    m = S.max(axis=1, keepdims=True)
    E = np.exp(S - m)
    den = E.sum(axis=1, keepdims=True)
    return E / den, (m + np.log(den))[:, 0]


def attention_from_keys(Q, Kp, V, scale=None):
    """Materialised causal attention of one sequence; returns O [L,Hq,d], LSE [L,Hq]."""
    Q = np.asarray(Q, dtype=np.float64); Kp = np.asarray(Kp, dtype=np.float64); V = np.asarray(V, dtype=np.float64)
    L, Hq, d = Q.shape
    G = Hq // Kp.shape[1]
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    O = np.zeros((L, Hq, d)); LSE = np.zeros((L, Hq))
    for hq in range(Hq):
        h = hq // G
        P, lse = _softmax_causal(Q[:, hq, :] @ Kp[:, h, :].T * scale)
        O[:, hq, :] = P @ V[:, h, :]
        LSE[:, hq] = lse
    return O, LSE


def attention_logit_bias(Q, K, V, mask, U, alpha=None, g=1.0, head_enable=None, scale=None):
    """Eq. 5 route: logits = A + B with B_ij = q_i^T (g P k_j) * scale on highlighted columns only."""
    Q = np.asarray(Q, dtype=np.float64); K = np.asarray(K, dtype=np.float64); V = np.asarray(V, dtype=np.float64)
    L, Hq, d = Q.shape
    G = Hq // K.shape[1]
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    hl = (np.asarray(mask) != 0).astype(np.float64)
    O = np.zeros((L, Hq, d)); LSE = np.zeros((L, Hq))
    for hq in range(Hq):
        h = hq // G
        A = Q[:, hq, :] @ K[:, h, :].T * scale
        if head_enable is None or head_enable[h]:
            Pm = dense_projector(U, h, alpha)
            Bias = (Q[:, hq, :] @ (g * Pm) @ K[:, h, :].T) * scale * hl[None, :]
        else:
            Bias = 0.0
        P, lse = _softmax_causal(A + Bias)
        O[:, hq, :] = P @ V[:, h, :]
        LSE[:, hq] = lse
    return O, LSE


def two_projector_edit(K, mask, U_pos, k_pos, U_neg, k_neg, g_pos, g_neg, head_enable=None):
    """The general SEKA key edit, Eq. 4 with the projectors of Eq. 2, on one sequence (K is [L, Hkv, d]):

        P+ = U+[:, :k+] U+[:, :k+]^T          (leading k+ left-singular vectors of the positive cross-covariance)
        P- = U-[:, k-:] U-[:, k-:]^T          (the vectors AFTER the leading k- ones of the negative cross-covariance)
        k' = k + (g+ P+ k + g- P- k) / 2      at highlighted tokens, other tokens untouched.

    U_pos and U_neg are [Hkv, d, d] (full orthogonal factors, one per KV head); k_pos and k_neg are the ranks chosen
    by the variance criterion of Eq. 3.  Dense d x d projectors, fp64, no shortcuts.
    """
    K = np.asarray(K, dtype=np.float64)
    out = K.copy()
    hl = np.asarray(mask) != 0
    for h in range(K.shape[1]):
        if head_enable is not None and not head_enable[h]:
            continue
        Up = np.asarray(U_pos[h], dtype=np.float64)[:, :k_pos]
        Un = np.asarray(U_neg[h], dtype=np.float64)[:, k_neg:]
        P_pos = Up @ Up.T
        P_neg = Un @ Un.T
        for t in np.nonzero(hl)[0]:
            k = K[t, h]
            out[t, h] = k + (g_pos * (P_pos @ k) + g_neg * (P_neg @ k)) / 2.0
    return out


def rank_by_variance(S, gamma):
    """Eq. 3: the smallest k whose leading singular values hold at least the fraction gamma of their sum."""
    S = np.asarray(S, dtype=np.float64)
    c = np.cumsum(S) / np.sum(S)
    return int(np.searchsorted(c, gamma - 1e-15) + 1)
