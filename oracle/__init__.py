"""fp64 CPU oracle for SEKA / AdaSEKA steered attention -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper over ``seka_oracle.c`` (compiled on first use with gcc).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library never does, and this package never imports the
CUDA library.  All tensors are packed ``[total_tokens, heads, d]`` numpy arrays
with ``cu_seqlens`` (host list of B+1 offsets) delimiting the sequences; every
input is upcast to float64 and nothing is rounded afterwards.

Functions follow the paper: ``route`` is Eq. 6 (Section 3.3), ``edit_keys`` is
the hook of Algorithm 1/2 with k' = k + g P k (Section 2, Eq. 7), and
``attention_rows`` is causal softmax attention with the score of Section 2;
``decode_attention`` is the attention of one generated token over the whole
(already edited) key cache, the situation after the hook of Algorithm 1 has run
"before generation"; ``learn_projections`` is the offline spectral learning of
Section 3.1 (cross-covariances, SVD, the rank rule of Eq. 3) with the
head-selection statistic of Section 3.4.
The reading of the routing query under GQA (sum over the group's query heads)
is PARITY UNPINNED: the paper does not fix it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "seka_oracle.c")
_LIB = os.path.join(_HERE, "libseka_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        u8p = ctypes.POINTER(ctypes.c_uint8)
        i32p = ctypes.POINTER(ctypes.c_int32)
        ci = ctypes.c_int
        lib.seka_oracle_route.argtypes = [ci, ci, ci, ci, ci, ci, dp, dp, dp, dp]
        lib.seka_oracle_route.restype = None
        lib.seka_oracle_edit_keys.argtypes = [ci, ci, ci, ci, ci, dp, u8p, dp, dp, ctypes.c_double, u8p, dp]
        lib.seka_oracle_edit_keys.restype = None
        lib.seka_oracle_attention_rows.argtypes = [ci, ci, ci, ci, dp, dp, dp, ctypes.c_double, ci, i32p, dp, dp]
        lib.seka_oracle_attention_rows.restype = None
        lib.seka_oracle_threads.argtypes = []
        lib.seka_oracle_threads.restype = ci
        _lib = lib
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _dp(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _u8p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8))


def threads() -> int:
    """OpenMP threads the oracle uses for its independent loops."""
    return int(_load().seka_oracle_threads())


def route(Q, cu_seqlens: Sequence[int], U, sigma, k_route: int = 0) -> np.ndarray:
    """AdaSEKA coefficients alpha[B, Hkv, M] from each sequence's last-token query (Eq. 6)."""
    lib = _load()
    Q = _f64(Q); U = _f64(U); sigma = _f64(sigma)
    M, Hkv, d, r = U.shape
    Hq = Q.shape[1]
    k_route = r if k_route in (0, None) else int(k_route)
    assert 1 <= k_route <= r and sigma.shape == (M, Hkv, r) and Hq % Hkv == 0
    B = len(cu_seqlens) - 1
    alpha = np.zeros((B, Hkv, M), dtype=np.float64)
    for b in range(B):
        last = int(cu_seqlens[b + 1]) - 1
        if last < int(cu_seqlens[b]):
            continue                      # a sequence without tokens has no last query: alpha = 0, nothing to steer
        q_last = np.ascontiguousarray(Q[last])
        out = np.zeros((Hkv, M), dtype=np.float64)
        lib.seka_oracle_route(Hq, Hkv, d, r, M, k_route, _dp(q_last), _dp(U), _dp(sigma), _dp(out))
        alpha[b] = out
    return alpha


def edit_keys(K, mask, cu_seqlens: Sequence[int], U, alpha=None, gain=None, head_enable=None) -> np.ndarray:
    """Edited keys k' = k + g * sum_m alpha_m U_m U_m^T k at highlighted tokens (Algorithm 1/2 hook)."""
    lib = _load()
    K = _f64(K); U = _f64(U)
    M, Hkv, d, r = U.shape
    assert K.shape[1:] == (Hkv, d)
    B = len(cu_seqlens) - 1
    mask = np.ascontiguousarray(np.asarray(mask) != 0, dtype=np.uint8)
    gain = np.ones(B) if gain is None else np.broadcast_to(np.asarray(gain, dtype=np.float64), (B,))
    he = None if head_enable is None else np.ascontiguousarray(np.asarray(head_enable) != 0, dtype=np.uint8)
    out = np.empty_like(K)
    for b in range(B):
        s, e = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        if e == s:
            continue
        Kb = np.ascontiguousarray(K[s:e]); mb = np.ascontiguousarray(mask[s:e])
        ab = None if alpha is None else _f64(np.asarray(alpha)[b])
        ob = np.empty_like(Kb)
        lib.seka_oracle_edit_keys(e - s, Hkv, d, r, M, _dp(Kb), _u8p(mb), _dp(U), _dp(ab),
                                  float(gain[b]), _u8p(he), _dp(ob))
        out[s:e] = ob
    return out


def attention_rows(Q, Kp, V, cu_seqlens: Sequence[int], rows=None, scale: Optional[float] = None):
    """Causal softmax attention over (already edited) keys for chosen query rows.

    ``rows`` is None (every row) or a list with one int array of in-sequence
    positions per sequence.  Returns ``(O, LSE, index)``: O [n, Hq, d] and
    LSE [n, Hq] stacked over sequences, and ``index`` [n] the packed token index
    of each returned row.
    """
    lib = _load()
    Q = _f64(Q); Kp = _f64(Kp); V = _f64(V)
    Hq, d = Q.shape[1:]
    Hkv = Kp.shape[1]
    scale = 1.0 / np.sqrt(d) if not scale else float(scale)
    B = len(cu_seqlens) - 1
    Os, Ls, idx = [], [], []
    for b in range(B):
        s, e = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        rb = np.arange(e - s, dtype=np.int32) if rows is None else np.ascontiguousarray(rows[b], dtype=np.int32)
        if rb.size == 0:
            continue
        assert rb.min() >= 0 and rb.max() < e - s
        Qb = np.ascontiguousarray(Q[s:e]); Kb = np.ascontiguousarray(Kp[s:e]); Vb = np.ascontiguousarray(V[s:e])
        O = np.empty((rb.size, Hq, d)); LSE = np.empty((rb.size, Hq))
        lib.seka_oracle_attention_rows(e - s, Hq, Hkv, d, _dp(Qb), _dp(Kb), _dp(Vb), scale, rb.size,
                                       rb.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), _dp(O), _dp(LSE))
        Os.append(O); Ls.append(LSE); idx.append(rb.astype(np.int64) + s)
    if not Os:
        return np.zeros((0, Hq, d)), np.zeros((0, Hq)), np.zeros((0,), dtype=np.int64)
    return np.concatenate(Os), np.concatenate(Ls), np.concatenate(idx)


def seka_attention(Q, K, V, mask, cu_seqlens, U, alpha=None, gain=None, head_enable=None,
                   rows=None, scale: Optional[float] = None):
    """The whole steered path: edit the highlighted keys, then causal attention."""
    Kp = edit_keys(K, mask, cu_seqlens, U, alpha, gain, head_enable)
    return attention_rows(Q, Kp, V, cu_seqlens, rows, scale)


def decode_attention(q, Kp, V, cu_seqlens: Sequence[int], scale: Optional[float] = None):
    """Attention of one new query token per sequence over its whole cache of (already edited) keys.

    Algorithm 1 edits the prompt's keys once, before generation; every generated token then attends to
    all cached tokens with the score of Section 2: for sequence b and query head h (KV head h // G)
        O[b, h] = sum_j softmax_j(q[b, h] . k'_j * scale) v_j,   j over the sequence's cached tokens.
    q is [B, Hq, d]; Kp and V are packed [T, Hkv, d].  Returns O [B, Hq, d] and LSE [B, Hq] (natural log);
    a sequence without cached tokens gives O = 0 and LSE = -inf.  Written as the definition, in fp64.
    """
    q = _f64(q); Kp = _f64(Kp); V = _f64(V)
    B, Hq, d = q.shape
    Hkv = Kp.shape[1]
    assert Hq % Hkv == 0 and len(cu_seqlens) == B + 1
    G = Hq // Hkv
    scale = 1.0 / np.sqrt(d) if not scale else float(scale)
    O = np.zeros((B, Hq, d)); LSE = np.full((B, Hq), -np.inf)
    for b in range(B):
        s, e = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        if e == s:
            continue
        for h in range(Hq):
            logits = (Kp[s:e, h // G, :] @ q[b, h]) * scale
            top = logits.max()
            w = np.exp(logits - top)
            den = w.sum()
            O[b, h] = (w / den) @ V[s:e, h // G, :]
            LSE[b, h] = top + np.log(den)
    return O, LSE


def seka_decode(q, K, V, mask, cu_seqlens, U, alpha=None, gain=None, head_enable=None, scale: Optional[float] = None):
    """The decode path: edit the highlighted cached keys once, then one decode step over the edited cache."""
    Kp = edit_keys(K, mask, cu_seqlens, U, alpha, gain, head_enable)
    return decode_attention(q, Kp, V, cu_seqlens, scale)


def learn_projections(h, h_pos, h_neg, gamma: float, answer_tokens=None):
    """Offline spectral learning of the projections (Section 3.1, Eq. 2-3, first loop of Algorithm 1) and the
    head-selection statistic of Section 3.4, for every (layer, head) slot at once.

    h, h_pos, h_neg are the neutral / positive / negative key embeddings [n, H, d] (H runs over all (layer, KV head)
    pairs).  Per slot:  Omega+ = h^T h+ / n,  Omega- = h^T h- / n  (d x d);  SVD of each (numpy / LAPACK, singular
    values descending);  k+ / k- = the smallest k whose leading singular values hold at least the fraction gamma of
    their sum;  D = mean over the answer tokens of ||h+_i - h-_i||_2  (answer_tokens: boolean [n], default all).
    Returns a dict of fp64 arrays: omega_pos, omega_neg [H, d, d]; U_pos, U_neg [H, d, d] (columns = left singular
    vectors); S_pos, S_neg [H, d]; k_pos, k_neg [H] (int); D [H].
    """
    h = _f64(h); h_pos = _f64(h_pos); h_neg = _f64(h_neg)
    n, H, d = h.shape
    assert h_pos.shape == h.shape and h_neg.shape == h.shape and n > 0 and 0.0 < gamma <= 1.0
    sel = np.ones(n, dtype=bool) if answer_tokens is None else np.asarray(answer_tokens) != 0
    out = {"omega_pos": np.zeros((H, d, d)), "omega_neg": np.zeros((H, d, d)),
           "U_pos": np.zeros((H, d, d)), "U_neg": np.zeros((H, d, d)),
           "S_pos": np.zeros((H, d)), "S_neg": np.zeros((H, d)),
           "k_pos": np.zeros(H, dtype=np.int64), "k_neg": np.zeros(H, dtype=np.int64), "D": np.zeros(H)}

    def smallest_rank(S):
        total = S.sum()
        run = 0.0
        for k in range(1, d + 1):
            run += S[k - 1]
            if run >= gamma * total:
                return k
        return d

    for s in range(H):
        for tag, other in (("pos", h_pos), ("neg", h_neg)):
            omega = h[:, s, :].T @ other[:, s, :] / n
            U, S, _ = np.linalg.svd(omega)
            out["omega_" + tag][s] = omega
            out["U_" + tag][s] = U
            out["S_" + tag][s] = S
            out["k_" + tag][s] = smallest_rank(S)
        diff = h_pos[sel, s, :] - h_neg[sel, s, :]
        out["D"][s] = np.sqrt((diff * diff).sum(axis=1)).mean() if sel.any() else 0.0
    return out
