"""Pins for the fp64 CPU oracle: everything the paper and the mathematics fix, none of it
computed by the oracle itself.  CPU only."""
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import brute
from paper_2603_01281_b200 import inputs

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")))


def tiny(seed=1, L=48, Hq=4, Hkv=2, d=16, r=4, M=1, lens=None, mask_kind="spans", gain=0.7, highlight=0.3):
    return inputs.make_custom(seed=seed, dtype="f32", lens=lens or [L], n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d,
                              rank=r, n_experts=M, mask_kind=mask_kind, gain=gain, highlight=highlight)


# ----------------------------------------------------------------- hand-derived examples

def test_route_hand_case():
    g = GOLD["route"]
    U = np.array(g["U"], dtype=np.float64)            # [M=2, Hkv=1, d=3, r=2]
    sigma = np.array(g["sigma"], dtype=np.float64)
    q = np.array(g["q"], dtype=np.float64).reshape(1, 1, 3)
    np.testing.assert_allclose(oracle.route(q, [0, 1], U, sigma, 2)[0, 0], g["alpha_K2"], atol=1e-15)
    np.testing.assert_allclose(oracle.route(q, [0, 1], U, sigma, 1)[0, 0], g["alpha_K1"], atol=1e-15)
    # the routing query is the LAST token of the sequence; earlier tokens must not matter
    qq = np.concatenate([np.full((3, 1, 3), 9.0), q], axis=0)
    np.testing.assert_allclose(oracle.route(qq, [0, 4], U, sigma, 2)[0, 0], g["alpha_K2"], atol=1e-15)
    # GQA: the group's query heads are summed
    qh = np.array(g["q_heads"], dtype=np.float64).reshape(1, 2, 3)
    np.testing.assert_allclose(oracle.route(qh, [0, 1], U, sigma, 2)[0, 0], g["alpha_K2"], atol=1e-15)


def test_edit_hand_case():
    g = GOLD["edit"]
    k = np.array(g["k"], dtype=np.float64).reshape(1, 1, 3)
    U1 = np.array(g["u1"]).reshape(1, 1, 3, 1)
    out = oracle.edit_keys(k, [1], [0, 1], U1, gain=[g["g"]])
    np.testing.assert_allclose(out[0, 0], g["k_edit_single"], atol=1e-14)
    U2 = np.stack([np.array(g["u1"]).reshape(1, 3, 1), np.array(g["u2"]).reshape(1, 3, 1)])
    out = oracle.edit_keys(k, [1], [0, 1], U2, alpha=np.array(g["alpha"], dtype=float).reshape(1, 1, 2), gain=[g["g"]])
    np.testing.assert_allclose(out[0, 0], g["k_edit_blend"], atol=1e-14)
    # unhighlighted token: untouched
    assert np.array_equal(oracle.edit_keys(k, [0], [0, 1], U1, gain=[g["g"]]), k)


def test_attention_hand_case():
    g = GOLD["attention"]
    Q = np.zeros((2, 1, 4)); Q[:, 0, 0] = 2.0
    K = np.zeros((2, 1, 4)); K[1, 0, 0] = math.log(3.0)
    V = np.zeros((2, 1, 4)); V[0, 0, :] = 4.0; V[1, 0, :] = 8.0
    O, LSE, idx = oracle.attention_rows(Q, K, V, [0, 2])
    np.testing.assert_allclose(O[1, 0], g["o1_plain"], atol=1e-14)
    np.testing.assert_allclose(O[0, 0], 4.0, atol=1e-14)
    np.testing.assert_allclose(LSE[:, 0], [0.0, math.log(4.0)], atol=1e-14)
    U = np.eye(4).reshape(1, 1, 4, 4)
    O, LSE, _ = oracle.seka_attention(Q, K, V, [0, 1], [0, 2], U, gain=[1.0])
    np.testing.assert_allclose(O[1, 0], g["o1_steered"], atol=1e-14)
    np.testing.assert_allclose(LSE[1, 0], math.log(10.0), atol=1e-14)


# ----------------------------------------------------------------- key edit: Appendix C closed forms

@pytest.mark.parametrize("g", [0.5, 1.0, -0.4, -5.0, 2.0])
def test_edit_closed_form_eq12(g):
    w = tiny(seed=3, gain=g)
    g = float(w.gain[0])          # the gain as stored (fp32)
    Kp = oracle.edit_keys(w.K, w.mask, w.cu_seqlens, w.U, gain=w.gain)
    K = w.K.astype(np.float64)
    hl = w.mask != 0
    assert hl.any() and (~hl).any()
    for h in range(w.n_kv_heads):
        U = w.U[0, h].astype(np.float64)
        # exactly orthonormal factor for the closed form (the stored fp32 U is only nearly so)
        Uo, _ = np.linalg.qr(U)
        Kpo = oracle.edit_keys(w.K, w.mask, w.cu_seqlens, np.broadcast_to(Uo, (1, w.n_kv_heads) + Uo.shape), gain=w.gain)
        par = K[hl, h] @ Uo @ Uo.T
        perp = K[hl, h] - par
        # Eq. 12: (I + g U U^T) x = x_perp + (1+g) x_par
        np.testing.assert_allclose(Kpo[hl, h], perp + (1 + g) * par, atol=1e-12)
        np.testing.assert_allclose(Kpo[hl, h] @ Uo, (1 + g) * (K[hl, h] @ Uo), atol=1e-12)
        np.testing.assert_allclose(np.sum(Kpo[hl, h] ** 2, -1),
                                   np.sum(perp ** 2, -1) + (1 + g) ** 2 * np.sum(par ** 2, -1), rtol=1e-12)
        # stored-U version: U (U^T k) as written
        np.testing.assert_allclose(Kp[hl, h], K[hl, h] + g * (K[hl, h] @ U) @ U.T, atol=1e-12)
    # every unhighlighted key is bit-identical
    assert np.array_equal(Kp[~hl], K[~hl])


def test_projector_idempotent_symmetric_and_full_rank_edit():
    rng = np.random.default_rng(0)
    U = inputs.orthonormal_bank(rng, 1, 2, 16, 16).astype(np.float64)
    Uq, _ = np.linalg.qr(U[0, 0])
    P = brute.dense_projector(Uq[None, None, :, :5], 0)
    np.testing.assert_allclose(P @ P, P, atol=1e-13)
    np.testing.assert_allclose(P, P.T, atol=0)
    # generated banks are orthonormal to fp32 accuracy
    np.testing.assert_allclose(U[0, 1].T @ U[0, 1], np.eye(16), atol=1e-6)
    # r = d with orthogonal U: k' = (1+g) k
    K = rng.standard_normal((5, 1, 16))
    Kp = oracle.edit_keys(K, np.ones(5), [0, 5], Uq[None, None], gain=[1.5])
    np.testing.assert_allclose(Kp, 2.5 * K, atol=1e-12)


def test_edit_head_enable_and_per_sequence_gain():
    w = tiny(seed=5, lens=[20, 33, 7], gain=[0.5, -1.0, 2.0], Hkv=2)
    he = np.array([1, 0], dtype=np.uint8)
    Kp = oracle.edit_keys(w.K, w.mask, w.cu_seqlens, w.U, gain=w.gain, head_enable=he)
    K = w.K.astype(np.float64)
    assert np.array_equal(Kp[:, 1], K[:, 1])             # unselected head untouched (Section 3.4)
    for b in range(3):
        s, e = w.cu_seqlens[b], w.cu_seqlens[b + 1]
        ref = brute.edited_keys(w.K[s:e], w.mask[s:e], w.U, g=float(w.gain[b]), head_enable=he)
        np.testing.assert_allclose(Kp[s:e], ref, atol=1e-12)


# ----------------------------------------------------------------- attention

def test_g0_and_empty_mask_are_textbook_causal_attention():
    w = tiny(seed=7, L=40, Hq=4, Hkv=2, d=16)
    Qt = torch.from_numpy(w.Q.astype(np.float64)).permute(1, 0, 2)[None]
    Kt = torch.from_numpy(w.K.astype(np.float64)).permute(1, 0, 2)[None].repeat_interleave(2, dim=1)
    Vt = torch.from_numpy(w.V.astype(np.float64)).permute(1, 0, 2)[None].repeat_interleave(2, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(Qt, Kt, Vt, is_causal=True)[0].permute(1, 0, 2).numpy()
    O0, _, _ = oracle.seka_attention(w.Q, w.K, w.V, w.mask, w.cu_seqlens, w.U, gain=[0.0])
    np.testing.assert_allclose(O0, ref, atol=1e-12)
    O1, _, _ = oracle.seka_attention(w.Q, w.K, w.V, np.zeros_like(w.mask), w.cu_seqlens, w.U, gain=[3.0])
    np.testing.assert_allclose(O1, ref, atol=1e-12)
    # GQA map: consecutive query heads share a KV head -- swapping which KV head a query head reads must break it
    bad = torch.nn.functional.scaled_dot_product_attention(
        Qt, Kt[:, [0, 2, 1, 3]], Vt[:, [0, 2, 1, 3]], is_causal=True)[0].permute(1, 0, 2).numpy()
    assert np.abs(bad - O0).max() > 1e-3


def test_rows_sum_to_one_first_row_and_lse():
    w = tiny(seed=8, L=37)
    ones = np.ones_like(w.V)
    O, LSE, idx = oracle.seka_attention(w.Q, w.K, ones, w.mask, w.cu_seqlens, w.U, gain=w.gain)
    np.testing.assert_allclose(O, 1.0, atol=1e-13)                    # softmax rows sum to 1
    O, LSE, idx = oracle.seka_attention(w.Q, w.K, w.V, w.mask, w.cu_seqlens, w.U, gain=w.gain)
    G = w.n_q_heads // w.n_kv_heads
    np.testing.assert_allclose(O[0], np.repeat(w.V[0].astype(np.float64), G, axis=0), atol=1e-13)   # o_0 = v_0
    # a future key must not matter (causality): perturb the last key/value, earlier rows unchanged
    K2 = w.K.copy(); V2 = w.V.copy(); K2[-1] += 5.0; V2[-1] -= 3.0
    O2, _, _ = oracle.seka_attention(w.Q, K2, V2, w.mask, w.cu_seqlens, w.U, gain=w.gain)
    assert np.array_equal(O2[:-1], O[:-1]) and not np.allclose(O2[-1], O[-1])


@pytest.mark.parametrize("M", [1, 3])
def test_brute_force_and_logit_bias_identity(M):
    # Eq. 5: attention over edited keys == attention over logits A + B, B the low-rank bias on highlighted columns
    w = tiny(seed=11 + M, L=53, Hq=6, Hkv=2, d=16, r=4, M=M, gain=1.3)
    rng = np.random.default_rng(2)
    alpha = rng.uniform(-1, 1, size=(1, w.n_kv_heads, M)) if M > 1 else None
    he = np.array([1, 1], dtype=np.uint8)
    O, LSE, _ = oracle.seka_attention(w.Q, w.K, w.V, w.mask, w.cu_seqlens, w.U, alpha=alpha, gain=w.gain, head_enable=he)
    a0 = None if alpha is None else alpha[0]
    Ob, Lb = brute.attention_from_keys(w.Q, brute.edited_keys(w.K, w.mask, w.U, a0, float(w.gain[0])), w.V)
    np.testing.assert_allclose(O, Ob, atol=1e-12); np.testing.assert_allclose(LSE, Lb, atol=1e-12)
    Oc, Lc = brute.attention_logit_bias(w.Q, w.K, w.V, w.mask, w.U, a0, float(w.gain[0]))
    np.testing.assert_allclose(O, Oc, atol=1e-12); np.testing.assert_allclose(LSE, Lc, atol=1e-12)


def test_query_side_duality():
    # Section 2: the same logits arise from editing the query, ((I + gP) q)^T k on highlighted columns
    w = tiny(seed=21, L=30, Hq=2, Hkv=2, d=16, r=5, gain=0.9)
    Kp = oracle.edit_keys(w.K, w.mask, w.cu_seqlens, w.U, gain=w.gain)
    hl = w.mask != 0
    for h in range(2):
        P = brute.dense_projector(w.U, h)
        Qe = w.Q[:, h].astype(np.float64) @ (np.eye(16) + float(w.gain[0]) * P).T
        S_key = w.Q[:, h].astype(np.float64) @ Kp[:, h].T
        S_dual = np.where(hl[None, :], Qe @ w.K[:, h].astype(np.float64).T, w.Q[:, h].astype(np.float64) @ w.K[:, h].astype(np.float64).T)
        np.testing.assert_allclose(S_key, S_dual, atol=1e-12)


def test_identity_projector_scales_highlighted_scores():
    # P = I: the scores of highlighted columns are multiplied by (1+g), the others unchanged
    w = tiny(seed=31, L=29, Hq=2, Hkv=1, d=8, r=8, gain=0.6)
    U = np.eye(8).reshape(1, 1, 8, 8)
    O, LSE, _ = oracle.seka_attention(w.Q, w.K, w.V, w.mask, w.cu_seqlens, U, gain=w.gain)
    hl = w.mask != 0
    for hq in range(2):
        S = w.Q[:, hq].astype(np.float64) @ w.K[:, 0].astype(np.float64).T / math.sqrt(8)
        S = np.where(hl[None, :], (1.0 + float(w.gain[0])) * S, S)
        P, lse = brute._softmax_causal(S)
        np.testing.assert_allclose(O[:, hq], P @ w.V[:, 0].astype(np.float64), atol=1e-12)
        np.testing.assert_allclose(LSE[:, hq], lse, atol=1e-12)


def test_varlen_sequences_are_independent_and_rows_subset():
    w = tiny(seed=41, lens=[17, 1, 40], Hq=4, Hkv=2, d=16, gain=[0.5, 1.0, 2.0])
    O, LSE, idx = oracle.seka_attention(w.Q, w.K, w.V, w.mask, w.cu_seqlens, w.U, gain=w.gain)
    assert list(idx) == list(range(58))
    for b in range(3):
        s, e = w.cu_seqlens[b], w.cu_seqlens[b + 1]
        Ob, _ = brute.attention_from_keys(w.Q[s:e], brute.edited_keys(w.K[s:e], w.mask[s:e], w.U, None, float(w.gain[b])), w.V[s:e])
        np.testing.assert_allclose(O[s:e], Ob, atol=1e-12)
    rows = [np.array([0, 16]), np.array([0]), np.array([5, 39])]
    Os, Ls, ids = oracle.seka_attention(w.Q, w.K, w.V, w.mask, w.cu_seqlens, w.U, gain=w.gain, rows=rows)
    np.testing.assert_allclose(Os, O[ids], atol=0); np.testing.assert_allclose(Ls, LSE[ids], atol=0)


def test_softmax_scale_override():
    w = tiny(seed=51, L=12, Hq=2, Hkv=2, d=16)
    O, _, _ = oracle.attention_rows(w.Q, w.K, w.V, w.cu_seqlens, scale=0.37)
    Ob, _ = brute.attention_from_keys(w.Q, w.K, w.V, scale=0.37)
    np.testing.assert_allclose(O, Ob, atol=1e-12)


# ----------------------------------------------------------------- AdaSEKA

def test_single_expert_unit_alpha_is_seka():
    w = tiny(seed=61, L=25)
    a = oracle.edit_keys(w.K, w.mask, w.cu_seqlens, w.U, gain=w.gain)
    b = oracle.edit_keys(w.K, w.mask, w.cu_seqlens, w.U, alpha=np.ones((1, w.n_kv_heads, 1)), gain=w.gain)
    assert np.array_equal(a, b)


def test_routing_of_an_empty_sequence_is_zero():
    w = tiny(seed=8, lens=[5, 0, 7], M=3, r=4)
    a = oracle.route(w.Q, w.cu_seqlens, w.U, w.sigma, 0)
    assert np.all(a[1] == 0.0) and np.all(np.abs(a[[0, 2]]).max(-1) == 1.0)
    # the neighbours are what they are without the empty sequence in between
    w2_cu = np.array([0, 5, 12])
    np.testing.assert_array_equal(a[[0, 2]], oracle.route(w.Q, w2_cu, w.U, w.sigma, 0))


def test_routing_invariants():
    w = inputs.make_custom(seed=71, dtype="f32", lens=[9, 14], n_q_heads=8, n_kv_heads=2, head_dim=16, rank=6,
                           n_experts=4, gain=1.0)
    a = oracle.route(w.Q, w.cu_seqlens, w.U, w.sigma, 5)
    assert a.shape == (2, 2, 4)
    np.testing.assert_allclose(np.abs(a).max(axis=-1), 1.0, atol=1e-15)          # max_m |alpha_m| = 1
    np.testing.assert_allclose(oracle.route(3.7 * w.Q.astype(np.float64), w.cu_seqlens, w.U, w.sigma, 5), a, atol=1e-12)
    np.testing.assert_allclose(oracle.route(-w.Q, w.cu_seqlens, w.U, w.sigma, 5), -a, atol=1e-12)
    # direct evaluation of Eq. 6 with matrix products
    for b in range(2):
        q = w.Q[w.cu_seqlens[b + 1] - 1].astype(np.float64).reshape(2, 4, 16).sum(axis=1)    # [Hkv, d]
        for h in range(2):
            s = np.array([(q[h] @ w.U[m, h].astype(np.float64)[:, :5]) @ w.sigma[m, h, :5].astype(np.float64) for m in range(4)])
            np.testing.assert_allclose(a[b, h], s / np.abs(s).max(), atol=1e-12)
    # k_route = 0 means every stored component
    np.testing.assert_allclose(oracle.route(w.Q, w.cu_seqlens, w.U, w.sigma, 0),
                               oracle.route(w.Q, w.cu_seqlens, w.U, w.sigma, 6), atol=0)
    # all-zero query: alpha = 0
    assert np.array_equal(oracle.route(np.zeros_like(w.Q), w.cu_seqlens, w.U, w.sigma, 5), np.zeros((2, 2, 4)))


def test_blend_factor_form_equals_dense_projector():
    w = inputs.make_custom(seed=81, dtype="f32", lens=[31], n_q_heads=4, n_kv_heads=2, head_dim=16, rank=4,
                           n_experts=4, gain=1.1, highlight=0.4)
    a = oracle.route(w.Q, w.cu_seqlens, w.U, w.sigma, 0)
    Kp = oracle.edit_keys(w.K, w.mask, w.cu_seqlens, w.U, alpha=a, gain=w.gain)
    np.testing.assert_allclose(Kp, brute.edited_keys(w.K, w.mask, w.U, a[0], float(w.gain[0])), atol=1e-12)


# ----------------------------------------------------------------- two-projector edit (Eq. 2-4)

def _two_bases(seed, Hkv, d):
    rng = np.random.default_rng(seed)
    Up = np.stack([np.linalg.qr(rng.standard_normal((d, d)))[0] for _ in range(Hkv)])
    Un = np.stack([np.linalg.qr(rng.standard_normal((d, d)))[0] for _ in range(Hkv)])
    return Up, Un


def test_two_projector_edit_closed_forms():
    from oracle import brute
    d, Hkv, L = 16, 2, 12
    Up, Un = _two_bases(5, Hkv, d)
    rng = np.random.default_rng(6)
    mask = np.zeros(L, dtype=np.uint8); mask[[1, 4, 5, 11]] = 1
    k_pos, k_neg, gp, gn = 3, 10, 0.8, -0.6
    # a key inside span(U+[:, :k+]) and orthogonal to span(U-[:, k-:]) is scaled by (1 + g+/2); build one by projecting
    h = 0
    Pn = Un[h][:, k_neg:] @ Un[h][:, k_neg:].T
    Pp = Up[h][:, :k_pos] @ Up[h][:, :k_pos].T
    K = rng.standard_normal((L, Hkv, d))
    out = brute.two_projector_edit(K, mask, Up, k_pos, Un, k_neg, gp, gn)
    hl = mask != 0
    assert np.array_equal(out[~hl], K[~hl])                                   # untouched rows
    for t in np.nonzero(hl)[0]:
        k = K[t, h]
        np.testing.assert_allclose(out[t, h], k + 0.5 * gp * Pp @ k + 0.5 * gn * Pn @ k, atol=1e-13)
        # components: along a leading positive vector the edit adds g+/2 of it (plus what P- sees of it)
        u = Up[h][:, 0]
        np.testing.assert_allclose(u @ out[t, h], u @ k + 0.5 * gp * (u @ k) + 0.5 * gn * (u @ (Pn @ k)), atol=1e-13)
    # g- = 0 reduces to the single-projector edit with gain g+/2 (checked against the C oracle)
    out1 = brute.two_projector_edit(K, mask, Up, k_pos, Un, k_neg, gp, 0.0)
    ref = oracle.edit_keys(K, mask, [0, L], Up[None, :, :, :k_pos], gain=gp / 2)
    np.testing.assert_allclose(out1, ref, atol=1e-13)
    # k- = 0 and g+ = 0: P- is the identity, every highlighted key is scaled by (1 + g-/2)
    out2 = brute.two_projector_edit(K, mask, Up, k_pos, Un, 0, 0.0, gn)
    np.testing.assert_allclose(out2[hl], (1 + gn / 2) * K[hl], atol=1e-13)
    # the trailing vectors are used, not the leading ones: swapping them changes the result
    out3 = brute.two_projector_edit(K, mask, Up, k_pos, Un[:, :, ::-1], k_neg, gp, gn)
    assert np.abs(out3 - out).max() > 1e-3


def test_rank_by_variance_rule():
    from oracle import brute
    S = np.array([4.0, 3.0, 2.0, 1.0])            # cumulative fractions 0.4, 0.7, 0.9, 1.0
    assert [brute.rank_by_variance(S, g) for g in (0.3, 0.4, 0.41, 0.7, 0.9, 0.95, 1.0)] == [1, 1, 2, 2, 3, 4, 4]


# ----------------------------------------------------------------- decode step over the edited cache

def _decode_case(seed=5, lens=(37, 1, 64), Hq=6, Hkv=2, d=16):
    rng = np.random.default_rng(seed)
    T = int(sum(lens))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    q = rng.standard_normal((len(lens), Hq, d))
    K = rng.standard_normal((T, Hkv, d))
    V = rng.standard_normal((T, Hkv, d))
    return q, K, V, cu


def test_decode_hand_case_and_pure_python_loops():
    # two cached tokens, scores 0 and ln 3 (scale 1/sqrt(4) = 1/2, q.k = 2 ln 3): weights 1/4 and 3/4
    q = np.zeros((1, 1, 4)); q[0, 0, 0] = 2.0
    K = np.zeros((2, 1, 4)); K[1, 0, 0] = math.log(3.0)
    V = np.zeros((2, 1, 4)); V[0, 0, :] = 4.0; V[1, 0, :] = 8.0
    O, LSE = oracle.decode_attention(q, K, V, [0, 2])
    np.testing.assert_allclose(O[0, 0], 7.0, atol=1e-14)
    np.testing.assert_allclose(LSE[0, 0], math.log(4.0), atol=1e-14)
    # scalar loops on a tiny random case, GQA group of 3
    q, K, V, cu = _decode_case(lens=(5, 3), Hq=6, Hkv=2, d=4)
    O, LSE = oracle.decode_attention(q, K, V, cu)
    for b in range(2):
        for h in range(6):
            num = [0.0] * 4; den = 0.0
            for t in range(int(cu[b]), int(cu[b + 1])):
                s = sum(q[b, h, c] * K[t, h // 3, c] for c in range(4)) / 2.0
                den += math.exp(s)
                for c in range(4):
                    num[c] += math.exp(s) * V[t, h // 3, c]
            np.testing.assert_allclose(O[b, h], [x / den for x in num], rtol=1e-12)
            np.testing.assert_allclose(LSE[b, h], math.log(den), rtol=1e-12)


def test_decode_is_the_last_row_of_causal_attention():
    # a generated token that attends to its whole cache is the last row of causal attention
    # (the C routine is a separate implementation)
    q, K, V, cu = _decode_case()
    Q = np.zeros((K.shape[0], q.shape[1], q.shape[2]))
    for b in range(q.shape[0]):
        Q[cu[b + 1] - 1] = q[b]
    rows = [np.array([cu[b + 1] - cu[b] - 1]) for b in range(q.shape[0])]
    O_ref, L_ref, _ = oracle.attention_rows(Q, K, V, cu, rows)
    O, LSE = oracle.decode_attention(q, K, V, cu)
    np.testing.assert_allclose(O, O_ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(LSE, L_ref, rtol=1e-12, atol=1e-13)


def test_decode_closed_forms():
    q, K, V, cu = _decode_case()
    O, LSE = oracle.decode_attention(q, K, V, cu)
    B, Hq, d = q.shape
    G = Hq // K.shape[1]
    # equal keys: uniform weights, the output is the mean value and LSE = score + ln L
    Ke = np.broadcast_to(K[:1], K.shape).copy()
    Oe, Le = oracle.decode_attention(q, Ke, V, cu)
    for b in range(B):
        s, e = int(cu[b]), int(cu[b + 1])
        for h in range(Hq):
            np.testing.assert_allclose(Oe[b, h], V[s:e, h // G].mean(axis=0), rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(Le[b, h], q[b, h] @ Ke[0, h // G] / math.sqrt(d) + math.log(e - s), rtol=1e-12)
    # adding one vector c to every key shifts all scores of a head alike: O unchanged, LSE + q.c * scale
    c = np.random.default_rng(9).standard_normal((K.shape[1], d))
    Os, Ls = oracle.decode_attention(q, K + c[None], V, cu)
    np.testing.assert_allclose(Os, O, rtol=1e-10, atol=1e-12)
    shift = np.einsum("bhd,hd->bh", q, np.repeat(c, G, axis=0)) / math.sqrt(d)
    np.testing.assert_allclose(Ls, LSE + shift, rtol=1e-12, atol=1e-12)
    # one key far along q dominates: the output is that token's value
    Kd = K.copy(); t = int(cu[0]) + 3
    Kd[t, 0] = 200.0 * q[0, 0] / np.linalg.norm(q[0, 0])
    Od, _ = oracle.decode_attention(q, Kd, V, cu)
    np.testing.assert_allclose(Od[0, 0], V[t, 0], atol=1e-9)
    # values enter linearly; a sequence with one cached token returns that token's value
    O2, _ = oracle.decode_attention(q, K, 2.0 * V + 1.0, cu)
    np.testing.assert_allclose(O2, 2.0 * O + 1.0, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(O[1], np.repeat(V[cu[1]], G, axis=0), atol=1e-14)
    # softmax scale override and an empty cache
    O3, _ = oracle.decode_attention(q, K, V, cu, scale=0.5)
    O4, _ = oracle.decode_attention(q * 0.5 * math.sqrt(d), K, V, cu)
    np.testing.assert_allclose(O3, O4, rtol=1e-12, atol=1e-13)
    Oz, Lz = oracle.decode_attention(q[:1], K[:0], V[:0], [0, 0])
    assert np.all(Oz == 0) and np.all(np.isneginf(Lz))


def test_decode_over_edited_cache_uses_edited_keys():
    # highlighted tokens with the identity projector (full rank) have their scores multiplied by 1 + g (Eq. 12)
    w = tiny(seed=4, L=40, d=8, r=8, gain=1.5)
    q = np.random.default_rng(2).standard_normal((1, w.n_q_heads, w.head_dim))
    U = np.broadcast_to(np.eye(8), (1, w.n_kv_heads, 8, 8)).copy()
    O, LSE = oracle.seka_decode(q, w.K, w.V, w.mask, w.cu_seqlens, U, gain=w.gain)
    Kp = w.K.astype(np.float64).copy()
    Kp[w.mask != 0] *= 1.0 + 1.5
    O_ref, L_ref = oracle.decode_attention(q, Kp, w.V, w.cu_seqlens)
    np.testing.assert_allclose(O, O_ref, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(LSE, L_ref, rtol=1e-10, atol=1e-12)


# ----------------------------------------------------------------- offline spectral learning (Section 3.1, Eq. 2-3, Section 3.4)

def test_learner_hand_case():
    # Omega+ = h^T h+ / 2 = diag(1.5, 1); Omega- = diag(0.5, 2): singular values sorted descending
    h = np.array([[1.0, 0.0], [0.0, 2.0]]).reshape(2, 1, 2)
    hp = np.array([[3.0, 0.0], [0.0, 1.0]]).reshape(2, 1, 2)
    hn = np.array([[1.0, 0.0], [0.0, 2.0]]).reshape(2, 1, 2)
    r = oracle.learn_projections(h, hp, hn, gamma=0.6)
    np.testing.assert_allclose(r["omega_pos"][0], np.diag([1.5, 1.0]), atol=1e-15)
    np.testing.assert_allclose(r["S_pos"][0], [1.5, 1.0], atol=1e-15)
    np.testing.assert_allclose(np.abs(r["U_pos"][0]), np.eye(2), atol=1e-15)
    np.testing.assert_allclose(r["S_neg"][0], [2.0, 0.5], atol=1e-15)
    np.testing.assert_allclose(np.abs(r["U_neg"][0]), [[0, 1], [1, 0]], atol=1e-15)      # the second axis leads
    assert r["k_pos"][0] == 1 and r["k_neg"][0] == 1                  # 1.5 / 2.5 = 0.6 and 2 / 2.5 = 0.8 reach gamma
    assert oracle.learn_projections(h, hp, hn, gamma=0.61)["k_pos"][0] == 2
    # D: ||h+ - h-|| per token = 2 and 1; mean 1.5; only the second token an answer token -> 1
    np.testing.assert_allclose(r["D"][0], 1.5, atol=1e-15)
    np.testing.assert_allclose(oracle.learn_projections(h, hp, hn, 0.6, answer_tokens=[0, 1])["D"][0], 1.0, atol=1e-15)


def test_learner_orientation_of_the_cross_covariance():
    # Section 3.1: Omega+ = h^T h+ / n and U+ = its LEFT singular vectors.  One token, h = e1, h+ = 2 e2, h- = 3 e3:
    # Omega+ = e1 (2 e2)^T has its only non-zero entry at (row 1, column 2), so the leading left vector is e1 (the
    # neutral direction) and the leading right vector e2.  The transposed product h+^T h / n would put the entry at
    # (2, 1) and return e2: this case tells the two apart (diagonal or symmetric Omega cannot).
    h = np.array([1.0, 0.0, 0.0]).reshape(1, 1, 3)
    hp = np.array([0.0, 2.0, 0.0]).reshape(1, 1, 3)
    hn = np.array([0.0, 0.0, 3.0]).reshape(1, 1, 3)
    r = oracle.learn_projections(h, hp, hn, gamma=0.5)
    expect_pos = np.zeros((3, 3)); expect_pos[0, 1] = 2.0
    expect_neg = np.zeros((3, 3)); expect_neg[0, 2] = 3.0
    np.testing.assert_allclose(r["omega_pos"][0], expect_pos, atol=1e-15)
    np.testing.assert_allclose(r["omega_neg"][0], expect_neg, atol=1e-15)
    np.testing.assert_allclose(r["S_pos"][0], [2.0, 0.0, 0.0], atol=1e-15)
    np.testing.assert_allclose(r["S_neg"][0], [3.0, 0.0, 0.0], atol=1e-15)
    np.testing.assert_allclose(np.abs(r["U_pos"][0][:, 0]), [1.0, 0.0, 0.0], atol=1e-15)
    np.testing.assert_allclose(np.abs(r["U_neg"][0][:, 0]), [1.0, 0.0, 0.0], atol=1e-15)
    assert r["k_pos"][0] == 1 and r["k_neg"][0] == 1
    # a second token makes the picture generic: h = (e1, e2), h+ = (2 e2, 5 e3): Omega+ = (e1 (2 e2)^T + e2 (5 e3)^T) / 2,
    # left vectors in order e2 (value 2.5), e1 (value 1); the transposed product would give e3, e2
    h2 = np.array([[1.0, 0, 0], [0, 1.0, 0]]).reshape(2, 1, 3)
    hp2 = np.array([[0, 2.0, 0], [0, 0, 5.0]]).reshape(2, 1, 3)
    r2 = oracle.learn_projections(h2, hp2, hp2, gamma=0.9)
    np.testing.assert_allclose(r2["S_pos"][0], [2.5, 1.0, 0.0], atol=1e-15)
    np.testing.assert_allclose(np.abs(r2["U_pos"][0][:, :2]), [[0, 1], [1, 0], [0, 0]], atol=1e-15)
    assert r2["k_pos"][0] == 2          # 2.5 / 3.5 < 0.9


def test_learner_recovers_a_planted_subspace_exactly():
    # neutral keys with h^T h / n = I exactly, positive keys h (I + a B B^T), negative keys h (I - b B B^T):
    # Omega+ = I + a B B^T and Omega- = I - b B B^T, whose spectra and subspaces are known in closed form
    rng = np.random.default_rng(3)
    n, d, r, a, b = 200, 12, 3, 2.0, 0.75
    qf, _ = np.linalg.qr(rng.standard_normal((n, d)))
    h = math.sqrt(n) * qf
    B, _ = np.linalg.qr(rng.standard_normal((d, r)))
    PB = B @ B.T
    hp = h @ (np.eye(d) + a * PB); hn = h @ (np.eye(d) - b * PB)
    gamma = 0.55          # 0.5 would put the threshold exactly on the sum of the three leading values
    out = oracle.learn_projections(h[:, None, :], hp[:, None, :], hn[:, None, :], gamma)
    np.testing.assert_allclose(out["omega_pos"][0], np.eye(d) + a * PB, atol=1e-12)
    np.testing.assert_allclose(out["S_pos"][0], [1 + a] * r + [1.0] * (d - r), atol=1e-12)
    np.testing.assert_allclose(out["S_neg"][0], [1.0] * (d - r) + [1 - b] * r, atol=1e-12)
    U = out["U_pos"][0]
    np.testing.assert_allclose(U.T @ U, np.eye(d), atol=1e-12)
    np.testing.assert_allclose(U[:, :r] @ U[:, :r].T, PB, atol=1e-10)                     # P+ of Eq. 2 with k+ = r
    Un = out["U_neg"][0]
    np.testing.assert_allclose(Un[:, d - r:] @ Un[:, d - r:].T, PB, atol=1e-10)           # P- of Eq. 2 with k- = d - r
    # Eq. 3 in closed form: the total is d + a r; k leading values of 1 + a, then ones
    total = d + a * r
    k_expect = next(k for k in range(1, d + 1) if (min(k, r) * (1 + a) + max(0, k - r)) >= gamma * total - 1e-12)
    assert out["k_pos"][0] == k_expect
    assert out["k_pos"][0] == brute.rank_by_variance(out["S_pos"][0], gamma)
    assert out["k_neg"][0] == brute.rank_by_variance(out["S_neg"][0], gamma)
    # D: h+ - h- = (a + b) h B B^T, so each token's distance is (a + b) ||B^T h_i||
    np.testing.assert_allclose(out["D"][0], ((a + b) * np.linalg.norm(h @ B, axis=1)).mean(), rtol=1e-12)


def test_learner_invariants_on_the_synthetic_embeddings():
    h, hp, hn, ans, bases, strength = inputs.contrastive_embeddings(seed=1, n=600, slots=5, head_dim=16, rank=3, dtype="f32")
    out = oracle.learn_projections(h, hp, hn, 0.7, answer_tokens=ans)
    for s in range(5):
        for tag in ("pos", "neg"):
            Om, U, S = out["omega_" + tag][s], out["U_" + tag][s], out["S_" + tag][s]
            assert np.all(np.diff(S) <= 1e-15) and np.all(S >= 0)
            np.testing.assert_allclose(U.T @ U, np.eye(16), atol=1e-12)
            np.testing.assert_allclose(Om @ Om.T @ U, U * (S * S), atol=1e-12)            # left singular vectors
            assert out["k_" + tag][s] == brute.rank_by_variance(S, 0.7)
    # repeating every token leaves the cross-covariances and D unchanged (the 1/n of Section 3.1)
    rep = oracle.learn_projections(np.tile(h, (2, 1, 1)), np.tile(hp, (2, 1, 1)), np.tile(hn, (2, 1, 1)), 0.7,
                                   answer_tokens=np.tile(ans, 2))
    np.testing.assert_allclose(rep["omega_pos"], out["omega_pos"], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(rep["D"], out["D"], rtol=1e-12)
    # slots are independent, and a head that does not react (strength 0) has the smallest distance
    one = oracle.learn_projections(h[:, 2:3], hp[:, 2:3], hn[:, 2:3], 0.7, answer_tokens=ans)
    np.testing.assert_array_equal(one["omega_neg"][0], out["omega_neg"][2])
    assert np.argmin(out["D"]) == 3 and strength[3] == 0.0
