"""GPU parity: the CUDA path (through the C ABI) against the fp64 CPU oracle on identical seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_01281_b200 import binding, inputs

import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load()          # raises if the compiled library is missing: there is no fallback


# ----------------------------------------------------------------- routing (Eq. 6)

@pytest.mark.parametrize("case", ["C3", "small_f32", "small_varlen"])
def test_route_matches_oracle(case):
    if case == "C3":
        w = inputs.make_workload("C3"); k_route = 0
    elif case == "small_f32":
        w = inputs.make_custom(seed=5, dtype="f32", lens=[40, 40], n_q_heads=8, n_kv_heads=2, head_dim=64, rank=16,
                               n_experts=3); k_route = 5
    else:
        w = inputs.make_custom(seed=6, dtype="bf16", lens=[17, 300, 1], n_q_heads=14, n_kv_heads=2, head_dim=128,
                               rank=8, n_experts=4); k_route = 8
    dev = H.device_tensors(w)
    shp = H.shape_of(w, dev)
    alpha = torch.full((w.batch, w.n_kv_heads, w.n_experts), float("nan"), device="cuda")
    binding.adaseka_route(shp, dev["Q"], dev["U"], dev["sigma"], k_route, alpha)
    ref = oracle.route(w.Q, w.cu_seqlens, w.U, w.sigma, k_route)
    np.testing.assert_allclose(alpha.cpu().numpy(), ref, atol=1e-5)
    assert np.allclose(np.abs(ref).max(-1), 1.0)


# ----------------------------------------------------------------- standalone key edit

def _check_edit(w, Kout, alpha=None, head_enable=None):
    ref = oracle.edit_keys(w.K, w.mask, w.cu_seqlens, w.U, alpha=alpha, gain=w.gain, head_enable=head_enable)
    got = Kout.double().cpu().numpy()
    hl = w.mask != 0
    # rows that are not highlighted (or belong to an unselected head) are bit-identical to the input
    assert np.array_equal(got[~hl], w.K[~hl].astype(np.float64))
    if head_enable is not None:
        off = np.asarray(head_enable) == 0
        assert np.array_equal(got[:, off], w.K[:, off].astype(np.float64))
    rowmax = np.abs(ref).max(axis=-1, keepdims=True)
    rel = np.abs(got - ref) / np.maximum(rowmax, 1e-30)
    # fp32: max relative error 1e-3 of the row's largest entry; bf16: one rounding of the result (2^-8 of row max)
    tol = 1e-3 if w.dtype == "f32" else 2.0 ** -8
    assert rel.max() <= tol, rel.max()
    return float(rel.max())


@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C4", "C5", "C2s100"])
def test_edit_keys_configs(name):
    w = inputs.make_workload(name)
    alpha = oracle.route(w.Q, w.cu_seqlens, w.U, w.sigma, 0) if w.n_experts > 1 else None
    dev = H.device_tensors(w)
    _check_edit(w, H.run_edit(w, dev, alpha=alpha), alpha=alpha)
    _check_edit(w, H.run_edit(w, dev, alpha=alpha, in_place=True), alpha=alpha)


def test_edit_keys_edge_cases():
    for kw in [dict(lens=[1], mask_kind="all"), dict(lens=[130, 0, 77], mask_kind="runs", highlight=0.5),
               dict(lens=[64], mask_kind="none"), dict(lens=[200], rank=1), dict(lens=[200], rank=64, n_experts=2)]:
        base = dict(seed=9, dtype="bf16", n_q_heads=4, n_kv_heads=2, head_dim=128, rank=16, gain=-0.5)
        base.update(kw)
        w = inputs.make_custom(**base)
        alpha = None
        if w.n_experts > 1:
            alpha = np.random.default_rng(1).uniform(-1, 1, size=(w.batch, w.n_kv_heads, w.n_experts))
        he = np.array([0, 1], dtype=np.uint8)
        _check_edit(w, H.run_edit(w, alpha=alpha, head_enable=he), alpha=alpha, head_enable=he)
    w = inputs.make_custom(seed=10, dtype="f32", lens=[50, 60], n_q_heads=2, n_kv_heads=2, head_dim=64, rank=7,
                           gain=[2.0, -5.0], highlight=0.3)
    assert _check_edit(w, H.run_edit(w)) < 1e-5


# ----------------------------------------------------------------- fused attention: small and edge cases

def _fused_vs_oracle(w, alpha=None, head_enable=None, rows=None, force_varlen=False, label=""):
    O, LSE = H.run_fused(w, alpha=alpha, head_enable=head_enable, force_varlen=force_varlen)
    Oref, Lref, idx = H.oracle_rows(w, rows, alpha=alpha, head_enable=head_enable)
    mx, mean = H.check_attention(O[idx], Oref, label)
    np.testing.assert_allclose(LSE[idx], Lref, atol=2e-2)
    return mx, mean


def test_fused_c1_full():
    w = inputs.make_workload("C1")
    _fused_vs_oracle(w, label="C1")


@pytest.mark.parametrize("d,Hq,Hkv,r", [(128, 4, 1, 32), (128, 7, 1, 64), (64, 2, 2, 16), (128, 2, 2, 128),
                                        (64, 4, 2, 1), (128, 2, 1, 8)])
@pytest.mark.parametrize("g", [0.5, -0.5, 2.0, -5.0])
def test_fused_small_shapes(d, Hq, Hkv, r, g):
    w = inputs.make_custom(seed=100 + r, dtype="bf16", lens=[300], n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, rank=r,
                           gain=g, highlight=0.2)
    # short rows with |1+g| up to 4 on up to all of the head dimension, at the stated tolerance
    _fused_vs_oracle(w, label="d%d r%d g%g" % (d, r, g))


@pytest.mark.parametrize("lens", [[1], [127], [128], [129], [257, 1, 0, 300], [5, 640]])
def test_fused_ragged_lengths(lens):
    w = inputs.make_custom(seed=7, dtype="bf16", lens=lens, n_q_heads=4, n_kv_heads=2, head_dim=128, rank=16,
                           gain=1.0, mask_kind="runs", highlight=0.3)
    _fused_vs_oracle(w, label=str(lens))


def test_fused_mask_patterns_and_head_enable():
    for kind in ["none", "all"]:
        w = inputs.make_custom(seed=8, dtype="bf16", lens=[384], n_q_heads=4, n_kv_heads=2, head_dim=128, rank=32,
                               gain=1.0, mask_kind=kind)
        _fused_vs_oracle(w, label=kind)
    w = inputs.make_custom(seed=8, dtype="bf16", lens=[384], n_q_heads=4, n_kv_heads=2, head_dim=128, rank=32,
                           gain=1.5, mask_kind="none")
    w.mask[127:130] = 1             # a span that straddles a key-tile boundary
    w.mask[383] = 1                 # the very last token
    he = np.array([1, 0], dtype=np.uint8)
    _fused_vs_oracle(w, head_enable=he, label="straddle")


def test_fused_unsteered_paths_are_bitwise_identical():
    # g = 0, an empty mask and "no steering arguments" all run the same arithmetic
    w = inputs.make_custom(seed=12, dtype="bf16", lens=[300, 200], n_q_heads=4, n_kv_heads=2, head_dim=128, rank=32,
                           gain=1.0, highlight=0.3)
    dev = H.device_tensors(w)
    base, _ = H.run_fused(w, dev, steer=False)
    w0 = inputs.make_custom(seed=12, dtype="bf16", lens=[300, 200], n_q_heads=4, n_kv_heads=2, head_dim=128, rank=32,
                            gain=0.0, highlight=0.3)
    dev0 = dict(dev); dev0["gain"] = torch.zeros_like(dev["gain"])
    g0, _ = H.run_fused(w0, dev0)
    devm = dict(dev); devm["mask"] = torch.zeros_like(dev["mask"])
    m0, _ = H.run_fused(w, devm)
    assert np.array_equal(base, g0) and np.array_equal(base, m0)
    steered, _ = H.run_fused(w, dev)
    assert not np.array_equal(base, steered)
    # the inputs are never modified
    assert torch.equal(dev["K"], torch.from_numpy(w.K).cuda().to(torch.bfloat16))


def test_fused_adaseka_blend_small():
    w = inputs.make_custom(seed=13, dtype="bf16", lens=[500, 140], n_q_heads=8, n_kv_heads=2, head_dim=128, rank=32,
                           n_experts=4, gain=1.0, highlight=0.15)
    dev = H.device_tensors(w)
    shp = H.shape_of(w, dev)
    alpha = torch.empty((w.batch, w.n_kv_heads, 4), device="cuda")
    binding.adaseka_route(shp, dev["Q"], dev["U"], dev["sigma"], 0, alpha)
    a = alpha.cpu().numpy().astype(np.float64)
    _fused_vs_oracle(w, alpha=a, label="adaseka")


def test_fused_fixed_layout_equals_packed_layout():
    w = inputs.make_custom(seed=14, dtype="bf16", lens=[256, 256], n_q_heads=2, n_kv_heads=1, head_dim=64, rank=16,
                           gain=1.0, highlight=0.2)
    a, _ = H.run_fused(w)
    b, _ = H.run_fused(w, force_varlen=True)
    assert np.array_equal(a, b)


def test_host_buffer_entry_point():
    w = inputs.make_custom(seed=15, dtype="bf16", lens=[300, 300], n_q_heads=4, n_kv_heads=2, head_dim=128, rank=32,
                           gain=1.0, highlight=0.2)
    dev = H.device_tensors(w)
    shp = H.shape_of(w, dev)
    ws = binding.new_workspace(shp)
    staging = torch.empty(binding.seka_host_staging_bytes(shp), dtype=torch.uint8, device="cuda")
    hQ, hK, hV = (dev[k].cpu().pin_memory() for k in "QKV")
    hmask = dev["mask"].cpu().pin_memory()
    hO = torch.empty_like(hQ).pin_memory()
    hlse = torch.empty((w.total_tokens, w.n_q_heads), dtype=torch.float32).pin_memory()
    binding.seka_attention_fwd_host(shp, hQ, hK, hV, hO, hlse, hmask, dev["U"], None, dev["gain"], None, staging, ws)
    assert binding.seka_poll_status(ws) == binding.SEKA_OK
    ref, lse = H.run_fused(w, dev)
    assert np.array_equal(hO.double().numpy(), ref) and np.array_equal(hlse.double().numpy(), lse)


def test_host_buffer_calls_back_to_back_share_a_staging_buffer():
    """Calls through host buffers overlap: the input copies of one run while the output of the one before is still on
    its way back, all through one staging buffer.  Different inputs, the same cut and then another cut (a batch of four,
    a batch of two, a packed batch), queued without a synchronisation in between: each result equals the device path's."""
    cases = []
    for seed, lens in ((21, [384] * 4), (22, [384] * 4), (23, [768] * 2), (24, [384] * 4), (25, [300, 41, 384]), (26, [384] * 4)):
        w = inputs.make_custom(seed=seed, dtype="bf16", lens=lens, n_q_heads=4, n_kv_heads=2, head_dim=128, rank=32,
                               gain=1.0, highlight=0.2)
        dev = H.device_tensors(w)
        cases.append((w, dev, H.shape_of(w, dev)))
    nbytes = max(binding.seka_host_staging_bytes(shp) for _, _, shp in cases)
    staging = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    ws = torch.zeros(max(binding.seka_workspace_bytes(shp) for _, _, shp in cases), dtype=torch.uint8, device="cuda")
    host = []
    for w, dev, shp in cases:
        hQ, hK, hV = (dev[k].cpu().pin_memory() for k in "QKV")
        host.append((hQ, hK, hV, dev["mask"].cpu().pin_memory(), torch.empty_like(hQ).pin_memory()))
    torch.cuda.synchronize()
    for (w, dev, shp), (hQ, hK, hV, hm, hO) in zip(cases, host):
        binding.seka_attention_fwd_host(shp, hQ, hK, hV, hO, None, hm, dev["U"], None, dev["gain"], None, staging, ws)
    torch.cuda.synchronize()
    assert binding.seka_poll_status(ws) == binding.SEKA_OK
    for (w, dev, shp), (_, _, _, _, hO) in zip(cases, host):
        ref, _ = H.run_fused(w, dev)
        assert np.array_equal(hO.double().numpy(), ref)


# ----------------------------------------------------------------- fused attention: the five configurations at full size

@pytest.mark.parametrize("name,nrows,nseq", [("C2", 256, None), ("C3", 256, None), ("C4", 256, None), ("C5", None, 8), ("C2s70", 128, None)])
def test_fused_full_size_sampled_rows(name, nrows, nseq):
    """The five configurations (and the 70 % stress mask) at full size, in the launch configuration the benchmark
    times.  The oracle evaluates complete query rows: `nrows` per sequence (always the first and last row, the rows at
    tile edges and the rows just after every span), or every row of `nseq` whole sequences (the packed batch)."""
    w = inputs.make_workload(name)
    alpha = None
    dev = H.device_tensors(w)
    if w.n_experts > 1:
        shp = H.shape_of(w, dev)
        a = torch.empty((w.batch, w.n_kv_heads, w.n_experts), device="cuda")
        binding.adaseka_route(shp, dev["Q"], dev["U"], dev["sigma"], 0, a)
        alpha = a.cpu().numpy().astype(np.float64)
        np.testing.assert_allclose(alpha, oracle.route(w.Q, w.cu_seqlens, w.U, w.sigma, 0), atol=1e-5)
    if nseq is None:
        rows = H.sampled_rows(w, nrows, seed=1)
    else:
        # whole sequences: the shortest, the longest and a seeded choice of the rest
        lens = np.diff(w.cu_seqlens)
        order = np.argsort(lens, kind="stable")
        pick = {int(order[0]), int(order[-1])}
        rng = np.random.default_rng(2)
        while len(pick) < nseq:
            pick.add(int(rng.integers(0, w.batch)))
        rows = [np.arange(int(lens[b]), dtype=np.int32) if b in pick else np.zeros(0, dtype=np.int32) for b in range(w.batch)]
    O, LSE = H.run_fused(w, dev, alpha=alpha)
    assert np.isfinite(O).all() and np.isfinite(LSE).all()          # every row was written
    Oref, Lref, idx = H.oracle_rows(w, rows, alpha=alpha)
    mx, mean = H.check_attention(O[idx], Oref, name)
    np.testing.assert_allclose(LSE[idx], Lref, atol=2e-2)
    print("%s: rows %d max abs %.3e mean abs %.3e" % (name, len(idx), mx, mean))


# ----------------------------------------------------------------- the two-projector edit of Eq. 4 through the bank interface

def test_two_projector_edit_maps_onto_the_expert_bank():
    """Eq. 4, k' = k + (g+ P+ k + g- P- k)/2 with P- built from the vectors after the leading k- ones (Eq. 2), is
    the blend sum_m alpha_m U_m U_m^T of two "experts": U_1 = U+[:, :k+], U_2 = U-[:, k-:] (zero-padded to a
    common width), alpha = (g+/2, g-/2), gain 1.  Edited keys and fused attention against the dense oracle."""
    from oracle import brute
    d, Hq, Hkv, L = 128, 4, 2, 300
    w = inputs.make_custom(seed=21, dtype="bf16", lens=[L], n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, rank=8,
                           gain=1.0, mask_kind="runs", highlight=0.25)
    rng = np.random.default_rng(22)
    Up = np.stack([np.linalg.qr(rng.standard_normal((d, d)))[0] for _ in range(Hkv)])
    Un = np.stack([np.linalg.qr(rng.standard_normal((d, d)))[0] for _ in range(Hkv)])
    k_pos, k_neg, g_pos, g_neg = 12, 100, 0.6, -0.4
    r = max(k_pos, d - k_neg)
    bank = np.zeros((2, Hkv, d, r), dtype=np.float32)
    bank[0, :, :, :k_pos] = Up[:, :, :k_pos]
    bank[1, :, :, :d - k_neg] = Un[:, :, k_neg:]
    alpha = np.tile(np.array([g_pos / 2, g_neg / 2]), (1, Hkv, 1))
    # the oracle consumes the bank as stored (fp32), like the kernels
    K_ref = brute.two_projector_edit(w.K, w.mask, bank[0].astype(np.float64)[:, :, :], k_pos,
                                     np.concatenate([np.zeros((Hkv, d, k_neg)), bank[1].astype(np.float64)[:, :, :d - k_neg]], axis=2),
                                     k_neg, g_pos, g_neg)
    dev = H.device_tensors(w)
    dev["U"] = torch.from_numpy(bank).cuda()
    shp = binding.make_shape(batch=1, max_seqlen=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, rank=r, n_experts=2,
                             dtype=torch.bfloat16)
    ws = binding.new_workspace(shp)
    a = torch.from_numpy(alpha.astype(np.float32)).cuda()
    Kout = torch.full_like(dev["K"], float("nan"))
    binding.seka_edit_keys(shp, dev["K"], Kout, dev["mask"], dev["U"], a, dev["gain"], None, ws)
    got = Kout.double().cpu().numpy()
    rel = np.abs(got - K_ref) / np.abs(K_ref).max(axis=-1, keepdims=True)
    assert rel.max() <= 2.0 ** -8, rel.max()
    hl = w.mask != 0
    assert np.array_equal(got[~hl], w.K[~hl].astype(np.float64))
    O = torch.full_like(dev["Q"], float("nan"))
    binding.seka_attention_fwd(shp, dev["Q"], dev["K"], dev["V"], O, None, dev["mask"], dev["U"], a, dev["gain"], None, ws)
    assert binding.seka_poll_status(ws) == binding.SEKA_OK
    Oref, _, idx = oracle.attention_rows(w.Q.astype(np.float64), K_ref, w.V.astype(np.float64), w.cu_seqlens, None)
    H.check_attention(O.double().cpu().numpy()[idx], Oref, "two projectors")


# ----------------------------------------------------------------- wide banks and many items per CTA

def test_wide_expert_banks():
    """Stacked rank M*r above the head dimension (the dense operator does not care), and a bank too large for the
    tensor-core edit kernel (M*d > 512), which takes the fp32 row kernel."""
    for M, r in [(3, 64), (5, 16)]:
        w = inputs.make_custom(seed=50 + M, dtype="bf16", lens=[260, 130], n_q_heads=4, n_kv_heads=2, head_dim=128, rank=r,
                               n_experts=M, gain=[0.5, -0.5], highlight=0.3)
        alpha = np.random.default_rng(M).uniform(-1, 1, size=(w.batch, w.n_kv_heads, M))
        _check_edit(w, H.run_edit(w, alpha=alpha), alpha=alpha)
        _fused_vs_oracle(w, alpha=alpha, label="M%d r%d" % (M, r))


def test_more_items_than_sms():
    """Fixed-length batch with more (row-tile, head-pair) items than the GPU has SMs: every persistent CTA walks
    several items (odd and even rounds), with steering on some sequences only and one KV head switched off."""
    w = inputs.make_custom(seed=60, dtype="bf16", lens=[2432, 2432], n_q_heads=8, n_kv_heads=2, head_dim=128, rank=16,
                           gain=[1.0, 0.0], highlight=0.2)
    he = np.array([1, 0], dtype=np.uint8)
    rows = H.sampled_rows(w, 40, seed=3)
    _fused_vs_oracle(w, head_enable=he, rows=rows, label="152 items")


@pytest.mark.parametrize("d", [64, 128])
def test_every_tile_highlighted_with_odd_group(d):
    """Odd group size (here MHA): an item pairs two consecutive row tiles, so the last key tile of an item is used
    by its second tile only.  With every token highlighted and many short sequences each persistent CTA walks items
    whose first and last key tiles are both edited, back to back: the softmax warps of the first tile then reach
    the next item's first edit while the previous item's last one is still being formed."""
    rng = np.random.default_rng(61)
    lens = [int(x) for x in rng.integers(130, 640, size=96)]
    w = inputs.make_custom(seed=61, dtype="bf16", lens=lens, n_q_heads=3, n_kv_heads=3, head_dim=d, rank=16,
                           mask_kind="all", gain=0.5)
    rows = H.sampled_rows(w, 6, seed=4)
    for _ in range(3):
        _fused_vs_oracle(w, rows=rows, label="all tiles hot, d=%d" % d)


@pytest.mark.parametrize("name", ["C5", "C4"])
def test_fused_output_is_repeatable(name):
    """The fused forward has no atomics and a static schedule: the same inputs give the same bits, launch after
    launch (a hand-off that sometimes came too early would show up here)."""
    w = inputs.make_workload(name)
    dev = H.device_tensors(w)
    shp = H.shape_of(w, dev)
    ws = binding.new_workspace(shp)
    O = torch.empty_like(dev["Q"])
    ref = None
    for _ in range(12 if name == "C5" else 4):
        O.fill_(float("nan"))
        binding.seka_attention_fwd(shp, dev["Q"], dev["K"], dev["V"], O, None, dev["mask"], dev["U"], None, dev["gain"], None, ws)
        torch.cuda.synchronize()
        if ref is None:
            ref = O.clone()
        else:
            assert torch.equal(O.view(torch.int16), ref.view(torch.int16))
    assert binding.seka_poll_status(ws) == binding.SEKA_OK


# ----------------------------------------------------------------- AdaSEKA in one call (routing inside the preparation launch)

@pytest.mark.parametrize("case", ["C3", "small_f32", "small_varlen", "wide_bank"])
def test_routed_forward_equals_route_then_forward(case):
    if case == "C3":
        w = inputs.make_workload("C3"); k_route = 0; he = None
    elif case == "wide_bank":      # 6 x 128 columns do not fit tensor memory: the one-launch preparation kernel
        w = inputs.make_custom(seed=7, dtype="bf16", lens=[260, 90], n_q_heads=4, n_kv_heads=2, head_dim=128, rank=8,
                               n_experts=6, gain=1.0); k_route = 0; he = None
    elif case == "small_f32":
        w = inputs.make_custom(seed=5, dtype="f32", lens=[200, 140], n_q_heads=8, n_kv_heads=2, head_dim=64, rank=16,
                               n_experts=3, gain=[0.8, 0.0]); k_route = 5; he = None
    else:
        w = inputs.make_custom(seed=6, dtype="bf16", lens=[17, 300, 1, 0, 129], n_q_heads=14, n_kv_heads=2, head_dim=128,
                               rank=8, n_experts=4, gain=1.0); k_route = 8; he = [1, 0]
    dev = H.device_tensors(w)
    shp = H.shape_of(w, dev)
    hed = None if he is None else torch.tensor(he, dtype=torch.uint8, device="cuda")
    launches0 = binding.seka_launch_count()
    # two calls
    alpha = torch.full((w.batch, w.n_kv_heads, w.n_experts), float("nan"), device="cuda")
    ws = binding.new_workspace(shp)
    O2 = torch.full_like(dev["Q"], float("nan")); lse2 = torch.empty((w.total_tokens, w.n_q_heads), device="cuda")
    binding.adaseka_route(shp, dev["Q"], dev["U"], dev["sigma"], k_route, alpha)
    binding.seka_attention_fwd(shp, dev["Q"], dev["K"], dev["V"], O2, lse2, dev["mask"], dev["U"], alpha, dev["gain"], hed, ws)
    launches_two = binding.seka_launch_count() - launches0
    # one call
    alpha1 = torch.full_like(alpha, float("nan"))
    ws1 = binding.new_workspace(shp)
    O1 = torch.full_like(dev["Q"], float("nan")); lse1 = torch.empty_like(lse2)
    binding.seka_attention_fwd_routed(shp, dev["Q"], dev["K"], dev["V"], O1, lse1, dev["mask"], dev["U"], dev["sigma"],
                                      k_route, alpha1, dev["gain"], hed, ws1)
    launches_one = binding.seka_launch_count() - launches0 - launches_two
    assert binding.seka_poll_status(ws1) == binding.SEKA_OK
    assert launches_one == launches_two - 1      # Eq. 6 runs in blocks of the preparation launch
    assert torch.equal(alpha1, alpha)
    assert torch.equal(O1.view(torch.int16 if O1.dtype == torch.bfloat16 else torch.int32),
                       O2.view(torch.int16 if O2.dtype == torch.bfloat16 else torch.int32))
    assert torch.equal(lse1, lse2)
    a_ref = oracle.route(w.Q, w.cu_seqlens, w.U, w.sigma, k_route)
    np.testing.assert_allclose(alpha1.cpu().numpy(), a_ref, atol=1e-5)
    if case != "C3":
        Oref, Lref, idx = H.oracle_rows(w, None, alpha=a_ref, head_enable=he)
        H.check_attention(O1.double().cpu().numpy()[idx], Oref, case)
