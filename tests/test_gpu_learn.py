"""GPU parity of the offline spectral learning (cross-covariances, SVD, rank rule, head-selection distance)
against the fp64 CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from oracle import brute
from paper_2603_01281_b200 import binding, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load()


def _to_dev(x):
    return torch.from_numpy(x).to(device="cuda", dtype=torch.bfloat16)


def _projector(U, lo, hi):
    return U[:, lo:hi] @ U[:, lo:hi].T


def _check_against_oracle(out, ref, n, d, gamma, label=""):
    """`out`: GPU results as float64 numpy; `ref`: oracle.learn_projections on the same embeddings."""
    slots = ref["D"].shape[0]
    for tag in ("pos", "neg"):
        Om, Om_ref = out["omega_" + tag], ref["omega_" + tag]
        # bf16 products are exact in fp32; what differs from fp64 is the fp32 accumulation over n tokens:
        # a random walk of n roundings of 2^-24 relative to partial sums of size ~ n E|x y| <= n, divided by n
        tol = 8.0 * np.sqrt(n) * 2.0 ** -24 * max(1.0, np.abs(Om_ref).max())
        assert np.abs(Om - Om_ref).max() <= tol, (label, tag, np.abs(Om - Om_ref).max(), tol)
        for s in range(slots):
            U, S = out["U_" + tag][s], out["S_" + tag][s]
            # the decomposition of the matrix the GPU holds: LAPACK on exactly that matrix
            U2, S2, _ = np.linalg.svd(Om[s])
            np.testing.assert_allclose(S, S2, rtol=2e-6, atol=2e-7 * S2[0])
            assert np.all(np.diff(S) <= 0)
            np.testing.assert_allclose(U.T @ U, np.eye(d), atol=5e-6)
            np.testing.assert_allclose(Om[s] @ Om[s].T @ U, U * (S2 * S2), atol=2e-5 * S2[0] ** 2)
            k = int(out["k_" + tag][s])
            assert k == brute.rank_by_variance(S2, gamma) or abs(np.cumsum(S2)[k - 1] / S2.sum() - gamma) < 1e-6
            # subspaces of Eq. 2 where the spectrum has a gap at the cut: leading k+ vectors, vectors after k-
            for cut in {k, d // 2}:
                gap = (S2[cut - 1] - S2[cut]) / S2[0] if cut < d else 1.0
                if gap > 1e-3:
                    lo, hi = (0, cut) if tag == "pos" else (cut, d)
                    err = np.abs(_projector(U, lo, hi) - _projector(U2, lo, hi)).max()
                    assert err <= 1e-5 / gap, (label, tag, s, cut, err, gap)
            # against the oracle's own run from the embeddings (fp64 all the way)
            np.testing.assert_allclose(S, ref["S_" + tag][s], rtol=1e-4, atol=1e-5 * ref["S_" + tag][s][0])
            kr = int(ref["k_" + tag][s])
            margin = abs(np.cumsum(ref["S_" + tag][s])[min(k, kr) - 1] / ref["S_" + tag][s].sum() - gamma)
            assert k == kr or margin < 1e-4, (label, tag, s, k, kr)
    np.testing.assert_allclose(out["D"], ref["D"], rtol=2e-5)


def _run(h, hp, hn, ans, gamma):
    res = binding.seka_learn_projections(_to_dev(h), _to_dev(hp), _to_dev(hn),
                                         None if ans is None else torch.from_numpy(ans).cuda(), gamma)
    return {k: v.double().cpu().numpy() for k, v in res.items() if k != "workspace"}, res


@pytest.mark.parametrize("n,slots,d", [(3000, 6, 128), (5000, 6, 64), (100, 2, 128), (4096, 4, 64), (129, 1, 128)])
def test_learner_small(n, slots, d):
    gamma = 0.7
    h, hp, hn, ans, _, strength = inputs.contrastive_embeddings(seed=n, n=n, slots=slots, head_dim=d, rank=8)
    out, _ = _run(h, hp, hn, ans, gamma)
    ref = oracle.learn_projections(h, hp, hn, gamma, answer_tokens=ans)
    _check_against_oracle(out, ref, n, d, gamma, label="n=%d d=%d" % (n, d))
    if slots >= 4:
        assert int(np.argmin(out["D"])) % 4 == 3 and strength[3] == 0.0      # the head that does not react


def test_learner_all_tokens_and_other_gamma():
    h, hp, hn, _, _, _ = inputs.contrastive_embeddings(seed=7, n=2500, slots=2, head_dim=128, rank=16)
    for gamma in (0.3, 1.0):
        out, _ = _run(h, hp, hn, None, gamma)
        ref = oracle.learn_projections(h, hp, hn, gamma)
        _check_against_oracle(out, ref, 2500, 128, gamma, label="gamma=%g" % gamma)
    assert np.all(out["k_pos"] == 128)                                       # gamma = 1 keeps every direction


def test_learned_projections_feed_the_key_edit():
    # the U the learner returns is what seka_edit_keys takes: leading k+ columns of one slot as a rank-k+ projector
    d, slots = 128, 2
    h, hp, hn, ans, _, _ = inputs.contrastive_embeddings(seed=11, n=3000, slots=slots, head_dim=d, rank=8)
    out, res = _run(h, hp, hn, ans, 0.5)
    k = int(out["k_pos"].max())
    w = inputs.make_custom(seed=12, dtype="bf16", lens=[300], n_q_heads=4, n_kv_heads=slots, head_dim=d, rank=k)
    U = res["U_pos"][:, :, :k].contiguous().unsqueeze(0)                     # [M=1, Hkv, d, r=k]
    K = torch.from_numpy(w.K).to(device="cuda", dtype=torch.bfloat16)
    shp = binding.make_shape(batch=1, max_seqlen=300, n_q_heads=4, n_kv_heads=slots, head_dim=d, rank=k)
    Kout = torch.empty_like(K)
    binding.seka_edit_keys(shp, K, Kout, torch.from_numpy(w.mask).cuda(), U, None, torch.ones(1, device="cuda"), None,
                           binding.new_workspace(shp))
    ref = oracle.edit_keys(w.K, w.mask, w.cu_seqlens, U.double().cpu().numpy(), gain=[1.0])
    got = Kout.double().cpu().numpy()
    rel = np.abs(got - ref) / np.abs(ref).max(-1, keepdims=True)
    assert rel.max() <= 2.0 ** -8


def test_learner_full_size_sampled_slots():
    # the benchmark's size: 32768 tokens x 288 slots (36 layers x 8 KV heads) x 128, generated on the device
    # (a planted low-rank lift per slot); the oracle evaluates a sample of the slots from the same values
    n, slots, d, gamma = 32768, 288, 128, 0.7
    gen = torch.Generator(device="cuda"); gen.manual_seed(260301283)
    h = torch.randn((n, slots, d), device="cuda", dtype=torch.float32, generator=gen).to(torch.bfloat16)
    B = torch.linalg.qr(torch.randn((slots, d, 8), device="cuda", generator=gen))[0]
    lift = torch.einsum("nsd,sdr,ser->nse", h.float(), B, B)
    a = torch.rand(slots, device="cuda", generator=gen)[None, :, None]
    hp = (h.float() + a * lift + 0.1 * torch.randn((n, slots, d), device="cuda", generator=gen)).to(torch.bfloat16)
    hn = (h.float() - 0.5 * a * lift + 0.1 * torch.randn((n, slots, d), device="cuda", generator=gen)).to(torch.bfloat16)
    del lift
    ans = (torch.rand(n, device="cuda", generator=gen) < 0.3).to(torch.uint8)
    res = binding.seka_learn_projections(h, hp, hn, ans, gamma)
    sample = [0, 101, 287]
    sub = lambda t: t[:, sample].float().cpu().numpy()
    ref = oracle.learn_projections(sub(h), sub(hp), sub(hn), gamma, answer_tokens=ans.cpu().numpy())
    out = {k: v[sample].double().cpu().numpy() for k, v in res.items() if k != "workspace"}
    _check_against_oracle(out, ref, n, d, gamma, label="full size")
    for k in ("U_pos", "U_neg", "S_pos", "S_neg", "omega_pos", "D"):
        assert torch.isfinite(res[k]).all()


def test_learner_rejects_what_it_does_not_cover():
    z = torch.zeros((64, 3, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.SekaError):
        binding.seka_learn_projections(z, z, z, None, 0.5)                  # odd number of 64-wide heads
    z = torch.zeros((64, 2, 32), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.SekaError):
        binding.seka_learn_projections(z, z, z, None, 0.5)                  # head_dim 32
