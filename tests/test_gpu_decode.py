"""GPU parity of the decode step over the (edited) key cache against the fp64 CPU oracle, through the C ABI.

The decode query of a sequence is the query of its last cached token (that token's key and value are the
last cached row), so the workloads of the prefill tests serve unchanged."""
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
    binding.load()


def _last_queries(w):
    last = w.cu_seqlens[1:].astype(np.int64) - 1
    q = np.zeros((w.batch, w.n_q_heads, w.head_dim), dtype=np.float32)
    ok = w.cu_seqlens[1:] > w.cu_seqlens[:-1]
    q[ok] = w.Q[last[ok]]
    return q


def _run_decode(w, dev, K_dev, q, fixed=False):
    shp = H.shape_of(w, dev, force_varlen=not fixed)
    n = binding.seka_decode_workspace_bytes(shp)
    assert n > 0
    ws = torch.zeros(n, dtype=torch.uint8, device="cuda")
    qd = torch.from_numpy(q).to(device="cuda", dtype=torch.bfloat16)
    O = torch.full_like(qd, float("nan"))
    lse = torch.full((w.batch, w.n_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    binding.seka_decode_attention(shp, qd, K_dev, dev["V"], O, lse, ws)
    st = binding.seka_poll_status(ws)
    assert st == binding.SEKA_OK, binding.status_string(st)
    return O.double().cpu().numpy(), lse.double().cpu().numpy()


def _check(O, LSE, Oref, Lref, label=""):
    # the tolerance of the prefill attention: bf16 output, max abs 1e-2 and mean abs 1e-3
    err = np.abs(O - Oref)
    assert err.max() <= 1e-2, (label, err.max())
    assert err.mean() <= 1e-3, (label, err.mean())
    fin = np.isfinite(Lref)
    np.testing.assert_allclose(LSE[fin], Lref[fin], atol=2e-2)
    assert np.array_equal(np.isneginf(LSE), np.isneginf(Lref))
    return float(err.max()), float(err.mean())


@pytest.mark.parametrize("d,Hq,Hkv", [(128, 8, 2), (128, 7, 1), (64, 4, 4), (128, 16, 1), (64, 24, 2), (128, 9, 1)])
def test_decode_plain_cache(d, Hq, Hkv):
    # no edit: the same bf16 keys on both sides; lengths below, at and above the 64-token stage and the chunk
    lens = [37, 1, 300, 64, 0, 700, 257, 63, 65, 1024]
    w = inputs.make_custom(seed=21, dtype="bf16", lens=lens, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, rank=8)
    dev = H.device_tensors(w)
    q = _last_queries(w)
    O, LSE = _run_decode(w, dev, dev["K"], q)
    Oref, Lref = oracle.decode_attention(q, w.K, w.V, w.cu_seqlens)
    assert np.all(O[4] == 0) and np.all(np.isneginf(LSE[4]))          # the empty cache
    _check(O, LSE, Oref, Lref, label="plain")


@pytest.mark.parametrize("L", [5000, 256, 1])
def test_decode_many_chunks_fixed_layout(L):
    # one long sequence is cut into many chunks (ragged last one); fixed-length layout without cu_seqlens
    w = inputs.make_custom(seed=22, dtype="bf16", lens=[L, L], n_q_heads=4, n_kv_heads=1, head_dim=128, rank=8)
    dev = H.device_tensors(w)
    q = _last_queries(w)
    Oref, Lref = oracle.decode_attention(q, w.K, w.V, w.cu_seqlens)
    for fixed in (True, False):
        O, LSE = _run_decode(w, dev, dev["K"], q, fixed=fixed)
        _check(O, LSE, Oref, Lref, label="L=%d fixed=%s" % (L, fixed))


def test_decode_scores_far_from_zero_and_scale_override():
    # large scores (the running maximum moves a lot between stages) and a caller-chosen softmax scale
    w = inputs.make_custom(seed=23, dtype="bf16", lens=[900, 130], n_q_heads=8, n_kv_heads=2, head_dim=64, rank=8)
    dev = H.device_tensors(w)
    q = inputs.round_to_bf16(3.0 * _last_queries(w))
    shp = H.shape_of(w, dev, force_varlen=True)
    shp.softmax_scale = 0.25
    ws = torch.zeros(binding.seka_decode_workspace_bytes(shp), dtype=torch.uint8, device="cuda")
    qd = torch.from_numpy(q).to(device="cuda", dtype=torch.bfloat16)
    O = torch.empty_like(qd)
    binding.seka_decode_attention(shp, qd, dev["K"], dev["V"], O, None, ws)
    assert binding.seka_poll_status(ws) == binding.SEKA_OK
    Oref, _ = oracle.decode_attention(q, w.K, w.V, w.cu_seqlens, scale=0.25)
    err = np.abs(O.double().cpu().numpy() - Oref)
    # peaked softmax: the output is close to single value rows of magnitude up to ~4, bf16 rounding 2^-8 relative
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())


@pytest.mark.parametrize("name", ["C2", "C5"])
def test_decode_over_edited_cache(name):
    # the path of Algorithm 1: edit the cached keys once in place, then decode over the edited cache
    w = inputs.make_workload(name)
    dev = H.device_tensors(w)
    Kp = H.run_edit(w, dev, in_place=True)
    q = _last_queries(w)
    O, LSE = _run_decode(w, dev, Kp, q)
    Oref, Lref = oracle.seka_decode(q, w.K, w.V, w.mask, w.cu_seqlens, w.U, gain=w.gain)
    mx, mean = _check(O, LSE, Oref, Lref, label=name)
    print("%s decode over edited cache: max abs %.3e mean abs %.3e" % (name, mx, mean))
    # and the decode alone, on exactly the cache the GPU holds
    O2ref, L2ref = oracle.decode_attention(q, Kp.float().cpu().numpy(), w.V, w.cu_seqlens)
    _check(O, LSE, O2ref, L2ref, label=name + " same cache")


def test_decode_full_size_cache_sampled_sequences():
    # the benchmark's decode workload: 64 cached sequences of 4096 tokens on the 8B shape (1 GiB of K and V);
    # the oracle evaluates a sample of the sequences
    B, L = 64, 4096
    w = inputs.make_workload("C2", batch=B, seqlen=L)
    dev = H.device_tensors(w)
    Kp = H.run_edit(w, dev, in_place=True)
    q = _last_queries(w)
    O, LSE = _run_decode(w, dev, Kp, q)
    assert np.isfinite(O).all() and np.isfinite(LSE).all()
    for b in (0, 17, 40, 63):
        s, e = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        Oref, Lref = oracle.seka_decode(q[b:b + 1], w.K[s:e], w.V[s:e], w.mask[s:e], [0, e - s], w.U,
                                        gain=w.gain[b:b + 1])
        _check(O[b:b + 1], LSE[b:b + 1], Oref, Lref, label="seq %d" % b)


def test_decode_rejects_what_it_does_not_cover():
    w = inputs.make_custom(seed=24, dtype="bf16", lens=[64], n_q_heads=34, n_kv_heads=2, head_dim=128, rank=8)
    dev = H.device_tensors(w)
    shp = H.shape_of(w, dev)
    assert binding.seka_decode_workspace_bytes(shp) == 0               # 17 query heads per KV head
    q = torch.zeros((1, 34, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.SekaError) as e:
        binding.seka_decode_attention(shp, q, dev["K"], dev["V"], torch.empty_like(q), None, ws)
    assert e.value.status == binding.SEKA_ERR_UNSUPPORTED
    w = inputs.make_custom(seed=24, dtype="bf16", lens=[64], n_q_heads=4, n_kv_heads=2, head_dim=128, rank=8)
    dev = H.device_tensors(w)
    shp = H.shape_of(w, dev)
    q = torch.zeros((1, 4, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.SekaError) as e:                        # workspace too small
        binding.seka_decode_attention(shp, q, dev["K"], dev["V"], torch.empty_like(q), None, ws[:256])
    assert e.value.status == binding.SEKA_ERR_WORKSPACE
