"""seka_edit_keys_static: the key-editing call for hosts that cannot allocate device memory.

A serving process that gave all of its memory to a KV-cache pool at start-up, or a plug-in running
inside someone else's stream callback, has no buffer to offer as workspace and may not call
cudaMalloc.  The variant keeps its scratch (the list of highlighted tokens) in a fixed array
inside the library.  It must give what seka_edit_keys gives, on a first call and on a second call
that finds the previous call's contents in the array.  Collected last on purpose (file name), so a
run that stops at the first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2603_01281_b200 import binding, inputs

import helpers as H

pytestmark = pytest.mark.gpu


def _both(w):
    dev = H.device_tensors(w)
    shp = H.shape_of(w, dev)
    ref = torch.full_like(dev["K"], float("nan"))
    binding.seka_edit_keys(shp, dev["K"], ref, dev["mask"], dev["U"], None, dev["gain"], None, binding.new_workspace(shp))
    got = torch.full_like(dev["K"], float("nan"))
    binding.seka_edit_keys_static(shp, dev["K"], got, dev["mask"], dev["U"], None, dev["gain"], None)
    torch.cuda.synchronize()
    return got.double().cpu().numpy(), ref.double().cpu().numpy()


def test_static_scratch_edit_matches_workspace_edit_twice():
    assert torch.cuda.is_available()
    # first call: many highlighted tokens; second call: fewer and elsewhere, so a stale list or a
    # counter that was not cleared would edit the wrong rows
    w1 = inputs.make_custom(seed=31, dtype="bf16", lens=[700, 300], n_q_heads=4, n_kv_heads=2, head_dim=128, rank=32,
                            gain=1.0, mask_kind="runs", highlight=0.6)
    w2 = inputs.make_custom(seed=32, dtype="bf16", lens=[500, 450], n_q_heads=4, n_kv_heads=2, head_dim=128, rank=32,
                            gain=[0.5, -1.5], mask_kind="spans", highlight=0.05)
    for w in (w1, w2):
        got, ref = _both(w)
        assert np.isfinite(got).all()
        rowmax = np.abs(ref).max(axis=-1, keepdims=True)
        # The other tests hold an edited bf16 key to 2^-8 of its row maximum against the exact edit.  The two
        # entry points no longer share their arithmetic (row kernel in fp32 here, tensor-core tiles there), so
        # each is held to that bound against the fp64 oracle, and to twice it against the other.
        exact = oracle.edit_keys(w.K, w.mask, w.cu_seqlens, w.U, gain=w.gain)
        emax = np.abs(exact).max(axis=-1, keepdims=True)
        assert (np.abs(got - exact) / emax).max() <= 2.0 ** -8
        assert (np.abs(ref - exact) / emax).max() <= 2.0 ** -8
        assert (np.abs(got - ref) / rowmax).max() <= 2.0 ** -7
        hl = w.mask != 0
        assert np.array_equal(got[~hl], w.K[~hl].astype(np.float64))    # untouched rows stay bit-identical


def test_static_scratch_rejects_oversize():
    s = binding.make_shape(batch=1, max_seqlen=binding.SEKA_STATIC_MAX_TOKENS + 1, n_q_heads=2, n_kv_heads=2,
                           head_dim=64, rank=8)
    one = ctypes.c_void_p(256)      # never dereferenced: the size check comes first
    st = binding.load().seka_edit_keys_static(ctypes.byref(s), one, one, one, one, None, one, None, None)
    assert st == binding.SEKA_ERR_UNSUPPORTED
