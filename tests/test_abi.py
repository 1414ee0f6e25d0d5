"""The C-ABI library loads without a GPU, exports every function the header declares, and rejects
bad arguments before launching anything.  CPU only (no compute call is made)."""
import ctypes
import os
import re

import pytest

from paper_2603_01281_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "seka.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b((?:seka|adaseka)_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_functions()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def shape(**kw):
    base = dict(batch=2, max_seqlen=256, total_tokens=0, n_q_heads=8, n_kv_heads=2, head_dim=128, rank=32,
                n_experts=1, dtype=binding.SEKA_BF16, softmax_scale=0.0, cu_seqlens=None)
    base.update(kw)
    return binding.SekaShape(*[base[f[0]] for f in binding.SekaShape._fields_])


def test_workspace_bytes_and_validation(lib):
    s = shape()
    n = binding.seka_workspace_bytes(s)
    assert n >= 256 + 2 * 2 * 128 * 128 * 2 + 2 * 2 + 512 * 4     # status, edit operators, tile flags, token list
    assert binding.seka_workspace_bytes(shape(dtype=binding.SEKA_F32)) > n       # bf16 staging of fp32 inputs
    assert binding.seka_workspace_bytes(shape(head_dim=96)) == 0
    assert binding.seka_workspace_bytes(shape(n_q_heads=7)) == 0
    assert binding.seka_host_staging_bytes(s) >= 512 * (8 + 2 + 2 + 8) * 128 * 2

    one = ctypes.c_void_p(256)       # never dereferenced: validation fails first
    bad = [shape(head_dim=96), shape(n_q_heads=7), shape(rank=0), shape(rank=200), shape(n_experts=0),
           shape(dtype=7), shape(batch=-1), shape(total_tokens=100)]
    for s_bad in bad:
        st = lib.seka_attention_fwd(ctypes.byref(s_bad), one, one, one, one, None, None, None, None, None, None,
                                    one, 1 << 30, None)
        assert st in (binding.SEKA_ERR_INVALID_ARG, binding.SEKA_ERR_UNSUPPORTED)
        assert lib.seka_edit_keys(ctypes.byref(s_bad), one, one, one, one, None, one, None, one, 1 << 30, None) != 0
        assert lib.adaseka_route(ctypes.byref(s_bad), one, one, one, 0, one, None) != 0
    # null tensors, misaligned tensors, short workspace
    s = shape()
    assert lib.seka_attention_fwd(ctypes.byref(s), None, one, one, one, None, None, None, None, None, None, one,
                                  1 << 30, None) == binding.SEKA_ERR_INVALID_ARG
    odd = ctypes.c_void_p(264)
    assert lib.seka_attention_fwd(ctypes.byref(s), odd, one, one, one, None, None, None, None, None, None, one,
                                  1 << 30, None) == binding.SEKA_ERR_INVALID_ARG
    assert lib.seka_attention_fwd(ctypes.byref(s), one, one, one, one, None, None, None, None, None, None, one,
                                  16, None) == binding.SEKA_ERR_WORKSPACE
    assert lib.seka_edit_keys(ctypes.byref(s), one, one, one, one, None, one, None, None, 0, None) == binding.SEKA_ERR_WORKSPACE
    assert lib.adaseka_route(ctypes.byref(s), one, one, one, 33, one, None) == binding.SEKA_ERR_INVALID_ARG
    # empty problems are fine and launch nothing
    assert lib.seka_attention_fwd(ctypes.byref(shape(batch=0)), None, None, None, None, None, None, None, None,
                                  None, None, None, 0, None) == binding.SEKA_OK
    assert binding.status_string(binding.SEKA_ERR_TIMEOUT).startswith("a bounded")
    assert binding.seka_launch_count() == 0


def test_decode_routed_and_learner_validation(lib):
    one = ctypes.c_void_p(256)
    s = shape()
    # decode: partial results per (sequence, KV head, chunk, group head): at least the status block and one chunk
    n = binding.seka_decode_workspace_bytes(s)
    assert n >= 256 + 2 * 2 * 4 * (128 + 2) * 4
    assert binding.seka_decode_workspace_bytes(shape(dtype=binding.SEKA_F32)) == 0        # bf16 caches only
    assert binding.seka_decode_workspace_bytes(shape(n_q_heads=34)) == 0                  # 17 heads per KV head
    assert binding.seka_decode_workspace_bytes(shape(head_dim=96)) == 0
    assert lib.seka_decode_attention(ctypes.byref(shape(n_q_heads=34)), one, one, one, one, None, one, 1 << 30,
                                     None) == binding.SEKA_ERR_UNSUPPORTED
    assert lib.seka_decode_attention(ctypes.byref(s), None, one, one, one, None, one, 1 << 30, None) == binding.SEKA_ERR_INVALID_ARG
    assert lib.seka_decode_attention(ctypes.byref(s), ctypes.c_void_p(264), one, one, one, None, one, 1 << 30,
                                     None) == binding.SEKA_ERR_INVALID_ARG
    assert lib.seka_decode_attention(ctypes.byref(s), one, one, one, one, None, one, 16, None) == binding.SEKA_ERR_WORKSPACE
    assert lib.seka_decode_attention(ctypes.byref(shape(batch=0)), None, None, None, None, None, None, 0, None) == binding.SEKA_OK
    # routed forward: needs mask, U and sigma, and k_route within the rank
    args = [one, one, one, one, None]
    assert lib.seka_attention_fwd_routed(ctypes.byref(s), *args, one, one, None, 0, None, one, None, one, 1 << 30,
                                         None) == binding.SEKA_ERR_INVALID_ARG
    assert lib.seka_attention_fwd_routed(ctypes.byref(s), *args, None, one, one, 0, None, one, None, one, 1 << 30,
                                         None) == binding.SEKA_ERR_INVALID_ARG
    assert lib.seka_attention_fwd_routed(ctypes.byref(s), *args, one, one, one, 33, None, one, None, one, 1 << 30,
                                         None) == binding.SEKA_ERR_INVALID_ARG
    assert lib.seka_attention_fwd_routed(ctypes.byref(s), *args, one, one, one, 0, None, one, None, one, 16,
                                         None) == binding.SEKA_ERR_WORKSPACE
    # learner
    L = binding.SekaLearnShape
    assert lib.seka_learn_workspace_bytes(ctypes.byref(L(1000, 4, 128, 0.7))) > 256 + 4 * 2 * 128 * 128 * 4
    for bad in (L(0, 4, 128, 0.7), L(1000, 0, 128, 0.7), L(1000, 4, 96, 0.7), L(1000, 3, 64, 0.7),
                L(1000, 4, 128, 0.0), L(1000, 4, 128, 1.5)):
        assert lib.seka_learn_workspace_bytes(ctypes.byref(bad)) == 0
        assert lib.seka_learn_projections(ctypes.byref(bad), *([one] * 14), 1 << 30, None) != 0
    ok = L(1000, 4, 128, 0.7)
    assert lib.seka_learn_projections(ctypes.byref(ok), None, *([one] * 13), 1 << 30, None) == binding.SEKA_ERR_INVALID_ARG
    assert lib.seka_learn_projections(ctypes.byref(ok), *([one] * 14), 16, None) == binding.SEKA_ERR_WORKSPACE
    assert binding.seka_launch_count() == 0
