"""Thin ctypes binding over ``libseka_b200.so`` (the C ABI declared in ``include/seka.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch supplies device memory and the current stream.  There is no fallback: if the
compiled library is missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libseka_b200.so")

SEKA_OK, SEKA_ERR_INVALID_ARG, SEKA_ERR_UNSUPPORTED, SEKA_ERR_WORKSPACE, SEKA_ERR_CUDA, SEKA_ERR_TIMEOUT = range(6)
SEKA_F32, SEKA_BF16 = 0, 1

EXPORTS = ["seka_workspace_bytes", "seka_edit_keys", "adaseka_route", "seka_attention_fwd",
           "seka_host_staging_bytes", "seka_attention_fwd_host", "seka_reset_status", "seka_poll_status",
           "seka_status_string", "seka_launch_count", "seka_edit_keys_static", "seka_decode_workspace_bytes",
           "seka_decode_attention", "seka_attention_fwd_routed", "seka_learn_workspace_bytes", "seka_learn_projections"]
SEKA_STATIC_MAX_TOKENS = 262144


class SekaShape(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("max_seqlen", ctypes.c_int32), ("total_tokens", ctypes.c_int32),
                ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("rank", ctypes.c_int32), ("n_experts", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float), ("cu_seqlens", ctypes.c_void_p)]


class SekaLearnShape(ctypes.Structure):
    _fields_ = [("n_tokens", ctypes.c_int32), ("n_slots", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("gamma", ctypes.c_float)]


class SekaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


_lib = None


def load() -> ctypes.CDLL:
    """Load the compiled CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("CUDA library %s is missing: run __graft_entry__.build() "
                               "(python -m paper_2603_01281_b200.build); there is no CPU fallback" % LIB_PATH)
        lib = ctypes.CDLL(LIB_PATH)
        vp, sp = ctypes.c_void_p, ctypes.POINTER(SekaShape)
        lib.seka_workspace_bytes.argtypes = [sp]; lib.seka_workspace_bytes.restype = ctypes.c_size_t
        lib.seka_host_staging_bytes.argtypes = [sp]; lib.seka_host_staging_bytes.restype = ctypes.c_size_t
        lib.seka_edit_keys.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        lib.seka_edit_keys.restype = ctypes.c_int
        lib.seka_edit_keys_static.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.seka_edit_keys_static.restype = ctypes.c_int
        lib.adaseka_route.argtypes = [sp, vp, vp, vp, ctypes.c_int32, vp, vp]
        lib.adaseka_route.restype = ctypes.c_int
        lib.seka_attention_fwd.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        lib.seka_attention_fwd.restype = ctypes.c_int
        lib.seka_attention_fwd_routed.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_int32, vp, vp, vp, vp,
                                                  ctypes.c_size_t, vp]
        lib.seka_attention_fwd_routed.restype = ctypes.c_int
        lib.seka_attention_fwd_host.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t,
                                                vp, ctypes.c_size_t, vp]
        lib.seka_attention_fwd_host.restype = ctypes.c_int
        lib.seka_decode_workspace_bytes.argtypes = [sp]; lib.seka_decode_workspace_bytes.restype = ctypes.c_size_t
        lib.seka_decode_attention.argtypes = [sp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        lib.seka_decode_attention.restype = ctypes.c_int
        lp = ctypes.POINTER(SekaLearnShape)
        lib.seka_learn_workspace_bytes.argtypes = [lp]; lib.seka_learn_workspace_bytes.restype = ctypes.c_size_t
        lib.seka_learn_projections.argtypes = [lp] + [vp] * 14 + [ctypes.c_size_t, vp]
        lib.seka_learn_projections.restype = ctypes.c_int
        lib.seka_reset_status.argtypes = [vp, vp]; lib.seka_reset_status.restype = ctypes.c_int
        lib.seka_poll_status.argtypes = [vp, vp]; lib.seka_poll_status.restype = ctypes.c_int
        lib.seka_status_string.argtypes = [ctypes.c_int]; lib.seka_status_string.restype = ctypes.c_char_p
        lib.seka_launch_count.argtypes = []; lib.seka_launch_count.restype = ctypes.c_uint64
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().seka_status_string(int(status)).decode()


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, where: str) -> None:
    if status != SEKA_OK:
        raise SekaError(status, where)


def make_shape(*, batch: int, max_seqlen: int, n_q_heads: int, n_kv_heads: int, head_dim: int, rank: int,
               n_experts: int = 1, dtype: torch.dtype = torch.bfloat16, total_tokens: int = 0,
               cu_seqlens: Optional[torch.Tensor] = None, softmax_scale: float = 0.0) -> SekaShape:
    """Fill the POD shape struct; ``cu_seqlens`` is a device int32 tensor [B+1] or None."""
    if cu_seqlens is not None:
        assert cu_seqlens.dtype == torch.int32 and cu_seqlens.is_cuda and cu_seqlens.is_contiguous()
    code = {torch.float32: SEKA_F32, torch.bfloat16: SEKA_BF16}[dtype]
    s = SekaShape(batch, max_seqlen, total_tokens, n_q_heads, n_kv_heads, head_dim, rank, n_experts, code,
                  softmax_scale, cu_seqlens.data_ptr() if cu_seqlens is not None else None)
    s._keepalive = cu_seqlens
    return s


def seka_workspace_bytes(shape: SekaShape) -> int:
    return int(load().seka_workspace_bytes(ctypes.byref(shape)))


def seka_host_staging_bytes(shape: SekaShape) -> int:
    return int(load().seka_host_staging_bytes(ctypes.byref(shape)))


def new_workspace(shape: SekaShape, device="cuda") -> torch.Tensor:
    """Allocate (with torch) and clear a workspace of the size the library asks for."""
    n = seka_workspace_bytes(shape)
    if n == 0:
        raise SekaError(SEKA_ERR_INVALID_ARG, "seka_workspace_bytes")
    ws = torch.zeros(n, dtype=torch.uint8, device=device)
    return ws


def seka_edit_keys(shape: SekaShape, K_in, K_out, mask, U, alpha, gain, head_enable, workspace) -> None:
    _check(load().seka_edit_keys(ctypes.byref(shape), _ptr(K_in), _ptr(K_out), _ptr(mask), _ptr(U), _ptr(alpha),
                                 _ptr(gain), _ptr(head_enable), _ptr(workspace),
                                 workspace.numel() if workspace is not None else 0, _stream()), "seka_edit_keys")


def seka_edit_keys_static(shape: SekaShape, K_in, K_out, mask, U, alpha, gain, head_enable) -> None:
    """seka_edit_keys for callers that cannot allocate: the scratch is a fixed array inside the library
    (at most SEKA_STATIC_MAX_TOKENS tokens; calls that overlap on the GPU race on it)."""
    _check(load().seka_edit_keys_static(ctypes.byref(shape), _ptr(K_in), _ptr(K_out), _ptr(mask), _ptr(U),
                                        _ptr(alpha), _ptr(gain), _ptr(head_enable), _stream()),
           "seka_edit_keys_static")


def adaseka_route(shape: SekaShape, Q, U, sigma, k_route: int, alpha_out) -> None:
    _check(load().adaseka_route(ctypes.byref(shape), _ptr(Q), _ptr(U), _ptr(sigma), int(k_route), _ptr(alpha_out),
                                _stream()), "adaseka_route")


def seka_attention_fwd(shape: SekaShape, Q, K, V, O, lse, mask, U, alpha, gain, head_enable, workspace) -> None:
    _check(load().seka_attention_fwd(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(lse), _ptr(mask),
                                     _ptr(U), _ptr(alpha), _ptr(gain), _ptr(head_enable), _ptr(workspace),
                                     workspace.numel() if workspace is not None else 0, _stream()),
           "seka_attention_fwd")


def seka_attention_fwd_routed(shape: SekaShape, Q, K, V, O, lse, mask, U, sigma, k_route: int, alpha_out, gain,
                              head_enable, workspace) -> None:
    """AdaSEKA in one call: the routing of Eq. 6 runs inside the operand-preparation launch."""
    _check(load().seka_attention_fwd_routed(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(lse),
                                            _ptr(mask), _ptr(U), _ptr(sigma), int(k_route), _ptr(alpha_out), _ptr(gain),
                                            _ptr(head_enable), _ptr(workspace),
                                            workspace.numel() if workspace is not None else 0, _stream()),
           "seka_attention_fwd_routed")


def seka_attention_fwd_host(shape: SekaShape, h_Q, h_K, h_V, h_O, h_lse, h_mask, U, alpha, gain, head_enable,
                            staging, workspace) -> None:
    """Host-buffer variant: h_* are CPU tensors (pinned for asynchronous copies)."""
    for t in (h_Q, h_K, h_V, h_O, h_lse, h_mask):
        assert t is None or not t.is_cuda
    _check(load().seka_attention_fwd_host(ctypes.byref(shape), _ptr(h_Q), _ptr(h_K), _ptr(h_V), _ptr(h_O),
                                          _ptr(h_lse), _ptr(h_mask), _ptr(U), _ptr(alpha), _ptr(gain),
                                          _ptr(head_enable), _ptr(staging), staging.numel(), _ptr(workspace),
                                          workspace.numel(), _stream()), "seka_attention_fwd_host")


def seka_decode_workspace_bytes(shape: SekaShape) -> int:
    return int(load().seka_decode_workspace_bytes(ctypes.byref(shape)))


def seka_decode_attention(shape: SekaShape, Q, K, V, O, lse, workspace) -> None:
    """One decode step over the (already edited) cache: Q and O are [B, Hq, d], K and V the packed caches."""
    _check(load().seka_decode_attention(ctypes.byref(shape), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(lse),
                                        _ptr(workspace), workspace.numel() if workspace is not None else 0,
                                        _stream()), "seka_decode_attention")


def seka_learn_projections(h, h_pos, h_neg, answer_tokens, gamma: float) -> dict:
    """Offline spectral learning for every slot of bf16 embeddings [n, slots, d]; allocates the outputs with torch
    and returns them in a dict (omega_pos, omega_neg, U_pos, U_neg, S_pos, S_neg, k_pos, k_neg, D)."""
    n, slots, d = h.shape
    assert h.dtype == torch.bfloat16 and h_pos.shape == h.shape and h_neg.shape == h.shape
    shp = SekaLearnShape(n, slots, d, gamma)
    nbytes = int(load().seka_learn_workspace_bytes(ctypes.byref(shp)))
    if nbytes == 0:
        raise SekaError(SEKA_ERR_UNSUPPORTED, "seka_learn_workspace_bytes")
    ws = torch.zeros(nbytes, dtype=torch.uint8, device=h.device)
    f32 = dict(dtype=torch.float32, device=h.device)
    out = {"omega_pos": torch.empty((slots, d, d), **f32), "omega_neg": torch.empty((slots, d, d), **f32),
           "U_pos": torch.empty((slots, d, d), **f32), "U_neg": torch.empty((slots, d, d), **f32),
           "S_pos": torch.empty((slots, d), **f32), "S_neg": torch.empty((slots, d), **f32),
           "k_pos": torch.empty(slots, dtype=torch.int32, device=h.device),
           "k_neg": torch.empty(slots, dtype=torch.int32, device=h.device), "D": torch.empty(slots, **f32)}
    _check(load().seka_learn_projections(ctypes.byref(shp), _ptr(h), _ptr(h_pos), _ptr(h_neg), _ptr(answer_tokens),
                                         _ptr(out["omega_pos"]), _ptr(out["omega_neg"]), _ptr(out["U_pos"]),
                                         _ptr(out["U_neg"]), _ptr(out["S_pos"]), _ptr(out["S_neg"]), _ptr(out["k_pos"]),
                                         _ptr(out["k_neg"]), _ptr(out["D"]), _ptr(ws), ws.numel(), _stream()),
           "seka_learn_projections")
    st = seka_poll_status(ws)
    if st != SEKA_OK:
        raise SekaError(st, "seka_learn_projections (device status)")
    out["workspace"] = ws
    return out


def seka_reset_status(workspace) -> None:
    _check(load().seka_reset_status(_ptr(workspace), _stream()), "seka_reset_status")


def seka_poll_status(workspace) -> int:
    return int(load().seka_poll_status(_ptr(workspace), _stream()))


def seka_launch_count() -> int:
    return int(load().seka_launch_count())
