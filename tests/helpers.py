"""Shared helpers for the GPU parity tests: move a synthetic workload to the device, call the
library through its binding, and evaluate the CPU oracle on the same inputs."""
import numpy as np
import torch

import oracle
from paper_2603_01281_b200 import binding, inputs

TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16}


def device_tensors(w, device="cuda"):
    dt = TORCH_DT[w.dtype]
    d = {
        "Q": torch.from_numpy(w.Q).to(device=device, dtype=dt),
        "K": torch.from_numpy(w.K).to(device=device, dtype=dt),
        "V": torch.from_numpy(w.V).to(device=device, dtype=dt),
        "mask": torch.from_numpy(w.mask).to(device),
        "U": torch.from_numpy(w.U).to(device),
        "gain": torch.from_numpy(w.gain).to(device),
        "cu": torch.from_numpy(w.cu_seqlens).to(device),
        "sigma": None if w.sigma is None else torch.from_numpy(w.sigma).to(device),
    }
    return d


def shape_of(w, dev, force_varlen=False):
    varlen = force_varlen or w.fixed_len is None
    return binding.make_shape(batch=w.batch, max_seqlen=w.max_seqlen, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                              head_dim=w.head_dim, rank=w.rank, n_experts=w.n_experts, dtype=TORCH_DT[w.dtype],
                              total_tokens=w.total_tokens if varlen else 0, cu_seqlens=dev["cu"] if varlen else None)


def run_fused(w, dev=None, alpha=None, head_enable=None, steer=True, want_lse=True, force_varlen=False):
    """seka_attention_fwd through the C ABI; returns (O float64 numpy, LSE float64 numpy or None)."""
    dev = dev or device_tensors(w)
    shp = shape_of(w, dev, force_varlen)
    ws = binding.new_workspace(shp)
    O = torch.full_like(dev["Q"], float("nan"))
    lse = torch.full((w.total_tokens, w.n_q_heads), float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    a = None if alpha is None else torch.as_tensor(np.asarray(alpha, dtype=np.float32)).cuda().contiguous()
    he = None if head_enable is None else torch.as_tensor(np.asarray(head_enable, dtype=np.uint8)).cuda()
    binding.seka_attention_fwd(shp, dev["Q"], dev["K"], dev["V"], O, lse, dev["mask"] if steer else None,
                               dev["U"] if steer else None, a, dev["gain"], he, ws)
    st = binding.seka_poll_status(ws)
    assert st == binding.SEKA_OK, binding.status_string(st)
    return O.double().cpu().numpy(), (None if lse is None else lse.double().cpu().numpy())


def run_edit(w, dev=None, alpha=None, head_enable=None, in_place=False):
    dev = dev or device_tensors(w)
    shp = shape_of(w, dev)
    ws = binding.new_workspace(shp)
    a = None if alpha is None else torch.as_tensor(np.asarray(alpha, dtype=np.float32)).cuda().contiguous()
    he = None if head_enable is None else torch.as_tensor(np.asarray(head_enable, dtype=np.uint8)).cuda()
    Kin = dev["K"].clone()
    Kout = Kin if in_place else torch.full_like(Kin, float("nan"))
    binding.seka_edit_keys(shp, Kin, Kout, dev["mask"], dev["U"], a, dev["gain"], he, ws)
    torch.cuda.synchronize()
    if not in_place:
        assert torch.equal(Kin, dev["K"]), "input keys were modified"
    return Kout


def oracle_rows(w, rows, alpha=None, head_enable=None):
    return oracle.seka_attention(w.Q, w.K, w.V, w.mask, w.cu_seqlens, w.U, alpha=alpha, gain=w.gain,
                                 head_enable=head_enable, rows=rows)


def check_attention(O_gpu, O_ref, label=""):
    """Stated tolerance for bf16 attention output on unit-variance inputs: max abs error 1e-2 and
    mean abs error 1e-3.  Where |o| > 1.28 the rounding of the bf16 output alone can reach 2^-8 |o|,
    so the per-element bound is max(1e-2, 2^-7 |o|) (one bf16 ulp, relative).  The bound is used as
    stated for every gain: the edited keys enter the score product with fp32 accuracy."""
    err = np.abs(O_gpu - O_ref)
    assert np.isfinite(O_gpu).all(), label + ": non-finite output"
    bound = np.maximum(1e-2, 2.0 ** -7 * np.abs(O_ref))
    worst = float((err / bound).max()) if err.size else 0.0
    assert worst <= 1.0, "%s: max abs err %.4g (ratio to bound %.3f)" % (label, err.max(), worst)
    assert err.size == 0 or err.mean() <= 1e-3, "%s: mean abs err %.4g" % (label, err.mean())
    return float(err.max()) if err.size else 0.0, float(err.mean()) if err.size else 0.0


def all_rows(w):
    return [np.arange(int(w.cu_seqlens[b + 1] - w.cu_seqlens[b]), dtype=np.int32) for b in range(w.batch)]


def sampled_rows(w, n, seed=0):
    rng = np.random.default_rng(seed)
    out = []
    for b in range(w.batch):
        s, e = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        out.append(inputs.sample_rows(rng, e - s, w.mask[s:e], n) if e > s else np.zeros(0, dtype=np.int32))
    return out
