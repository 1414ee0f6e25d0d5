"""The bounded-wait failure path of the fused forward, exercised without faulting or hanging the GPU.

Every device-side wait of the kernel has a limit; when one runs out the CTA raises its abort flag, every role
leaves its loop, the loads and products already issued are waited for, tensor memory is freed, the kernel returns and
the workspace status word holds SEKA_ERR_TIMEOUT.  The test makes a wait run out by the host-set hook in the status
block: the producer of CTA 0 leaves out one V/K pair of its first work item altogether (neither the byte count nor the
copy is issued, so nothing is in flight when the CTA gives up), with the wait limit set to a few milliseconds for
that launch."""
import numpy as np
import pytest
import torch

from paper_2603_01281_b200 import binding, inputs

import helpers as H

pytestmark = pytest.mark.gpu

HOOK_SKIP_PAIR_WORD, WAIT_LIMIT_US_WORD = 4, 5      # int32 words of the 256-byte status block at the head of the workspace


@pytest.mark.parametrize("d", [128, 64])
def test_wait_runs_out_and_the_workspace_recovers(d):
    binding.load()
    # two row tiles of one head pair: CTA 0 takes the item with two key tiles, CTA 1 the one with a single tile
    w = inputs.make_custom(seed=31, dtype="bf16", lens=[256], n_q_heads=2, n_kv_heads=1, head_dim=d, rank=16,
                           gain=1.0, highlight=0.2)
    dev = H.device_tensors(w)
    shp = H.shape_of(w, dev)
    ws = binding.new_workspace(shp)
    words = ws[:256].view(torch.int32)
    O = torch.full_like(dev["Q"], float("nan"))

    def call():
        binding.seka_attention_fwd(shp, dev["Q"], dev["K"], dev["V"], O, None, dev["mask"], dev["U"], None, dev["gain"], None, ws)

    # a normal launch first: the hook words are zero, the status stays clear
    call()
    assert binding.seka_poll_status(ws) == binding.SEKA_OK
    good = O.clone()

    words[HOOK_SKIP_PAIR_WORD] = 1            # leave out V(0) / K(1) of CTA 0's first item
    words[WAIT_LIMIT_US_WORD] = 5000          # every wait of this launch gives up after 5 ms
    torch.cuda.synchronize()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record(); call(); t1.record()
    st = binding.seka_poll_status(ws)         # synchronises: the kernel has returned
    assert st == binding.SEKA_ERR_TIMEOUT, binding.status_string(st)
    where = int(words[1].item())
    assert where in (24, 25, 26, 28, 29, 40, 41), where      # the relay (operands never landed) or a role that waited on it
    assert t0.elapsed_time(t1) < 2000.0       # bounded: milliseconds, not the default two seconds per wait

    # a launch on the failed workspace does nothing (the status is sticky until it is reset)
    O.fill_(float("nan"))
    call()
    assert binding.seka_poll_status(ws) == binding.SEKA_ERR_TIMEOUT
    assert torch.isnan(O.float()).all()

    # reset (this also clears the hook words): the context is intact and the next launch is right again
    binding.seka_reset_status(ws)
    call()
    assert binding.seka_poll_status(ws) == binding.SEKA_OK
    assert torch.equal(O.view(torch.int16), good.view(torch.int16))
    Oref, _, idx = H.oracle_rows(w, None)
    H.check_attention(O.double().cpu().numpy()[idx], Oref, "after recovery")
