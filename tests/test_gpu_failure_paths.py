"""Failure detection on the GPU, in forms that fault, trap or hang nothing: a bounded device-side wait that is made
to run out reports through the status word and leaves the context usable; a list id that the host corrupts is
clamped by the kernel and reported; both codes are cleared by the next da2_prepare."""
import numpy as np
import pytest
import torch

import da2_inputs
import paper_2609_32628_b200 as da2
from helpers import run_gpu

pytestmark = pytest.mark.gpu

W = da2_inputs.Workload


def test_bounded_wait_that_runs_out_reports_timeout_and_the_context_survives():
    w = W("probe", 1, 2, 64, 2, 16, 16, 0.1, 0.2, 0.3, seed=41)
    q, k, v = da2_inputs.make_qkv(w, "cuda")
    plan, ws, out = run_gpu(w, q, k, v)
    assert da2.da2_device_status(plan, ws) == 0
    # a wait on a barrier that nothing completes, limited to about a millisecond of GPU clock cycles
    da2.da2_probe_bounded_wait(plan, ws, 2_000_000)
    torch.cuda.synchronize()                       # the kernel returned by itself
    assert da2.da2_device_status(plan, ws) == 5    # DA2_ERR_TIMEOUT
    # the same context keeps working: a normal call clears the word and gives the same bits as before
    out2 = torch.full_like(out, float("nan"))
    da2.da2_prepare(plan, q, k, v, ws)
    da2.da2_attention_fwd(plan, q, k, v, ws, out2)
    torch.cuda.synchronize()
    assert da2.da2_device_status(plan, ws) == 0
    assert torch.equal(out2.view(torch.int16), out.view(torch.int16))
    with pytest.raises(da2.Da2Error):
        da2.da2_probe_bounded_wait(plan, ws, 0)    # the limit itself is validated


def test_list_id_out_of_range_is_clamped_and_reported():
    w = W("badlist", 1, 2, 64, 2, 16, 16, 0.1, 0.2, 0.3, seed=42)
    q, k, v = da2_inputs.make_qkv(w, "cuda")
    plan, ws, out = run_gpu(w, q, k, v)
    I = plan.info
    ids = ws[I.off_ids:I.off_ids + 2 * int(I.ids_per_head) * I.B * I.H].view(torch.int16)
    ids[3] = np.int16(I.R + 7)                     # host-made corruption of one key-block id of head 0, row 0
    bad = torch.full_like(out, float("nan"))
    da2.da2_attention_fwd(plan, q, k, v, ws, bad)
    torch.cuda.synchronize()                       # nothing out of range was read: the kernel used block 0 instead
    assert da2.da2_device_status(plan, ws) == 6    # DA2_ERR_INTERNAL
    assert torch.isfinite(bad.float()).all()
    # rows that do not use the corrupted list are untouched
    tok_row0 = torch.arange(8, device="cuda")[:, None] * w.Wg + torch.arange(8, device="cuda")[None, :]
    mask = torch.ones(w.N, dtype=torch.bool, device="cuda")
    mask[tok_row0.flatten()] = False
    assert torch.equal(bad[0, 0][mask].view(torch.int16), out[0, 0][mask].view(torch.int16))
    assert torch.equal(bad[0, 1].view(torch.int16), out[0, 1].view(torch.int16))
    da2.da2_prepare(plan, q, k, v, ws)             # rewrites the lists and clears the word
    da2.da2_attention_fwd(plan, q, k, v, ws, bad)
    torch.cuda.synchronize()
    assert da2.da2_device_status(plan, ws) == 0
    assert torch.equal(bad.view(torch.int16), out.view(torch.int16))
