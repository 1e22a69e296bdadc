"""da2_draft_map_noalloc -- the draft map for callers that cannot allocate device memory (no cudaMalloc inside a
serving loop, or a memory pool owned by someone else): its scratch is a fixed array inside the library instead of the
caller's workspace.  Checked against the regular path (da2_prepare's map in the workspace), on two calls in a row with
different problem sizes so that what the first call left in the shared scratch cannot leak into the second.

Collected last on purpose (file name), and passes alone in a fresh process as well as after the other tests."""
import numpy as np
import pytest
import torch

import da2_inputs
import oracle
import paper_2609_32628_b200 as da2

pytestmark = pytest.mark.gpu


def _regular_path(w):
    q, k, v = da2_inputs.make_qkv(w, "cuda")
    plan = da2.da2_plan(w.B, w.H, w.T, w.Hg, w.Wg, w.head_dim, w.frac16, w.frac8, w.frac4, lam=w.lam)
    ws = torch.empty(int(plan.info.workspace_bytes), dtype=torch.uint8, device="cuda")
    da2.da2_prepare(plan, q, k, v, ws)
    torch.cuda.synchronize()
    I = plan.info
    BH, R, d = w.B * w.H, I.R, w.head_dim
    desc = [ws[I.off_desc[i]:I.off_desc[i] + BH * R * d * 4].view(torch.float32).view(BH, R, d).clone()
            for i in range(4)]
    ref = ws[I.off_map:I.off_map + BH * R * R * 4].view(torch.float32).view(BH, R, R).clone()
    return desc, ref, float(I.lambda_), float(I.softmax_scale)


def test_noalloc_draft_map_matches_regular_path_twice_in_a_row():
    cases = [da2_inputs.Workload("na_big", 1, 3, 128, 3, 20, 28, 0.0, 0.2, 0.3, seed=31),   # R = 36
             da2_inputs.WORKLOADS["tiny"]]                                                   # R = 16, d = 64
    prepared = [_regular_path(w) for w in cases]
    outs = []
    for desc, ref, lam, scale in prepared:   # the two no-alloc calls run back to back
        out = torch.full_like(ref, float("nan"))
        da2.da2_draft_map_noalloc(*desc, lam, scale, out)
        outs.append(out)
    torch.cuda.synchronize()
    for out, (desc, ref, lam, scale) in zip(outs, prepared):
        assert torch.isfinite(out).all()
        assert torch.equal(out, ref)   # the same kernels on the same descriptors: identical bits
        assert np.allclose(out.sum(-1).cpu().numpy(), 1.0, atol=1e-5)
        # and against the CPU oracle's draft map of the same descriptors (the tolerance of the regular parity tests)
        exp = oracle.draft(*(t.cpu().numpy() for t in desc), lam, scale)
        assert np.allclose(out.cpu().numpy(), exp, rtol=2e-5, atol=1e-12)


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    BH, R, d = 2, 1024, 64   # 2 * 1024 * 1024 > 2**20
    x = torch.zeros(1, device="cuda")
    desc = [torch.zeros(16, device="cuda") for _ in range(4)]
    lib = da2.load_library()
    fn = lib.da2_draft_map_noalloc
    import ctypes
    fn.restype = ctypes.c_int
    vp = ctypes.c_void_p
    fn.argtypes = [vp, vp, vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_float, ctypes.c_float,
                   vp, vp]
    rc = fn(*(int(t.data_ptr()) for t in desc), BH, R, d, 0.2, 0.125, int(x.data_ptr()), None)
    assert rc == 3  # DA2_ERR_WORKSPACE_TOO_SMALL, nothing launched
    rc = fn(*(int(t.data_ptr()) for t in desc), 40000, 5, d, 0.2, 0.125, int(x.data_ptr()), None)
    assert rc == 2  # DA2_ERR_UNSUPPORTED: more heads than a launch dimension holds, nothing launched
