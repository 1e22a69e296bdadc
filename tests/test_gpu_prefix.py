"""GPU parity with prefix (text) tokens (App. C.1): prefix interactions lie outside the region budget -- every video
query keeps all prefix keys, every prefix query attends to all keys -- and run in the 16-bit tier.  The CUDA path gets
the joint tensors [B, H, P + N, d] (prefix first); the oracle runs its video-only stages on the video part and its
attention on the joint sequence."""
import numpy as np
import pytest
import torch

import da2_inputs
import oracle
import paper_2609_32628_b200 as da2
from helpers import Workspace, compare_lists, oracle_all, rel_l2, scale_of

pytestmark = pytest.mark.gpu

W = da2_inputs.Workload


def _joint_inputs(w, P, seed):
    """Video tokens from the workload's generator, P prefix tokens (plain seeded normals) in front of them."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    vid = da2_inputs.make_qkv(w, "cuda")
    out = []
    for x in vid:
        pre = torch.randn(w.B, w.H, P, w.head_dim, generator=g).to(torch.bfloat16).cuda()
        out.append(torch.cat([pre, x], dim=2).contiguous())
    return out


@pytest.mark.parametrize("name,P", [("p3", 77), ("p3", 128), ("p64", 200), ("p8only", 40)])
def test_prefix_tokens_parity(name, P):
    w = {"p3": W("p3", 1, 2, 128, 3, 12, 20, 0.15, 0.25, 0.30, seed=51),      # three tiers + prefix, ragged tiles
         "p64": W("p64", 2, 2, 64, 2, 16, 16, 0.0, 0.2, 0.3, seed=52),        # d = 64, no budgeted 16-bit tier
         "p8only": W("p8only", 1, 1, 128, 2, 16, 16, 0.0, 0.5, 0.0, seed=53)}[name]
    q, k, v = _joint_inputs(w, P, 1000 + P)
    BH, d = w.B * w.H, w.head_dim
    plan = da2.da2_plan(w.B, w.H, w.T, w.Hg, w.Wg, d, w.frac16, w.frac8, w.frac4, lam=w.lam, n_prefix=P)
    I = plan.info
    R, Rp = I.R, I.R_prefix
    Rt = R + Rp
    assert I.n_prefix == P and Rp == -(-P // 64) and I.tier_active[2] == 1
    ws = torch.zeros(int(I.workspace_bytes), dtype=torch.uint8, device="cuda")
    out = torch.full_like(q, float("nan"))
    da2.da2_prepare(plan, q, k, v, ws)
    da2.da2_attention_fwd(plan, q, k, v, ws, out)
    torch.cuda.synchronize()
    assert da2.da2_device_status(plan, ws) == 0
    assert torch.isfinite(out.float()).all()       # every row of the joint tensor was written

    # ---- oracle: video-only stages on the video part
    vid = lambda t: t[:, :, P:].contiguous()
    ref = oracle_all(w, vid(q), vid(k), vid(v))
    plv = ref["pl"]
    pl = oracle.plan_with_prefix(plv, P)
    ids_x, cnt_x = oracle.lists_with_prefix(ref["ids"], ref["counts"], R, Rp)
    V = Workspace(plan, ws)
    for i, nm in enumerate(("qavg", "qmax", "kavg", "kmax")):
        assert np.array_equal(V.desc(i), ref[nm]), nm

    # ---- lists of the joint sequence, row by row
    cnt = ws[I.off_counts:I.off_counts + BH * Rt * 16].cpu().numpy().view(np.int32).reshape(BH, Rt, 4)
    ids_raw = ws[I.off_ids:I.off_ids + BH * int(I.ids_per_head) * 2].cpu().numpy().view(np.uint16)
    ids_raw = ids_raw.reshape(BH, int(I.ids_per_head))
    ids_g = np.full((BH, Rt, Rt), -1, np.int32)
    for h in range(BH):
        for a in range(Rt):
            n, o = int(cnt[h, a, :3].sum()), int(cnt[h, a, 3])
            ids_g[h, a, :n] = ids_raw[h, o:o + n]
    cnt_g = np.ascontiguousarray(cnt[:, :, :3])
    A_x = np.zeros((BH, Rt, Rt), np.float32)       # scores of the video pairs; prefix entries cannot be near-ties
    A_x[:, :R, :R] = ref["A"]
    bad, excused = compare_lists(A_x, ids_x, cnt_x, ids_g, cnt_g)
    print(f"[{w.name} P={P}] list rows differing by near-ties: {len(bad)} (entries excused: {excused})")
    assert all(a < R for _, a in bad)

    # ---- bf16 records of all blocks incl. the prefix blocks
    qb, kb, vb = (oracle.bf16_bits(t.reshape(BH, P + w.N, d).cpu()) for t in (q, k, v))
    qr = ws[I.off_qrec[2]:I.off_qrec[2] + BH * Rt * I.qrec_bytes[2]].cpu().numpy().view(np.uint16)
    kvr = ws[I.off_kvrec[2]:I.off_kvrec[2] + BH * Rt * I.kvrec_bytes[2]].cpu().numpy().view(np.uint16)
    qr = qr.reshape(BH, Rt, d // 8, 64, 8).transpose(0, 1, 3, 2, 4).reshape(BH, Rt, 64, d)
    kvr = kvr.reshape(BH, Rt, 2 * 64 * d)
    kr = kvr[:, :, :64 * d].reshape(BH, Rt, d // 8, 64, 8).transpose(0, 1, 3, 2, 4).reshape(BH, Rt, 64, d)
    vr = kvr[:, :, 64 * d:].reshape(BH, Rt, 8, d, 8).transpose(0, 1, 2, 4, 3).reshape(BH, Rt, 64, d)
    st = np.maximum(pl.slot_token, 0)
    valid = (pl.slot_token >= 0)[None, :, :, None]
    for rec, x in ((qr, qb), (kr, kb), (vr, vb)):
        assert np.array_equal(rec, np.where(valid, x[:, st], 0))

    # ---- attention on every row of the joint sequence
    ops = oracle.pad_operands(oracle.quantize_all(ref["q"], ref["k"], ref["v"], plv), Rt)
    sel = [(h, a) for h in range(BH) for a in range(Rt) if (h, a) not in set(bad)]
    exp = oracle.attention(qb, kb, vb, pl, ids_x, cnt_x, ops, scale_of(w), sel)
    o = out.reshape(BH, P + w.N, d).float().cpu().numpy()
    got = np.zeros_like(exp)
    for i, (h, a) in enumerate(sel):
        tok = pl.slot_token[a]
        got[i] = np.where((tok >= 0)[:, None], o[h, np.maximum(tok, 0)], 0.0)
    err, mx = rel_l2(got, exp.astype(np.float64)), float(np.abs(got - exp).max())
    pre = [i for i, (h, a) in enumerate(sel) if a >= R]
    dense = oracle.dense(qb, kb, vb, pl, scale_of(w), [sel[i] for i in pre])
    print(f"[{w.name} P={P}] attention vs oracle: rel L2 {err:.3e}, max abs {mx:.3e} on {len(sel)} blocks; prefix rows "
          f"vs dense fp64: rel L2 {rel_l2(got[pre], dense):.3e}")
    assert err <= 1e-2 and mx <= 2e-2
    assert rel_l2(got[pre], dense) <= 1e-2


def test_prefix_needs_row_scope_and_zero_prefix_changes_nothing():
    with pytest.raises(da2.Da2Error) as e:
        da2.da2_plan(1, 1, 2, 16, 16, 64, 0.0, 0.2, 0.2, rank_scope=1, n_prefix=10)
    assert e.value.code == 2
    a = da2.da2_plan(1, 2, 2, 16, 16, 64, 0.1, 0.2, 0.2).info
    b = da2.da2_plan(1, 2, 2, 16, 16, 64, 0.1, 0.2, 0.2, n_prefix=0).info
    assert bytes(a) == bytes(b)
