"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Bars: descriptors, codes and scales bit-exact; lists exact except near-ties within 1e-5 relative (counted and
printed); attention output rel. L2 <= 1e-2 and max abs <= 2e-2 against the oracle's quantisation-emulated result.
"""
import dataclasses

import numpy as np
import pytest
import torch

import da2_inputs
import oracle
import paper_2609_32628_b200 as da2
from helpers import Workspace, compare_lists, oracle_all, oracle_operands, rel_l2, run_gpu, scale_of

pytestmark = pytest.mark.gpu

W = da2_inputs.Workload
SMALL = {
    # the tiny correctness configuration
    "tiny": da2_inputs.WORKLOADS["tiny"],
    # ragged edge tiles (12 = 8+4 rows, 20 = 8+8+4 columns), d = 128, all three tiers at once
    "ragged3": W("ragged3", 1, 2, 128, 3, 12, 20, 0.15, 0.25, 0.30, seed=11),
    # d = 64 with all three tiers, ragged in both directions
    "ragged64": W("ragged64", 1, 3, 64, 2, 9, 13, 0.2, 0.2, 0.3, seed=12),
    # single-tier endpoints
    "all8": W("all8", 1, 1, 128, 2, 16, 16, 0.0, 1.0, 0.0, seed=13),
    "all16": W("all16", 1, 1, 128, 2, 16, 16, 1.0, 0.0, 0.0, seed=14),
    "all4": W("all4", 1, 1, 128, 2, 16, 16, 0.0, 0.0, 1.0, seed=15),
    # a 4 -> 16 switch with no 8-bit phase
    "skip8": W("skip8", 1, 2, 64, 2, 16, 16, 0.25, 0.0, 0.5, seed=16),
    # batch of two (heads of different batch entries are independent problems), all three tiers
    "batch2": W("batch2", 2, 2, 64, 2, 16, 16, 0.1, 0.2, 0.3, seed=17),
}


def _inputs(w, device="cuda"):
    return da2_inputs.make_qkv(w, device)


def _check_prepare(w, plan, ws, ref, heads=None, g_fixed=None, dv_fixed=None):
    V = Workspace(plan, ws, heads)
    I = plan.info
    # descriptors: bit-exact
    for i, name in enumerate(("qavg", "qmax", "kavg", "kmax")):
        assert np.array_equal(V.desc(i), ref[name]), name
    # draft map: fp32 evaluation of a softmax mixture
    A = V.draft_map()
    assert np.allclose(A, ref["A"], rtol=2e-5, atol=1e-12)
    ids_g, cnt_g = V.lists()
    bad_rows, excused = compare_lists(ref["A"], ref["ids"], ref["counts"], ids_g, cnt_g)
    print(f"[{w.name}] list rows differing by near-ties: {len(bad_rows)} (entries excused: {excused})")
    if I.rank_scope == 0:
        k4, k8, k16 = (int(x) for x in I.quota)
        assert (cnt_g == np.array([k4, k8, k16])).all()
    else:
        assert (cnt_g.reshape(len(V.heads), -1, 3).sum(1) == np.array([int(x) for x in I.quota])).all()
    # operand records: bit-exact codes and scales
    pl = ref["pl"]
    if I.tier_active[1]:
        for which, x in (("q", ref["q"]), ("k", ref["k"])):
            codes, delta = oracle.quant_int8(x, pl)
            assert np.array_equal(V.q_or_k_int8(which), codes), f"int8 {which} codes"
            assert np.array_equal(V.dq8() if which == "q" else V.dk8(), delta), f"int8 {which} scales"
        if dv_fixed is None:
            codes, dc = oracle.quant_v_e4m3(ref["v"], pl)
        else:   # carried-over per-channel scales: the workspace still holds them, the codes follow them
            dc = np.ascontiguousarray(np.asarray(dv_fixed, np.float32)[V.heads])
            codes = oracle.quant_v_e4m3_given(ref["v"], pl, dc)
        assert np.array_equal(V.dv8(), dc)
        assert np.array_equal(V.v_e4m3(), codes), "e4m3 v codes"
    if I.tier_active[0]:
        if g_fixed is None:
            g = np.stack([oracle.nvfp4_global_scale(ref[n]) for n in ("q", "k", "v")], 1)
        else:   # caller-fixed per-tensor scales: the workspace must hold exactly those, and the codes follow them
            g = np.stack([np.asarray(x, np.float32)[V.heads] for x in g_fixed], 1)
        assert np.array_equal(V.gscale(), g)
        for i, which in enumerate(("q", "k")):
            codes, sf = oracle.quant_nvfp4_qk(ref[which], pl, np.ascontiguousarray(g[:, i]))
            gc, gsf = V.q_or_k_fp4(which)
            assert np.array_equal(gsf, sf), f"nvfp4 {which} scales"
            assert np.array_equal(gc, codes), f"nvfp4 {which} codes"
        codes, sf = oracle.quant_nvfp4_v(ref["v"], pl, np.ascontiguousarray(g[:, 2]))
        gc, gsf = V.v_fp4()
        assert np.array_equal(gsf, sf), "nvfp4 v scales"
        assert np.array_equal(gc, codes), "nvfp4 v codes"
    if I.tier_active[2]:
        st = np.maximum(pl.slot_token, 0)
        valid = (pl.slot_token >= 0)[None, :, :, None]
        for rec, x in zip(V.bf16_records(), (ref["q"], ref["k"], ref["v"])):
            exp = np.where(valid, x[:, st], 0)
            assert np.array_equal(rec, exp)
    return bad_rows


def _check_attention(w, out, ref, sel, bad_rows, heads=None, g_fixed=None, dv_fixed=None):
    """sel: [(head index within ref, block)]; rows whose lists differ by near-ties are left out."""
    pl = ref["pl"]
    sel = [s for s in sel if tuple(s) not in set(bad_rows)]
    ops = oracle_operands(ref, g_fixed, heads, dv_fixed)
    exp = oracle.attention(ref["q"], ref["k"], ref["v"], pl, ref["ids"], ref["counts"], ops, scale_of(w), sel)
    dense = oracle.dense(ref["q"], ref["k"], ref["v"], pl, scale_of(w), sel)
    o = out.reshape(-1, w.N, w.head_dim)
    hs = list(range(o.shape[0])) if heads is None else list(heads)
    got = np.zeros_like(exp)
    for i, (h, a) in enumerate(sel):
        tok = pl.slot_token[a]
        rows = o[hs[h], torch.from_numpy(np.maximum(tok, 0)).to(o.device).long()].float().cpu().numpy()
        got[i] = np.where((tok >= 0)[:, None], rows, 0.0)
    assert np.isfinite(got).all()
    err, mx = rel_l2(got, exp.astype(np.float64)), float(np.abs(got - exp).max())
    err_d = rel_l2(got, dense)
    print(f"[{w.name}] attention vs oracle: rel L2 {err:.3e}, max abs {mx:.3e}; vs dense fp64: rel L2 {err_d:.3e} "
          f"(oracle vs dense {rel_l2(exp, dense):.3e}) on {len(sel)} query blocks")
    # bars: rel. L2 <= 1e-2 and max abs <= 2e-2.  The output is bf16: where |O| >= 4 its spacing (2^-5 and up) is
    # wider than 2e-2, so a value whose exact result lies next to a rounding boundary can only differ by one unit
    # in the last place or not at all; there the bar is that one unit (counted and printed).
    diff = np.abs(got - exp)
    ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(exp), 1e-30))) - 7)
    wide = (np.abs(exp) >= 4.0) & (diff > 2e-2)
    if wide.any():
        print(f"[{w.name}] {int(wide.sum())} outputs with |O| >= 4 differ by one bf16 unit in the last place")
    assert err <= 1e-2 and (diff <= np.where(np.abs(exp) >= 4.0, np.maximum(ulp, 2e-2), 2e-2)).all()
    return err, mx


@pytest.mark.parametrize("name", list(SMALL))
def test_small_configs_full_parity(name):
    w = SMALL[name]
    q, k, v = _inputs(w)
    plan, ws, out = run_gpu(w, q, k, v)
    ref = oracle_all(w, q, k, v)
    bad = _check_prepare(w, plan, ws, ref)
    R = plan.info.R
    sel = [(h, a) for h in range(w.B * w.H) for a in range(R)]
    _check_attention(w, out, ref, sel, bad)
    # every valid output element was written (the buffer was NaN-filled) -- padding does not exist in raster order
    assert torch.isfinite(out.float()).all()


@pytest.mark.parametrize("name", ["tiny", "ragged3", "ragged64"])
def test_head_scope_parity(name):
    """Alg. 1 as printed: one ranking over all R*R pairs of a head; rows may keep different numbers of blocks."""
    w = SMALL[name]
    q, k, v = _inputs(w)
    plan, ws, out = run_gpu(w, q, k, v, rank_scope=1)
    ref = oracle_all(w, q, k, v, rank_scope=1)
    bad = _check_prepare(w, plan, ws, ref)
    sel = [(h, a) for h in range(w.B * w.H) for a in range(plan.info.R)]
    _check_attention(w, out, ref, sel, bad)


def test_head_scope_empty_rows_give_zero():
    """A head-level budget can leave a query block without any key block: those rows return zero (App. C.1)."""
    w = W("sparsehead", 1, 1, 64, 2, 16, 16, 0.0, 0.02, 0.02, seed=21)
    q, k, v = _inputs(w)
    plan, ws, out = run_gpu(w, q, k, v, rank_scope=1)
    ref = oracle_all(w, q, k, v, rank_scope=1)
    bad = _check_prepare(w, plan, ws, ref)
    empty = [a for a in range(plan.info.R) if ref["counts"][0, a].sum() == 0]
    assert empty, "the case is built to have empty rows"
    pl = ref["pl"]
    for a in empty:
        if (0, a) in set(bad):
            continue
        assert (out[0, 0, torch.from_numpy(pl.slot_token[a]).long().cuda()] == 0).all()
    sel = [(0, a) for a in range(plan.info.R)]
    _check_attention(w, out, ref, sel, bad)


@pytest.mark.parametrize("lam", [0.0, 1.0])
def test_lambda_endpoints(lam):
    w = SMALL["ragged64"]
    q, k, v = _inputs(w)
    plan, ws, out = run_gpu(w, q, k, v, lam=lam)
    ref = oracle_all(w, q, k, v, lam=lam)
    bad = _check_prepare(w, plan, ws, ref)
    _check_attention(w, out, ref, [(0, 0), (1, 3), (2, 5)], bad)


def test_zero_budget_gives_zero_output():
    w = W("nothing", 1, 1, 64, 1, 16, 16, 0.0, 0.0, 0.0, seed=22)
    q, k, v = _inputs(w)
    plan, ws, out = run_gpu(w, q, k, v)
    assert (out == 0).all()


def test_determinism():
    w = SMALL["ragged3"]
    q, k, v = _inputs(w)
    # zero-filled workspaces so that bytes the library never writes compare equal
    _, ws1, o1 = run_gpu(w, q, k, v, zero_ws=True)
    _, ws2, o2 = run_gpu(w, q, k, v, zero_ws=True)
    assert torch.equal(o1, o2)
    assert torch.equal(ws1, ws2)


def test_argument_errors_are_reported_before_any_launch():
    w = SMALL["tiny"]
    q, k, v = _inputs(w)
    plan = da2.da2_plan(w.B, w.H, w.T, w.Hg, w.Wg, w.head_dim, 0.0, 0.25, 0.25)
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(da2.Da2Error) as e:
        da2.da2_prepare(plan, q, k, v, small)
    assert e.value.code == 3
    ws = torch.empty(int(plan.info.workspace_bytes), dtype=torch.uint8, device="cuda")
    with pytest.raises(da2.Da2Error) as e:
        da2.da2_attention_fwd(plan, q, k, v, ws, q)  # output aliases an input
    assert e.value.code == 1


def _sampled_parity(name, nheads=2, nblocks=16, rank_scope=0, g_fixed=None, partition=0):
    """Full-size workload in the launch configuration the benchmark times; the oracle follows on sampled heads
    (every stage before attention in full for those heads) and on sampled query blocks for the attention output.
    The sample always holds the first and the last head (the last head's records lie beyond 2^31 bytes in the
    larger workspaces), both query blocks of two CTA pairs, one block of every edge-tile class and the last block."""
    w = da2_inputs.WORKLOADS[name]
    q, k, v = _inputs(w)
    plan, ws, out = run_gpu(w, q, k, v, rank_scope=rank_scope, g_fixed=g_fixed, partition=partition)
    BH, R = w.B * w.H, plan.info.R
    rng = np.random.default_rng(w.seed)
    heads = {0, BH - 1}
    while len(heads) < min(nheads, BH):
        heads.add(int(rng.integers(BH)))
    heads = sorted(heads)[:max(nheads, 1)] if nheads < 2 else sorted(heads)
    ref = oracle_all(w, q, k, v, heads=heads, rank_scope=rank_scope, balanced=bool(partition))
    bad = _check_prepare(w, plan, ws, ref, heads=heads, g_fixed=g_fixed)
    R_f, ntx = plan.info.R_f, plan.info.ntx
    pair0, pair1 = 2 * int(rng.integers(R // 2)), 2 * int(rng.integers(R // 2))
    blocks = {0, ntx - 1, R_f - ntx, R_f - 1, R - 1, pair0, pair0 + 1, pair1, pair1 + 1}
    while len(blocks) < min(nblocks, R):
        blocks.add(int(rng.integers(R)))
    sel = [(hi, int(a)) for hi in range(len(heads)) for a in sorted(blocks)]
    _check_attention(w, out, ref, sel, bad, heads=heads, g_fixed=g_fixed)


def test_wan1p3b_480p_sampled_parity():
    _sampled_parity("wan1p3b_480p", nheads=3, nblocks=16)


def test_wan1p3b_480p_head_scope_sampled_parity():
    """Alg. 1 as printed (one ranking over all R*R pairs of a head) at a full-size configuration: rows of very
    different lengths, the scheduling order, CSR-style list offsets."""
    _sampled_parity("wan1p3b_480p", nheads=2, nblocks=16, rank_scope=1)


def test_wan14b_720p_head_scope_sampled_parity():
    """The head-level budget on the bench workload (the configuration whose timing the measured table quotes): rows
    from 11 to 1260 blocks long, paired by the scheduling order."""
    _sampled_parity("wan14b_720p", nheads=2, nblocks=8, rank_scope=1)


@pytest.mark.parametrize("name", ["ragged3", "ragged64", "batch2"])
@pytest.mark.parametrize("rank_scope", [0, 1])
def test_balanced_partition_full_parity(name, rank_scope):
    """The balanced ragged partition of App. C.2 (capacity 64) instead of fixed tiles: fewer blocks (12 x 20: 4
    instead of 6 per frame; 9 x 13: 2 instead of 4), regions of 58 to 64 tokens packed into the first slots of their
    blocks; every stage against the oracle on its own balanced plan, in both ranking scopes."""
    w = SMALL[name]
    q, k, v = _inputs(w)
    plan, ws, out = run_gpu(w, q, k, v, rank_scope=rank_scope, partition=1)
    ref = oracle_all(w, q, k, v, rank_scope=rank_scope, balanced=True)
    assert plan.info.R == ref["pl"].R < oracle.plan(w.T, w.Hg, w.Wg).R or name == "batch2"
    bad = _check_prepare(w, plan, ws, ref)
    sel = [(h, a) for h in range(w.B * w.H) for a in range(plan.info.R)]
    _check_attention(w, out, ref, sel, bad)
    assert torch.isfinite(out.float()).all()


@pytest.mark.parametrize("name", ["wan1p3b_480p", "wan14b_720p"])
def test_balanced_partition_sampled_parity(name):
    """Full-size configurations on the balanced partition: 25 instead of 28 blocks per 30 x 52 frame, 57 instead of 60
    per 45 x 80 frame."""
    _sampled_parity(name, nheads=2, nblocks=16, partition=1)


def test_hunyuan_720p_sampled_parity():
    _sampled_parity("hunyuan_720p", nheads=2, nblocks=16)


def test_wan14b_720p_sampled_parity():
    """The benchmark's workload (20 % 8-bit + 40 % 4-bit, K outlier channels) in the benchmark's launch configuration."""
    _sampled_parity("wan14b_720p", nheads=2, nblocks=16)


def test_wan14b_720p_bf16_8bit_variant_sampled_parity():
    _sampled_parity("wan14b_720p_hi", nheads=2, nblocks=16)


@pytest.mark.parametrize("grid,high,low", [(2, 0.10, 0.40), (1, 0.0, 0.40), (3, 0.20, 0.0), (0, 0.05, 0.60)])
def test_sweep_point_sampled_parity(grid, high, low):
    """Points of the budget sweep (24 heads, d = 128): a mixed point, a point without the 8-bit tier, a point
    without the 4-bit tier, and the smallest grid at the largest 4-bit share."""
    w = da2_inputs.sweep_workload(grid, high, low)
    da2_inputs.WORKLOADS[w.name] = w
    _sampled_parity(w.name, nheads=2, nblocks=12)


@pytest.mark.parametrize("name", ["sweep_131k_all8", "sweep_131k_allbf16"])
def test_sweep_dense_endpoints_sampled_parity(name):
    """The two zero-sparsity endpoints of the sweep at the largest grid (131,072 tokens): every key block retained in
    the 8-bit tier, and every key block retained in bf16 (which the oracle's pins tie to dense attention)."""
    _sampled_parity(name, nheads=2, nblocks=8)


def test_caller_fixed_nvfp4_scales():
    """g_q, g_k, g_v supplied by the caller (App. C.3: a given positive per-tensor scale): the workspace holds exactly
    those scales, codes and group scales are the oracle's for the same g, and so is the attention output.  One of
    the scales is deliberately too small, so that the largest groups saturate at the top scale code."""
    w = SMALL["ragged3"]
    BH = w.B * w.H
    g_fixed = ([0.004, 0.0035], [0.0011, 0.005], [0.003, 0.0042])
    assert all(len(g) == BH for g in g_fixed)
    q, k, v = _inputs(w)
    plan, ws, out = run_gpu(w, q, k, v, g_fixed=g_fixed)
    ref = oracle_all(w, q, k, v)
    bad = _check_prepare(w, plan, ws, ref, g_fixed=g_fixed)
    sel = [(h, a) for h in range(BH) for a in range(plan.info.R)]
    _check_attention(w, out, ref, sel, bad, g_fixed=g_fixed)


def test_quantiser_codes_on_a_lattice_of_bf16_patterns():
    """The quantisers get their quotients from a hoisted reciprocal and two fused multiply-adds instead of a division
    per element; the codes must still be the oracle's (which divides) bit for bit.  Inputs here are not smooth fields
    but bf16 bit patterns drawn over 19 binades with every mantissa, both signs and signed zeros, under caller-fixed
    NVFP4 scales with awkward significands, so that quotients land on and next to rounding boundaries of every
    format."""
    w = SMALL["ragged3"]
    BH = w.B * w.H
    gen = torch.Generator().manual_seed(2024)
    def lattice():
        shape = (w.B, w.H, w.N, w.head_dim)
        sign = torch.randint(0, 2, shape, generator=gen, dtype=torch.int32) << 15
        expo = (torch.randint(127 - 12, 127 + 7, shape, generator=gen, dtype=torch.int32)) << 7
        mant = torch.randint(0, 128, shape, generator=gen, dtype=torch.int32)
        bits = sign | expo | mant
        zero = torch.rand(shape, generator=gen) < 0.02
        bits = torch.where(zero, sign, bits)  # +0 and -0
        return bits.to(torch.int16).view(torch.bfloat16).cuda()
    q, k, v = lattice(), lattice(), lattice()
    g_fixed = ([0.0123456, 0.0301], [0.0271828, 0.0099999], [0.0314159, 0.0200001])
    assert all(len(g) == BH for g in g_fixed)
    plan, ws, out = run_gpu(w, q, k, v, g_fixed=g_fixed)
    ref = oracle_all(w, q, k, v)
    _check_prepare(w, plan, ws, ref, g_fixed=g_fixed)


@pytest.mark.parametrize("mode,n_divisors", [(0, 1 << 16), (1, 1 << 12), (2, 1)])
def test_quantiser_arithmetic_selfcheck(mode, n_divisors):
    """The device functions behind the quantisers' quotients (hoisted reciprocal + two fused multiply-adds) and the
    INT8 rounding (one add and a truncation) against the IEEE division and roundf: every bf16 numerator of magnitude
    at least 2^-100 against 65,536 pseudo-random divisors and 4,096 divisors with significands of all ones, and every
    float below 2^23 through the rounding.  No mismatch is allowed."""
    bad = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    da2.da2_selfcheck_quantiser_arithmetic(mode, n_divisors, 20260101, bad)
    torch.cuda.synchronize()
    assert int(bad.item()) == 0


def test_refresh_operands_keeps_the_selection():
    """da2_refresh_operands: new operands under the lists of an earlier call (the selection is reused)."""
    w1 = SMALL["ragged64"]
    w2 = W("ragged64b", w1.B, w1.H, w1.head_dim, w1.T, w1.Hg, w1.Wg, w1.frac16, w1.frac8, w1.frac4, seed=112)
    q1, k1, v1 = _inputs(w1)
    q2, k2, v2 = _inputs(w2)
    plan, ws, _ = run_gpu(w1, q1, k1, v1, zero_ws=True)
    ref1 = oracle_all(w1, q1, k1, v1)
    bad = _check_prepare(w1, plan, ws, ref1)
    I = plan.info
    keep = [(I.off_map, I.off_counts - I.off_map), (I.off_counts, I.off_ids - I.off_counts),
            (I.off_ids, I.B * I.H * I.ids_per_head * 2)]
    before = [ws[o:o + n].clone() for o, n in keep]
    out = torch.full_like(q2, float("nan"))
    da2.da2_refresh_operands(plan, q2, k2, v2, ws)
    da2.da2_attention_fwd(plan, q2, k2, v2, ws, out)
    torch.cuda.synchronize()
    assert da2.da2_device_status(plan, ws) == 0
    for (o, n), b in zip(keep, before):
        assert torch.equal(ws[o:o + n], b), "the draft map, counts and ids must not change"
    # operands, scales and descriptors are those of the new inputs: the oracle's, bit for bit
    ref2 = oracle_all(w2, q2, k2, v2)
    mixed = dict(ref2)
    mixed.update(A=ref1["A"], ids=ref1["ids"], counts=ref1["counts"], tags=ref1["tags"])
    assert _check_prepare(w2, plan, ws, mixed) == bad
    sel = [(h, a) for h in range(w1.B * w1.H) for a in range(I.R)]
    _check_attention(w2, out, mixed, sel, bad)
    assert torch.isfinite(out.float()).all()


@pytest.mark.parametrize("reselect", [True, False])
def test_prepare_cached_scales_is_one_pass_with_carried_over_scales(reselect):
    """da2_prepare_cached_scales: descriptors and every operand record of NEW inputs in one pass, quantised with the
    NVFP4 per-tensor and E4M3 per-channel scales an earlier da2_prepare left in the workspace (Sec. 3.3, fused
    gathering + pooling + quantisation).  The new Q and K (and four channels of V) are 1.6 times larger, so values
    beyond the carried-over range occur and must saturate as the casts define.  Everything is compared with the oracle fed the same
    scales; the scales in the workspace must not change."""
    w1 = SMALL["ragged3"]
    w2 = W("ragged3b", w1.B, w1.H, w1.head_dim, w1.T, w1.Hg, w1.Wg, w1.frac16, w1.frac8, w1.frac4, seed=211)
    q1, k1, v1 = _inputs(w1)
    q2, k2, v2 = _inputs(w2)
    q2, k2 = ((x.float() * 1.6).to(torch.bfloat16) for x in (q2, k2))
    gain = torch.ones(w1.head_dim, device="cuda")
    gain[[5, 40, 77, 100]] = 1.6          # a few value channels leave the carried-over range as well
    v2 = (v2.float() * gain).to(torch.bfloat16)
    plan, ws, _ = run_gpu(w1, q1, k1, v1, zero_ws=True)
    ref1 = oracle_all(w1, q1, k1, v1)
    bad1 = _check_prepare(w1, plan, ws, ref1)
    V1 = Workspace(plan, ws)
    g1, dv1 = V1.gscale().copy(), V1.dv8().copy()
    g_fixed = (g1[:, 0], g1[:, 1], g1[:, 2])
    out = torch.full_like(q2, float("nan"))
    da2.da2_prepare_cached_scales(plan, q2, k2, v2, ws, reselect=reselect)
    assert da2.da2_last_launch_count(plan) == (3 if reselect else 1)   # one pass over Q, K, V (+ draft map, ranking)
    da2.da2_attention_fwd(plan, q2, k2, v2, ws, out)
    torch.cuda.synchronize()
    assert da2.da2_device_status(plan, ws) == 0
    ref2 = oracle_all(w2, q2, k2, v2)
    if not reselect:   # the earlier call's selection stays
        ref2.update(A=ref1["A"], ids=ref1["ids"], counts=ref1["counts"], tags=ref1["tags"])
    bad = _check_prepare(w2, plan, ws, ref2, g_fixed=g_fixed, dv_fixed=dv1)
    if not reselect:
        assert bad == bad1
    sel = [(h, a) for h in range(w1.B * w1.H) for a in range(plan.info.R)]
    _check_attention(w2, out, ref2, sel, bad, g_fixed=g_fixed, dv_fixed=dv1)
    assert torch.isfinite(out.float()).all()


def test_prepare_and_attention_replay_from_a_cuda_graph():
    """The two calls only enqueue kernels and a memset on the caller's stream (no allocation, no synchronisation), so
    a captured graph of them replays to the same bits as the eager calls."""
    w = SMALL["ragged64"]
    q, k, v = _inputs(w)
    plan, ws, out = run_gpu(w, q, k, v, zero_ws=True)
    ws2 = torch.zeros_like(ws)
    out2 = torch.full_like(out, float("nan"))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):                      # warm-up on the capture stream (function attributes, modules)
        da2.da2_prepare(plan, q, k, v, ws2)
        da2.da2_attention_fwd(plan, q, k, v, ws2, out2)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        da2.da2_prepare(plan, q, k, v, ws2)
        da2.da2_attention_fwd(plan, q, k, v, ws2, out2)
    for _ in range(2):
        out2.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert da2.da2_device_status(plan, ws2) == 0
        assert torch.equal(out2.view(torch.int16), out.view(torch.int16))


def test_graph_replay_with_caller_fixed_scales():
    """With caller-fixed NVFP4 scales da2_prepare hands them over as kernel arguments (no copy from pageable host
    memory), so the call can still be captured; the replay gives the bits of the eager call."""
    w = SMALL["ragged3"]
    g_fixed = ([0.004, 0.0035], [0.0011, 0.005], [0.003, 0.0042])
    q, k, v = _inputs(w)
    plan, ws, out = run_gpu(w, q, k, v, zero_ws=True, g_fixed=g_fixed)
    ws2 = torch.zeros_like(ws)
    out2 = torch.full_like(out, float("nan"))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        da2.da2_prepare(plan, q, k, v, ws2)
        da2.da2_attention_fwd(plan, q, k, v, ws2, out2)
    graph.replay()
    torch.cuda.synchronize()
    assert da2.da2_device_status(plan, ws2) == 0
    assert torch.equal(out2.view(torch.int16), out.view(torch.int16))
    assert torch.equal(ws2, ws)


def test_host_pipeline_equals_the_direct_call():
    """HostPipeline (head groups through three streams, host tensors in and out) gives the bits of one direct call."""
    w = W("pipe", 1, 5, 64, 2, 16, 24, 0.1, 0.2, 0.3, seed=31)
    q, k, v = _inputs(w)
    plan, ws, out = run_gpu(w, q, k, v)
    hq, hk, hv = (x.cpu().pin_memory() for x in (q, k, v))
    for groups in (1, 2, 3, 5, "ramp"):   # 3 groups of 5 heads: sizes 2, 2, 1 (two plans)
        hout = torch.full_like(hq, float("nan")).pin_memory()
        pipe = da2.HostPipeline(w.B, w.H, w.T, w.Hg, w.Wg, w.head_dim, w.frac16, w.frac8, w.frac4, lam=w.lam,
                                groups=groups)
        for _ in range(2):
            pipe.run(hq, hk, hv, hout)
        torch.cuda.synchronize()
        assert pipe.status() == 0
        assert torch.equal(hout.view(torch.int16), out.cpu().view(torch.int16)), groups


def test_c_abi_host_entry_equals_the_direct_call():
    """da2_attention_host (the C ABI's own pipelined host-buffer path) gives the bits of one direct call, for the
    default group ramp and for fixed group counts, also with a prefix and the balanced partition."""
    for kw in (dict(), dict(n_prefix=70, partition=1)):
        w = W("hostc", 1, 5, 64, 2, 16, 24, 0.1, 0.2, 0.3, seed=33)
        P = kw.get("n_prefix", 0)
        q, k, v = _inputs(w)
        if P:
            g = torch.Generator(device="cpu").manual_seed(7)
            q, k, v = (torch.cat([torch.randn(w.B, w.H, P, w.head_dim, generator=g).to(torch.bfloat16).cuda(), x], 2)
                       .contiguous() for x in (q, k, v))
        plan = da2.da2_plan(w.B, w.H, w.T, w.Hg, w.Wg, w.head_dim, w.frac16, w.frac8, w.frac4, lam=w.lam, **kw)
        ws = torch.empty(int(plan.info.workspace_bytes), dtype=torch.uint8, device="cuda")
        out = torch.full_like(q, float("nan"))
        da2.da2_prepare(plan, q, k, v, ws)
        da2.da2_attention_fwd(plan, q, k, v, ws, out)
        torch.cuda.synchronize()
        hq, hk, hv = (x.cpu().pin_memory() for x in (q, k, v))
        cfg = da2.make_config(w.B, w.H, w.T, w.Hg, w.Wg, w.head_dim, w.frac16, w.frac8, w.frac4, lam=w.lam, **kw)
        for groups in (0, 1, 3):
            arena = torch.empty(da2.da2_attention_host_arena_bytes(cfg, groups), dtype=torch.uint8, device="cuda")
            hout = torch.full_like(hq, float("nan")).pin_memory()
            da2.da2_attention_host(cfg, hq, hk, hv, hout, arena, groups)
            assert torch.equal(hout.view(torch.int16), out.cpu().view(torch.int16)), (kw, groups)
        small = torch.empty(1024, dtype=torch.uint8, device="cuda")
        with pytest.raises(da2.Da2Error) as e:
            da2.da2_attention_host(cfg, hq, hk, hv, hout, small, 0)
        assert e.value.code == 3


def test_scheduling_order_sorts_rows_by_list_length(rank_scope=1):
    """The order region pairs query blocks of equal list length: a permutation of the blocks of each head, by
    decreasing length, lower index first among equals, padded with 0xFFFF when R is odd."""
    w = SMALL["ragged3"]
    q, k, v = _inputs(w)
    plan, ws, _ = run_gpu(w, q, k, v, rank_scope=rank_scope)
    I = plan.info
    BH, R = I.B * I.H, I.R
    Rp = 2 * ((R + 1) // 2)
    order = ws[I.off_order:I.off_order + BH * Rp * 2].cpu().numpy().view(np.uint16).reshape(BH, Rp)
    counts = ws[I.off_counts:I.off_counts + BH * R * 16].cpu().numpy().view(np.int32).reshape(BH, R, 4)
    L = counts[:, :, :3].sum(-1)
    for h in range(BH):
        expect = sorted(range(R), key=lambda a: (-int(L[h, a]), a))
        assert order[h, :R].tolist() == expect
        if Rp > R:
            assert order[h, R] == 0xFFFF
