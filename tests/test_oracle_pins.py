"""Pins for the CPU oracle: every oracle function is checked against something other
than itself -- closed forms, library routines, brute force on tiny inputs, invariants
and bounds that the paper or the mathematics fix.  No GPU involved."""
import itertools
import math

import numpy as np
import pytest
import torch

import oracle


def rand_bf16(rng, shape, scale=1.0):
    x = torch.from_numpy((rng.standard_normal(shape) * scale).astype(np.float32)).to(torch.bfloat16)
    return x


def bits(t):
    return oracle.bf16_bits(t)


def f64(t):
    return t.to(torch.float64).numpy()


# ------------------------------------------------------------------ plan
@pytest.mark.parametrize("grid", [(4, 16, 16), (2, 30, 52), (1, 45, 80), (3, 5, 9), (1, 8, 8)])
def test_plan_partition_and_counts(grid):
    T, Hg, Wg = grid
    pl = oracle.plan(T, Hg, Wg)
    nty, ntx = -(-Hg // 8), -(-Wg // 8)
    assert pl.R == T * nty * ntx
    assert int(pl.n_valid.sum()) == T * Hg * Wg
    toks = pl.slot_token[pl.slot_token >= 0]
    assert np.array_equal(np.sort(toks), np.arange(T * Hg * Wg))  # slot map is a bijection onto tokens
    assert (pl.n_valid >= 1).all()
    # inverse map o slot map = identity, and the slot really is the (ly, lx) position inside tile (ty, tx)
    for a in range(pl.R):
        for j in range(64):
            tok = pl.slot_token[a, j]
            if tok < 0:
                continue
            t, rem = divmod(int(tok), Hg * Wg)
            y, x = divmod(rem, Wg)
            assert a == (t * nty + y // 8) * ntx + x // 8 and j == (y % 8) * 8 + (x % 8)


@pytest.mark.parametrize("grid", [(1, 30, 52), (1, 45, 80), (1, 16, 16)])
def test_plan_perimeter_identity(grid):
    """App. C.2 Eq. 'region-perimeter': sum of region perimeters = 2(H+W) + 2 E_cut, by brute-force edge count."""
    T, Hg, Wg = grid
    pl = oracle.plan(T, Hg, Wg)
    region = np.full((Hg, Wg), -1)
    for a in range(pl.R):
        for j in range(64):
            tok = pl.slot_token[a, j]
            if tok >= 0:
                region[tok // Wg, tok % Wg] = a
    per = 0
    cut = 0
    for y in range(Hg):
        for x in range(Wg):
            for dy, dx in ((0, 1), (1, 0), (0, -1), (-1, 0)):
                yy, xx = y + dy, x + dx
                if not (0 <= yy < Hg and 0 <= xx < Wg):
                    per += 1
                elif region[yy, xx] != region[y, x]:
                    per += 1
                    cut += 1
    cut //= 2
    assert per == 2 * (Hg + Wg) + 2 * cut


def _frame_regions(pl, Hg, Wg):
    """Region id of every cell of frame 0, from the slot table."""
    Rf = pl.R // pl.T
    region = np.full(Hg * Wg, -1)
    for a in range(Rf):
        toks = pl.slot_token[a][pl.slot_token[a] >= 0]
        assert (region[toks] == -1).all()
        region[toks] = a
    assert (region >= 0).all()
    return region.reshape(Hg, Wg), Rf


def _perimeter_by_edges(region):
    """Sum over regions of their unit boundary edges, counted cell by cell."""
    H, W = region.shape
    per = 0
    cut = 0
    for y in range(H):
        for x in range(W):
            for dy, dx in ((0, 1), (1, 0), (0, -1), (-1, 0)):
                yy, xx = y + dy, x + dx
                if not (0 <= yy < H and 0 <= xx < W):
                    per += 1
                elif region[yy, xx] != region[y, x]:
                    per += 1
                    cut += 1
    return per, cut // 2


@pytest.mark.parametrize("grid", [(2, 30, 52), (1, 45, 80), (3, 12, 20), (1, 9, 13), (1, 32, 32), (1, 7, 5)])
@pytest.mark.parametrize("C", [64, 128])
def test_balanced_partition_invariants(grid, C):
    """App. C.2: R_f = ceil(HW / C) regions per frame, less than one block of padding per frame
    (Eq. 'ragged-padding'), balanced sizes, every region connected (scipy's component labelling), the slot table a
    bijection that repeats frame by frame, and Eq. 'region-perimeter' by brute-force edge count."""
    from scipy import ndimage
    T, Hg, Wg = grid
    pl = oracle.plan_balanced(T, Hg, Wg, C)
    HW = Hg * Wg
    Rf = -(-HW // C)
    assert pl.R == T * Rf and pl.S == C
    assert 0 <= Rf * C - HW < C
    assert int(pl.n_valid.sum()) == T * HW and pl.n_valid.max() - pl.n_valid.min() <= 1 and pl.n_valid.max() <= C
    toks = pl.slot_token[pl.slot_token >= 0]
    assert np.array_equal(np.sort(toks), np.arange(T * HW))
    for a in range(pl.R):   # valid slots come first, padding after them
        assert (pl.slot_token[a, :pl.n_valid[a]] >= 0).all() and (pl.slot_token[a, pl.n_valid[a]:] == -1).all()
    for t in range(1, T):   # the same partition in every frame
        assert np.array_equal(pl.slot_token[t * Rf:(t + 1) * Rf][pl.slot_token[:Rf] >= 0],
                              pl.slot_token[:Rf][pl.slot_token[:Rf] >= 0] + t * HW)
    region, _ = _frame_regions(pl, Hg, Wg)
    for a in range(Rf):
        _, ncomp = ndimage.label(region == a)
        assert ncomp == 1, f"region {a} is not connected"
    per, cut = _perimeter_by_edges(region)
    assert per == 2 * (Hg + Wg) + 2 * cut
    assert pl.choice[2] == per
    # the winner is no worse than the always-admissible candidate of single-row bands, written out here
    strips = np.empty(HW, int)
    order = [y * Wg + (x if y % 2 == 0 else Wg - 1 - x) for y in range(Hg) for x in range(Wg)]
    n, rem = divmod(HW, Rf)
    pos = 0
    for a in range(Rf):
        for _ in range(n + (a < rem)):
            strips[order[pos]] = a
            pos += 1
    assert per <= _perimeter_by_edges(strips.reshape(Hg, Wg))[0]


def test_balanced_partition_against_fixed_tiles_and_exhaustive_search():
    """(i) Where 8 x 8 tiles divide the frame, the balanced partition of capacity 64 IS the tile partition.
    (ii) On the 720p latent frame it needs 57 blocks instead of 60 and its perimeter does not exceed the tiles'.
    (iii) On tiny frames an exhaustive search over ALL partitions into connected regions of the balanced sizes finds
    no smaller perimeter than the chosen candidate's."""
    for Hg, Wg in ((16, 16), (32, 48)):
        a, _ = _frame_regions(oracle.plan_balanced(1, Hg, Wg, 64), Hg, Wg)
        b, _ = _frame_regions(oracle.plan(1, Hg, Wg), Hg, Wg)
        # same partition up to the numbering of the regions
        pairs = set(zip(a.ravel().tolist(), b.ravel().tolist()))
        assert len(pairs) == a.max() + 1 == b.max() + 1
    bal, fix = oracle.plan_balanced(1, 45, 80, 64), oracle.plan(1, 45, 80)
    assert (bal.R, fix.R) == (57, 60)
    assert bal.choice[2] <= _perimeter_by_edges(_frame_regions(fix, 45, 80)[0])[0]

    def best_perimeter(H, W, sizes):
        best = [None]
        grid = [-1] * (H * W)

        def neighbours(c):
            y, x = divmod(c, W)
            return [cc for cc, ok in (((y - 1) * W + x, y > 0), ((y + 1) * W + x, y < H - 1),
                                      (y * W + x - 1, x > 0), (y * W + x + 1, x < W - 1)) if ok]

        def grow(a, cells, frontier_min):
            if len(cells) == sizes[a]:
                place(a + 1)
                return
            cand = sorted({n for c in cells for n in neighbours(c) if grid[n] == -1 and n > frontier_min})
            for n in cand:       # canonical growth: only cells above the region's first cell, each set once
                grid[n] = a
                grow(a, cells + [n], frontier_min)
                grid[n] = -1
            return

        seen = set()

        def place(a):
            if a == len(sizes):
                key = tuple(grid)
                if key in seen:
                    return
                seen.add(key)
                per = _perimeter_by_edges(np.array(grid).reshape(H, W))[0]
                best[0] = per if best[0] is None else min(best[0], per)
                return
            first = grid.index(-1)      # the region that owns the first free cell is placed next
            grid[first] = a
            grow(a, [first], first)
            grid[first] = -1

        place(0)
        return best[0]

    for (H, W, C) in ((4, 4, 4), (2, 6, 4), (3, 4, 4), (3, 3, 3)):
        pl = oracle.plan_balanced(1, H, W, C)
        sizes = sorted(pl.n_valid.tolist(), reverse=True)
        # the exhaustive search lets any region take any of the balanced sizes: try every ordering of sizes
        cands = {best_perimeter(H, W, list(p)) for p in set(itertools.permutations(sizes))}
        assert pl.choice[2] == min(c for c in cands if c is not None), (H, W, C)


def test_quotas_match_budget_tables():
    # exact retained-block counts per query-block row for the named workloads
    assert oracle.quotas(0.0, 0.25, 0.25, 16) == (0, 4, 4)
    assert oracle.quotas(0.0, 0.10, 0.30, 588) == (0, 59, 176)
    assert oracle.quotas(0.0, 0.05, 0.20, 1980) == (0, 99, 396)
    assert oracle.quotas(0.0, 0.20, 0.40, 1260) == (0, 252, 504)
    assert oracle.quotas(0.20, 0.40, 0.0, 1260) == (252, 504, 0)
    for M in (7, 16, 588, 1260 * 1260):
        for f in ((0.1, 0.2, 0.3), (0.0, 0.0, 1.0), (0.33, 0.33, 0.34), (0, 0, 0)):
            k = oracle.quotas(*f, M)
            assert min(k) >= 0 and sum(k) == math.floor(sum(f) * M + 0.5) and sum(k) <= M


# ------------------------------------------------------------ descriptors
def test_avg_pool_is_mean_pair_logit():
    """Remark 3.2: Qavg_a . Kavg_b / sqrt(d) equals the mean token-pair logit between the regions."""
    rng = np.random.default_rng(1)
    T, Hg, Wg, d = 1, 11, 13, 16
    pl = oracle.plan(T, Hg, Wg)
    q, k = rand_bf16(rng, (1, pl.N, d)), rand_bf16(rng, (1, pl.N, d))
    qavg, qmax = oracle.pool(bits(q), pl)
    kavg, kmax = oracle.pool(bits(k), pl)
    Q, K = f64(q)[0], f64(k)[0]
    for a in range(pl.R):
        ta = pl.slot_token[a][pl.slot_token[a] >= 0]
        assert np.array_equal(qmax[0, a], Q[ta].max(axis=0).astype(np.float32))
        assert (qmax[0, a] >= qavg[0, a]).all()
        for b in range(pl.R):
            tb = pl.slot_token[b][pl.slot_token[b] >= 0]
            mean_logit = (Q[ta] @ K[tb].T).mean() / math.sqrt(d)
            got = float(qavg[0, a].astype(np.float64) @ kavg[0, b].astype(np.float64)) / math.sqrt(d)
            assert abs(got - mean_logit) < 1e-5  # descriptors are stored in fp32


def test_constant_field_descriptors_and_uniform_map():
    T, Hg, Wg, d = 2, 12, 9, 8
    pl = oracle.plan(T, Hg, Wg)
    q = torch.full((1, pl.N, d), 0.75, dtype=torch.bfloat16)
    k = rand_bf16(np.random.default_rng(2), (1, pl.N, d))
    qavg, qmax = oracle.pool(bits(q), pl)
    assert np.array_equal(qavg, qmax) and (qavg == 0.75).all()
    # constant K too -> every logit equal -> A == 1/R -> ties everywhere -> lowest indices win (App. C.1)
    kc = torch.full((1, pl.N, d), -0.5, dtype=torch.bfloat16)
    r = oracle.run_pipeline(bits(q), bits(kc), bits(kc), pl, lam=0.2, scale=1.0, frac16=0.25, frac8=0.25, frac4=0.25)
    assert np.allclose(r["A"], 1.0 / pl.R, rtol=1e-6)
    k16, k8, k4 = r["quotas"]
    for a in range(pl.R):
        assert list(r["ids"][0, a, :k4]) == list(range(k16 + k8, k16 + k8 + k4))
        assert list(r["ids"][0, a, k4:k4 + k8]) == list(range(k16, k16 + k8))
        assert list(r["ids"][0, a, k4 + k8:k4 + k8 + k16]) == list(range(k16))
    del k


def test_draft_map_rows_and_lambda_endpoints():
    rng = np.random.default_rng(3)
    pl = oracle.plan(2, 16, 16)
    d = 32
    q, k = rand_bf16(rng, (2, pl.N, d)), rand_bf16(rng, (2, pl.N, d))
    qavg, qmax = oracle.pool(bits(q), pl)
    kavg, kmax = oracle.pool(bits(k), pl)
    s = 1 / math.sqrt(d)
    for lam in (0.0, 0.2, 1.0):
        A = oracle.draft(qavg, qmax, kavg, kmax, lam, s)
        assert np.allclose(A.sum(-1), 1.0, atol=1e-6)
        p1 = torch.softmax(torch.from_numpy(qavg.astype(np.float64)) @ torch.from_numpy(kavg.astype(np.float64)).transpose(1, 2) * s, -1)
        p2 = torch.softmax(torch.from_numpy(qmax.astype(np.float64)) @ torch.from_numpy(kmax.astype(np.float64)).transpose(1, 2) * s, -1)
        ref = ((1 - lam) * p1 + lam * p2).numpy()
        assert np.allclose(A, ref, rtol=1e-6, atol=1e-9)
    # lambda = 0 recovers average-only guidance (Remark 3.2)
    A0 = oracle.draft(qavg, qmax, kavg, kmax, 0.0, s)
    A0b = oracle.draft(qavg, qavg * 0 + 7, kavg, kmax * 3, 0.0, s)
    assert np.array_equal(A0, A0b)


# ---------------------------------------------------------------- ranking
def test_rank_row_equals_library_stable_sort():
    rng = np.random.default_rng(4)
    BH, R = 3, 37
    A = rng.random((BH, R, R)).astype(np.float32)
    A[:, :, 5] = A[:, :, 11]  # exact ties
    A[1, 3, :] = 0.25
    k16, k8, k4 = 3, 7, 11
    tags = oracle.rank_row(A, k16, k8, k4)
    for bh in range(BH):
        for a in range(R):
            order = np.argsort(-A[bh, a], kind="stable")
            exp = np.zeros(R, np.uint8)
            exp[order[:k16]] = 16
            exp[order[k16:k16 + k8]] = 8
            exp[order[k16 + k8:k16 + k8 + k4]] = 4
            assert np.array_equal(tags[bh, a], exp)
            assert (tags[bh, a] == 16).sum() == k16 and (tags[bh, a] == 8).sum() == k8 and (tags[bh, a] == 4).sum() == k4
    ids, counts = oracle.lists(tags)
    assert (counts == np.array([k4, k8, k16])).all()
    for seg, (lo, hi) in zip((4, 8, 16), ((0, k4), (k4, k4 + k8), (k4 + k8, k4 + k8 + k16))):
        got = ids[2, 5, lo:hi]
        assert np.array_equal(got, np.nonzero(tags[2, 5] == seg)[0])  # ascending ids inside a segment
    assert (ids[:, :, k4 + k8 + k16:] == -1).all()


def test_rank_head_equals_library_stable_sort_and_allows_empty_rows():
    rng = np.random.default_rng(5)
    BH, R = 2, 19
    A = rng.random((BH, R, R)).astype(np.float32)
    A[0, 4, :] = 0.0  # a row that loses every pair under a head-level budget
    A[1, :, 3] = A[1, :, 9]
    T16, T8, T4 = oracle.quotas(0.05, 0.1, 0.2, R * R)
    tags = oracle.rank_head(A, T16, T8, T4)
    for bh in range(BH):
        order = np.argsort(-A[bh].reshape(-1), kind="stable")
        exp = np.zeros(R * R, np.uint8)
        exp[order[:T16]] = 16
        exp[order[T16:T16 + T8]] = 8
        exp[order[T16 + T8:T16 + T8 + T4]] = 4
        assert np.array_equal(tags[bh].reshape(-1), exp)
        s = A[bh].reshape(-1)
        t = tags[bh].reshape(-1)
        assert s[t == 16].min() >= s[t == 8].max() >= s[t == 8].min() >= s[t == 4].max() >= s[t == 4].min() >= s[t == 0].max()
    assert (tags[0, 4] == 0).all()
    _, counts = oracle.lists(tags)
    assert counts[0].sum() == T16 + T8 + T4 and counts[0, 4].sum() == 0


def test_rank_order_minimises_weighted_error_bound():
    """Theorem 3.6 by enumeration: with eps16=0 <= eps8 <= eps4, giving 16 bits to the largest masses,
    8 bits to the next and 4 bits to the rest minimises sum W*eps -- which is the order Algorithm 1 applies."""
    rng = np.random.default_rng(6)
    W = rng.random(7).astype(np.float32)
    eps = {16: 0.0, 8: 0.3, 4: 1.1}
    tags = oracle.rank_row(np.ascontiguousarray(np.tile(W, (1, 7, 1))), 2, 2, 3)[0, 0]
    cost = sum(float(W[i]) * eps[int(tags[i])] for i in range(7))
    best = min(sum(float(W[i]) * eps[p] for i, p in enumerate(perm))
               for perm in set(itertools.permutations([16, 16, 8, 8, 4, 4, 4])))
    assert cost <= best + 1e-12


# ----------------------------------------------------------- small formats
E2M1_VALUES = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]  # 1 sign, 2 exponent, 1 mantissa bit


def test_e2m1_exhaustive():
    for c in range(16):
        v = oracle.decode_e2m1(c)
        assert abs(v) == E2M1_VALUES[c & 7] and (v < 0 or math.copysign(1, v) < 0) == bool(c & 8)
        assert oracle.cast_e2m1(v) == c
    for i in range(7):
        mid = (E2M1_VALUES[i] + E2M1_VALUES[i + 1]) / 2
        even = i if i % 2 == 0 else i + 1
        assert oracle.cast_e2m1(mid) == even and oracle.cast_e2m1(-mid) == (even | 8)
        assert oracle.cast_e2m1(np.nextafter(np.float32(mid), np.float32(100))) == i + 1
        assert oracle.cast_e2m1(np.nextafter(np.float32(mid), np.float32(-100))) == i
    assert oracle.cast_e2m1(6.0) == 7 and oracle.cast_e2m1(1e9) == 7 and oracle.cast_e2m1(-7.0) == 15
    # brute force nearest on a dense sweep
    for x in np.linspace(-7, 7, 2801):
        c = oracle.cast_e2m1(float(np.float32(x)))
        dists = [abs(abs(float(np.float32(x))) - v) for v in E2M1_VALUES]
        assert dists[c & 7] == min(dists)


def test_e4m3_exhaustive_against_format_definition_and_torch():
    vals = []
    for c in range(256):
        if (c & 0x7f) == 0x7f:
            continue
        e, m = (c >> 3) & 0xf, c & 7
        mag = m * 2.0 ** -9 if e == 0 else (1 + m / 8) * 2.0 ** (e - 7)
        v = oracle.decode_e4m3(c)
        assert abs(v) == mag
        assert oracle.cast_e4m3(v) == c or (mag == 0 and oracle.cast_e4m3(v) in (0, 0x80))
        if not (c & 0x80):
            vals.append(mag)
    assert max(vals) == 448.0 and vals[1] == 2.0 ** -9
    for i in range(len(vals) - 1):
        mid = (vals[i] + vals[i + 1]) / 2
        even = i if i % 2 == 0 else i + 1
        assert oracle.cast_e4m3(mid) == even
        assert oracle.cast_e4m3(float(np.nextafter(np.float32(mid), np.float32(1e9)))) == i + 1
        assert oracle.cast_e4m3(float(np.nextafter(np.float32(mid), np.float32(-1)))) == i
    assert oracle.cast_e4m3(448.0) == 0x7e and oracle.cast_e4m3(470.0) == 0x7e and oracle.cast_e4m3(1e30) == 0x7e
    assert oracle.cast_e4m3(-1e30) == 0xfe
    # library routine: torch's float8_e4m3fn conversion (round to nearest even) inside the finite range
    rng = np.random.default_rng(7)
    xs = np.concatenate([rng.standard_normal(20000) * 30, rng.standard_normal(20000) * 0.01, rng.uniform(-448, 448, 20000)])
    xs = xs.astype(np.float32)
    xs = xs[np.abs(xs) <= 448]
    ref = torch.from_numpy(xs).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([oracle.cast_e4m3(float(x)) for x in xs], np.uint8)
    assert np.array_equal(got, ref)


# --------------------------------------------------------------- quantisers
def test_int8_quantiser_bounds_and_ties_away_from_zero():
    rng = np.random.default_rng(8)
    pl = oracle.plan(1, 12, 10)
    d = 32
    x = rand_bf16(rng, (2, pl.N, d), 3.0)
    codes, delta = oracle.quant_int8(bits(x), pl)
    X = f64(x)
    assert codes.min() >= -127 and codes.max() <= 127
    for bh in range(2):
        for a in range(pl.R):
            tok = pl.slot_token[a]
            valid = tok >= 0
            blk = X[bh, tok[valid]]
            dl = float(delta[bh, a])
            assert dl == np.float32(np.float32(np.abs(blk).max().astype(np.float32) / np.float32(127)) + np.float32(1e-7))
            rec = dl * codes[bh, a][valid].astype(np.float64)
            assert np.abs(rec - blk).max() <= dl / 2 * (1 + 1e-6)                       # scalar bound
            assert np.linalg.norm(rec - blk, axis=1).max() <= math.sqrt(d) * dl / 2 * (1 + 1e-6)  # vector bound
            assert (codes[bh, a][~valid] == 0).all()
            assert np.abs(codes[bh, a]).max() == 127  # the block maximum maps to full scale
    # amax = 254 -> delta = fl32(2 + 1e-7) = 2 exactly, so x/delta hits exact .5 ties
    pl1 = oracle.plan(1, 8, 8)
    y = torch.zeros(1, 64, 16, dtype=torch.bfloat16)
    y[0, 0, 0] = 254.0
    y[0, 1, :6] = torch.tensor([1.0, -1.0, 3.0, -3.0, 5.0, 7.0], dtype=torch.bfloat16)
    c, dl = oracle.quant_int8(bits(y), pl1)
    assert float(dl[0, 0]) == 2.0 and c[0, 0, 0, 0] == 127
    assert list(c[0, 0, 1, :6]) == [1, -1, 2, -2, 3, 4]  # 0.5->1, -0.5->-1, 1.5->2, -1.5->-2, 2.5->3, 3.5->4


def test_v_e4m3_quantiser():
    rng = np.random.default_rng(9)
    pl = oracle.plan(2, 9, 8)
    d = 16
    v = rand_bf16(rng, (2, pl.N, d), 2.0)
    v[:, :, 3] = 0  # an all-zero channel is encoded as zero
    codes, dc = oracle.quant_v_e4m3(bits(v), pl)
    V = f64(v)
    for bh in range(2):
        assert np.array_equal(dc[bh], (np.abs(V[bh]).max(0).astype(np.float32) / np.float32(2.25)))
        assert dc[bh, 3] == 0 and (codes[bh, :, :, 3] == 0).all()
    # reconstruction: the channel maximum lands on 2.25 exactly, relative error <= 2^-4 for normal codes
    for bh in range(2):
        for a in range(pl.R):
            for j in range(64):
                tok = pl.slot_token[a, j]
                if tok < 0:
                    assert (codes[bh, a, j] == 0).all()
                    continue
                for c in range(d):
                    if dc[bh, c] == 0:
                        continue
                    rec = float(dc[bh, c]) * oracle.decode_e4m3(int(codes[bh, a, j, c]))
                    x = V[bh, tok, c]
                    assert abs(rec - x) <= max(abs(x) * 2.0 ** -4, float(dc[bh, c]) * 2.0 ** -10) * (1 + 1e-6)
    amax_code = oracle.cast_e4m3(2.25)
    assert oracle.decode_e4m3(amax_code) == 2.25


def test_v_e4m3_quantiser_with_a_given_scale():
    """The given-scale variant: (i) fed the tensor's own max/2.25 it returns the codes of the self-scaled quantiser,
    (ii) under any other scale every code is torch's float8_e4m3fn cast of fl32(V / delta) (saturating at 448, which
    a too small scale reaches), (iii) a zero scale skips the channel."""
    rng = np.random.default_rng(29)
    pl = oracle.plan(2, 12, 20)
    v = rand_bf16(rng, (2, pl.N, 16), 3.0)
    codes_self, dc = oracle.quant_v_e4m3(bits(v), pl)
    assert np.array_equal(oracle.quant_v_e4m3_given(bits(v), pl, dc), codes_self)
    other = (dc * rng.uniform(0.002, 3.0, dc.shape)).astype(np.float32)
    other[1, 5] = 0.0
    other[0, 3] = dc[0, 3] * np.float32(0.001)   # far too small: the larger values of this channel saturate
    codes = oracle.quant_v_e4m3_given(bits(v), pl, other)
    vf = v.float().numpy()
    st = np.maximum(pl.slot_token, 0)
    valid = (pl.slot_token >= 0)[None, :, :, None]
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = (vf[:, st] / other[:, None, None, :]).astype(np.float32)
    ratio = np.clip(np.nan_to_num(ratio, nan=0.0, posinf=448.0, neginf=-448.0), -448.0, 448.0)
    ref = torch.from_numpy(ratio).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    live = valid & (other > 0)[:, None, None, :]
    assert np.array_equal(np.where(live, codes, 0), np.where(live, ref, 0))
    assert (codes[~np.broadcast_to(live, codes.shape)] == 0).all()
    assert (np.abs(ratio[np.broadcast_to(live, ratio.shape)]) >= 448.0).any()   # the saturating branch is exercised


def test_nvfp4_quantisers():
    rng = np.random.default_rng(10)
    pl = oracle.plan(1, 16, 12)
    d = 32
    x = rand_bf16(rng, (2, pl.N, d), 1.5)
    x[0, pl.slot_token[1, :16], 5] = 0  # for the V-style grouping: one all-zero group
    x[1, 7, 16:32] = 0                  # for the Q/K-style grouping: one all-zero group
    X = f64(x)
    g = oracle.nvfp4_global_scale(bits(x))
    assert np.array_equal(g, (np.abs(X).reshape(2, -1).max(1).astype(np.float32) / np.float32(2688)))
    assert 2688 == 6 * 448
    for kind in ("qk", "v"):
        if kind == "qk":
            codes, sf = oracle.quant_nvfp4_qk(bits(x), pl, g)
        else:
            codes, sf = oracle.quant_nvfp4_v(bits(x), pl, g)
        assert codes.max() <= 15
        top = 0
        for bh in range(2):
            for a in range(pl.R):
                tok = pl.slot_token[a]
                blk = np.where((tok >= 0)[:, None], X[bh, np.maximum(tok, 0)], 0.0)  # [64, d], padding = 0
                groups = []
                if kind == "qk":
                    for j in range(64):
                        for gi in range(d // 16):
                            groups.append((blk[j, gi * 16:(gi + 1) * 16], codes[bh, a, j, gi * 16:(gi + 1) * 16], sf[bh, a, j, gi]))
                else:
                    for gi in range(4):
                        for c in range(d):
                            groups.append((blk[gi * 16:(gi + 1) * 16, c], codes[bh, a, gi * 16:(gi + 1) * 16, c], sf[bh, a, gi, c]))
                for vals, cc, s in groups:
                    sigma = oracle.decode_e4m3(int(s))
                    top = max(top, sigma)
                    if np.abs(vals).max() == 0:
                        assert s == 0
                    if sigma == 0:
                        assert (cc == 0).all()
                        continue
                    step = float(g[bh]) * sigma
                    rec = np.array([step * oracle.decode_e2m1(int(c)) for c in cc])
                    # E2M1 spacing is at most 2 (between 4 and 6): |x - rec| <= step, and <= step/4 below 2*step
                    inside = np.abs(vals) <= 6 * step
                    assert (np.abs(rec - vals)[inside] <= step * (1 + 1e-6)).all()
                    small = np.abs(vals) <= 2 * step
                    assert (np.abs(rec - vals)[small] <= step / 4 * (1 + 1e-6)).all()
                    # the local scale is amax/(6 g) rounded to E4M3: the group maximum lands within one E4M3 step of 6
                    assert np.abs(vals).max() / step <= 6 * (1 + 2.0 ** -4) * (1 + 1e-6) or sigma == 448
        assert top == 448.0  # the head's largest group uses the largest scale


def test_p8_constants():
    """App. C.3: offset 8.807 amplifies by about 448; eta is its inverse to fp32 precision."""
    amp = 2.0 ** 8.807
    eta = float(np.float32(0.0022326917))
    assert abs(amp - 447.8898) < 1e-3 and amp < 448.0
    assert abs(1 / eta - 447.8899) < 1e-3
    assert abs(eta * amp - 1.0) < 5e-7


# ---------------------------------------------------------------- attention
def _setup(rng, T, Hg, Wg, d, BH=1, scale_q=1.0):
    pl = oracle.plan(T, Hg, Wg)
    q, k, v = (rand_bf16(rng, (BH, pl.N, d), scale_q), rand_bf16(rng, (BH, pl.N, d)), rand_bf16(rng, (BH, pl.N, d)))
    return pl, q, k, v


def _all_blocks_lists(BH, R, tier):
    ids = np.tile(np.arange(R, dtype=np.int32), (BH, R, 1))
    counts = np.zeros((BH, R, 3), np.int32)
    counts[:, :, {4: 0, 8: 1, 16: 2}[tier]] = R
    return ids, counts


def test_all_blocks_16bit_reduces_to_dense_attention():
    rng = np.random.default_rng(11)
    pl, q, k, v = _setup(rng, 2, 12, 10, 32, BH=2, scale_q=2.0)
    ids, counts = _all_blocks_lists(2, pl.R, 16)
    sel = [(0, 0), (0, pl.R - 1), (1, 3)]
    s = 1 / math.sqrt(32)
    got = oracle.attention(bits(q), bits(k), bits(v), pl, ids, counts, None, s, sel)
    ref = oracle.dense(bits(q), bits(k), bits(v), pl, s, sel)
    # independent library routine for the dense reference itself
    P = torch.softmax(q.double() @ k.double().transpose(1, 2) * s, -1) @ v.double()
    for i, (bh, a) in enumerate(sel):
        tok = pl.slot_token[a]
        assert np.allclose(ref[i][tok >= 0], P[bh, tok[tok >= 0]].numpy(), rtol=1e-10, atol=1e-12)
        assert (got[i][tok < 0] == 0).all()
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert rel < 4e-3  # only bf16 rounding of the weights and of the output separates them


def test_block_order_irrelevant_without_weight_quantisation_and_subset_is_renormalised():
    rng = np.random.default_rng(12)
    pl, q, k, v = _setup(rng, 1, 16, 16, 16)
    R = pl.R
    ids = np.full((1, R, R), -1, np.int32)
    counts = np.zeros((1, R, 3), np.int32)
    keep = [2, 0, 3]  # deliberately not ascending: order must not matter beyond rounding
    ids[0, :, :3] = keep
    counts[0, :, 2] = 3
    s = 0.25
    got = oracle.attention(bits(q), bits(k), bits(v), pl, ids, counts, None, s, [(0, 1)])[0]
    Q, K, V = f64(q)[0], f64(k)[0], f64(v)[0]
    tk = np.concatenate([pl.slot_token[b] for b in keep])
    P = torch.softmax(torch.from_numpy(Q[pl.slot_token[1]] @ K[tk].T * s), -1).numpy()
    ref = P @ V[tk]
    assert np.abs(got - ref).max() < 2e-2 and np.linalg.norm(got - ref) / np.linalg.norm(ref) < 4e-3


def test_empty_support_returns_zero():
    rng = np.random.default_rng(13)
    pl, q, k, v = _setup(rng, 1, 8, 16, 16)
    ids = np.full((1, pl.R, 4), -1, np.int32)
    counts = np.zeros((1, pl.R, 3), np.int32)
    out = oracle.attention(bits(q), bits(k), bits(v), pl, ids, counts, None, 0.25, [(0, 0), (0, 1)])
    assert (out == 0).all()


def _lossless_inputs(rng, pl, d):
    """Q, K, V whose INT8 and NVFP4 encodings are exact, so only the weight conversion is lossy."""
    N = pl.N
    # values in {-6..6 on the E2M1 grid} * 42: amax 252 -> g = 252/2688 = 0.09375, every group holds a +-6*42
    grid = np.array([0.5, 1, 1.5, 2, 3, 4, 6, 0, -0.5, -1, -1.5, -2, -3, -4, -6]) * 42.0
    x = grid[rng.integers(0, len(grid), (3, 1, N, d))]
    x[:, :, :, ::16] = 252.0 * np.sign(rng.standard_normal((3, 1, N, d // 16)) + 1e-9)  # per-token channel groups
    for a in range(pl.R):  # per-channel key-slot groups of V: make slot 0 of every 16-slot group full scale
        for gi in range(4):
            tok = pl.slot_token[a, gi * 16]
            x[2, 0, tok, :] = 252.0
    return [torch.from_numpy(t.astype(np.float32)).to(torch.bfloat16) for t in x]


def test_lossless_operands_give_exact_logits_and_values():
    rng = np.random.default_rng(14)
    pl = oracle.plan(1, 16, 16)
    d = 32
    q, k, v = _lossless_inputs(rng, pl, d)
    ops = oracle.quantize_all(bits(q), bits(k), bits(v), pl)
    assert float(ops.gq[0]) == 252.0 / 2688.0
    s = 1e-4
    Q, K, V = f64(q)[0], f64(k)[0], f64(v)[0]
    for tier in (4, 16):
        ids, counts = _all_blocks_lists(1, pl.R, tier)
        dbg = oracle.attention_row_debug(bits(q), bits(k), bits(v), pl, ids, counts, ops, s, 0, 1, 9)
        u = pl.slot_token[1, 9]
        exact = K @ Q[u] * s
        assert np.allclose(dbg["shat"], exact, rtol=1e-12, atol=1e-12)
        assert np.allclose(dbg["vhat"], V, rtol=0, atol=0)
        assert (dbg["tier"] == tier).all()
    # INT8: block amax 252 -> delta = fl32(252/127 + 1e-7) is not a power of two, so check the bound instead
    ids, counts = _all_blocks_lists(1, pl.R, 8)
    dbg = oracle.attention_row_debug(bits(q), bits(k), bits(v), pl, ids, counts, ops, s, 0, 1, 9)
    dq, dk = float(ops.dq8[0, 1]), ops.dk8[0].astype(np.float64)
    u = pl.slot_token[1, 9]
    exact = K @ Q[u] * s
    blk_of = np.empty(pl.N, int)
    for a in range(pl.R):
        blk_of[pl.slot_token[a]] = a
    # Eq. 'v2-logit-quant' with |dQ| <= sqrt(d) dq/2, |dK| <= sqrt(d) dk/2
    nq, nk = np.linalg.norm(Q[u]), np.linalg.norm(K, axis=1)
    eq, ek = math.sqrt(d) * dq / 2, math.sqrt(d) * dk[blk_of] / 2
    bound = (nq * ek + nk * eq + eq * ek) * s
    assert (np.abs(dbg["shat"] - exact) <= bound * (1 + 1e-9)).all()
    assert np.abs(dbg["shat"] - exact).max() > 0  # the path really is quantised


@pytest.mark.parametrize("tier", [4, 8])
def test_zero_query_closed_form(tier):
    """Q = 0: every weight is 1.  8-bit path: E4M3(2^8.807) = 448, so the numerator weight is eta*448;
    4-bit path: sigma_P = 448, code 6, numerator weight exactly 1.  The output is that weight times the mean
    of the reconstructed values (here exactly representable), normalised by the fp32 denominator."""
    rng = np.random.default_rng(15)
    pl = oracle.plan(1, 16, 16)
    d = 32
    _, k, v = _lossless_inputs(rng, pl, d)
    if tier == 8:  # E4M3-exact values: integers * 2^k with channel max 2.25 * 2^6 = 144
        v = torch.from_numpy((rng.integers(-4, 5, (1, pl.N, d)) * 16.0).astype(np.float32)).to(torch.bfloat16)
        v[0, 0, :] = 144.0
    q = torch.zeros_like(k)
    ops = oracle.quantize_all(bits(q), bits(k), bits(v), pl)
    ids, counts = _all_blocks_lists(1, pl.R, tier)
    out = oracle.attention(bits(q), bits(k), bits(v), pl, ids, counts, ops, 0.1, [(0, 2)])[0]
    mean_v = f64(v)[0].mean(0)
    wq = float(np.float32(0.0022326917)) * 448.0 if tier == 8 else 1.0
    ref = torch.from_numpy((wq * mean_v).astype(np.float32)).to(torch.bfloat16).float().numpy()
    assert np.array_equal(out, np.tile(ref, (64, 1)))


def _mixed_lists(rng, BH, R, n4, n8, n16):
    ids = np.full((BH, R, R), -1, np.int32)
    counts = np.zeros((BH, R, 3), np.int32)
    for bh in range(BH):
        for a in range(R):
            perm = rng.permutation(R)[:n4 + n8 + n16]
            segs = [np.sort(perm[:n4]), np.sort(perm[n4:n4 + n8]), np.sort(perm[n4 + n8:])]
            ids[bh, a, :n4 + n8 + n16] = np.concatenate(segs)
            counts[bh, a] = (n4, n8, n16)
    return ids, counts


def test_encoded_units_enter_exit_match_common_units():
    """Eq. 'precision-state-conversion': carrying the 8-bit phase in encoded units with Enter/Exit gives the same
    normalised output as accumulating in common units; phase count gives at most two switches."""
    rng = np.random.default_rng(16)
    pl, q, k, v = _setup(rng, 2, 16, 16, 32, BH=2, scale_q=2.0)
    ops = oracle.quantize_all(bits(q), bits(k), bits(v), pl)
    s = 1 / math.sqrt(32)
    for n4, n8, n16 in ((2, 3, 1), (0, 4, 0), (3, 2, 0), (0, 2, 2)):
        ids, counts = _mixed_lists(rng, 2, pl.R, n4, n8, n16)
        assert max(sum(1 for n in (n4, n8, n16) if n) - 1, 0) <= 2
        sel = [(0, 0), (1, 5)]
        a_ = oracle.attention(bits(q), bits(k), bits(v), pl, ids, counts, ops, s, sel, encoded_units=False)
        b_ = oracle.attention(bits(q), bits(k), bits(v), pl, ids, counts, ops, s, sel, encoded_units=True)
        # identical up to the factor eta*2^8.807 = 1 - 1.6e-7 on the 8-bit share of the denominator: at most a
        # final bf16 rounding flip
        assert np.abs(a_ - b_).max() <= 2.0 ** -8 * np.abs(a_).max()
        assert (a_ != b_).mean() < 0.01


@pytest.mark.parametrize("mix", [(3, 2, 1), (0, 4, 2), (5, 0, 0), (0, 6, 0)])
def test_reconstruction_identity_and_error_bound(mix):
    """(i) The output equals sum(what * vhat)/ell rebuilt from the per-key reconstructions (App. B.3,
    Eq. 'v2-reconstructed-output'); (ii) Lemma 3.3, block form: |O_dense - O| <= 2 Vmax delta_u +
    e^{alpha_u} sum_b m_ub c_ub with alpha, nu, omega measured from the reconstructed operands."""
    rng = np.random.default_rng(17)
    d = 32
    pl, q, k, v = _setup(rng, 1, 16, 24, d, scale_q=1.5)
    ops = oracle.quantize_all(bits(q), bits(k), bits(v), pl)
    s = 1 / math.sqrt(d)
    ids, counts = _mixed_lists(rng, 1, pl.R, *mix)
    Q, K, V = f64(q)[0], f64(k)[0], f64(v)[0]
    vmax = np.linalg.norm(V, axis=1).max()
    blk_of = np.empty(pl.N, int)
    for a in range(pl.R):
        blk_of[pl.slot_token[a]] = a
    for (a, ju) in ((0, 0), (3, 17), (5, 63)):
        dbg = oracle.attention_row_debug(bits(q), bits(k), bits(v), pl, ids, counts, ops, s, 0, a, ju)
        u = pl.slot_token[a, ju]
        kept = ~np.isnan(dbg["shat"])
        assert kept.sum() == 64 * sum(mix)
        hf = dbg["h_final"]
        w_fin = np.where(kept, np.exp(np.where(kept, dbg["shat"], 0) - hf), 0.0)
        what_fin = np.where(kept, dbg["what"] * np.exp(np.where(kept, dbg["h_at"], 0) - hf), 0.0)
        assert abs(w_fin.sum() - dbg["ell"]) <= 1e-6 * dbg["ell"]       # denominator uses unquantised weights
        o_rec = (what_fin[:, None] * dbg["vhat"]).sum(0) / dbg["ell"]
        assert np.abs(o_rec - dbg["out"]).max() <= 2.0 ** -8 * max(1.0, np.abs(o_rec).max())
        # bound
        s_exact = K @ Q[u] * s
        p_dense = np.exp(s_exact - s_exact.max())
        p_dense /= p_dense.sum()
        o_dense = p_dense @ V
        delta_u = p_dense[~kept].sum()
        z = np.where(kept, np.exp(s_exact - s_exact[kept].max()), 0.0)
        m_v = z / z.sum()
        total = 0.0
        alphas = []
        for b in np.unique(blk_of[kept]):
            in_b = kept & (blk_of == b)
            alpha = np.abs(dbg["shat"][in_b] - s_exact[in_b]).max()
            nu = np.linalg.norm(dbg["vhat"][in_b] - V[in_b], axis=1).max()
            omega = np.abs(what_fin[in_b] - w_fin[in_b]).sum() / w_fin[in_b].sum()
            c_ub = 2 * vmax * (math.exp(alpha) - 1) + math.exp(alpha) * (nu + (vmax + nu) * omega)
            total += m_v[in_b].sum() * c_ub
            alphas.append(alpha)
        bound = 2 * vmax * delta_u + math.exp(max(alphas)) * total
        err = np.linalg.norm(o_dense - o_rec)
        assert err <= bound * (1 + 1e-9)
        # weight conversion stays within the formats' relative precision (bf16: 2^-9, E4M3: 2^-4, NVFP4 group: coarse)
        t = dbg["tier"]
        rel = np.abs(what_fin - w_fin)[kept] / w_fin[kept]
        assert (rel[t[kept] == 16] <= 2.0 ** -8).all()
        big8 = (t[kept] == 8) & (dbg["what"][kept] > 0.0022326917 * 2.0 ** -6)
        assert (rel[big8] <= 2.0 ** -4 + 1e-3).all()
        # NVFP4 weights: the error is at most half the widest E2M1 gap in units of the group scale, i.e. about a
        # sixth of the largest weight of the row's block at the time it was processed (<= 1)
        assert (np.abs(dbg["what"] - np.where(kept, np.exp(np.where(kept, dbg["shat"] - dbg["h_at"], 0)), 0.0))[kept][t[kept] == 4]
                <= (1 + 2.0 ** -3) / 6.0).all()



_E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def _e2m1_nearest_even(x: float) -> float:
    """Nearest E2M1 magnitude by exhaustive search; a tie goes to the neighbour with the even code."""
    dist = np.abs(_E2M1_VALUES - x)
    best = np.flatnonzero(dist == dist.min())
    if len(best) == 2:
        return float(_E2M1_VALUES[best[0] if best[0] % 2 == 0 else best[1]])
    return float(_E2M1_VALUES[best[0]])


@pytest.mark.parametrize("grid,mix", [((1, 12, 20), (4, 1, 1)), ((2, 16, 16), (6, 0, 0)), ((1, 9, 17), (3, 2, 0))])
def test_online_nvfp4_weight_quantiser_is_the_printed_formula(grid, mix):
    """Eq. 'v2-nvfp4-probability' on non-uniform weights, rebuilt outside the oracle: groups are the 16 consecutive
    key slots 16g..16g+15 of a block (padding counts as 0), sigma_P = E4M3(448 max_G w) through torch's
    float8_e4m3fn cast, the code is the nearest E2M1 value of 2688 w / sigma_P (ties to the even code, by search),
    and the weight the numerator uses is sigma_P / 2688 times that value; a zero scale zeroes the group."""
    rng = np.random.default_rng(23)
    d = 32
    pl, q, k, v = _setup(rng, *grid, d, scale_q=2.5)
    ops = oracle.quantize_all(bits(q), bits(k), bits(v), pl)
    s = 1 / math.sqrt(d)
    ids, counts = _mixed_lists(rng, 1, pl.R, *mix)
    n_checked = n_zero_groups = n_nonuniform = 0
    for (a, ju) in ((0, 0), (pl.R - 1, 0), (1, 9)):
        if pl.slot_token[a, ju] < 0:
            continue
        dbg = oracle.attention_row_debug(bits(q), bits(k), bits(v), pl, ids, counts, ops, s, 0, a, ju)
        for b in ids[0, a, :mix[0]]:
            for g in range(4):
                toks = pl.slot_token[b, 16 * g:16 * g + 16]
                valid = toks >= 0
                if not valid.any():
                    continue
                tv = toks[valid]
                assert (dbg["tier"][tv] == 4).all()
                w = np.zeros(16, np.float32)
                w[valid] = np.exp(dbg["shat"][tv] - dbg["h_at"][tv]).astype(np.float32)
                gm = np.float32(w.max())
                sigma = float(torch.tensor([np.float32(448.0) * gm], dtype=torch.float32)
                              .to(torch.float8_e4m3fn).to(torch.float32)[0])
                expect = np.zeros(16)
                if sigma > 0.0:
                    for i in range(16):
                        r = np.float32(2688.0 * float(w[i]) / sigma)
                        expect[i] = sigma / 2688.0 * _e2m1_nearest_even(float(r))
                else:
                    n_zero_groups += 1
                assert np.array_equal(dbg["what"][tv], expect[valid]), (a, ju, b, g)
                # coarse bound of the format: half of the widest E2M1 gap (4..6) in units of sigma_P/2688 ~ max/6
                assert (np.abs(expect[valid] - w[valid]) <= float(gm) / 6.0 * (1 + 2.0 ** -3) + 1e-30).all()
                n_checked += int(valid.sum())
                n_nonuniform += int(len(np.unique(expect[valid])) > 1)
    assert n_checked > 200 and n_nonuniform > 10


def _prefix_case(rng, P, mix, d=32, grid=(2, 12, 20)):
    """Joint tensors [P prefix | video], the video-only stages on the video part, lists and plan of the joint
    sequence."""
    plv = oracle.plan(*grid)
    q, k, v = (rand_bf16(rng, (1, P + plv.N, d), 1.5), rand_bf16(rng, (1, P + plv.N, d)),
               rand_bf16(rng, (1, P + plv.N, d)))
    vid = lambda t: np.ascontiguousarray(bits(t)[:, P:])
    ops = oracle.quantize_all(vid(q), vid(k), vid(v), plv)
    ids, counts = _mixed_lists(rng, 1, plv.R, *mix)
    pl = oracle.plan_with_prefix(plv, P)
    ids_x, cnt_x = oracle.lists_with_prefix(ids, counts, plv.R, pl.R - plv.R)
    return plv, pl, q, k, v, oracle.pad_operands(ops, pl.R), ids, counts, ids_x, cnt_x


def test_prefix_plan_is_a_partition_of_the_joint_sequence():
    plv = oracle.plan(2, 12, 20)
    for P in (0, 1, 64, 77, 200):
        pl = oracle.plan_with_prefix(plv, P)
        toks = pl.slot_token[pl.slot_token >= 0]
        assert np.array_equal(np.sort(toks), np.arange(P + plv.N))
        assert pl.R == plv.R + -(-P // 64) and pl.N == P + plv.N
        assert np.array_equal(pl.slot_token[:plv.R][plv.slot_token >= 0], plv.slot_token[plv.slot_token >= 0] + P)
        if P:
            assert np.array_equal(pl.slot_token[plv.R:].reshape(-1)[:P], np.arange(P))


def test_prefix_keys_alone_and_prefix_queries_dense():
    """App. C.1.  (i) With every video block skipped, a video query attends to the prefix keys alone: its output is
    dense softmax attention over those P keys (fp64, written out here).  (ii) A prefix query is non-sparse: its row
    equals dense attention over the whole joint sequence.  Only the bf16 rounding of the weights (16-bit tier) and of
    the output separates the two sides."""
    rng = np.random.default_rng(31)
    P, d = 77, 32
    plv, pl, q, k, v, ops, ids, counts, ids_x, cnt_x = _prefix_case(rng, P, (0, 0, 0), d)
    s = 1 / math.sqrt(d)
    Q, K, V = f64(q)[0], f64(k)[0], f64(v)[0]
    sel = [(0, 0), (0, 5), (0, plv.R - 1)]
    out = oracle.attention(bits(q), bits(k), bits(v), pl, ids_x, cnt_x, ops, s, sel)
    for i, (_, a) in enumerate(sel):
        for j in range(64):
            u = pl.slot_token[a, j]
            if u < 0:
                assert (out[i, j] == 0).all()
                continue
            lg = K[:P] @ Q[u] * s
            w = np.exp(lg - lg.max())
            ref = (w / w.sum()) @ V[:P]
            assert np.abs(out[i, j] - ref).max() <= 2.0 ** -7 * max(1.0, np.abs(ref).max())
    pre_rows = [(0, a) for a in range(plv.R, pl.R)]
    got = oracle.attention(bits(q), bits(k), bits(v), pl, ids_x, cnt_x, ops, s, pre_rows)
    dense = oracle.dense(bits(q), bits(k), bits(v), pl, s, pre_rows)
    assert np.abs(got - dense).max() <= 2.0 ** -7 * max(1.0, np.abs(dense).max())
    assert (got[-1, P - 64:] == 0).all()          # slots of the last prefix block beyond token P-1 are padding


def test_prefix_blocks_sit_outside_the_budget_and_vanish_without_prefix():
    """(i) P = 0 leaves the joint tables identical to the video ones and the output bit-identical.  (ii) With a
    prefix, every video row keeps exactly its ranked blocks plus all prefix blocks, the latter in the 16-bit segment
    (last in the phase order), so the budget counts of the quantised tiers do not change.  (iii) The output equals
    the per-key reconstruction sum(what * vhat) / ell over the retained video keys AND the P prefix keys."""
    rng = np.random.default_rng(32)
    d = 32
    plv, pl0, q, k, v, ops0, ids, counts, ids0, cnt0 = _prefix_case(rng, 0, (3, 2, 1), d)
    s = 1 / math.sqrt(d)
    sel = [(0, 1), (0, 4)]
    base = oracle.attention(bits(q), bits(k), bits(v), plv, ids, counts, ops0, s, sel)
    same = oracle.attention(bits(q), bits(k), bits(v), pl0, ids0, cnt0, ops0, s, sel)
    assert pl0.R == plv.R and np.array_equal(base, same)
    P = 100
    plv, pl, q, k, v, ops, ids, counts, ids_x, cnt_x = _prefix_case(rng, P, (3, 2, 1), d)
    Rp = pl.R - plv.R
    assert Rp == 2
    assert np.array_equal(cnt_x[0, :plv.R, :2], counts[0, :, :2])
    assert (cnt_x[0, :plv.R, 2] == counts[0, :, 2] + Rp).all()
    for a in range(plv.R):
        n = int(cnt_x[0, a].sum())
        assert ids_x[0, a, n - Rp:n].tolist() == [plv.R, plv.R + 1]
    for (a, ju) in ((0, 0), (3, 17)):
        dbg = oracle.attention_row_debug(bits(q), bits(k), bits(v), pl, ids_x, cnt_x, ops, s, 0, a, ju)
        kept = ~np.isnan(dbg["shat"])
        assert kept[:P].all() and kept.sum() == P + sum(int(plv.n_valid[b]) for b in ids[0, a, :6])
        assert (dbg["tier"][:P] == 16).all()
        hf = dbg["h_final"]
        what_fin = np.where(kept, dbg["what"] * np.exp(np.where(kept, dbg["h_at"], 0) - hf), 0.0)
        o_rec = (what_fin[:, None] * dbg["vhat"]).sum(0) / dbg["ell"]
        assert np.abs(o_rec - dbg["out"]).max() <= 2.0 ** -8 * max(1.0, np.abs(o_rec).max())


def test_prop_3_4_bound_difference_identity():
    """Prop. 3.4: B_v2 - B_v1 = -2 Vmax tau + (tau8 eps8 + tau4 eps4)/(1 - delta_v2)."""
    rng = np.random.default_rng(18)
    for _ in range(100):
        vmax, d2, t8, t4, e8, e4 = rng.random(6)
        if d2 + t8 + t4 >= 1:
            continue
        tau = t8 + t4
        b1 = 2 * vmax * (d2 + tau)
        m8, m4 = t8 / (1 - d2), t4 / (1 - d2)
        b2 = 2 * vmax * d2 + m8 * e8 + m4 * e4
        assert abs((b2 - b1) - (-2 * vmax * tau + (t8 * e8 + t4 * e4) / (1 - d2))) < 1e-12
        assert (b2 < b1) == (t8 * e8 + t4 * e4 < 2 * vmax * tau * (1 - d2))


def _golden():
    import os
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, value = line.split()[:2]
                vals[name] = float(value)
    return vals


def test_golden_constants():
    """The constants the paper prints (tests/golden/paper_constants.txt) against what the oracle computes with."""
    g = _golden()
    # format ranges: the largest codes decode to the printed maxima, and their product is the NVFP4 range
    assert oracle.decode_e2m1(7) == g["e2m1_max"] and oracle.decode_e2m1(15) == -g["e2m1_max"]
    assert oracle.decode_e4m3(0x7E) == g["e4m3_max"] and oracle.cast_e4m3(1e9) == 0x7E
    assert g["e2m1_max"] * g["e4m3_max"] == g["nvfp4_range"]
    # INT8: a block whose largest magnitude is `levels` gets delta = 1 + eps (to fp32) and the code `levels`
    pl = oracle.plan(1, 8, 8)
    x = np.zeros((1, 64, 16), np.float32)
    x[0, 5, 3] = g["int8_levels"]
    x[0, 6, 2] = -1.0
    codes, delta = oracle.quant_int8(oracle.bf16_bits(torch.from_numpy(x).to(torch.bfloat16)), pl)
    assert float(delta[0, 0]) == float(np.float32(np.float32(1.0) + np.float32(g["int8_epsilon"])))
    assert codes.reshape(64, 16)[5, 3] == g["int8_levels"] and codes.reshape(64, 16)[6, 2] == -1
    # E4M3 V: the per-channel scale is the channel maximum over the printed divisor
    v = np.zeros((1, 64, 16), np.float32)
    v[0, 9, 4] = 4.5
    _, dc = oracle.quant_v_e4m3(oracle.bf16_bits(torch.from_numpy(v).to(torch.bfloat16)), pl)
    assert float(dc[0, 4]) == float(np.float32(4.5) / np.float32(g["v_e4m3_divisor"])) and float(dc[0, 0]) == 0.0
    # NVFP4: per-head scale = amax / 2688
    assert float(oracle.nvfp4_global_scale(oracle.bf16_bits(torch.from_numpy(x).to(torch.bfloat16)))[0]) == \
        float(np.float32(g["int8_levels"]) / np.float32(g["nvfp4_range"]))
    # 8-bit weights: the offset amplifies a weight of 1 to just below the E4M3 maximum, and eta undoes it
    amp = 2.0 ** g["p8_exponent_offset"]
    assert g["e4m3_max"] - 0.2 < amp < g["e4m3_max"]
    assert abs(g["p8_eta"] * amp - 1.0) < 5e-7
    assert oracle.decode_e4m3(oracle.cast_e4m3(amp)) == g["e4m3_max"]
