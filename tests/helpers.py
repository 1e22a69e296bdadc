"""Test-side helpers: run the CUDA path through the C ABI, run the oracle on the same bits, and undo the
documented record layouts (pure index permutations, see include/da2.h) so both can be compared element-wise."""
from __future__ import annotations

import math

import numpy as np
import torch

import da2_inputs
import oracle
import paper_2609_32628_b200 as da2


def scale_of(w) -> float:
    return float(np.float32(1.0) / np.sqrt(np.float32(w.head_dim)))


def run_gpu(w, q, k, v, rank_scope=0, lam=None, zero_ws=False, g_fixed=None, partition=0):
    """q,k,v CUDA bf16 [B,H,N,d].  g_fixed: optional (g_q, g_k, g_v) host arrays [B*H] of caller-fixed NVFP4
    per-tensor scales.  Returns (plan, workspace uint8 tensor, out)."""
    gq, gk, gv = (None, None, None) if g_fixed is None else g_fixed
    plan = da2.da2_plan(w.B, w.H, w.T, w.Hg, w.Wg, w.head_dim, w.frac16, w.frac8, w.frac4,
                        lam=w.lam if lam is None else lam, rank_scope=rank_scope, g_q=gq, g_k=gk, g_v=gv,
                        partition=partition)
    ws = (torch.zeros if zero_ws else torch.empty)(int(plan.info.workspace_bytes), dtype=torch.uint8, device=q.device)
    out = torch.full_like(q, float("nan"))
    da2.da2_prepare(plan, q, k, v, ws)
    da2.da2_attention_fwd(plan, q, k, v, ws, out)
    torch.cuda.synchronize()
    assert da2.da2_device_status(plan, ws) == 0
    return plan, ws, out


def region(ws, off, nbytes, dtype):
    return ws[off:off + nbytes].cpu().numpy().view(dtype)


class Workspace:
    """Logical views of a da2 workspace (CPU numpy), heads optionally restricted."""

    def __init__(self, plan, ws, heads=None):
        self.I = I = plan.info
        self.ws = ws
        self.BH = I.B * I.H
        self.heads = list(range(self.BH)) if heads is None else list(heads)
        self.R, self.d = I.R, I.head_dim

    def _per_head(self, off, per_head_bytes, dtype):
        parts = [region(self.ws, off + h * per_head_bytes, per_head_bytes, dtype) for h in self.heads]
        return np.stack(parts)

    def desc(self, i):
        return self._per_head(self.I.off_desc[i], self.R * self.d * 4, np.float32).reshape(-1, self.R, self.d)

    def draft_map(self):
        return self._per_head(self.I.off_map, self.R * self.R * 4, np.float32).reshape(-1, self.R, self.R)

    def gscale(self):
        return self._per_head(self.I.off_gscale, 16, np.float32)[:, :3]

    def dq8(self):
        return self._per_head(self.I.off_dq8, self.R * 4, np.float32)

    def dk8(self):
        return self._per_head(self.I.off_dk8, self.R * 4, np.float32)

    def dv8(self):
        return self._per_head(self.I.off_dv8, self.d * 4, np.float32)

    def lists(self):
        """-> ids int32 [H', R, R] (-1 padded), counts int32 [H', R, 3]."""
        cnt = self._per_head(self.I.off_counts, self.R * 16, np.int32).reshape(-1, self.R, 4)
        ids_raw = self._per_head(self.I.off_ids, int(self.I.ids_per_head) * 2, np.uint16)
        ids = np.full((len(self.heads), self.R, self.R), -1, np.int32)
        for h in range(len(self.heads)):
            for a in range(self.R):
                n = int(cnt[h, a, :3].sum())
                o = int(cnt[h, a, 3])
                ids[h, a, :n] = ids_raw[h, o:o + n]
        return ids, np.ascontiguousarray(cnt[:, :, :3])

    # ---- records -> logical block order [H', R, 64, d]
    def _rec(self, off, rec_bytes):
        return self._per_head(off, self.R * rec_bytes, np.uint8).reshape(len(self.heads), self.R, rec_bytes)

    def q_or_k_int8(self, which):
        d = self.d
        rec = self._rec(self.I.off_qrec[1], self.I.qrec_bytes[1]) if which == "q" else \
            self._rec(self.I.off_kvrec[1], self.I.kvrec_bytes[1])[:, :, :64 * d]
        x = rec.reshape(-1, self.R, d // 16, 64, 16).transpose(0, 1, 3, 2, 4).reshape(-1, self.R, 64, d)
        return np.ascontiguousarray(x).view(np.int8)

    def v_e4m3(self):
        d = self.d
        rec = self._rec(self.I.off_kvrec[1], self.I.kvrec_bytes[1])[:, :, 64 * d:]
        x = rec.reshape(-1, self.R, 4, d, 16).transpose(0, 1, 2, 4, 3).reshape(-1, self.R, 64, d)
        return np.ascontiguousarray(x)

    @staticmethod
    def _nibbles(b):
        return np.stack([b & 0xf, b >> 4], axis=-1).reshape(*b.shape[:-1], b.shape[-1] * 2)

    def q_or_k_fp4(self, which):
        d = self.d
        img = 64 * d // 2
        natom = d // 64
        rec = self._rec(self.I.off_qrec[0], self.I.qrec_bytes[0]) if which == "q" else \
            self._rec(self.I.off_kvrec[0], self.I.kvrec_bytes[0])
        codes = self._nibbles(rec[:, :, :img].reshape(-1, self.R, d // 32, 64, 16))      # [.., kc, r, 32]
        codes = codes.transpose(0, 1, 3, 2, 4).reshape(-1, self.R, 64, d)
        atoms = rec[:, :, img:img + natom * 512].reshape(-1, self.R, natom, 32, 4, 4)    # [atom, r%32, r/32, g]
        sf = atoms.transpose(0, 1, 4, 3, 2, 5).reshape(-1, self.R, 128, natom * 4)[:, :, :64]
        return np.ascontiguousarray(codes), np.ascontiguousarray(sf)

    def v_fp4(self):
        d = self.d
        base = 64 * d // 2 + (d // 64) * 512
        rec = self._rec(self.I.off_kvrec[0], self.I.kvrec_bytes[0])[:, :, base:]
        codes = self._nibbles(rec[:, :, :d * 32].reshape(-1, self.R, 2, d, 16))          # [.., kc, c, 32 slots]
        codes = codes.transpose(0, 1, 2, 4, 3).reshape(-1, self.R, 64, d)
        atom = rec[:, :, d * 32:d * 32 + 512].reshape(-1, self.R, 32, 4, 4)              # [c%32, c/32, g]
        sf = atom.transpose(0, 1, 4, 3, 2).reshape(-1, self.R, 4, 128)[:, :, :, :d]      # [g, c]
        return np.ascontiguousarray(codes), np.ascontiguousarray(sf)

    def bf16_records(self):
        """-> (q, k, v) uint16 bit patterns in block order [H', R, 64, d]."""
        d = self.d
        qr = self._rec(self.I.off_qrec[2], self.I.qrec_bytes[2]).view(np.uint16)
        kvr = self._rec(self.I.off_kvrec[2], self.I.kvrec_bytes[2]).view(np.uint16)
        unq = lambda r: r.reshape(-1, self.R, d // 8, 64, 8).transpose(0, 1, 3, 2, 4).reshape(-1, self.R, 64, d)
        vt = kvr[:, :, 64 * d:].reshape(-1, self.R, 8, d, 8).transpose(0, 1, 2, 4, 3).reshape(-1, self.R, 64, d)
        return unq(qr), unq(kvr[:, :, :64 * d]), vt


def oracle_all(w, q, k, v, heads=None, rank_scope=0, lam=None, balanced=False):
    """Runs every oracle stage on CPU copies of q, k, v (optionally a subset of flat heads)."""
    sel = slice(None) if heads is None else list(heads)
    bits = lambda t: np.ascontiguousarray(oracle.bf16_bits(t.reshape(-1, w.N, w.head_dim).cpu())[sel])
    qb, kb, vb = bits(q), bits(k), bits(v)
    pl = oracle.plan_balanced(w.T, w.Hg, w.Wg, 64) if balanced else oracle.plan(w.T, w.Hg, w.Wg)
    lam32 = float(np.float32(w.lam if lam is None else lam))
    r = oracle.run_pipeline(qb, kb, vb, pl, lam=lam32, scale=scale_of(w), frac16=w.frac16, frac8=w.frac8,
                            frac4=w.frac4, head_scope=bool(rank_scope))
    r.update(pl=pl, q=qb, k=kb, v=vb)
    return r


def oracle_operands(ref, g_fixed=None, heads=None, dv_fixed=None):
    """Every quantised operand set of the oracle; with g_fixed = (g_q, g_k, g_v) [BH] the NVFP4 quantisers take those
    per-tensor scales instead of deriving them (App. C.3: g_X is a given positive per-tensor scale)."""
    pl = ref["pl"]
    ops = oracle.quantize_all(ref["q"], ref["k"], ref["v"], pl)
    if g_fixed is not None:
        sel = slice(None) if heads is None else list(heads)
        gq, gk, gv = (np.ascontiguousarray(np.asarray(g, np.float32)[sel]) for g in g_fixed)
        ops.gq, ops.gk, ops.gv = gq, gk, gv
        ops.q4, ops.sfq = oracle.quant_nvfp4_qk(ref["q"], pl, gq)
        ops.k4, ops.sfk = oracle.quant_nvfp4_qk(ref["k"], pl, gk)
        ops.v4, ops.sfv = oracle.quant_nvfp4_v(ref["v"], pl, gv)
    if dv_fixed is not None:   # carried-over E4M3 per-channel value scales [BH, d]
        sel = slice(None) if heads is None else list(heads)
        ops.dv8 = np.ascontiguousarray(np.asarray(dv_fixed, np.float32)[sel])
        ops.v8 = oracle.quant_v_e4m3_given(ref["v"], pl, ops.dv8)
    return ops


def compare_lists(A, ids_o, cnt_o, ids_g, cnt_g, rel=1e-5):
    """Exact comparison of per-row lists; a difference is excused only if every swapped entry's score lies within
    `rel` of a tier boundary score.  Returns (rows_differing, excused_entries); raises on a real mismatch."""
    BH, R, _ = A.shape
    bad_rows, excused = [], 0
    for h in range(BH):
        for a in range(R):
            no, ng = int(cnt_o[h, a].sum()), int(cnt_g[h, a].sum())
            if np.array_equal(cnt_o[h, a], cnt_g[h, a]) and np.array_equal(ids_o[h, a, :no], ids_g[h, a, :ng]):
                continue
            bad_rows.append((h, a))
            row = A[h, a].astype(np.float64)
            tag_o = np.zeros(R, np.int8)
            tag_g = np.zeros(R, np.int8)
            for ids, cnt, tag in ((ids_o, cnt_o, tag_o), (ids_g, cnt_g, tag_g)):
                pos = 0
                for s, tier in enumerate((4, 8, 16)):
                    n = int(cnt[h, a, s])
                    seg = ids[h, a, pos:pos + n]
                    assert (np.diff(seg) > 0).all(), "ids must ascend inside a segment"
                    tag[seg] = tier
                    pos += n
            # boundary scores of the oracle's assignment
            bounds = [row[tag_o == t].min() for t in (16, 8, 4) if (tag_o == t).any()]
            for idx in np.nonzero(tag_o != tag_g)[0]:
                ok = any(abs(row[idx] - b) <= rel * b for b in bounds)
                assert ok, f"list mismatch at head {h} row {a} key block {idx} not explained by a near-tie"
                excused += 1
    return bad_rows, excused


def rel_l2(x, ref):
    return float(np.linalg.norm(x.astype(np.float64) - ref) / max(np.linalg.norm(ref), 1e-30))
