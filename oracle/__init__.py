"""Python face of the CPU oracle (oracle/da2_oracle.c).  TEST INFRASTRUCTURE ONLY.

Nothing in the product package may import this module.  It compiles the plain C
oracle with gcc on first use and wraps each function with numpy marshalling;
there is no arithmetic of the method in this file.

Citations (paper sections/equations) are on the C functions.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "da2_oracle.c")
_LIB = os.path.join(_HERE, "libda2_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle into oracle/libda2_oracle.so (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
                               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_decode_e4m3.restype = ctypes.c_float
        _lib.orc_decode_e4m3.argtypes = [ctypes.c_uint8]
        _lib.orc_decode_e2m1.restype = ctypes.c_float
        _lib.orc_decode_e2m1.argtypes = [ctypes.c_uint8]
        _lib.orc_cast_e4m3.restype = ctypes.c_uint8
        _lib.orc_cast_e4m3.argtypes = [ctypes.c_float]
        _lib.orc_cast_e2m1.restype = ctypes.c_uint8
        _lib.orc_cast_e2m1.argtypes = [ctypes.c_float]
        _lib.orc_plan.restype = ctypes.c_int
        _lib.orc_plan_balanced.restype = ctypes.c_int
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    return int(env) if env else (os.cpu_count() or 1)


def _p(a: Optional[np.ndarray]):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be contiguous"
    return a.ctypes.data_as(ctypes.c_void_p)


def _i64(v):
    return ctypes.c_int64(int(v))


def _i(v):
    return ctypes.c_int(int(v))


def _d(v):
    return ctypes.c_double(float(v))


def bf16_bits(t) -> np.ndarray:
    """torch bf16 tensor (CPU) -> contiguous numpy uint16 view of its bits."""
    import torch
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


# ---------------------------------------------------------------- scalar casts
def cast_e4m3(x: float) -> int:
    return int(lib().orc_cast_e4m3(ctypes.c_float(x)))


def decode_e4m3(c: int) -> float:
    return float(lib().orc_decode_e4m3(ctypes.c_uint8(c)))


def cast_e2m1(x: float) -> int:
    return int(lib().orc_cast_e2m1(ctypes.c_float(x)))


def decode_e2m1(c: int) -> float:
    return float(lib().orc_decode_e2m1(ctypes.c_uint8(c)))


# ------------------------------------------------------------------------ plan
@dataclass
class Plan:
    T: int
    Hg: int
    Wg: int
    th: int
    tw: int
    R: int
    S: int
    slot_token: np.ndarray  # int32 [R, S], -1 = padding
    n_valid: np.ndarray     # int32 [R]
    n_prefix: int = 0       # prefix (text) tokens in front of the video tokens; their blocks follow the video regions
    R_video: int = -1       # number of video regions (== R without a prefix)

    @property
    def N(self) -> int:
        return self.T * self.Hg * self.Wg + self.n_prefix


def plan(T: int, Hg: int, Wg: int, th: int = 8, tw: int = 8) -> Plan:
    R = lib().orc_plan(_i(T), _i(Hg), _i(Wg), _i(th), _i(tw), None, None)
    S = th * tw
    st = np.empty((R, S), np.int32)
    nv = np.empty((R,), np.int32)
    lib().orc_plan(_i(T), _i(Hg), _i(Wg), _i(th), _i(tw), _p(st), _p(nv))
    return Plan(T, Hg, Wg, th, tw, R, S, st, nv)


def plan_balanced(T: int, Hg: int, Wg: int, C: int = 64) -> Plan:
    """Balanced ragged minimum-perimeter partition (App. C.2): R_f = ceil(Hg*Wg/C) connected regions per frame whose
    sizes differ by at most one; .choice = (transposed, bands, perimeter of one frame)."""
    R = lib().orc_plan_balanced(_i(T), _i(Hg), _i(Wg), _i(C), None, None, None)
    st = np.empty((R, C), np.int32)
    nv = np.empty((R,), np.int32)
    choice = (ctypes.c_int64 * 3)()
    lib().orc_plan_balanced(_i(T), _i(Hg), _i(Wg), _i(C), _p(st), _p(nv), choice)
    pl = Plan(T, Hg, Wg, 0, 0, R, C, st, nv, 0, R)
    pl.choice = (int(choice[0]), int(choice[1]), int(choice[2]))
    return pl


# ---------------------------------------------------------------- prefix tokens
# App. C.1: "prefix interactions lie outside the video-region budget": a video query keeps every valid prefix key,
# a prefix query attends to everything.  Readings: the P prefix tokens come first in the token order, followed by the
# video tokens in raster order; prefix tokens form ceil(P/S) blocks of S consecutive tokens that follow the video
# regions in the block numbering; prefix interactions run in the 16-bit tier (they are "retained prefix
# interactions" of a precision set, Sec. 3.2, and no lower format is named for them), i.e. last in the phase order.
def plan_with_prefix(pl: Plan, P: int) -> Plan:
    """Block table of the joint sequence [P prefix tokens | video tokens]: video regions (token ids shifted by P),
    then the prefix blocks."""
    assert pl.n_prefix == 0
    if P == 0:
        return Plan(pl.T, pl.Hg, pl.Wg, pl.th, pl.tw, pl.R, pl.S, pl.slot_token, pl.n_valid, 0, pl.R)
    Rp = -(-P // pl.S)
    st = np.full((pl.R + Rp, pl.S), -1, np.int32)
    st[:pl.R] = np.where(pl.slot_token >= 0, pl.slot_token + P, -1)
    for j in range(Rp):
        toks = np.arange(j * pl.S, min(P, (j + 1) * pl.S), dtype=np.int32)
        st[pl.R + j, :len(toks)] = toks
    nv = (st >= 0).sum(1).astype(np.int32)
    return Plan(pl.T, pl.Hg, pl.Wg, pl.th, pl.tw, pl.R + Rp, pl.S, st, nv, P, pl.R)


def lists_with_prefix(ids: np.ndarray, counts: np.ndarray, R: int, Rp: int):
    """Lists of the joint sequence from the ranked video lists ids [BH,R,*], counts [BH,R,3]: every video row gets
    all prefix blocks appended to its 16-bit segment, every prefix row keeps all blocks in the 16-bit tier."""
    BH = ids.shape[0]
    Rt = R + Rp
    out = np.full((BH, Rt, Rt), -1, np.int32)
    cnt = np.zeros((BH, Rt, 3), np.int32)
    pre = np.arange(R, Rt, dtype=np.int32)
    for h in range(BH):
        for a in range(R):
            n = int(counts[h, a].sum())
            out[h, a, :n] = ids[h, a, :n]
            out[h, a, n:n + Rp] = pre
            cnt[h, a] = counts[h, a] + np.array([0, 0, Rp], np.int32)
        for a in range(R, Rt):
            out[h, a] = np.arange(Rt, dtype=np.int32)
            cnt[h, a] = (0, 0, Rt)
    return out, cnt


def pad_operands(ops: "Operands", Rt: int) -> "Operands":
    """Per-block operand arrays padded with empty entries for the prefix blocks (which only ever run in the 16-bit
    tier and therefore have no quantised operands)."""
    def pad(x):
        if x.ndim < 2 or x.shape[1] == Rt:
            return x
        shape = list(x.shape)
        shape[1] = Rt - x.shape[1]
        return np.ascontiguousarray(np.concatenate([x, np.zeros(shape, x.dtype)], 1))
    keep = {"dv8", "gq", "gk", "gv"}   # per head (and channel), not per block
    return Operands(**{k: (v if k in keep else pad(v)) for k, v in ops.__dict__.items()})


def quotas(f16: float, f8: float, f4: float, M: int):
    out = (ctypes.c_int64 * 3)()
    lib().orc_quotas(_d(f16), _d(f8), _d(f4), _i64(M), out)
    return int(out[0]), int(out[1]), int(out[2])


# ----------------------------------------------------------------- pool/draft
def pool(x: np.ndarray, pl: Plan):
    """x: uint16 bf16 bits [BH, N, d] -> (avg, max) fp32 [BH, R, d]."""
    BH, N, d = x.shape
    avg = np.empty((BH, pl.R, d), np.float32)
    mx = np.empty((BH, pl.R, d), np.float32)
    lib().orc_pool(_p(x), _i64(BH), _i64(N), _i(d), _i(pl.R), _i(pl.S), _p(pl.slot_token), _p(avg), _p(mx))
    return avg, mx


def draft(qavg, qmax, kavg, kmax, lam: float, scale: float) -> np.ndarray:
    BH, R, d = qavg.shape
    A = np.empty((BH, R, R), np.float32)
    lib().orc_draft(_p(qavg), _p(qmax), _p(kavg), _p(kmax), _i64(BH), _i(R), _i(d), _d(lam), _d(scale), _p(A))
    return A


def rank_row(A: np.ndarray, k16: int, k8: int, k4: int) -> np.ndarray:
    BH, R, _ = A.shape
    tags = np.empty((BH, R, R), np.uint8)
    lib().orc_rank_row(_p(A), _i64(BH), _i(R), _i64(k16), _i64(k8), _i64(k4), _p(tags))
    return tags


def rank_head(A: np.ndarray, T16: int, T8: int, T4: int) -> np.ndarray:
    BH, R, _ = A.shape
    tags = np.empty((BH, R, R), np.uint8)
    lib().orc_rank_head(_p(A), _i64(BH), _i(R), _i64(T16), _i64(T8), _i64(T4), _p(tags))
    return tags


def lists(tags: np.ndarray, stride: Optional[int] = None):
    """tags uint8 [BH,R,R] -> ids int32 [BH,R,stride] (4-bit | 8-bit | 16-bit, ascending), counts [BH,R,3]."""
    BH, R, _ = tags.shape
    stride = R if stride is None else stride
    ids = np.empty((BH, R, stride), np.int32)
    counts = np.empty((BH, R, 3), np.int32)
    lib().orc_lists(_p(tags), _i64(BH * R), _i(R), _i(stride), _p(ids), _p(counts))
    return ids, counts


# ------------------------------------------------------------------ quantisers
def quant_int8(x: np.ndarray, pl: Plan):
    BH, N, d = x.shape
    codes = np.empty((BH, pl.R, pl.S, d), np.int8)
    delta = np.empty((BH, pl.R), np.float32)
    lib().orc_quant_int8(_p(x), _i64(BH), _i64(N), _i(d), _i(pl.R), _i(pl.S), _p(pl.slot_token), _p(codes), _p(delta))
    return codes, delta


def quant_v_e4m3(v: np.ndarray, pl: Plan):
    BH, N, d = v.shape
    codes = np.empty((BH, pl.R, pl.S, d), np.uint8)
    delta_c = np.empty((BH, d), np.float32)
    lib().orc_quant_v_e4m3(_p(v), _i64(BH), _i64(N), _i(d), _i(pl.R), _i(pl.S), _p(pl.slot_token), _p(codes),
                           _p(delta_c))
    return codes, delta_c


def quant_v_e4m3_given(v: np.ndarray, pl: Plan, delta_c: np.ndarray) -> np.ndarray:
    """E4M3 codes of V under a given per-(head, channel) scale delta_c [BH, d] (0 = channel skipped)."""
    BH, N, d = v.shape
    codes = np.empty((BH, pl.R, pl.S, d), np.uint8)
    dc = np.ascontiguousarray(delta_c, np.float32)
    lib().orc_quant_v_e4m3_given(_p(v), _i64(BH), _i64(N), _i(d), _i(pl.R), _i(pl.S), _p(pl.slot_token), _p(dc),
                                 _p(codes))
    return codes


def nvfp4_global_scale(x: np.ndarray) -> np.ndarray:
    BH, N, d = x.shape
    g = np.empty((BH,), np.float32)
    lib().orc_nvfp4_global_scale(_p(x), _i64(BH), _i64(N), _i(d), _p(g))
    return g


def quant_nvfp4_qk(x: np.ndarray, pl: Plan, g: np.ndarray):
    BH, N, d = x.shape
    codes = np.empty((BH, pl.R, pl.S, d), np.uint8)
    sf = np.empty((BH, pl.R, pl.S, d // 16), np.uint8)
    lib().orc_quant_nvfp4_qk(_p(x), _i64(BH), _i64(N), _i(d), _i(pl.R), _i(pl.S), _p(pl.slot_token), _p(g),
                             _p(codes), _p(sf))
    return codes, sf


def quant_nvfp4_v(v: np.ndarray, pl: Plan, g: np.ndarray):
    BH, N, d = v.shape
    codes = np.empty((BH, pl.R, pl.S, d), np.uint8)
    sf = np.empty((BH, pl.R, pl.S // 16, d), np.uint8)
    lib().orc_quant_nvfp4_v(_p(v), _i64(BH), _i64(N), _i(d), _i(pl.R), _i(pl.S), _p(pl.slot_token), _p(g),
                            _p(codes), _p(sf))
    return codes, sf


@dataclass
class Operands:
    """Every quantised operand set of one (Q, K, V) triple, in logical block order."""
    q8: np.ndarray
    k8: np.ndarray
    dq8: np.ndarray
    dk8: np.ndarray
    v8: np.ndarray
    dv8: np.ndarray
    q4: np.ndarray
    k4: np.ndarray
    v4: np.ndarray
    sfq: np.ndarray
    sfk: np.ndarray
    sfv: np.ndarray
    gq: np.ndarray
    gk: np.ndarray
    gv: np.ndarray


def quantize_all(q: np.ndarray, k: np.ndarray, v: np.ndarray, pl: Plan) -> Operands:
    q8, dq8 = quant_int8(q, pl)
    k8, dk8 = quant_int8(k, pl)
    v8, dv8 = quant_v_e4m3(v, pl)
    gq, gk, gv = nvfp4_global_scale(q), nvfp4_global_scale(k), nvfp4_global_scale(v)
    q4, sfq = quant_nvfp4_qk(q, pl, gq)
    k4, sfk = quant_nvfp4_qk(k, pl, gk)
    v4, sfv = quant_nvfp4_v(v, pl, gv)
    return Operands(q8, k8, dq8, dk8, v8, dv8, q4, k4, v4, sfq, sfk, sfv, gq, gk, gv)


# ------------------------------------------------------------------- attention
def _attn_common(q, k, v, pl, ids, counts, ops: Optional[Operands]):
    BH, N, d = q.shape
    ids2 = np.ascontiguousarray(ids.reshape(BH * pl.R, -1), np.int32)
    cnt2 = np.ascontiguousarray(counts.reshape(BH * pl.R, 3), np.int32)
    o = ops
    g = lambda name: _p(getattr(o, name)) if o is not None else None
    args = [_p(q), _p(k), _p(v), _i64(BH), _i64(N), _i(d), _i(pl.R), _i(pl.S), _p(pl.slot_token), _p(ids2),
            _p(cnt2), _i(ids2.shape[1]), g("q8"), g("k8"), g("dq8"), g("dk8"), g("v8"), g("dv8"), g("q4"),
            g("k4"), g("v4"), g("sfq"), g("sfk"), g("sfv"), g("gq"), g("gk"), g("gv")]
    return args, (ids2, cnt2)


def attention(q, k, v, pl: Plan, ids, counts, ops: Optional[Operands], scale: float,
              sel: Sequence[Sequence[int]], encoded_units: bool = False) -> np.ndarray:
    """Phased mixed-precision attention for query blocks sel=[(bh, a), ...] -> fp32 [nsel, S, d]."""
    args, keep = _attn_common(q, k, v, pl, ids, counts, ops)
    sel_a = np.ascontiguousarray(np.asarray(sel, np.int32).reshape(-1, 2))
    out = np.zeros((sel_a.shape[0], pl.S, q.shape[2]), np.float32)
    lib().orc_attention(*args, _d(scale), _i(1 if encoded_units else 0), _p(sel_a), _i(sel_a.shape[0]), _p(out))
    return out


def attention_row_debug(q, k, v, pl: Plan, ids, counts, ops: Optional[Operands], scale: float,
                        bh: int, a: int, ju: int):
    args, keep = _attn_common(q, k, v, pl, ids, counts, ops)
    N, d = q.shape[1], q.shape[2]
    out = np.zeros((d,), np.float32)
    shat = np.empty((N,), np.float64)
    h_at = np.empty((N,), np.float64)
    what = np.empty((N,), np.float64)
    vhat = np.zeros((N, d), np.float64)
    tier = np.empty((N,), np.int32)
    hf = np.zeros((1,), np.float64)
    ell = np.zeros((1,), np.float64)
    lib().orc_attention_row_debug(*args, _d(scale), _i64(bh), _i(a), _i(ju), _p(out), _p(shat), _p(h_at), _p(what),
                                  _p(vhat), _p(tier), _p(hf), _p(ell))
    return dict(out=out, shat=shat, h_at=h_at, what=what, vhat=vhat, tier=tier, h_final=float(hf[0]),
                ell=float(ell[0]))


def dense(q, k, v, pl: Plan, scale: float, sel: Sequence[Sequence[int]]) -> np.ndarray:
    """fp64 dense softmax attention for the query tokens of blocks sel -> fp64 [nsel, S, d]."""
    BH, N, d = q.shape
    sel_a = np.ascontiguousarray(np.asarray(sel, np.int32).reshape(-1, 2))
    out = np.zeros((sel_a.shape[0], pl.S, d), np.float64)
    lib().orc_dense(_p(q), _p(k), _p(v), _i64(BH), _i64(N), _i(d), _i(pl.S), _p(pl.slot_token), _d(scale),
                    _p(sel_a), _i(sel_a.shape[0]), _p(out))
    return out


def run_pipeline(q, k, v, pl: Plan, *, lam: float, scale: float, frac16: float, frac8: float, frac4: float,
                 head_scope: bool = False):
    """Pool -> draft -> rank -> lists for bf16-bit arrays q,k [BH,N,d]. Returns dict of every stage."""
    qavg, qmax = pool(q, pl)
    kavg, kmax = pool(k, pl)
    A = draft(qavg, qmax, kavg, kmax, lam, scale)
    if head_scope:
        t16, t8, t4 = quotas(frac16, frac8, frac4, pl.R * pl.R)
        tags = rank_head(A, t16, t8, t4)
    else:
        t16, t8, t4 = quotas(frac16, frac8, frac4, pl.R)
        tags = rank_row(A, t16, t8, t4)
    ids, counts = lists(tags)
    return dict(qavg=qavg, qmax=qmax, kavg=kavg, kmax=kmax, A=A, tags=tags, ids=ids, counts=counts,
                quotas=(t16, t8, t4))
