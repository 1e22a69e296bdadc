"""Operator-level ablations on synthetic inputs: error against dense attention and latency of the call for a grid of
precision budgets and draft-map mixing weights (the shape of the paper's budget / lambda studies, Sec. 4 and Fig. 5,
without its models or datasets).

    python ablation.py [--grid T,Hg,Wg] [--heads H] [--blocks 8] [--steps 3]

A report script beside bench.py, not part of the library.  Every line is one configuration run through da2_prepare +
da2_attention_fwd on cuda:0.  The error is the relative L2 distance to dense softmax attention written out as its
definition with fp64 PyTorch matmuls, for a sample of query blocks of every head.  Prints a markdown table.
"""
from __future__ import annotations

import argparse
import math
import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
import da2_inputs  # noqa: E402
from paper_2609_32628_b200 import binding as da2  # noqa: E402

BUDGETS = (  # (share of 16-bit, 8-bit, 4-bit key blocks per query-block row)
    (1.0, 0.0, 0.0), (0.0, 1.0, 0.0), (0.0, 0.0, 1.0),          # dense endpoints of each format
    (0.6, 0.0, 0.0), (0.0, 0.6, 0.0), (0.0, 0.0, 0.6),          # one format, 60 % of the blocks
    (0.2, 0.4, 0.0), (0.0, 0.2, 0.4), (0.1, 0.2, 0.3),          # two and three simultaneous tiers, 60 %
    (0.0, 0.1, 0.4), (0.0, 0.05, 0.2), (0.05, 0.1, 0.15),       # sparser calls
)
LAMBDAS = (0.0, 0.2, 0.5, 1.0)  # weight of the max-pooled branch in the draft map (0: average branch only)


def dense_rows(q, k, v, rows, scale):
    """softmax(q_rows k^T * scale) v for token index tensor `rows` [n] of every head; fp64, head by head."""
    out = []
    for h in range(q.shape[1]):
        s = (q[0, h, rows].double() @ k[0, h].double().t()) * scale
        out.append(torch.softmax(s, dim=-1) @ v[0, h].double())
    return torch.stack(out).float()


def block_tokens(w, blocks):
    """Raster token indices of the given 8 x 8 spatial blocks (frame-major block numbering), ragged edges clipped."""
    nty, ntx = (w.Hg + 7) // 8, (w.Wg + 7) // 8
    out = []
    for b in blocks:
        t, r = divmod(b, nty * ntx)
        ty, tx = divmod(r, ntx)
        for y in range(ty * 8, min(ty * 8 + 8, w.Hg)):
            for x in range(tx * 8, min(tx * 8 + 8, w.Wg)):
                out.append((t * w.Hg + y) * w.Wg + x)
    return torch.tensor(out, dtype=torch.long)


def run(w, q, k, v, f16, f8, f4, lam, steps, rows, ref):
    plan = da2.da2_plan(w.B, w.H, w.T, w.Hg, w.Wg, w.head_dim, f16, f8, f4, lam=lam)
    ws = torch.empty(int(plan.info.workspace_bytes), dtype=torch.uint8, device=q.device)
    out = torch.empty_like(q)
    for _ in range(2):
        da2.da2_prepare(plan, q, k, v, ws)
        da2.da2_attention_fwd(plan, q, k, v, ws, out)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        da2.da2_prepare(plan, q, k, v, ws)
        da2.da2_attention_fwd(plan, q, k, v, ws, out)
    e1.record()
    torch.cuda.synchronize()
    if da2.da2_device_status(plan, ws) != 0:
        raise RuntimeError("device status")
    got = out[0, :, rows.to(q.device)].float()
    err = float((got - ref).norm() / ref.norm())
    da2.da2_plan_destroy(plan)
    return err, e0.elapsed_time(e1) / steps


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--grid", default="16,48,48")
    ap.add_argument("--heads", type=int, default=8)
    ap.add_argument("--blocks", type=int, default=8, help="query blocks per head in the error sample")
    ap.add_argument("--steps", type=int, default=3)
    a = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device (there is no CPU path)")
    T, Hg, Wg = (int(x) for x in a.grid.split(","))
    w = da2_inputs.Workload("ablation", 1, a.heads, 128, T, Hg, Wg, 0.0, 0.2, 0.4, seed=7)
    q, k, v = da2_inputs.make_qkv(w, "cuda")
    R = T * ((Hg + 7) // 8) * ((Wg + 7) // 8)
    blocks = [int(i * R / a.blocks + R / (2 * a.blocks)) for i in range(a.blocks)]
    rows = block_tokens(w, blocks)
    scale = 1.0 / math.sqrt(w.head_dim)
    ref = dense_rows(q, k, v, rows.to(q.device), scale)
    print(f"grid {T}x{Hg}x{Wg} = {w.N} tokens, {a.heads} heads, d=128; error on {len(rows)} query rows per head\n")
    print("| 16-bit / 8-bit / 4-bit share | lambda | rel. L2 error vs dense | ms per call |")
    print("|---|---|---|---|")
    for f16, f8, f4 in BUDGETS:
        err, ms = run(w, q, k, v, f16, f8, f4, 0.2, a.steps, rows, ref)
        print(f"| {f16:g} / {f8:g} / {f4:g} | 0.2 | {err:.4f} | {ms:.2f} |")
    for lam in LAMBDAS:
        for f16, f8, f4 in ((0.0, 0.1, 0.4), (0.0, 0.05, 0.2)):
            err, ms = run(w, q, k, v, f16, f8, f4, lam, a.steps, rows, ref)
            print(f"| {f16:g} / {f8:g} / {f4:g} | {lam:g} | {err:.4f} | {ms:.2f} |")


if __name__ == "__main__":
    main()
