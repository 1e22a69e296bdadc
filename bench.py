#!/usr/bin/env python
"""Benchmark of the da2 hot path: one step = da2_prepare (pool, draft map, ranking, operand records) +
da2_attention_fwd (phased mixed-precision block-sparse attention) over one batch of synthetic Q/K/V.

    python bench.py --gpus 1 --steps 5 --warmup 3            # this implementation
    python bench.py --impl reference --steps 1 --warmup 0    # the CPU oracle on the host cores (bounded sample)

Prints ONE JSON line (rank 0).  value = dense-equivalent TFLOP/s of the whole call (4*N^2*d*B*H flops of dense
attention divided by the time of one step), inputs resident in HBM; e2e = the same through the C ABI with host
buffers (pinned H2D of Q, K, V and D2H of the output inside the timed region).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import da2_inputs

NOMINAL_RATIO = {0: 4.0, 1: 2.0, 2: 1.0}  # dense tensor peak relative to bf16: NVFP4, 8-bit, bf16
METRIC = "dense-equivalent TFLOP/s per attention call (draft + operand prep + phased attention)"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16=p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                    bf16_burst=p["bf16_tflops"], source="measured")
    return dict(hbm_gbs=6650.0, bf16=1400.0, bf16_burst=1590.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "200"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in self.rows if len(r) >= 6 for n, v in zip(names, r[2:6]) if v.lower() == "active"})
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def flop_counts(w, plan, ws):
    """Dense-equivalent flops, and per-tier flops of the retained block pairs: padded (64 x 64 tokens per pair) and
    valid-token counts, from the lists the prepare step wrote (accounting only, uses torch ops)."""
    I = plan.info
    BH, R, d = w.B * w.H, I.R, w.head_dim
    dense = 4.0 * w.N * w.N * d * BH
    cnt = ws[I.off_counts:I.off_counts + BH * R * 16].view(torch.int32).view(BH, R, 4).long()
    padded = [float(cnt[:, :, t].sum().item()) * 4 * 64 * 64 * d for t in range(3)]
    # valid tokens per block
    if I.partition == 0:
        nty, ntx = I.nty, I.ntx
        vr = torch.tensor([min(8, w.Hg - 8 * ty) for ty in range(nty)], device=ws.device)
        vc = torch.tensor([min(8, w.Wg - 8 * tx) for tx in range(ntx)], device=ws.device)
        nv = (vr[:, None] * vc[None, :]).reshape(-1).repeat(w.T).double()  # [R]
    else:   # balanced ragged partition: region r of a frame holds part_n + (r < part_rem) tokens
        nv = (I.part_n + (torch.arange(I.R_f, device=ws.device) < I.part_rem).long()).repeat(w.T).double()
    valid = [0.0, 0.0, 0.0]
    if I.rank_scope == 0:
        stride = int(I.ids_per_head) // R
        ids = ws[I.off_ids:I.off_ids + BH * int(I.ids_per_head) * 2].view(torch.int16).view(BH, R, stride)
        ids = ids.long() & 0xffff
        k4, k8, k16 = (int(x) for x in I.quota)
        lo = 0
        for t, n in enumerate((k4, k8, k16)):
            if n:
                keys = nv[ids[:, :, lo:lo + n]].sum(-1)           # [BH, R]
                valid[t] = float((keys * nv[None, :]).sum().item()) * 4 * d
            lo += n
    else:
        # head-level budget: rows of unequal length; entry e of row a sits at ids[head][offset_a + e]
        per_head = int(I.ids_per_head)
        ids_all = (ws[I.off_ids:I.off_ids + BH * per_head * 2].view(torch.int16).view(BH, per_head).long()) & 0xffff
        rows = torch.arange(R, device=ws.device)
        for h in range(BH):
            n3, off = cnt[h, :, :3], cnt[h, :, 3]
            n = n3.sum(-1)
            total = int(n.sum().item())
            if total == 0:
                continue
            row_of = torch.repeat_interleave(rows, n)
            start = torch.repeat_interleave(torch.cumsum(n, 0) - n, n)
            within = torch.arange(total, device=ws.device) - start
            key = ids_all[h, torch.repeat_interleave(off, n) + within]
            tier = (within >= torch.repeat_interleave(n3[:, 0], n)).long() + \
                   (within >= torch.repeat_interleave(n3[:, 0] + n3[:, 1], n)).long()
            pair = nv[row_of] * nv[key]
            for t in range(3):
                valid[t] += float(pair[tier == t].sum().item()) * 4 * d
    return dense, padded, valid


MMA_KINDS = ("bf16", "int8", "e4m3", "nvfp4")
MMA_K = (16, 32, 32, 64)


def mma_peaks(iters: int = 4000):
    """tcgen05.mma microbenchmark on every SM: TFLOP/s and cycles per instruction per kind at M = 128 and
    N = 64, 128, 256 (operands in shared memory)."""
    import paper_2609_32628_b200 as da2
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    out = torch.zeros(4, dtype=torch.int64, device=dev)
    rows = []
    for kind, name in enumerate(MMA_KINDS):
        for n in (64, 128, 256):
            for _ in range(2):
                da2.da2_tcgen05_peak(kind, n, iters, sms, out)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            da2.da2_tcgen05_peak(kind, n, iters, sms, out)
            e1.record()
            torch.cuda.synchronize()
            cyc, instr, fail = (int(x) for x in out[:3].tolist())
            assert fail == 0, "the microbenchmark's bounded wait gave up"
            ms = e0.elapsed_time(e1)
            flops = 2.0 * 128 * n * MMA_K[kind] * instr * sms
            rows.append({"kind": name, "n": n, "tflops": flops / (ms * 1e-3) / 1e12, "cycles_per_mma": cyc / instr,
                         "ms": ms})
    return {"sms": sms, "iters": iters, "rows": rows}


def sweep(steps: int = 5, warmup: int = 3):
    """The budget sweep: five grids (8k to 131k tokens, 24 heads, d = 128) x high tier {0, 5, 10, 20} % (8-bit) x low
    tier {0, 20, 40, 60} % (NVFP4) without the empty 0/0 point, plus the two dense endpoints (every block 8-bit, every
    block bf16) per grid.  Each point is timed as a full call (da2_prepare + da2_attention_fwd), one JSON line each."""
    import paper_2609_32628_b200 as da2
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = measured_peaks()
    for gi in range(len(da2_inputs.SWEEP_GRIDS)):
        points = [(h, l, False) for h in (0.0, 0.05, 0.10, 0.20) for l in (0.0, 0.20, 0.40, 0.60) if h + l > 0]
        points += [(1.0, 0.0, False), (1.0, 0.0, True)]
        base = da2_inputs.sweep_workload(gi, 0.05, 0.20)
        q, k, v = da2_inputs.make_qkv(base, dev)
        out = torch.empty_like(q)
        for high, low, bf16 in points:
            w = da2_inputs.sweep_workload(gi, high, low, high_is_bf16=bf16)
            plan = da2.da2_plan(w.B, w.H, w.T, w.Hg, w.Wg, w.head_dim, w.frac16, w.frac8, w.frac4, lam=w.lam)
            ws = torch.empty(int(plan.info.workspace_bytes), dtype=torch.uint8, device=dev)
            for _ in range(warmup):
                da2.da2_prepare(plan, q, k, v, ws)
                da2.da2_attention_fwd(plan, q, k, v, ws, out)
            torch.cuda.synchronize()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * steps + 1)]
            ev[0].record()
            for i in range(steps):
                da2.da2_prepare(plan, q, k, v, ws)
                ev[2 * i + 1].record()
                da2.da2_attention_fwd(plan, q, k, v, ws, out)
                ev[2 * i + 2].record()
            torch.cuda.synchronize()
            assert da2.da2_device_status(plan, ws) == 0
            ms = ev[0].elapsed_time(ev[-1]) / steps
            attn = float(np.mean([ev[2 * i + 1].elapsed_time(ev[2 * i + 2]) for i in range(steps)]))
            dense, padded, valid = flop_counts(w, plan, ws)
            t_roof = sum(valid[t] / (peaks["bf16"] * 1e12 * NOMINAL_RATIO[t]) for t in range(3)) * 1e3
            print(json.dumps({"grid": [w.T, w.Hg, w.Wg], "tokens": w.N, "high": high, "low": low,
                              "high_tier": "bf16" if bf16 else "8-bit", "ms_call": ms, "ms_attention": attn,
                              "dense_equiv_tflops": dense / (ms * 1e-3) / 1e12,
                              "frac_of_measured_roofline": t_roof / attn if attn > 0 else None}), flush=True)
            del ws, plan
        del q, k, v, out
        torch.cuda.empty_cache()


def microbench_peaks():
    """Per-kind tensor peaks (TFLOP/s, best N) from the committed microbenchmark summary, or None."""
    path = os.path.join(ROOT, "profiles", "tcgen05_mma_peaks.md")
    if not os.path.exists(path):
        return None
    best = {}
    for ln in open(path):
        if ln.startswith("kind="):
            f = dict(x.split("=") for x in ln.split())
            best[f["kind"]] = max(best.get(f["kind"], 0.0), float(f["tflops"]))
    return best or None


def rank_workload(name: str, rank: int):
    """Weak scaling: every rank runs the whole named workload on its own batch element (heads and batch elements never
    mix on this path, so there is no collective); only the input seed differs per rank."""
    base = da2_inputs.WORKLOADS[name]
    return da2_inputs.Workload(**{**base.__dict__, "seed": base.seed + 1000 * rank})


def max_over_ranks(value: float, world: int, device) -> float:
    """Step time of the job = the slowest rank's."""
    if world <= 1:
        return float(value)
    t = torch.tensor([value], device=device, dtype=torch.float64)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def run_da2(args, rank, world, local_rank):
    import paper_2609_32628_b200 as da2
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    w = rank_workload(args.workload, rank)
    q, k, v = da2_inputs.make_qkv(w, dev)
    plan = da2.da2_plan(w.B, w.H, w.T, w.Hg, w.Wg, w.head_dim, w.frac16, w.frac8, w.frac4, lam=w.lam,
                        rank_scope=args.rank_scope, partition=args.partition)
    ws = torch.empty(int(plan.info.workspace_bytes), dtype=torch.uint8, device=dev)
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream()

    def step():
        da2.da2_prepare(plan, q, k, v, ws, stream)
        n1 = da2.da2_last_launch_count(plan)
        da2.da2_attention_fwd(plan, q, k, v, ws, out, stream)
        return n1 + da2.da2_last_launch_count(plan)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    assert da2.da2_device_status(plan, ws) == 0, "device status after warm-up"
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    launches = 0
    barrier()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for s in range(args.steps):
        ev[s][0].record(stream)
        da2.da2_prepare(plan, q, k, v, ws, stream)
        launches += da2.da2_last_launch_count(plan)
        ev[s][1].record(stream)
        da2.da2_attention_fwd(plan, q, k, v, ws, out, stream)
        launches += da2.da2_last_launch_count(plan)
        ev[s][2].record(stream)
    t1.record(stream)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = t0.elapsed_time(t1)
    prep_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    attn_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]))
    assert da2.da2_device_status(plan, ws) == 0, "device status after the timed region"
    ms_per_step = max_over_ranks(total_ms / args.steps, world, dev)
    # the single-pass preparation (scales carried over from the call above), reported beside the two-pass one
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    da2.da2_prepare_cached_scales(plan, q, k, v, ws, True, stream)
    c0.record(stream)
    for _ in range(3):
        da2.da2_prepare_cached_scales(plan, q, k, v, ws, True, stream)
    c1.record(stream)
    torch.cuda.synchronize()
    prep_cached_ms = c0.elapsed_time(c1) / 3

    # ---- end to end through the public API with pinned HOST buffers: every step copies Q, K, V to the device and the
    # output back.  Two ways: one call for all heads (copies and kernels in series on one stream), and the library's
    # HostPipeline (groups of heads through three streams, so that the copies hide behind the kernels).
    hq, hk, hv = (x.cpu().pin_memory() for x in (q, k, v))
    hout = torch.empty_like(hq).pin_memory()
    dq, dk, dv = (torch.empty_like(x) for x in (q, k, v))
    e2e_steps = max(1, min(args.steps, 3))

    def serial_step():
        dq.copy_(hq, non_blocking=True)
        dk.copy_(hk, non_blocking=True)
        dv.copy_(hv, non_blocking=True)
        da2.da2_prepare(plan, dq, dk, dv, ws, stream)
        da2.da2_attention_fwd(plan, dq, dk, dv, ws, out, stream)
        hout.copy_(out, non_blocking=True)

    def timed(step_fn):
        step_fn()
        barrier()
        a0 = torch.cuda.Event(enable_timing=True)
        a1 = torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        for _ in range(e2e_steps):
            step_fn()
        a1.record(stream)
        barrier()
        return max_over_ranks(a0.elapsed_time(a1) / e2e_steps, world, dev)

    e2e_serial_ms = timed(serial_step)
    del dq, dk, dv
    pipe = da2.HostPipeline(w.B, w.H, w.T, w.Hg, w.Wg, w.head_dim, w.frac16, w.frac8, w.frac4, lam=w.lam,
                            rank_scope=args.rank_scope, groups="ramp", device=dev, partition=args.partition)
    groups = [b - a for a, b in pipe.ranges]
    e2e_ms = timed(lambda: pipe.run(hq, hk, hv, hout))
    assert pipe.status() == 0, "device status after the end-to-end region"
    e2e_launches = pipe.launches
    del pipe
    torch.cuda.empty_cache()
    # the same pipeline inside the C ABI (da2_attention_host: synchronous, so timed on the host clock)
    cfg = da2.make_config(w.B, w.H, w.T, w.Hg, w.Wg, w.head_dim, w.frac16, w.frac8, w.frac4, lam=w.lam,
                          rank_scope=args.rank_scope, partition=args.partition)
    arena = torch.empty(da2.da2_attention_host_arena_bytes(cfg), dtype=torch.uint8, device=dev)
    da2.da2_attention_host(cfg, hq, hk, hv, hout, arena)
    barrier()
    tc0 = time.perf_counter()
    for _ in range(e2e_steps):
        da2.da2_attention_host(cfg, hq, hk, hv, hout, arena)
    e2e_c_ms = max_over_ranks((time.perf_counter() - tc0) * 1e3 / e2e_steps, world, dev)
    del arena
    if rank != 0:
        return None

    dense, padded, valid = flop_counts(w, plan, ws)
    peaks = measured_peaks()
    t_roof_ms = sum(valid[t] / (peaks["bf16"] * 1e12 * NOMINAL_RATIO[t]) for t in range(3)) * 1e3
    t_roof_nominal_ms = sum(padded[t] / (2.25e15 * NOMINAL_RATIO[t]) for t in range(3)) * 1e3
    total_valid = sum(valid)
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "attention_kernel_dram_traffic.txt")
    if os.path.exists(tpath):
        for ln in open(tpath):
            if ln.startswith("workload=" + args.workload + " "):
                traffic = int(ln.split("dram_bytes_per_launch=")[1].split()[0])
    roofline = {
        "kernel": "attention_kernel (da2_attention_fwd)", "bound": "tensor",
        "achieved": total_valid / (attn_ms * 1e-3) / 1e12,
        "peak": total_valid / (t_roof_ms * 1e-3) / 1e12 if t_roof_ms > 0 else None,
        "unit": "TFLOP/s", "frac": t_roof_ms / attn_ms if attn_ms > 0 else None, "traffic": traffic,
        "peak_source": f"{peaks['source']} bf16 sustained {peaks['bf16']} TFLOP/s x nominal ratio per dtype "
                       "(8-bit x2, NVFP4 x4), mixed by the phases' valid-token flops",
        "ms_kernel": attn_ms, "ms_roofline": t_roof_ms,
        "flops_valid": {"nvfp4": valid[0], "int8_e4m3": valid[1], "bf16": valid[2]},
        "flops_padded": {"nvfp4": padded[0], "int8_e4m3": padded[1], "bf16": padded[2]},
        "frac_of_nominal_padded": t_roof_nominal_ms / attn_ms if attn_ms > 0 else None,
        "frac_of_nominal_valid": sum(valid[t] / (2.25e15 * NOMINAL_RATIO[t]) for t in range(3)) * 1e3 / attn_ms
                                 if attn_ms > 0 else None,
        "ms_prepare": prep_ms, "ms_prepare_cached_scales": prep_cached_ms,
    }
    mb = microbench_peaks()
    if mb and attn_ms > 0:
        # this GPU's own tcgen05 peaks per kind (best tile shape of the committed microbenchmark); the 8-bit tier is
        # half INT8 (scores) and half E4M3 (values)
        t_mb = (valid[0] / (mb["nvfp4"] * 1e12) + valid[1] * 0.5 / (mb["int8"] * 1e12) +
                valid[1] * 0.5 / (mb["e4m3"] * 1e12) + valid[2] / (mb["bf16"] * 1e12)) * 1e3
        roofline["frac_of_microbenchmark_peaks"] = t_mb / attn_ms
        roofline["microbenchmark_peaks_tflops"] = mb
    line = {
        "metric": METRIC, "value": dense * world / (ms_per_step * 1e-3) / 1e12, "unit": "TFLOP/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "nvfp4+int8/e4m3+bf16 (fp32 softmax)",
        "data": "synthetic",
        "config": {"workload": args.workload, "B": w.B * world, "H": w.H, "head_dim": w.head_dim,
                   "grid": [w.T, w.Hg, w.Wg], "tokens": w.N, "budget_16_8_4": [w.frac16, w.frac8, w.frac4],
                   "rank_scope": "row" if args.rank_scope == 0 else "head",
                   "partition": "8x8 tiles" if args.partition == 0 else "balanced ragged, capacity 64",
                   "l2": "inputs larger than L2 (Q, K, V and operand records are several GB per step)"},
        "e2e": {"value": dense * world / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": 3 * q.numel() * 2, "d2h_bytes_per_step": out.numel() * 2,
                "how": f"HostPipeline: groups of {groups} heads, copy-in, copy-out and two alternating compute streams, "
                       f"{e2e_launches} kernels per step",
                "c_abi_host_entry_ms_per_step": e2e_c_ms,
                "serial_ms_per_step": e2e_serial_ms,
                "serial_value": dense * world / (e2e_serial_ms * 1e-3) / 1e12},
        "gpu_launches": launches, "clocks": clocks, "roofline": roofline,
    }
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(args.workload, args.rank_scope, nblocks=args.cpu_blocks)
    return line


def cpu_baseline(workload: str, rank_scope: int = 0, nblocks: int = 16):
    """The oracle, as it stands, on the host cores: one head through every stage before attention, plus the
    attention of a few query blocks; scaled to the whole call by heads and by query blocks."""
    import oracle
    w = da2_inputs.WORKLOADS[workload]
    q, k, v = da2_inputs.make_qkv(w, "cpu", heads=[0])
    bits = lambda t: oracle.bf16_bits(t.reshape(-1, w.N, w.head_dim))
    qb, kb, vb = bits(q), bits(k), bits(v)
    scale = float(np.float32(1.0) / np.sqrt(np.float32(w.head_dim)))
    t0 = time.perf_counter()
    pl = oracle.plan(w.T, w.Hg, w.Wg)
    r = oracle.run_pipeline(qb, kb, vb, pl, lam=float(np.float32(w.lam)), scale=scale, frac16=w.frac16,
                            frac8=w.frac8, frac4=w.frac4, head_scope=bool(rank_scope))
    ops = oracle.quantize_all(qb, kb, vb, pl)
    t1 = time.perf_counter()
    rng = np.random.default_rng(0)
    blocks = sorted(rng.choice(pl.R, min(nblocks, pl.R), replace=False).tolist())
    oracle.attention(qb, kb, vb, pl, r["ids"], r["counts"], ops, scale, [(0, a) for a in blocks])
    t2 = time.perf_counter()
    BH = w.B * w.H
    est = (t1 - t0) * BH + (t2 - t1) / len(blocks) * pl.R * BH
    dense = 4.0 * w.N * w.N * w.head_dim * BH
    return {"value": dense / est / 1e12, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle",
            "sample": f"1 of {BH} heads through pool/draft/rank/quantise ({t1 - t0:.2f} s) + attention of "
                      f"{len(blocks)} of {pl.R} query blocks of that head ({t2 - t1:.2f} s); scaled by heads and "
                      f"query blocks to an estimated {est:.0f} s per call",
            "seconds_measured": t2 - t0, "seconds_per_call_estimated": est}


def run_reference(args):
    """The reference arm of this benchmark is the CPU oracle on the host cores (there is no other implementation of
    the method to run): each step is a bounded sample of the workload, scaled to the whole call."""
    vals = []
    for _ in range(args.warmup):
        cpu_baseline(args.workload, args.rank_scope, nblocks=max(2, args.cpu_blocks // 4))
    last = None
    for _ in range(max(1, args.steps)):
        last = cpu_baseline(args.workload, args.rank_scope, nblocks=args.cpu_blocks)
        vals.append(last["value"])
    w = da2_inputs.WORKLOADS[args.workload]
    value = float(np.mean(vals))
    est_ms = last["seconds_per_call_estimated"] * 1e3
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": est_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64 (fp32 where the formats fix it)", "data": "synthetic",
        "config": {"workload": args.workload, "B": w.B, "H": w.H, "head_dim": w.head_dim,
                   "grid": [w.T, w.Hg, w.Wg], "tokens": w.N, "budget_16_8_4": [w.frac16, w.frac8, w.frac4],
                   "rank_scope": "row" if args.rank_scope == 0 else "head"},
        "cpu_baseline": {**last, "value": value},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="da2", choices=["da2", "reference"])
    ap.add_argument("--workload", default="wan14b_720p", choices=sorted(da2_inputs.WORKLOADS))
    ap.add_argument("--rank-scope", type=int, default=0, choices=[0, 1])
    ap.add_argument("--partition", type=int, default=0, choices=[0, 1],
                    help="0: fixed 8x8 tiles (the benchmark configurations); 1: balanced ragged partition (App. C.2)")
    ap.add_argument("--cpu-blocks", type=int, default=16)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--mma-peaks", action="store_true",
                    help="run the tcgen05.mma microbenchmark (per-kind tensor peaks) instead of the benchmark")
    ap.add_argument("--sweep", action="store_true",
                    help="time every point of the budget sweep (one JSON line per point) instead of the benchmark")
    args = ap.parse_args()
    if args.sweep:
        sweep(args.steps, max(3, args.warmup))
        return
    if args.mma_peaks:
        res = mma_peaks()
        for r in res["rows"]:
            print(f"kind={r['kind']} n={r['n']} tflops={r['tflops']:.1f} cycles_per_mma={r['cycles_per_mma']:.1f}")
        print(json.dumps(res))
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "da2":
        # started as a plain script: launch the N ranks (one process per GPU) and let rank 0 print the line
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)))
        return
    if args.warmup < 3:
        args.warmup = 3
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        line = run_da2(args, rank, world, local_rank)
        if rank == 0:
            print(json.dumps(line))
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
