"""Seeded synthetic inputs for the DraftAttention2 attention path.

This module holds no arithmetic of the method itself: it only manufactures
Q/K/V tensors and names the workload shapes.  Both the CPU oracle tests and
the CUDA path are fed from here, so the two sides always see the same bits
(generate once on one device, copy to the other).

Recipe (per tensor X in {Q, K, V}, per head and channel): an i.i.d. N(0,1)
field on the T x Hg x Wg latent grid is blurred with a separable Gaussian
(sigma = 2 tokens along t, h and w; taps exp(-k^2/8), radius 8, normalised,
mirrored at the borders), divided by its own population standard deviation,
and 0.5 * N(0,1) i.i.d. noise is added before the cast to bf16.  The result is
spatiotemporally smooth like video-DiT activations, which is what makes 8x8
spatial pooling informative.

Random numbers are counter based: a 64-bit mixing hash of
(seed, tensor id, head, channel, token) feeds Box-Muller, so the values do
not depend on generation order or chunking.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, Tuple

import torch

_MASK64 = (1 << 64) - 1


def _to_i64(v: int) -> int:
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


_C1 = _to_i64(0xBF58476D1CE4E5B9)
_C2 = _to_i64(0x94D049BB133111EB)
_GOLD = 0x9E3779B97F4A7C15


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on int64 tensors (wrapping arithmetic)."""
    x = (x ^ _lsr(x, 30)) * _C1
    x = (x ^ _lsr(x, 27)) * _C2
    return x ^ _lsr(x, 31)


def _normal(key: int, n: int, device) -> torch.Tensor:
    """n standard normals (fp32) for the stream `key`, element i <- hash(key, i)."""
    idx = torch.arange(n, dtype=torch.int64, device=device)
    h = _mix64(idx * _to_i64(_GOLD) + _to_i64(key))
    u1 = ((_lsr(h, 40) & 0xFFFFFF) + 1).to(torch.float32) * (1.0 / 16777216.0)
    u2 = (_lsr(h, 16) & 0xFFFFFF).to(torch.float32) * (1.0 / 16777216.0)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def _stream_key(seed: int, tensor_id: int, head: int, kind: int) -> int:
    k = (seed * 0x100000001B3 + tensor_id) & _MASK64
    k = (k * 0x100000001B3 + head) & _MASK64
    k = (k * 0x100000001B3 + kind) & _MASK64
    # scramble once more on the host so nearby keys give unrelated streams
    k ^= k >> 30
    k = (k * 0xBF58476D1CE4E5B9) & _MASK64
    k ^= k >> 27
    k = (k * 0x94D049BB133111EB) & _MASK64
    k ^= k >> 31
    return k


def _blur_matrix(n: int, sigma: float, radius: int, device) -> torch.Tensor:
    """Dense [n, n] matrix of a normalised Gaussian blur with mirrored borders."""
    taps = [math.exp(-(k * k) / (2.0 * sigma * sigma)) for k in range(-radius, radius + 1)]
    tot = sum(taps)
    m = torch.zeros(n, n, dtype=torch.float64)
    period = 2 * n
    for i in range(n):
        for t, k in zip(taps, range(-radius, radius + 1)):
            j = (i + k) % period
            if j >= n:
                j = period - 1 - j
            m[i, j] += t / tot
    return m.to(torch.float32).to(device)


@dataclass(frozen=True)
class Workload:
    """One named problem: shapes, budgets and the input seed."""
    name: str
    B: int
    H: int
    head_dim: int
    T: int
    Hg: int
    Wg: int
    frac16: float
    frac8: float
    frac4: float
    seed: int
    lam: float = 0.2
    k_outlier_channels: Tuple[int, ...] = ()
    k_outlier_gain: float = 1.0

    @property
    def N(self) -> int:
        return self.T * self.Hg * self.Wg


WORKLOADS: Dict[str, Workload] = {
    # tiny correctness case
    "tiny": Workload("tiny", 1, 2, 64, 4, 16, 16, 0.0, 0.25, 0.25, seed=0),
    # Wan2.1-1.3B-shaped 480p
    "wan1p3b_480p": Workload("wan1p3b_480p", 1, 12, 128, 21, 30, 52, 0.0, 0.10, 0.30, seed=1),
    # HunyuanVideo-shaped 720p
    "hunyuan_720p": Workload("hunyuan_720p", 1, 24, 128, 33, 45, 80, 0.0, 0.05, 0.20, seed=2),
    # Wan2.1-14B-shaped 720p, few-step budgets, with K outlier channels
    "wan14b_720p": Workload("wan14b_720p", 1, 40, 128, 21, 45, 80, 0.0, 0.20, 0.40, seed=3,
                            k_outlier_channels=(3, 35, 67, 99), k_outlier_gain=20.0),
    # same, bf16 high tier and 8-bit low tier
    "wan14b_720p_hi": Workload("wan14b_720p_hi", 1, 40, 128, 21, 45, 80, 0.20, 0.40, 0.0, seed=3,
                               k_outlier_channels=(3, 35, 67, 99), k_outlier_gain=20.0),
}

SWEEP_GRIDS = ((8, 32, 32), (16, 32, 32), (16, 48, 48), (16, 64, 64), (32, 64, 64))


def sweep_workload(grid_index: int, high: float, low: float, *, high_is_bf16: bool = False) -> Workload:
    """Sweep point: H=24, d=128, cubic-ish grid; `high` = 8-bit (or bf16) share, `low` = 4-bit share."""
    T, Hg, Wg = SWEEP_GRIDS[grid_index]
    f16, f8 = (high, 0.0) if high_is_bf16 else (0.0, high)
    return Workload(f"sweep{grid_index}_{high:g}_{low:g}", 1, 24, 128, T, Hg, Wg, f16, f8, low,
                    seed=100 + grid_index)


def _register_sweep():
    """Budget sweep at the largest and smallest grids plus the dense endpoints, as named workloads."""
    names = {0: "8k", 1: "16k", 2: "37k", 3: "65k", 4: "131k"}
    for gi in (0, 2, 4):
        for high, low in ((0.05, 0.20), (0.10, 0.40), (0.20, 0.60)):
            w = sweep_workload(gi, high, low)
            WORKLOADS[f"sweep_{names[gi]}_{int(high * 100)}_{int(low * 100)}"] = Workload(
                **{**w.__dict__, "name": f"sweep_{names[gi]}_{int(high * 100)}_{int(low * 100)}"})
    # single-tier calls at the middle grid (every block kept in one format): small enough for a profiler capture
    for name, w in (("sweep_37k_all4", sweep_workload(2, 0.0, 1.0)), ("sweep_37k_all8", sweep_workload(2, 1.0, 0.0)),
                    ("sweep_37k_allbf16", sweep_workload(2, 1.0, 0.0, high_is_bf16=True))):
        WORKLOADS[name] = Workload(**{**w.__dict__, "name": name})
    w = sweep_workload(4, 1.0, 0.0)
    WORKLOADS["sweep_131k_all8"] = Workload(**{**w.__dict__, "name": "sweep_131k_all8"})
    w = sweep_workload(4, 1.0, 0.0, high_is_bf16=True)
    WORKLOADS["sweep_131k_allbf16"] = Workload(**{**w.__dict__, "name": "sweep_131k_allbf16"})


_register_sweep()


def make_tensor(w: Workload, tensor_id: int, device="cpu", heads=None) -> torch.Tensor:
    """bf16 [B, H', N, d] tensor number `tensor_id` (0=Q, 1=K, 2=V) of workload `w`.

    `heads` optionally restricts to a list of flat (b*H+h) head indices (H' = len(heads), B' = 1).
    """
    dev = torch.device(device)
    d, N = w.head_dim, w.N
    head_ids = list(range(w.B * w.H)) if heads is None else list(heads)
    mt = _blur_matrix(w.T, 2.0, 8, dev)
    mh = _blur_matrix(w.Hg, 2.0, 8, dev)
    mw = _blur_matrix(w.Wg, 2.0, 8, dev)
    out = torch.empty(len(head_ids), N, d, dtype=torch.bfloat16, device=dev)
    for i, hd in enumerate(head_ids):
        z = _normal(_stream_key(w.seed, tensor_id, hd, 0), d * N, dev).view(d, w.T, w.Hg, w.Wg)
        z = torch.einsum("ctyx,st->csyx", z, mt)
        z = torch.einsum("ctyx,sy->ctsx", z, mh)
        z = torch.einsum("ctyx,sx->ctys", z, mw)
        z = z.reshape(d, N)
        std = z.to(torch.float64).pow(2).mean(dim=1).sub(z.to(torch.float64).mean(dim=1).pow(2)).sqrt()
        z = z / std.to(torch.float32).unsqueeze(1)
        z = z + 0.5 * _normal(_stream_key(w.seed, tensor_id, hd, 1), d * N, dev).view(d, N)
        if tensor_id == 1 and w.k_outlier_channels:
            z[list(w.k_outlier_channels)] *= w.k_outlier_gain
        out[i] = z.t().to(torch.bfloat16)
    if heads is None:
        return out.view(w.B, w.H, N, d)
    return out.view(1, len(head_ids), N, d)


def make_qkv(w: Workload, device="cpu", heads=None):
    """(Q, K, V), each bf16 [B, H, N, d] in raster token order u = (t*Hg + y)*Wg + x."""
    return tuple(make_tensor(w, i, device, heads) for i in range(3))
