"""Seeded synthetic workloads: sizes, segment layouts and gradient distributions.

This module only produces INPUTS (gradients, initial points, segment offsets).  It holds
none of the optimizer's or the compressors' arithmetic and is the one module that both the
CUDA library's tests/benchmark and the CPU oracle's tests may use: both sides receive the
same bytes.

The five workloads are shaped like the models the paper trains (ResNet-18/50, BERT-base,
GPT-2-XL sized parameter vectors); the paper's datasets are not needed for an optimizer
step, only the sizes and the gradient statistics matter.
"""
from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch

SIGN, TOPK, IDENTITY, RANDK = 0, 1, 2, 3


def _gen(device, *key):
    """A torch generator on `device` seeded by a tuple of small integers."""
    s = 0x9E3779B97F4A7C15
    for v in key:
        s = ((s ^ (int(v) + 0x632BE59BD9B4E019)) * 0xD6E8FEB86659FD93) & 0x7FFFFFFFFFFFFFFF
    g = torch.Generator(device=device)
    g.manual_seed(s)
    return g


def loguniform_segments(d, q, lo, hi, seed):
    """q contiguous segment sizes, log-uniform in [lo, hi], rescaled to sum to d.

    Sizes are rounded to integers and NOT aligned to any vector or word width; the last
    segment absorbs the rounding remainder.  Returns int64 offsets of length q+1."""
    rng = np.random.default_rng(seed)
    raw = np.exp(rng.uniform(np.log(lo), np.log(hi), size=q))
    sizes = np.maximum(1, np.floor(raw * (d / raw.sum()))).astype(np.int64)
    sizes[-1] += d - sizes.sum()
    if sizes[-1] < 1:
        raise ValueError("segment recipe does not fit d")
    off = np.zeros(q + 1, dtype=np.int64)
    off[1:] = np.cumsum(sizes)
    return off


def cyclic_segments(d, sizes):
    """Repeat `sizes` until d is filled; the last segment is truncated."""
    off = [0]
    i = 0
    while off[-1] < d:
        off.append(min(d, off[-1] + sizes[i % len(sizes)]))
        i += 1
    return np.asarray(off, dtype=np.int64)


@dataclass
class Workload:
    name: str
    d: int
    n: int
    compressor: int
    steps: int
    k: int = 0
    offsets: Optional[np.ndarray] = None     # None = one flat segment
    dist: str = "normal"                     # normal | segnormal | spiky | student3
    std: float = 1.0
    seed: int = 0
    beta1: float = 0.9
    beta2: float = 0.999
    lr: float = 1e-3
    eps: float = 1e-8
    sigma_seg: Optional[np.ndarray] = field(default=None, repr=False)

    @property
    def q(self):
        return 1 if self.offsets is None else len(self.offsets) - 1

    def x0(self, device="cpu"):
        """Initial point x_1 ~ N(0, 0.02^2)."""
        return torch.randn(self.d, generator=_gen(device, self.seed, 7777), device=device,
                           dtype=torch.float32) * 0.02

    def _row_scale(self, device):
        """Per-coordinate multiplier that is fixed over steps and workers (or None)."""
        if self.dist == "segnormal":
            sizes = np.diff(self.offsets)
            sig = torch.as_tensor(self.sigma_seg, dtype=torch.float32, device=device)
            return torch.repeat_interleave(sig, torch.as_tensor(sizes, device=device))
        if self.dist == "spiky":
            u = torch.rand(self.d, generator=_gen(device, self.seed, 4242), device=device)
            return torch.where(u < 1e-3, 100.0, 1.0).to(torch.float32)
        return None

    def grads(self, step, device="cpu", out=None):
        """The n stochastic gradients of iteration `step` (1-based), n x d float32."""
        if out is None:
            out = torch.empty((self.n, self.d), dtype=torch.float32, device=device)
        device = out.device
        scale = self._row_scale(device)
        chunk = 1 << 26
        for i in range(self.n):
            g = _gen(device, self.seed, step, i)
            row = out[i]
            if self.dist == "student3":
                for a in range(0, self.d, chunk):
                    b = min(self.d, a + chunk)
                    z = torch.randn(4, b - a, generator=g, device=device)
                    chi = (z[1] * z[1] + z[2] * z[2] + z[3] * z[3]) / 3.0
                    row[a:b] = z[0] / torch.sqrt(chi) * self.std
            else:
                row.normal_(0.0, self.std, generator=g)
                if scale is not None:
                    row.mul_(scale)
        return out


def random_sets(d, k, rows, seed, step):
    """Rand-k draws: `rows` independent uniformly random k-subsets of range(d), each listed in
    increasing order (uint32, rows x k).  Inputs of the method, not part of it."""
    out = np.empty((rows, k), dtype=np.uint32)
    for r in range(rows):
        rng = np.random.default_rng([seed, step, r, 991])
        if k * 4 > d:
            pick = rng.permutation(d)[:k]
        else:                                  # rejection-free for k << d: draw, dedupe, top up
            pick = np.unique(rng.integers(0, d, size=int(k * 1.2) + 16))
            while pick.size < k:
                pick = np.unique(np.concatenate([pick, rng.integers(0, d, size=k)]))
            pick = rng.permutation(pick)[:k]
        out[r] = np.sort(pick).astype(np.uint32)
    return out


def workload(name, scale=1.0, steps=None, seed=0):
    """One of the five configurations, optionally with d scaled down (same structure).

    C1 d=65,536 n=4 sign flat, N(0,1); C2 d=11.2M n=8 sign over 62 log-uniform segments,
    N(0, sigma_seg) with sigma log-uniform in [1e-4, 1e-1]; C3 d=25.6M n=16 top-k with
    k = 1% of d, N(0,1) with 0.1% of the coordinates times 100; C4 d=110M n=8 sign over
    transformer-shaped segments, 1e-3 * Student-t(3); C5 d=1.5G n=4 sign flat, N(0, 1e-2).
    """
    name = name.upper()
    if name == "C1":
        w = Workload("C1", int(65536 * scale), 4, SIGN, 10, dist="normal", std=1.0)
    elif name == "C2":
        d = int(11_200_000 * scale)
        off = loguniform_segments(d, 62, 64, 2.4e6, seed + 11)
        rng = np.random.default_rng(seed + 12)
        sig = np.exp(rng.uniform(np.log(1e-4), np.log(1e-1), size=62)).astype(np.float32)
        w = Workload("C2", d, 8, SIGN, 100, offsets=off, dist="segnormal", sigma_seg=sig)
    elif name == "C3":
        d = int(25_600_000 * scale)
        w = Workload("C3", d, 16, TOPK, 50, k=max(1, d // 100), dist="spiky")
    elif name == "C4":
        d = int(110_000_000 * scale)
        sizes = [max(1, int(s * scale)) for s in (768 * 768, 768 * 3072, 30522 * 768)]
        w = Workload("C4", d, 8, SIGN, 50, offsets=cyclic_segments(d, sizes),
                     dist="student3", std=1e-3)
    elif name == "C5":
        w = Workload("C5", int(1_500_000_000 * scale), 4, SIGN, 20, dist="normal", std=1e-2)
    else:
        raise ValueError("unknown workload " + name)
    w.seed = seed
    if steps is not None:
        w.steps = steps
    return w
