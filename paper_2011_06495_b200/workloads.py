"""Seeded synthetic inputs shaped like the paper's workloads.

The paper trains ResNet-18 (d = 11,173,962 parameters) on CIFAR-10 with N = 10
workers and sparsity K = phi*d, phi between 1e-2 and 1e-3 (Section 4.1).  Neither
the data set nor real gradients are needed to exercise the majority-vote step, so
this module draws gradients with the same sizes and a layer-like scale structure
from seeded generators.  It holds no arithmetic of the method itself: it only
fills `grads` (and the initial `err`) tensors, on the CPU or on a CUDA device.
The tests hand the very same bytes to the CUDA library and to the CPU oracle.

Layer structure: a real per-tensor shape list is not available, so the d
coordinates are split into L contiguous segments whose sizes are proportional to
10**U(1.8, 6.4) (rescaled to sum to d, each at least 16, boundaries deliberately
unaligned) and each segment gets its own standard deviation, log-uniform in
[std_lo, std_hi].
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch

BASE_SEED = 201106495


@dataclass(frozen=True)
class Workload:
    name: str
    N: int
    d: int
    K: int
    steps: int
    kind: str                      # "iid" | "correlated" | "student_t"
    config_id: int
    segments: int = 1
    std_lo: float = 1.0
    std_hi: float = 1.0
    rho: float = 0.0               # cross-worker correlation (share of the common component's variance)
    err0_std: float = 0.0
    round_decimals: Optional[int] = None
    tie_free: bool = False         # redraw coinciding magnitudes until every row is tie-free
    note: str = ""

    def seed(self, step: int = 0) -> int:
        return BASE_SEED + 1000 * self.config_id + step


def resnet_like(name: str) -> Workload:
    """The four named configurations (c1..c4)."""
    d18, d50 = 11_173_962, 25_557_032
    table = {
        "c1": Workload("c1", N=4, d=10_000, K=100, steps=1, kind="iid", config_id=1, tie_free=True,
                       note="tie-free unit Gaussians"),
        "c1_ties": Workload("c1_ties", N=4, d=10_000, K=100, steps=1, kind="iid", config_id=1,
                            round_decimals=1, note="magnitudes rounded to one decimal"),
        "c2": Workload("c2", N=10, d=d18, K=d18 // 100, steps=20, kind="iid", config_id=2,
                       segments=62, std_lo=1e-4, std_hi=1e-1, note="ResNet-18-sized, independent workers"),
        "c3": Workload("c3", N=25, d=d18, K=d18 // 1000, steps=20, kind="correlated", config_id=3,
                       segments=62, std_lo=1e-4, std_hi=1e-1, rho=0.5,
                       note="ResNet-18-sized, half of the variance shared by all workers"),
        "c4": Workload("c4", N=8, d=d50, K=d50 // 4000, steps=50, kind="student_t", config_id=4,
                       segments=161, std_lo=1e-5, std_hi=1e-1, note="ResNet-50-sized, Student-t (nu=3)"),
    }
    return table[name]


def sweep_cells():
    """The 27 cells of the sweep (c5): N x d x K/d, correlation 0.3, err ~ N(0, 0.01^2)."""
    cells = []
    cid = 0
    for N in (4, 16, 64):
        for d in (1 << 20, 1 << 24, 1 << 27):
            for ratio in (1e-2, 1e-3, 2.5e-4):
                K = int(math.floor(d * ratio))
                cells.append(Workload(f"c5_N{N}_d{d}_K{K}", N=N, d=d, K=K, steps=1, kind="correlated",
                                      config_id=500 + cid, rho=0.3, err0_std=0.01,
                                      note="sweep cell"))
                cid += 1
    return cells


def scaled(w: Workload, d: int, K: Optional[int] = None, N: Optional[int] = None, steps: Optional[int] = None) -> Workload:
    """The same recipe at another size (used for quick tests)."""
    ratio = w.K / w.d
    return Workload(f"{w.name}_d{d}", N=N or w.N, d=d, K=K or max(1, int(d * ratio)), steps=steps or w.steps,
                    kind=w.kind, config_id=w.config_id, segments=min(w.segments, max(1, d // 16)),
                    std_lo=w.std_lo, std_hi=w.std_hi, rho=w.rho, err0_std=w.err0_std,
                    round_decimals=w.round_decimals, note=w.note + " (rescaled)")


def layer_segments(w: Workload):
    """Returns (bounds int64[L+1], std float64[L]) drawn once per workload."""
    L = w.segments
    if L <= 1:
        return np.array([0, w.d], dtype=np.int64), np.array([w.std_hi], dtype=np.float64)
    rng = np.random.default_rng(w.seed(0) ^ 0x5EED)
    raw = 10.0 ** rng.uniform(1.8, 6.4, size=L)
    sizes = np.maximum(16, np.floor(raw * (w.d / raw.sum())).astype(np.int64))
    sizes[np.argmax(sizes)] += w.d - sizes.sum()
    assert sizes.min() >= 1 and sizes.sum() == w.d
    std = 10.0 ** rng.uniform(math.log10(w.std_lo), math.log10(w.std_hi), size=L)
    bounds = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    return bounds, std


def std_vector(w: Workload, device="cpu") -> torch.Tensor:
    """Per-coordinate standard deviation, float32 [d]."""
    bounds, std = layer_segments(w)
    sizes = torch.from_numpy(np.diff(bounds))
    v = torch.repeat_interleave(torch.from_numpy(std.astype(np.float32)), sizes)
    return v.to(device)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def initial_err(w: Workload, device="cpu", out: Optional[torch.Tensor] = None) -> torch.Tensor:
    err = out if out is not None else torch.empty((w.N, w.d), dtype=torch.float32, device=device)
    if w.err0_std == 0.0:
        err.zero_()
    else:
        g = _gen(err.device, w.seed(0) + 999_983)
        for n in range(w.N):
            err[n].normal_(0.0, w.err0_std, generator=g)
    return err


def gradients(w: Workload, step: int, device="cpu", out: Optional[torch.Tensor] = None,
              std: Optional[torch.Tensor] = None) -> torch.Tensor:
    """grads [N, d] float32 for one step, filled row by row (bounded temporaries)."""
    grads = _gradients(w, step, device, out, std, 0)
    if w.tie_free:      # redraw the later member(s) of every group of equal magnitudes until none is left
        g = _gen(grads.device, w.seed(step) + 7919)
        for n in range(w.N):
            row = grads[n]
            for _ in range(100):
                mag, order = row.abs().sort(stable=True)
                dup = torch.zeros(w.d, dtype=torch.bool, device=row.device)
                dup[order[1:]] = mag[1:] == mag[:-1]
                k = int(dup.sum())
                if k == 0:
                    break
                row[dup] = torch.empty(k, dtype=torch.float32, device=row.device).normal_(generator=g)
            else:
                raise RuntimeError("could not make the row tie-free")
    return grads


def _gradients(w: Workload, step: int, device, out, std, attempt: int) -> torch.Tensor:
    grads = out if out is not None else torch.empty((w.N, w.d), dtype=torch.float32, device=device)
    dev = grads.device
    g = _gen(dev, w.seed(step) + 7919 * attempt)
    if std is None and w.segments > 1:
        std = std_vector(w, dev)
    common = None
    if w.kind == "correlated":
        common = torch.empty(w.d, dtype=torch.float32, device=dev).normal_(generator=g)
        common.mul_(math.sqrt(w.rho))
    for n in range(w.N):
        row = grads[n]
        row.normal_(generator=g)
        if w.kind == "correlated":
            row.mul_(math.sqrt(1.0 - w.rho)).add_(common)
        elif w.kind == "student_t":
            chi = torch.zeros(w.d, dtype=torch.float32, device=dev)
            tmp = torch.empty(w.d, dtype=torch.float32, device=dev)
            for _ in range(3):
                tmp.normal_(generator=g)
                chi.addcmul_(tmp, tmp)
            row.div_(chi.div_(3.0).sqrt_())
        if std is not None:
            row.mul_(std)
        if w.round_decimals is not None:
            s = 10.0 ** w.round_decimals
            row.mul_(s).round_().div_(s)
    return grads
