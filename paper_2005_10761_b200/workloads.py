"""Seeded synthetic gradients shaped like the paper's workloads.

The paper trains ResNet-18/34 and a 2x1500 LSTM (Section IV) and motivates
rTop-k by gradients that are "skewed and sparse": few large entries, many near
zero (Section II-C).  Its datasets are not available, so these generators stand
in for real gradients: same vector lengths, same worker counts, heavy-tailed /
spike-and-bulk magnitude profiles.

This module holds input recipes only -- none of the method's arithmetic -- and is
the one piece shared by the CUDA tests, the CPU oracle's tests and the benchmark.
Every tensor is produced by a ``torch.Generator`` seeded from (seed, worker,
step), one row (worker) at a time, on whichever device is asked for.  CPU and
CUDA generators give different streams: generate once, then copy.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional, Sequence, Tuple

import torch


def round_up(x: int, m: int) -> int:
    return (x + m - 1) // m * m


@dataclass(frozen=True)
class Workload:
    """One configuration: W workers, length-d vectors, top-r then k-of-r."""
    name: str
    d: int
    W: int
    r: int
    k: int
    steps: int = 1
    grad_dtype: str = "f32"            # "f32" | "bf16"
    recipe: str = "spike_bulk"         # spike_bulk | spike_bulk_persistent | laplace_skew | student_t | bernoulli
    seed: int = 0
    # per-tensor (segmented) selection: offsets [S+1], r and k per tensor
    seg_off: Optional[Tuple[int, ...]] = None
    seg_r: Optional[Tuple[int, ...]] = None
    seg_k: Optional[Tuple[int, ...]] = None
    bulk_sigma: float = 1e-3           # "N(0, 1e-6)" read as variance 1e-6
    spike_prob: float = 0.01

    @property
    def ld(self) -> int:
        """Row stride in elements: padded so every row starts 16-byte aligned."""
        return round_up(self.d, 8)

    @property
    def k_total(self) -> int:
        return sum(self.seg_k) if self.seg_k is not None else self.k


def _ratio(d: int, frac_num: int, frac_den: int) -> int:
    return max(1, d * frac_num // frac_den)


def ratios(d: int, r_den: int = 100, k_den: int = 1000) -> Tuple[int, int]:
    """r = floor(d / r_den), k = floor(d / k_den), clamped to 1 <= k <= r."""
    r = _ratio(d, 1, r_den)
    k = min(r, _ratio(d, 1, k_den))
    return r, k


_LSTM_TENSORS = (10000 * 1500, 6000 * 1500, 6000 * 1500, 6000 * 1500, 6000 * 1500, 1500 * 10000)


def _segments(sizes: Sequence[int]):
    off = [0]
    for s in sizes:
        off.append(off[-1] + s)
    rr = tuple(max(1, s // 100) for s in sizes)
    kk = tuple(max(1, s // 1000) for s in sizes)
    return tuple(off), rr, kk


def configs() -> dict:
    """The named configurations (vector sizes of ResNet-18, ResNet-50, the PTB LSTM)."""
    c = {}
    c["c1"] = Workload("c1", d=1 << 20, W=4, r=16384, k=1024, steps=1, seed=0)
    d2 = 11_173_962
    r2, k2 = ratios(d2)
    c["c2"] = Workload("c2", d=d2, W=8, r=r2, k=k2, steps=10, recipe="spike_bulk_persistent", seed=2)
    # the paper's own example setting: n = 5 nodes, k = 0.1% d, r = 0.5% d (Section IV-A)
    c["c2_n5"] = Workload("c2_n5", d=d2, W=5, r=d2 * 5 // 1000, k=d2 // 1000, steps=1,
                          recipe="spike_bulk_persistent", seed=5)
    d3 = 25_557_032
    r3, k3 = ratios(d3)
    c["c3_f32"] = Workload("c3_f32", d=d3, W=16, r=r3, k=k3, steps=10, recipe="laplace_skew", seed=3)
    c["c3_bf16"] = replace(c["c3_f32"], name="c3_bf16", grad_dtype="bf16")
    off, rr, kk = _segments(_LSTM_TENSORS)
    c["c4"] = Workload("c4", d=off[-1], W=8, r=sum(rr), k=sum(kk), steps=1, recipe="student_t",
                       seed=4, seg_off=off, seg_r=rr, seg_k=kk)
    d5 = 1 << 28
    for W in (1, 4, 16, 32):
        for r_den in (100, 1000):
            r5 = d5 // r_den
            for k_div in (10, 4):
                name = f"c5_W{W}_r{r_den}_k{k_div}"
                c[name] = Workload(name, d=d5, W=W, r=r5, k=max(1, r5 // k_div), seed=5)
        c[f"c5_W{W}_topk"] = Workload(f"c5_W{W}_topk", d=d5, W=W, r=d5 // 100, k=d5 // 100, seed=5)
        c[f"c5_W{W}_randk"] = Workload(f"c5_W{W}_randk", d=d5, W=W, r=d5, k=d5 // 1000, seed=5)
    return c


def scaled(cfg: Workload, d: int, W: Optional[int] = None, name: Optional[str] = None) -> Workload:
    """The same recipe and ratios at another length (for small parity cases), or with another row count."""
    if cfg.seg_off is not None:                       # per-tensor sizes are tied to the length: only the rows change
        assert d == cfg.d
        return replace(cfg, W=W or cfg.W, name=name or cfg.name)
    r = max(1, cfg.r * d // cfg.d)
    k = max(1, min(r, cfg.k * d // cfg.d))
    return replace(cfg, d=d, W=W or cfg.W, r=r, k=k, name=name or f"{cfg.name}_d{d}")


def _gen(device, *seed_parts: int) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for p in seed_parts:
        s = (s * 6364136223846793005 + 1442695040888963407 + int(p)) % (1 << 63)
    g.manual_seed(s)
    return g


def _row(cfg: Workload, w: int, step: int, device) -> torch.Tensor:
    d = cfg.d
    f32 = dict(dtype=torch.float32, device=device)
    if cfg.recipe == "spike_bulk":
        g = _gen(device, cfg.seed, w, step, 1)
        x = torch.randn(d, generator=g, **f32) * cfg.bulk_sigma
        mask = torch.rand(d, generator=g, **f32) < cfg.spike_prob
        x = torch.where(mask, torch.randn(d, generator=g, **f32), x)
        return x
    if cfg.recipe == "spike_bulk_persistent":
        # half of the spike positions are drawn once per worker, half anew each step
        g = _gen(device, cfg.seed, w, step, 1)
        gp = _gen(device, cfg.seed, w, 0, 2)
        x = torch.randn(d, generator=g, **f32) * cfg.bulk_sigma
        fixed = torch.rand(d, generator=gp, **f32) < (cfg.spike_prob / 2)
        fresh = torch.rand(d, generator=g, **f32) < (cfg.spike_prob / 2)
        x = torch.where(fixed | fresh, torch.randn(d, generator=g, **f32), x)
        return x
    if cfg.recipe == "laplace_skew":
        # Laplace(0,1) magnitudes times a per-coordinate log-normal(0, sigma=2) skew that is
        # the same for every worker and step (a property of the coordinate)
        gs = _gen(device, cfg.seed, 0, 0, 3)
        skew = torch.exp(2.0 * torch.randn(d, generator=gs, **f32))
        g = _gen(device, cfg.seed, w, step, 1)
        u = torch.rand(d, generator=g, **f32).clamp_(1e-30, 1.0)
        sign = torch.where(torch.rand(d, generator=g, **f32) < 0.5, -1.0, 1.0)
        return (-torch.log(u)) * sign * skew
    if cfg.recipe == "student_t":
        g = _gen(device, cfg.seed, w, step, 1)
        z = torch.randn(d, generator=g, **f32)
        chi = torch.zeros(d, **f32)
        for _ in range(3):
            chi += torch.randn(d, generator=g, **f32) ** 2
        return 0.01 * z / torch.sqrt(chi / 3.0)
    if cfg.recipe == "bernoulli":
        # signed, scaled sparse Bernoulli sample plus a bounded continuous perturbation
        # (Section II-C, refinements (i)-(iii)); theta decays with the coordinate
        gs = _gen(device, cfg.seed, 0, 0, 4)
        theta = torch.rand(d, generator=gs, **f32) ** 8
        g = _gen(device, cfg.seed, w, step, 1)
        on = (torch.rand(d, generator=g, **f32) < theta).to(torch.float32)
        sign = torch.where(torch.rand(d, generator=gs, **f32) < 0.5, -1.0, 1.0)
        return on * sign + (torch.rand(d, generator=g, **f32) - 0.5) * 0.5
    raise ValueError(f"unknown recipe {cfg.recipe!r}")


def gradient(cfg: Workload, step: int, device="cpu", out: Optional[torch.Tensor] = None,
             workers: Optional[Sequence[int]] = None) -> torch.Tensor:
    """Rows ``workers`` (default all W) of step ``step``'s gradient, shape [n, ld] in the
    configuration's dtype (float32, or bfloat16 rounded to nearest from the float32 draw).
    Padding columns d..ld-1 are zero."""
    ws = list(range(cfg.W)) if workers is None else list(workers)
    dt = torch.float32 if cfg.grad_dtype == "f32" else torch.bfloat16
    if out is None:
        out = torch.zeros((len(ws), cfg.ld), dtype=dt, device=device)
    assert out.shape == (len(ws), cfg.ld) and out.dtype == dt
    for n, w in enumerate(ws):
        out[n, : cfg.d] = _row(cfg, w, step, out.device).to(dt)
        if cfg.ld > cfg.d:
            out[n, cfg.d:] = 0
    return out


def zero_residual(cfg: Workload, device="cpu", rows: Optional[int] = None) -> torch.Tensor:
    """m^0 = 0 (Algorithm 1, initialisation)."""
    return torch.zeros((rows or cfg.W, cfg.ld), dtype=torch.float32, device=device)
