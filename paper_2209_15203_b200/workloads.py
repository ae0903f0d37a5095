"""Seeded synthetic workloads (inputs only — none of the method's arithmetic).

The paper trains MLPs/CNNs/VGG19 on MNIST, Fashion-MNIST and CIFAR10 with
N = 20..100 simulated workers and K = d - floor((1 - 0.001) d) (Section 4).
Those datasets are not available offline, so the five workloads below stand in
for the gradients such runs produce: flat fp32 vectors cut into contiguous
"layer" blocks whose scales differ by orders of magnitude, Gaussian or
heavy-tailed (Student-t, nu = 3) inside a block, with one adversarial workload
that plants exact zeros and large groups of equal magnitudes around the K-th
value.  Everything is drawn from seeded torch generators; the same bytes are
handed to the CUDA library and (copied to the host) to the CPU oracle.

This module is imported by the tests, the benchmark and the smoke check.  It
imports neither the CUDA binding nor the oracle.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Optional, Tuple

import torch

BASE_SEED = 220915203


def k_from_ratio(d: int, num: int, den: int) -> int:
    """K = d - floor((1 - num/den) d), evaluated in integers (Section 4's formula
    with 0.001 -> num/den, which avoids the off-by-one a float 0.999 can give)."""
    return d - ((den - num) * d) // den


@dataclass(frozen=True)
class Workload:
    cid: int                      # configuration number (1..5 benchmark workloads, 6..10 paper shapes)
    name: str
    N: int                        # workers (rows)
    d: int                        # vector length
    K_up: int
    K_down: Tuple[int, ...]       # one or several downlink K (config 4 sweeps)
    steps: int
    modes: Tuple[int, ...]        # 0 = unidirectional, 1 = bidirectional
    dist: str                     # "student" | "gauss"
    blocks: int                   # number of layer blocks (0 = no block layout)
    sigma_lo: float
    sigma_hi: float
    p_kind: str                   # "uniform" | "dirichlet"
    adversarial: bool = False     # zeros + planted ties (config 4)
    alpha: float = 0.1
    w_std: float = 0.02


def _cfg(cid: int, d: Optional[int] = None) -> Workload:
    if cid == 1:
        d = d or 100_000
        K = max(1, d // 100)
        return Workload(1, "tiny", 4, d, K, (K,), 10, (0, 1), "student", 0, 1e-3, 1e-3, "uniform")
    if cid == 2:
        d = d or 11_700_000
        K = k_from_ratio(d, 1, 1000)
        return Workload(2, "resnet18-sized", 16, d, K, (K,), 20, (1,), "gauss", 60, 1e-5, 1e-2, "uniform")
    if cid == 3:
        d = d or 25_600_000
        K = k_from_ratio(d, 1, 1000)
        return Workload(3, "resnet50-sized", 32, d, K, (K,), 20, (0, 1), "student", 160, 1e-6, 1e-2, "dirichlet")
    if cid == 4:
        d = d or 11_700_000
        return Workload(4, "ties-and-zeros", 64, d, k_from_ratio(d, 1, 10000),
                        (k_from_ratio(d, 1, 10000), k_from_ratio(d, 1, 1000), k_from_ratio(d, 1, 100)),
                        10, (1,), "gauss", 60, 1e-5, 1e-2, "uniform", adversarial=True)
    if cid == 5:
        d = d or 124_000_000
        K = k_from_ratio(d, 1, 10000)
        return Workload(5, "gpt2-small-sized", 8, d, K, (K,), 10, (1,), "gauss", 150, 1e-6, 1e-3, "uniform")
    # Shapes of the paper's own experiments (Section 4): N in {20, 50, 100} workers, the models'
    # parameter counts, K = d - floor((1 - 0.001) d), same K up and down.  Synthetic values.
    if cid == 6:   # MLP [784,256,128,64,10] on Fashion-MNIST, 100 workers
        d = d or 242_762
        K = k_from_ratio(d, 1, 1000)
        return Workload(6, "paper-fmnist-mlp", 100, d, K, (K,), 10, (0, 1), "student", 8, 1e-4, 1e-2, "uniform")
    if cid == 7:   # VGG19 on CIFAR10, 20 workers
        d = d or 20_040_522
        K = k_from_ratio(d, 1, 1000)
        return Workload(7, "paper-vgg19", 20, d, K, (K,), 10, (0, 1), "gauss", 40, 1e-5, 1e-2, "uniform")
    if cid == 8:   # CNN on MNIST, 50 workers
        d = d or 1_199_882
        K = k_from_ratio(d, 1, 1000)
        return Workload(8, "paper-mnist-cnn", 50, d, K, (K,), 10, (0, 1), "gauss", 8, 1e-4, 1e-2, "dirichlet")
    if cid == 9:   # CNN on Fashion-MNIST, 20 workers: the smallest model
        d = d or 29_034
        K = k_from_ratio(d, 1, 1000)
        return Workload(9, "paper-fmnist-cnn", 20, d, K, (K,), 10, (0, 1), "student", 6, 1e-4, 1e-2, "uniform")
    if cid == 10:  # MLP [784,64,10] on MNIST, 100 workers
        d = d or 50_890
        K = k_from_ratio(d, 1, 1000)
        return Workload(10, "paper-mnist-mlp", 100, d, K, (K,), 10, (0, 1), "gauss", 4, 1e-4, 1e-2, "uniform")
    raise ValueError("unknown configuration %r" % cid)


def workload(cid: int, d: Optional[int] = None, N: Optional[int] = None) -> Workload:
    """Configuration ``cid`` at full size, or the same recipe at another d / N
    (the K's are re-derived from the configuration's ratios)."""
    w = _cfg(cid, d)
    if N is not None:
        w = replace(w, N=N)
    return w


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _aux_seed(wl: Workload, which: int) -> int:
    return BASE_SEED + 10007 * wl.cid + 900000 + which


def block_sizes(wl: Workload) -> torch.Tensor:
    """Sizes of the contiguous layer blocks: proportional to exp(U(0, ln 1e4)),
    made integer by largest remainder, at least one element each."""
    B = min(wl.blocks, wl.d)
    g = _gen("cpu", _aux_seed(wl, 1))
    wts = torch.exp(torch.rand(B, generator=g, dtype=torch.float64) * math.log(1e4))
    free = wl.d - B                      # one element is reserved for every block
    share = wts / wts.sum() * free
    base = torch.floor(share).to(torch.int64)
    rem = free - int(base.sum())
    order = torch.argsort(share - base.to(torch.float64), descending=True, stable=True)
    base[order[:rem]] += 1
    return base + 1


def scale_vector(wl: Workload, device) -> Optional[torch.Tensor]:
    """Per-element scale sigma_b of the block an element falls in (fp32, [d]),
    fixed per configuration and shared by all workers and steps."""
    if wl.blocks == 0:
        return None
    sizes = block_sizes(wl)
    g = _gen("cpu", _aux_seed(wl, 1) + 50)
    u = torch.rand(sizes.numel(), generator=g, dtype=torch.float64)
    sig = torch.exp(math.log(wl.sigma_lo) + u * (math.log(wl.sigma_hi) - math.log(wl.sigma_lo)))
    return torch.repeat_interleave(sig.to(torch.float32).to(device), sizes.to(device))


def make_p(wl: Workload) -> torch.Tensor:
    """Worker weights p_q (fp32, host): uniform 1/N or Dirichlet(1)."""
    if wl.p_kind == "uniform":
        return torch.full((wl.N,), 1.0 / wl.N, dtype=torch.float32)
    g = _gen("cpu", _aux_seed(wl, 2))
    e = -torch.log1p(-torch.rand(wl.N, generator=g, dtype=torch.float64))
    return (e / e.sum()).to(torch.float32)


def make_w(wl: Workload, device) -> torch.Tensor:
    g = _gen(device, _aux_seed(wl, 3))
    return torch.randn(wl.d, generator=g, device=device, dtype=torch.float32) * wl.w_std


def _student_row(d: int, g: torch.Generator, device) -> torch.Tensor:
    z = torch.randn(d, generator=g, device=device, dtype=torch.float32)
    s = torch.zeros(d, device=device, dtype=torch.float32)
    for _ in range(3):
        c = torch.randn(d, generator=g, device=device, dtype=torch.float32)
        s.addcmul_(c, c)
    return z * torch.sqrt(3.0 / s)


def _plant(wl: Workload, G: torch.Tensor, step: int, device) -> None:
    """Configuration 4: exact zeros (a quarter of them -0.0) and, on 1 % of the
    positions, one of 16 magnitudes taken from that row's own 2K largest, so
    that big groups of equal magnitudes straddle the K-th value.  Workers 2m
    and 2m+1 share the planted positions and magnitudes with opposite signs,
    which makes some aggregated entries cancel to exactly zero."""
    d, K = wl.d, wl.K_up
    g = _gen(device, _aux_seed(wl, 4) + 131 * step)
    pos = mags = sgn = None
    for q in range(wl.N):
        row = G[q]
        zero = torch.rand(d, generator=g, device=device) < 0.05
        neg = torch.rand(d, generator=g, device=device) < 0.25
        row[zero] = 0.0
        row[zero & neg] = -0.0
        if q % 2 == 0 or pos is None:
            n_pl = min(d, max(16, d // 100))
            pos = torch.randperm(d, generator=g, device=device)[:n_pl]
            top = torch.topk(row.abs(), min(d, 2 * K)).values
            pick = torch.randint(0, top.numel(), (16,), generator=g, device=device)
            which = torch.randint(0, 16, (n_pl,), generator=g, device=device)
            mags = top[pick][which]
            sgn = torch.where(torch.rand(n_pl, generator=g, device=device) < 0.5, -1.0, 1.0).to(torch.float32)
            row[pos] = mags * sgn
        else:
            row[pos] = -(mags * sgn)


def make_grads(wl: Workload, step: int, device, out: Optional[torch.Tensor] = None,
               scale: Optional[torch.Tensor] = None, agree: Optional[float] = None) -> torch.Tensor:
    """The N workers' vectors for one step, fp32 [N][d] on ``device``.

    By default the rows are drawn independently.  With ``agree`` = c the workers see noisy
    copies of one shared vector, row_q = base * (1 + c * z_q) with z_q standard normal, the way
    workers that sample the same loss do: their K largest coordinates then mostly coincide."""
    seed = BASE_SEED + 10007 * wl.cid + step
    g = _gen(device, seed)
    G = out if out is not None else torch.empty((wl.N, wl.d), device=device, dtype=torch.float32)
    if scale is None:
        scale = scale_vector(wl, device)
    if agree is not None:
        base = _student_row(wl.d, g, device) if wl.dist == "student" else \
            torch.randn(wl.d, generator=g, device=device, dtype=torch.float32)
        base *= scale if scale is not None else wl.sigma_lo
        for q in range(wl.N):
            z = torch.randn(wl.d, generator=g, device=device, dtype=torch.float32)
            z.mul_(agree).add_(1.0).mul_(base)
            G[q].copy_(z)
            del z
        if wl.adversarial:
            _plant(wl, G, step, device)
        return G
    for q in range(wl.N):
        if wl.dist == "student":
            row = _student_row(wl.d, g, device)
        else:
            row = torch.randn(wl.d, generator=g, device=device, dtype=torch.float32)
        if scale is not None:
            row *= scale
        else:
            row *= wl.sigma_lo
        G[q].copy_(row)
        del row
    if wl.adversarial:
        _plant(wl, G, step, device)
    return G


def checksum(t: torch.Tensor) -> int:
    """64-bit wrap-around sum of the tensor's 32-bit words (for run logs)."""
    v = t.contiguous().view(torch.int32).to(torch.int64)
    return int(v.sum().item()) & 0xFFFFFFFFFFFFFFFF


def describe(wl: Workload) -> Dict[str, object]:
    return {"workload": "config%d:%s" % (wl.cid, wl.name), "N": wl.N, "d": wl.d, "K_up": wl.K_up,
            "K_down": list(wl.K_down), "dist": wl.dist, "blocks": wl.blocks, "p": wl.p_kind}
