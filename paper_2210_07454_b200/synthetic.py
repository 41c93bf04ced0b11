"""Seeded synthetic gradient workloads shaped like the paper's DNN experiments.

This module holds no optimiser arithmetic: it only names the workload configurations and draws the random
gradients they are made of (on any torch device).  It imports neither the CUDA binding nor the CPU oracle.

The second parameter of every distribution is its scale (standard deviation, Laplace b, Student-t scale).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    d: int
    n: int
    r: int
    c: int
    k: int
    steps: int
    recipe: str
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.99
    eps: float = 1e-8
    seed: int = 0           # hash seed


WORKLOADS = {
    # d ~ 60k parameters (LeNet-5-sized), planted heavy coordinates
    "C1": Workload("C1", 65_536, 4, 5, 2_048, 512, 10, "planted"),
    # ResNet-18-sized
    "C2": Workload("C2", 11_200_000, 8, 5, 100_000, 112_000, 20, "laplace_shared_t"),
    # ResNet-50-sized ("about 25M parameters"), per-layer scales
    "C3": Workload("C3", 25_600_000, 8, 5, 250_000, 256_000, 20, "layer_scales"),
    # ResNet-50-sized, 32 workers with non-identical distributions
    "C4": Workload("C4", 25_600_000, 32, 7, 500_000, 128_000, 20, "worker_shift"),
    # GPT-2-small-sized
    "C5": Workload("C5", 124_000_000, 16, 5, 1_000_000, 124_000, 10, "sparse_heavy"),
}


def scaled(w: Workload, factor: int, name: str | None = None) -> Workload:
    """The same recipe at 1/factor of the size (d, c, k divided; d kept a multiple of 64, k >= 1)."""
    d = max(64, (w.d // factor) // 64 * 64)
    return Workload(name or f"{w.name}/{factor}", d, w.n, w.r, max(32, w.c // factor), max(1, min(d, w.k // factor)),
                    w.steps, w.recipe, w.lr, w.beta1, w.beta2, w.eps, w.seed)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


class GradientSource:
    """Draws the gradients of every step of one workload.  `cfg_id` separates the seed spaces of workloads:
    data seed = 1000*cfg_id + step, structure seed = 1000*cfg_id + 999."""

    def __init__(self, w: Workload, device="cpu", cfg_id: int | None = None):
        self.w, self.device = w, torch.device(device)
        self.cfg_id = cfg_id if cfg_id is not None else (int(w.name[1]) if w.name[:1] == "C" and w.name[1:2].isdigit() else 9)
        gs = _gen(self.device, 1000 * self.cfg_id + 999)
        d = w.d
        self.struct = {}
        if w.recipe == "planted":
            self.struct["pos"] = torch.randperm(d, generator=gs, device=self.device)[: min(256, d)]
        elif w.recipe == "laplace_shared_t":
            self.struct["pos"] = torch.randperm(d, generator=gs, device=self.device)[: max(1, d // 100)]
        elif w.recipe == "layer_scales":
            expo = torch.rand(50, generator=gs, device=self.device) * 4.0 - 5.0       # log10 scale in [-5,-1]
            self.struct["sigma"] = torch.pow(10.0, expo)
        elif w.recipe == "sparse_heavy":
            self.struct["pos"] = torch.randperm(d, generator=gs, device=self.device)[: max(1, d // 1000)]
        elif w.recipe == "worker_shift":
            pass                                          # per-worker means are regenerated from their seed
        else:
            raise ValueError(w.recipe)

    def x0(self) -> torch.Tensor:
        g = _gen(self.device, 1000 * self.cfg_id + 998)
        return torch.randn(self.w.d, generator=g, device=self.device, dtype=torch.float32) * 0.02

    def grads(self, step: int, out: torch.Tensor | None = None) -> torch.Tensor:
        """(n, d) float32 gradients of step `step` (1-based)."""
        w, dev = self.w, self.device
        n, d = w.n, w.d
        g = _gen(dev, 1000 * self.cfg_id + step)
        if out is None:
            out = torch.empty((n, d), dtype=torch.float32, device=dev)
        if w.recipe == "planted":
            out.normal_(0.0, 1e-3, generator=g)
            pos = self.struct["pos"]
            mag = torch.rand((n, pos.numel()), generator=g, device=dev) * 0.5 + 0.5
            sgn = torch.randint(0, 2, (n, pos.numel()), generator=g, device=dev).float() * 2 - 1
            out[:, pos] = mag * sgn
        elif w.recipe == "laplace_shared_t":
            u = torch.rand((n, d), generator=g, device=dev) - 0.5                     # Laplace(0, 1e-3) by inversion
            out.copy_(-1e-3 * torch.sign(u) * torch.log1p(-2 * u.abs().clamp(max=0.4999999)))
            del u
            pos = self.struct["pos"]
            z = torch.randn(pos.numel(), generator=g, device=dev)                     # Student-t(3) = z / sqrt(chi2_3/3)
            chi = torch.randn((3, pos.numel()), generator=g, device=dev).pow(2).sum(0)
            out[:, pos] += (1e-2 * z / torch.sqrt(chi / 3.0))[None, :]
        elif w.recipe == "layer_scales":
            out.normal_(0.0, 1.0, generator=g)
            blk = (d + 49) // 50
            sig = self.struct["sigma"].repeat_interleave(blk)[:d]
            out.mul_(sig[None, :])
        elif w.recipe == "worker_shift":
            out.normal_(0.0, 1e-3, generator=g)
            for i in range(n):
                gm = _gen(dev, 1000 * self.cfg_id + 900 + i)
                out[i] += torch.randn(d, generator=gm, device=dev) * 1e-3
        elif w.recipe == "sparse_heavy":
            out.normal_(0.0, 1e-4, generator=g)
            pos = self.struct["pos"]
            out[:, pos] += torch.randn((n, pos.numel()), generator=g, device=dev) * 1e-1
        return out
