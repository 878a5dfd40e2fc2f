"""Seeded synthetic inputs shaped like the paper's Top-10/5/3-of-768 workloads.

This module only draws random tensors; it holds none of the method's
arithmetic, so both the CUDA path and the CPU checker can be fed from it.

Recipe (stand-in for the paper's training batches, Section 4.1 / Table A:
E = 768 routed experts, K in {3, 5, 10}, hidden 1024-2048):
  hidden states  x = bf16(g + mu_c),  g ~ N(0, 1) iid, cluster c uniform over
                 C clusters per token, mu_c[h] ~ N(0, sigma_c^2) drawn once per
                 (workload, layer) -- the cluster shifts make expert loads
                 imbalanced;
  router weights W_r[e][h] ~ N(0, 0.02^2) in bf16, drawn once per (workload,
                 layer); a seeded 5 % of the experts have their row scaled by 3
                 before the cast;
  drift          (deep-stack workload) mu_c(t) = mu_A + t/(steps-1) (mu_B - mu_A).
Bias and previous error start at zero (Algorithm 1 line 1).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

BASE_SEED = 260939137


@dataclass(frozen=True)
class Workload:
    name: str
    L: int            # router layers per step
    T: int            # tokens per layer per step
    H: int            # hidden size
    E: int            # routed experts
    K: int            # experts per token
    clusters: int     # C
    sigma_c: float    # std of the cluster mean shifts
    scaled_frac: float  # fraction of experts whose W_r row is scaled x3
    steps: int
    drift: bool = False
    wid: int = 0      # enters the seed

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = {
    "tiny_top3": Workload("tiny_top3", 1, 1024, 256, 768, 3, 8, 1.5, 0.0, 20, wid=1),
    "top10_single": Workload("top10_single", 1, 16384, 2048, 768, 10, 16, 1.0, 0.05, 200, wid=2),
    "top3_single": Workload("top3_single", 1, 16384, 2048, 768, 3, 16, 1.0, 0.05, 200, wid=3),
    "top5_single": Workload("top5_single", 1, 16384, 2048, 768, 5, 16, 1.0, 0.05, 200, wid=3),
    "top10_deep": Workload("top10_deep", 48, 16384, 2048, 768, 10, 16, 1.0, 0.05, 500, drift=True, wid=4),
    "top10_large": Workload("top10_large", 60, 65536, 4096, 768, 10, 32, 1.0, 0.05, 100, wid=5),
    # the paper's second routing shape (Table A, medium model): Top-8 of 256 experts, hidden 2048, 28 layers
    "top8_of_256": Workload("top8_of_256", 28, 16384, 2048, 256, 8, 16, 1.0, 0.05, 100, wid=6),
}


def _gen(device, *parts: int) -> torch.Generator:
    seed = BASE_SEED
    for p in parts:
        seed = (seed * 1000003 + int(p) + 12345) % (2 ** 62)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def router_weights(wl: Workload, layer: int, device="cpu") -> torch.Tensor:
    """W_r for one layer: [E][H] bf16."""
    g = _gen(device, wl.wid, layer, 1)
    w = torch.randn(wl.E, wl.H, generator=g, device=device, dtype=torch.float32) * 0.02
    n_scaled = int(round(wl.scaled_frac * wl.E))
    if n_scaled > 0:
        g2 = _gen("cpu", wl.wid, layer, 2)
        pick = torch.randperm(wl.E, generator=g2)[:n_scaled].to(device)
        w[pick] *= 3.0
    return w.to(torch.bfloat16)


def cluster_means(wl: Workload, layer: int, which: int = 0, device="cpu") -> torch.Tensor:
    """mu_c: [C][H] fp32. which = 0 start set, 1 end set (drifting workloads)."""
    g = _gen(device, wl.wid, layer, 3 + which)
    return torch.randn(wl.clusters, wl.H, generator=g, device=device, dtype=torch.float32) * wl.sigma_c


def hidden_states(wl: Workload, layer: int, step: int, device="cpu", tokens: int | None = None) -> torch.Tensor:
    """x for one layer and step: [T][H] bf16 (fresh batch per step)."""
    T = wl.T if tokens is None else tokens
    mu = cluster_means(wl, layer, 0, device)
    if wl.drift:
        mu_b = cluster_means(wl, layer, 1, device)
        frac = 0.0 if wl.steps <= 1 else step / float(wl.steps - 1)
        mu = mu + frac * (mu_b - mu)
    g = _gen(device, wl.wid, layer, 7, step)
    c = torch.randint(0, wl.clusters, (T,), generator=g, device=device)
    x = torch.randn(T, wl.H, generator=g, device=device, dtype=torch.float32)
    x += mu[c]
    return x.to(torch.bfloat16)


def stacked_inputs(wl: Workload, step: int, device="cpu", tokens: int | None = None):
    """(x [L][T][H] bf16, W_r [L][E][H] bf16) for one step."""
    xs = torch.stack([hidden_states(wl, l, step, device, tokens) for l in range(wl.L)])
    ws = torch.stack([router_weights(wl, l, device) for l in range(wl.L)])
    return xs.contiguous(), ws.contiguous()


def bf16_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 array of its bit patterns (host)."""
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view("uint16")
