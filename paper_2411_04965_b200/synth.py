"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no arithmetic of the method itself (no quantiser, no
contraction): it only draws random tensors.  Both the CPU oracle's tests and
the CUDA path's tests and benchmark take their inputs from here.

Recipes (the paper's activations come from trained models on C4, which are not
available; these stand in for them):
  * latent weights: N(0, 0.02^2) in fp32;
  * ternary-valued latents: codes with P(-1)=P(0)=P(+1)=1/3 times 0.024, so
    that the absmean scale is 0.016 and every code survives ternarisation;
  * inputs to attention / FFN: N(0,1) with ceil(1 %) of the channels (fixed
    across tokens) multiplied by 20;
  * intermediate states: Student-t with 3 degrees of freedom.
"""
from __future__ import annotations

import math

import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def latent_weights(N: int, K: int, seed: int, device="cpu", std: float = 0.02) -> torch.Tensor:
    g = _gen(seed, device)
    return torch.randn(N, K, generator=g, device=device, dtype=torch.float32) * std


def ternary_latents(N: int, K: int, seed: int, device="cpu", magnitude: float = 0.024) -> torch.Tensor:
    g = _gen(seed, device)
    codes = torch.randint(-1, 2, (N, K), generator=g, device=device, dtype=torch.int8)
    return codes.to(torch.float32) * magnitude


def outlier_channels(K: int, seed: int, frac: float = 0.01, count: int | None = None) -> torch.Tensor:
    n = count if count is not None else max(1, math.ceil(frac * K))
    g = _gen(seed + 7919, "cpu")
    return torch.randperm(K, generator=g)[:n].sort().values


def gaussian_outlier_activations(M: int, K: int, seed: int, device="cpu", frac: float = 0.01,
                                 scale: float = 20.0, count: int | None = None) -> torch.Tensor:
    g = _gen(seed, device)
    x = torch.randn(M, K, generator=g, device=device, dtype=torch.float32)
    ch = outlier_channels(K, seed, frac, count).to(device)
    x[:, ch] *= scale
    return x


def student_t3(M: int, K: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, device)
    z = torch.randn(M, K, generator=g, device=device, dtype=torch.float32)
    chi = torch.zeros(M, K, device=device, dtype=torch.float32)
    for _ in range(3):
        chi += torch.randn(M, K, generator=g, device=device, dtype=torch.float32) ** 2
    return z / torch.sqrt(chi / 3.0)


def norm_gains(H: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, device)
    return 1.0 + 0.1 * torch.randn(H, generator=g, device=device, dtype=torch.float32)


def kv_cache(B: int, n_heads: int, ctx_cap: int, head_dim: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, device)
    return torch.randn(B, n_heads, ctx_cap, head_dim, generator=g, device=device, dtype=torch.float32)
