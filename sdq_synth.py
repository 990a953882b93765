"""Seeded synthetic inputs shaped like the linear layers of OPT-6.7B / LLaMA-7B.

This module serves both the CPU oracle's tests and the CUDA path's tests/benchmarks.  It holds none
of the method's arithmetic: it only draws random weights and activations and rounds them to bf16.

Recipe (stands in for real checkpoints and text, which are not available offline):
  * weights  W[N, K]  ~ Student-t(df=4) * 0.02   (heavy tails supply the weight outliers)
  * activations X[M, K] ~ N(0, 1), with a fixed seeded set of "outlier channels" multiplied by 30
Both are rounded to bf16 (round to nearest even) and returned as torch tensors.
"""
from __future__ import annotations

import numpy as np
import torch


def _gen(seed: int, device: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_weight(N: int, K: int, seed: int, device: str = "cpu", scale: float = 0.02) -> torch.Tensor:
    """Student-t(df=4)*scale weights [N, K] in bf16: t = z * sqrt(4 / v), v ~ chi-square(4)."""
    g = _gen(seed, device)
    out = torch.empty((N, K), dtype=torch.bfloat16, device=device)
    rows = max(1, (1 << 24) // K)
    for r0 in range(0, N, rows):
        r1 = min(N, r0 + rows)
        z = torch.randn((r1 - r0, K), generator=g, device=device, dtype=torch.float32)
        u = torch.rand((2, r1 - r0, K), generator=g, device=device, dtype=torch.float32).clamp_min_(1e-30)
        v = -2.0 * torch.log(u[0] * u[1])              # chi-square with 4 degrees of freedom
        out[r0:r1] = (z * torch.sqrt(4.0 / v) * scale).to(torch.bfloat16)
    return out


def outlier_channels(K: int, n_channels: int, seed: int) -> torch.Tensor:
    g = _gen(seed + 7919, "cpu")
    return torch.randperm(K, generator=g)[:n_channels]


def make_act(M: int, K: int, seed: int, n_outlier_channels: int | None = None, device: str = "cpu",
             gain: float = 30.0) -> torch.Tensor:
    """N(0,1) activations [M, K] in bf16 with `n_outlier_channels` channels scaled by `gain`
    (default K/128 channels)."""
    if n_outlier_channels is None:
        n_outlier_channels = max(1, K // 128)
    g = _gen(seed + 104729, device)
    x = torch.randn((M, K), generator=g, device=device, dtype=torch.float32)
    ch = outlier_channels(K, n_outlier_channels, seed).to(device)
    x[:, ch] *= gain
    return x.to(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 torch tensor -> numpy uint16 bit patterns (CPU)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
