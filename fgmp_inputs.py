"""Seeded synthetic inputs shaped like the Llama-2 linear layers the paper evaluates.

This module holds no arithmetic of the method: it only draws tensors.  Both the CPU
oracle (in tests) and the CUDA library (tests, benchmark) consume exactly these bits.

Recipe (stand-in for real Llama-2 activations/weights/Fisher information, which need the
model and its calibration set):
  * activations X [M, K]: N(0, 1); a fixed fraction of input channels (columns), chosen at
    random, is multiplied by an outlier factor; then rounded to bf16.
  * weights W [N, K]: N(0, std 0.02), rounded to bf16.
  * activation Fisher information, per input channel [K]: LogNormal(0, sigma).
  * weight Fisher information, per element [N, K]: LogNormal(0, sigma), i.i.d.
Each tensor has its own generator stream (seed * 1000 + stream id) so that changing one
shape does not change another tensor's values.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

STREAM_X, STREAM_OUTLIER, STREAM_W, STREAM_FX, STREAM_FW = range(5)


def _gen(seed: int, stream: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 1000 + stream)
    return g


def activations(M: int, K: int, seed: int, outlier_frac: float, outlier_factor: float,
                n_outlier: int | None = None) -> torch.Tensor:
    """bf16 [M, K] on CPU."""
    x = torch.randn(M, K, generator=_gen(seed, STREAM_X), dtype=torch.float32)
    n_out = n_outlier if n_outlier is not None else int(round(outlier_frac * K))
    if n_out > 0:
        perm = torch.randperm(K, generator=_gen(seed, STREAM_OUTLIER))
        x[:, perm[:n_out]] *= outlier_factor
    return x.to(torch.bfloat16)


def weights(N: int, K: int, seed: int, std: float = 0.02) -> torch.Tensor:
    """bf16 [N, K] on CPU."""
    w = torch.randn(N, K, generator=_gen(seed, STREAM_W), dtype=torch.float32) * std
    return w.to(torch.bfloat16)


def fisher_channels(K: int, seed: int, sigma: float) -> torch.Tensor:
    """float32 [K]."""
    return torch.exp(torch.randn(K, generator=_gen(seed, STREAM_FX), dtype=torch.float32) * sigma)


def fisher_elements(N: int, K: int, seed: int, sigma: float) -> torch.Tensor:
    """float32 [N, K]."""
    return torch.exp(torch.randn(N, K, generator=_gen(seed, STREAM_FW), dtype=torch.float32) * sigma)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """uint16 view (numpy) of a CPU bf16 tensor."""
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def tensor_scale(t: torch.Tensor) -> float:
    """The FP32 per-tensor NVFP4 scale a calibration pass would hand to the quantizer:
    amax / (6 * 448), as an fp32 division.  An input of the method, not part of it."""
    amax = np.float32(t.abs().max().float().item())
    return float(amax / np.float32(2688.0))


@dataclass
class Workload:
    name: str
    M: int
    N: int
    K: int
    outlier_frac: float
    outlier_factor: float
    fisher_sigma: float
    fp8_fraction: float
    n_outlier: int | None = None
    seed: int = 0

    def x(self) -> torch.Tensor:
        return activations(self.M, self.K, self.seed, self.outlier_frac, self.outlier_factor,
                           self.n_outlier)

    def w(self) -> torch.Tensor:
        return weights(self.N, self.K, self.seed)

    def fx(self) -> torch.Tensor:
        return fisher_channels(self.K, self.seed, self.fisher_sigma)

    def fw(self) -> torch.Tensor:
        return fisher_elements(self.N, self.K, self.seed, self.fisher_sigma)


def tiny(seed: int = 0) -> Workload:
    """Config 1: M=64, K=256, N=256, two outlier channels x20, LogNormal(0,1), 10% FP8."""
    return Workload("tiny", 64, 256, 256, 0.0, 20.0, 1.0, 0.10, n_outlier=2, seed=seed)


def llama(name: str, M: int, N: int, K: int, fp8_fraction: float = 0.10, seed: int = 0) -> Workload:
    """Configs 2-5: 1% outlier channels x30, LogNormal(0, 1.5)."""
    return Workload(name, M, N, K, 0.01, 30.0, 1.5, fp8_fraction, seed=seed)


LLAMA2_7B_LAYER = [  # (name, N, K) of the seven linears of one decoder layer
    ("q_proj", 4096, 4096), ("k_proj", 4096, 4096), ("v_proj", 4096, 4096), ("o_proj", 4096, 4096),
    ("fc1", 11008, 4096), ("gate", 11008, 4096), ("fc2", 4096, 11008),
]
