"""Seeded synthetic LASAD workloads (shapes, value distributions, decay spread).

This module only *draws inputs*: it holds none of the operator's arithmetic and is the one
module that both the CUDA tests/benchmark and the CPU oracle's tests may use.  Shapes follow the
paper's model table (Table 1: width/heads give 64 channels per head) and its 16x tokenizer
(256 tokens for a 256-pixel image, Section 4.1); values are seeded Gaussians standing in for
the projected activations of a trained model.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    dtype: str          # "f32" | "bf16": type of q, k, v, o (state and decay are always fp32)
    B: int
    H: int
    grid_h: int
    grid_w: int
    d: int              # d_k = d_v
    prefix_len: int     # leading non-grid tokens (class token)
    seed: int
    decay_kind: str     # "uniform" (U[lo,hi], seeded) | "geometric" (1-decay log-spaced)
    decay_lo: float
    decay_hi: float

    @property
    def T(self) -> int:
        return self.prefix_len + self.grid_h * self.grid_w

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def scaled(self, B: int | None = None, H: int | None = None) -> "Workload":
        """Same recipe at a reduced batch / head count (for oracle-sized parity cases)."""
        return dataclasses.replace(self, B=B or self.B, H=H or self.H,
                                   name=f"{self.name}[B={B or self.B},H={H or self.H}]")


WORKLOADS = {
    # single layer, fp32, 16x16 grid: prefill plus 256 sequential decode steps
    "config1": Workload("config1", "f32", 1, 4, 16, 16, 32, 0, 1, "uniform", 0.8, 0.99),
    # LlamaGen-B-shaped layer (width 768, 12 heads), 256-pixel image
    "config2": Workload("config2", "bf16", 32, 12, 16, 16, 64, 0, 3, "geometric", 0.9, 0.999),
    # LlamaGen-L-shaped layer (width 1024, 16 heads), 384-pixel image
    "config3": Workload("config3", "bf16", 64, 16, 24, 24, 64, 0, 4, "geometric", 0.9, 0.999),
    # LlamaGen-XL-shaped decode sweep (width 1280, 20 heads), class-token prefix of length 1
    "config4": Workload("config4", "bf16", 256, 20, 16, 16, 64, 1, 5, "geometric", 0.9, 0.999),
    # LlamaGen-XXL-shaped high-resolution prefill (width 1536, 24 heads)
    "config5a": Workload("config5a", "bf16", 8, 24, 64, 64, 64, 0, 6, "geometric", 0.9, 0.999),
    "config5b": Workload("config5b", "bf16", 8, 24, 96, 96, 64, 0, 6, "geometric", 0.9, 0.999),
}


def make_decay(wl: Workload) -> torch.Tensor:
    """Per-head decay constants, fp32 [H]."""
    if wl.decay_kind == "uniform":
        g = torch.Generator().manual_seed(wl.seed + 1)
        u = torch.rand(wl.H, generator=g, dtype=torch.float64)
        return (wl.decay_lo + (wl.decay_hi - wl.decay_lo) * u).to(torch.float32)
    if wl.decay_kind == "geometric":
        # 1 - decay spaced geometrically from 1-lo down to 1-hi
        a, b = math.log10(1.0 - wl.decay_lo), math.log10(1.0 - wl.decay_hi)
        e = torch.linspace(a, b, wl.H, dtype=torch.float64) if wl.H > 1 else torch.tensor([a], dtype=torch.float64)
        return (1.0 - torch.pow(torch.tensor(10.0, dtype=torch.float64), e)).to(torch.float32)
    raise ValueError(wl.decay_kind)


def make_qkv(wl: Workload, T: int | None = None):
    """q, k, v as CPU tensors [B,T,H,d] in the workload's I/O dtype: N(0,1)/sqrt(d), seeded."""
    T = wl.T if T is None else T
    g = torch.Generator().manual_seed(wl.seed)
    out = []
    for _ in range(3):
        x = torch.randn(wl.B, T, wl.H, wl.d, generator=g, dtype=torch.float32)
        x.mul_(1.0 / math.sqrt(wl.d))
        out.append(x.to(wl.torch_dtype))
    return tuple(out)


def make_state(wl: Workload, seed_offset: int = 100) -> torch.Tensor:
    """A seeded non-zero incoming state, fp32 [B,H,d,d] (for hand-off / decode cases)."""
    g = torch.Generator().manual_seed(wl.seed + seed_offset)
    return torch.randn(wl.B, wl.H, wl.d, wl.d, generator=g, dtype=torch.float32)


def make_gate(wl: Workload, T: int | None = None) -> torch.Tensor:
    """A data-dependent gate lambda [B,T,H,d] in the workload's I/O dtype, standing in for the
    Sigmoid(Linear(x)) of a trained layer: a seeded logistic-normal with its mass near 1
    (median 0.88), where forget gates of trained gated linear attention layers sit."""
    T = wl.T if T is None else T
    g = torch.Generator().manual_seed(wl.seed + 7)
    z = torch.randn(wl.B, T, wl.H, wl.d, generator=g, dtype=torch.float32)
    return torch.sigmoid(z + 2.0).to(wl.torch_dtype)
