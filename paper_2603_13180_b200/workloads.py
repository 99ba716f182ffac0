"""Seeded synthetic inputs for the MXNorm hot path.

This module holds input recipes only - none of the method's arithmetic - so that
the CPU oracle's tests and the CUDA path's tests can draw identical bytes from it.
Tensors are generated on the CPU in fp32 with a seeded ``torch.Generator`` and
rounded once to bf16 (round-to-nearest-even); the bf16 bit pattern is the contract.

The shapes and distributions stand in for the paper's workloads: Llama-3 hidden
sizes (1B: 2048, 8B: 4096) at batch 4 x sequence 4096 tokens, Gaussian benchmark
inputs, and a few "outlier feature" channels whose magnitude is far above the rest
(the activation pattern the paper's loss-spike analysis describes).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    T: int
    D: int
    seed: int
    outlier_frac: float = 0.0   # fraction of channels multiplied by ``outlier_gain``
    outlier_gain: float = 20.0
    has_gain: bool = False      # bf16 norm gain ~ N(1, std 0.1)
    has_grad: bool = False      # bf16 upstream gradient ~ N(0, std 1e-2)
    kind: str = "mxfp8"         # "mxfp8" | "nvfp4" | "bwd"
    swizzled_scales: bool = False


CONFIGS = {
    "C1": Workload("C1", 2048, 768, seed=0),
    "C2": Workload("C2", 16384, 2048, seed=0, outlier_frac=0.001, has_gain=True),
    "C3": Workload("C3", 16384, 4096, seed=0, outlier_frac=0.001, has_gain=True,
                   swizzled_scales=True),
    "C4": Workload("C4", 16384, 4096, seed=0, outlier_frac=0.001, kind="nvfp4"),
    "C5": Workload("C5", 16384, 4096, seed=1, outlier_frac=0.001, has_gain=True, has_grad=True,
                   kind="bwd"),
}


def make_inputs(w: Workload, T: int | None = None) -> dict:
    """Returns CPU bf16 tensors {"x": [T, D], "gain": [D] | None, "grad": [T, D] | None}.

    ``T`` overrides the row count (rows are drawn in order from one generator, so the first
    rows of a short draw do NOT equal the first rows of the full one; a test that samples
    the full-size case slices the full tensor instead)."""
    T = w.T if T is None else T
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed)
    z = torch.randn(T, w.D, generator=g, dtype=torch.float32)
    row_scale = torch.exp(torch.randn(T, 1, generator=g, dtype=torch.float32))  # lognormal(0, 1)
    x = z * row_scale
    n_out = int(round(w.outlier_frac * w.D))
    if n_out > 0:
        cols = torch.randperm(w.D, generator=g)[:n_out]
        x[:, cols] *= w.outlier_gain
    out = {"x": x.to(torch.bfloat16).contiguous(), "gain": None, "grad": None}
    if w.has_gain:
        out["gain"] = (1.0 + 0.1 * torch.randn(w.D, generator=g, dtype=torch.float32)).to(torch.bfloat16)
    if w.has_grad:
        out["grad"] = (1e-2 * torch.randn(T, w.D, generator=g, dtype=torch.float32)).to(torch.bfloat16).contiguous()
    return out


def gaussian(T: int, D: int, seed: int, row_scale_sigma: float = 0.0) -> torch.Tensor:
    """Plain i.i.d. N(0,1) rows (the paper's kernel-benchmark input), optional lognormal row scale."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    x = torch.randn(T, D, generator=g, dtype=torch.float32)
    if row_scale_sigma > 0:
        x = x * torch.exp(row_scale_sigma * torch.randn(T, 1, generator=g, dtype=torch.float32))
    return x.to(torch.bfloat16).contiguous()


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 CPU tensor -> numpy uint16 bit patterns (no copy of values, same bytes)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray) -> torch.Tensor:
    """numpy uint16 bit patterns -> bf16 CPU tensor."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (RN-even) via torch and return the bit patterns."""
    return bits(torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16))
