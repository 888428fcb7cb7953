"""Seeded synthetic stochastic gradients standing in for DNN gradients.

The paper's experiments train ResNets on image datasets that are not available
offline; what the compression step sees of them is one dense gradient vector
per worker per iteration.  The recipes below draw such vectors with the value
distributions of the benchmark configurations (Gaussian, heavy-tailed Student-t,
bf16 Gaussian with sparse outliers).  One tensor is drawn once and the very same
bytes are handed to whichever implementation consumes them.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Optional

import torch

from .layouts import (Layout, flat_layout, gpt2_small_layout, resnet18_layout,
                      resnet50_layout)


@dataclass(frozen=True)
class Workload:
    name: str
    num_workers: int
    layout: Callable[[], Layout]
    dist: str            # "normal", "student_t3", "bf16_outliers"
    scale: float         # std (normal / bf16), multiplier (student-t)
    compressor: str      # "sign" or "topk"
    topk_frac: tuple     # (num, den), used when compressor == "topk"
    lr: float
    steps: int
    grad_dtype: str      # "f32" or "bf16"


WORKLOADS = {
    "c1": Workload("c1", 4, lambda: flat_layout(65536), "normal", 1.0, "sign", (0, 1), 0.1, 20, "f32"),
    "c2": Workload("c2", 8, resnet18_layout, "normal", 0.01, "sign", (0, 1), 0.05, 50, "f32"),
    "c3": Workload("c3", 16, resnet50_layout, "student_t3", 1e-3, "topk", (1, 100), 0.1, 50, "f32"),
    "c4": Workload("c4", 32, gpt2_small_layout, "bf16_outliers", 1e-2, "sign", (0, 1), 1e-3, 20, "bf16"),
}


def gradient_seed(base_seed: int, worker: int, step: int) -> int:
    """Distinct stream per (worker, step); plain integer mixing, no arithmetic of the method."""
    return (int(base_seed) * 1_000_003 + int(step)) * 4099 + int(worker) + 17


def _draw_row(dist: str, scale: float, d: int, gen: torch.Generator, device) -> torch.Tensor:
    if dist == "normal":
        return torch.randn(d, generator=gen, device=device, dtype=torch.float32) * scale
    if dist == "student_t3":
        z = torch.randn(d, generator=gen, device=device, dtype=torch.float32)
        c = torch.zeros(d, device=device, dtype=torch.float32)
        for _ in range(3):
            w = torch.randn(d, generator=gen, device=device, dtype=torch.float32)
            c += w * w
        return z / torch.sqrt(c / 3.0) * scale
    if dist == "bf16_outliers":
        g = torch.randn(d, generator=gen, device=device, dtype=torch.float32) * scale
        u = torch.rand(d, generator=gen, device=device, dtype=torch.float32)
        sgn = torch.where(torch.rand(d, generator=gen, device=device) < 0.5, -1.0, 1.0)
        g = torch.where(u < 1e-3, sgn * 0.1, g)
        return g.to(torch.bfloat16)  # round to nearest even
    raise ValueError(f"unknown distribution {dist!r}")


def make_gradients(dist: str, scale: float, num_workers: int, d: int, step: int,
                   base_seed: int = 0, device="cpu",
                   out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """[num_workers, d] gradients for one iteration, row i seeded by (base_seed, i, step)."""
    dtype = torch.bfloat16 if dist == "bf16_outliers" else torch.float32
    if out is None:
        out = torch.empty((num_workers, d), dtype=dtype, device=device)
    assert out.shape == (num_workers, d) and out.dtype == dtype
    gen = torch.Generator(device=device)
    for i in range(num_workers):
        gen.manual_seed(gradient_seed(base_seed, i, step))
        out[i].copy_(_draw_row(dist, scale, d, gen, device))
    return out
