"""Seeded synthetic workloads: LLaMA-shaped parameter lists and gradient recipes.

This module holds no arithmetic of the optimizer; it only names shapes and draws inputs.
Both the CUDA library's tests/benchmark and the CPU oracle's tests consume the arrays it
returns, so the two sides always see identical inputs.

Shapes follow the LLaMA size table of the paper's pre-training appendix (hidden size,
intermediate size, layer count).  Per layer: q, k, v, o are hidden x hidden; gate and up
are hidden x intermediate (stored wide); down is intermediate x hidden (stored tall).
The real workload behind the paper's numbers is C4 pre-training gradients; these draws
stand in for them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch


def llama_linear_shapes(layers: int, hidden: int, intermediate: int) -> list[tuple[int, int]]:
    per_layer = [(hidden, hidden)] * 4 + [(hidden, intermediate)] * 2 + [(intermediate, hidden)]
    return per_layer * layers


@dataclass
class Workload:
    name: str
    shapes: list
    dtype: str                # "f32" | "bf16"
    rank: int
    mode: str                 # "channel" | "tensor"
    T: int
    steps: int
    lr: float = 1e-2
    wd: float = 0.0
    alpha: float = 1.0
    gamma: float = 1.01
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    seed: int = 42            # Philox seed of the projection
    data_seed: int = 0
    grad: str = "normal"      # "normal" | "row_scaled" | "student_t3" | "outlier_cols"
    grad_scale: float = 1e-3
    w_std: float = 0.02
    extra: dict = field(default_factory=dict)

    @property
    def params(self) -> int:
        return sum(r * c for r, c in self.shapes)


def workload(name: str) -> Workload:
    """The named configurations (single matrix, 60M, 350M, 1B, 7B APOLLO, 7B Mini)."""
    if name == "single":
        return Workload("single", [(512, 1376)], "f32", 128, "channel", T=5, steps=10)
    if name == "llama60m_mini":
        return Workload("llama60m_mini", llama_linear_shapes(8, 512, 1376), "bf16", 1, "tensor", T=200,
                        steps=20, alpha=math.sqrt(128.0), grad="row_scaled")
    if name == "llama350m":
        return Workload("llama350m", llama_linear_shapes(24, 1024, 2736), "bf16", 256, "channel", T=10,
                        steps=20, grad="student_t3")
    if name == "llama1b":
        return Workload("llama1b", llama_linear_shapes(24, 2048, 5461), "bf16", 512, "channel", T=20,
                        steps=50, wd=0.01, grad="outlier_cols")
    if name == "llama7b":
        return Workload("llama7b", llama_linear_shapes(32, 4096, 11008), "bf16", 256, "channel", T=10, steps=20)
    if name == "llama7b_mini":
        return Workload("llama7b_mini", llama_linear_shapes(32, 4096, 11008), "bf16", 1, "tensor", T=10,
                        steps=20, alpha=math.sqrt(128.0))
    raise KeyError(name)


def torch_dtype(dtype: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]


def _gen(device, *seed_parts: int) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for p in seed_parts:
        s = (s * 6364136223846793005 + 1442695040888963407 + int(p)) % (1 << 63)
    g.manual_seed(s)
    return g


def make_weight(wl: Workload, mat: int, device="cpu") -> torch.Tensor:
    rows, cols = wl.shapes[mat]
    g = _gen(device, wl.data_seed, 1, mat)
    w = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32) * wl.w_std
    return w.to(torch_dtype(wl.dtype))


def make_grad(wl: Workload, mat: int, step: int, device="cpu") -> torch.Tensor:
    """Gradient of matrix `mat` at step `step`; redrawn every step, independent of W."""
    rows, cols = wl.shapes[mat]
    g = _gen(device, wl.data_seed, 2, mat, step)
    x = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
    if wl.grad == "normal":
        pass
    elif wl.grad == "row_scaled":
        # per-row factor, log-uniform in [0.1, 10]; fixed over steps
        gr = _gen(device, wl.data_seed, 3, mat)
        f = torch.pow(10.0, torch.rand(rows, 1, generator=gr, device=device) * 2.0 - 1.0)
        x = x * f
    elif wl.grad == "student_t3":
        # normal / sqrt(chi2_3 / 3)
        chi = torch.randn(3, rows, cols, generator=g, device=device, dtype=torch.float32).square_().sum(0)
        x = x / torch.sqrt(chi / 3.0)
    elif wl.grad == "outlier_cols":
        # a fixed random 1 % of the columns carries 50x the scale
        gc = _gen(device, wl.data_seed, 4, mat)
        mask = torch.rand(1, cols, generator=gc, device=device) < 0.01
        x = x * torch.where(mask, 50.0, 1.0)
    else:
        raise KeyError(wl.grad)
    return (x * wl.grad_scale).to(torch_dtype(wl.dtype))
