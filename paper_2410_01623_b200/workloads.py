"""Seeded synthetic workloads: LLaMA-shaped lists of 2-D weight matrices and
their gradients.

This module only DRAWS inputs (shapes, random numbers, scale factors).  It holds
none of the optimizer's arithmetic and is the one module that both the CUDA
library's callers and the CPU checker's callers may use, so that both sides
receive byte-identical tensors.

Shapes follow the paper's table of LLaMA architectures for pre-training
(Appendix B.1: hidden / intermediate sizes 512/1376, 1024/2736, 2048/5461,
4096/11008) and the ranks of its pre-training table (128, 256, 512; 1024 for
7B).  Per layer the 2-D weights are q, k, v, o (hidden x hidden) and
gate, up (hidden x mlp), down (mlp x hidden).

Gradients stand in for real training gradients (the paper trains on C4, which
is not used here): G_t = Z_t * diag(c) with Z_t iid N(0,1) drawn fresh each step
and c_j = exp(N(0,1)) one log-normal scale per column, fixed over steps.  Some
workloads multiply a fixed 1 % of the columns by 20 (outlier columns) and some
multiply the whole gradient by 10 on given steps (spikes, which make the
norm-growth limiter act).  Weights start as N(0, 0.02^2).
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence, Tuple

import torch

BASE_SEED = 20241001


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    shapes: Tuple[Tuple[int, int], ...]      # (m, n) of every matrix, in order
    r: int
    dtype: str                               # "f32" | "bf16": storage of W, G, P
    steps: int
    T: int                                   # projection refresh gap (0 = never)
    lr: float = 1e-2
    alpha: float = 0.25
    gamma: float = 1.01
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    spike_steps: Tuple[int, ...] = ()        # 1-based steps whose G is multiplied by 10
    outlier_frac: float = 0.0                # fraction of columns multiplied by 20
    layers: int = 1

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


def llama_shapes(layers: int, hidden: int, mlp: int) -> Tuple[Tuple[int, int], ...]:
    per_layer = [(hidden, hidden)] * 4 + [(hidden, mlp)] * 2 + [(mlp, hidden)]
    return tuple(per_layer * layers)


def workload(name: str, layers: Optional[int] = None) -> Workload:
    """The five named workloads.  `layers` overrides the layer count (used to
    run a full-size shape list that is only a few layers long)."""
    if name == "single-60m":
        return Workload(name, ((512, 1376),), r=128, dtype="f32", steps=10, T=0,
                        spike_steps=(6,))
    if name == "llama-60m":
        L = layers or 8
        return Workload(name, llama_shapes(L, 512, 1376), r=128, dtype="f32", steps=50,
                        T=20, layers=L)
    if name == "llama-350m":
        L = layers or 24
        return Workload(name, llama_shapes(L, 1024, 2736), r=256, dtype="bf16", steps=100,
                        T=50, layers=L)
    if name == "llama-1b":
        L = layers or 24
        return Workload(name, llama_shapes(L, 2048, 5461), r=512, dtype="bf16", steps=50,
                        T=25, outlier_frac=0.01, layers=L)
    if name == "llama-7b":
        L = layers or 32
        return Workload(name, llama_shapes(L, 4096, 11008), r=1024, dtype="bf16", steps=50,
                        T=200, alpha=0.0625, spike_steps=(25, 50), layers=L)
    raise KeyError(name)


WORKLOAD_NAMES = ("single-60m", "llama-60m", "llama-350m", "llama-1b", "llama-7b")


def _seed(*parts: int) -> int:
    h = BASE_SEED
    for p in parts:
        h = (h * 1_000_003 + int(p) + 0x9E3779B97F4A7C15) % (1 << 62)
    return h


def _gen(device, *parts: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed(*parts))
    return g


def initial_weight(wl: Workload, idx: int, device="cpu") -> torch.Tensor:
    m, n = wl.shapes[idx]
    w = torch.randn(m, n, generator=_gen(device, 1, idx), device=device, dtype=torch.float32)
    return (w * 0.02).to(wl.torch_dtype)


def column_scale(wl: Workload, idx: int, device="cpu") -> torch.Tensor:
    """One fixed scale per column of G: log-normal(0,1), with a seeded subset of
    the columns multiplied by 20 when the workload has outlier columns."""
    m, n = wl.shapes[idx]
    c = torch.exp(torch.randn(n, generator=_gen(device, 2, idx), device=device,
                              dtype=torch.float32))
    if wl.outlier_frac > 0.0:
        u = torch.rand(n, generator=_gen(device, 3, idx), device=device, dtype=torch.float32)
        c = torch.where(u < wl.outlier_frac, c * 20.0, c)
    return c


def gradient(wl: Workload, idx: int, step: int, device="cpu",
             scale: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Gradient of matrix `idx` at 1-based step `step`."""
    m, n = wl.shapes[idx]
    if scale is None:
        scale = column_scale(wl, idx, device)
    z = torch.randn(m, n, generator=_gen(device, 4, idx, step), device=device,
                    dtype=torch.float32)
    g = z * scale[None, :]
    if step in wl.spike_steps:
        g = g * 10.0
    return g.to(wl.torch_dtype)


def random_projection(wl: Workload, idx: int, device="cpu") -> torch.Tensor:
    """A seeded matrix with orthonormal columns (the Q factor of a Gaussian
    matrix), d x r with d = min(m, n), in the workload's storage type."""
    m, n = wl.shapes[idx]
    d = min(m, n)
    a = torch.randn(d, wl.r, generator=_gen("cpu", 5, idx), dtype=torch.float64)
    q, _ = torch.linalg.qr(a)
    return q.to(wl.torch_dtype).contiguous().to(device)


def planted_gradient(m: int, n: int, r: int, seed: int, gap: float = 4.0,
                     device="cpu") -> torch.Tensor:
    """A float32 matrix whose r leading singular values sit a factor `gap` above
    the rest: U diag(s) V^T with seeded orthonormal U, V, s_i in [1, 2] * gap for
    i < r and in [0.5, 1] below.  Stands in for real gradients, whose spectrum
    decays, when the refreshed subspace itself is compared."""
    d = min(m, n)
    g = torch.Generator(device="cpu")
    g.manual_seed(_seed(6, seed))
    u, _ = torch.linalg.qr(torch.randn(m, d, generator=g, dtype=torch.float64))
    v, _ = torch.linalg.qr(torch.randn(n, d, generator=g, dtype=torch.float64))
    s = torch.cat([gap * (1.0 + torch.rand(r, generator=g, dtype=torch.float64)),
                   0.5 + 0.5 * torch.rand(d - r, generator=g, dtype=torch.float64)])
    s, _ = torch.sort(s, descending=True)
    return ((u * s[None, :]) @ v.T).to(torch.float32).to(device)
