"""Helpers of the GPU parity tests: run the CUDA library and the fp64 oracle on
the same seeded inputs and compare element by element."""
from __future__ import annotations

import math
from typing import List, Optional, Sequence

import numpy as np
import torch

from oracle import fira_oracle as fo
from paper_2410_01623_b200 import binding as fb
from paper_2410_01623_b200 import workloads as wk

# Tolerances on ||W_gpu - W_oracle||_F / ||W_oracle||_F (per matrix, max over steps):
# 1e-5 for the all-fp32 path, 2e-2 for bf16 storage / bf16 tensor-core products.
TOL_W = {"f32": 1e-5, "bf16": 2e-2}
# The same ratio on the accumulated update W_t - W_0, which is far more sensitive
# (W itself barely moves in a few steps).  fp32: products and norms in fp32 over up
# to a few thousand terms.  bf16: one bf16 rounding of the low-rank operand of the
# back-projection (2^-9 per element, averaged over r terms) plus storage rounding
# flips of W.
TOL_DW = {"f32": 2e-4, "bf16": 3e-2}


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def rel_err(a: np.ndarray, b: np.ndarray) -> float:
    den = float(np.linalg.norm(b))
    return float(np.linalg.norm(a - b)) / (den if den > 0 else 1.0)


def oracle_hyper(hp: fb.Hparams) -> fo.Hyper:
    return fo.Hyper(lr=hp.lr, beta1=hp.beta1, beta2=hp.beta2, eps=hp.eps, alpha=hp.alpha,
                    gamma=hp.gamma, alpha_lowrank_only=bool(hp.flags & fb.FLAG_ALPHA_LOWRANK_ONLY),
                    scaling=("matrix" if hp.flags & fb.FLAG_MATRIX_SCALING else
                             "none" if hp.flags & fb.FLAG_NO_SCALING else "column"),
                    residual=not (hp.flags & fb.FLAG_NO_RESIDUAL),
                    psi=("rmsprop" if hp.flags & fb.FLAG_PSI_RMSPROP else
                         "adagrad" if hp.flags & fb.FLAG_PSI_ADAGRAD else "adam"))


class Trajectory:
    """Steps the library and the oracle side by side over one matrix list."""

    def __init__(self, shapes, r, dtype: torch.dtype, hp: fb.Hparams, W0: Sequence[torch.Tensor],
                 device="cuda", check: Optional[Sequence[int]] = None):
        self.dtype = dtype
        self.kind = "bf16" if dtype == torch.bfloat16 else "f32"
        self.hp = hp
        self.shapes = list(shapes)
        self.f = fb.Fira(shapes, r, dtype, hp, device)
        self.W = [w.to(device).contiguous() for w in W0]
        self.check = list(range(len(shapes))) if check is None else list(check)
        self.W0 = {i: to_np64(W0[i]) for i in self.check}
        self.Wo = {i: to_np64(W0[i]) for i in self.check}
        self.st = {i: fo.new_state(*self.shapes[i], self.f.ranks[i]) for i in self.check}
        self.ohp = oracle_hyper(hp)
        self.max_w = 0.0
        self.max_dw = 0.0
        self.lams: List[List[float]] = []

    def oracle_projection(self, i):
        # the oracle is given exactly the stored projection values
        return to_np64(self.f.get_projection(i))

    def step(self, Gs: Sequence[torch.Tensor], lr: Optional[float] = None, compare=True):
        Gd = [g.to(self.W[0].device).contiguous() for g in Gs]
        projs = {i: self.oracle_projection(i) for i in self.check}
        self.f.step(self.W, Gd, lr)
        torch.cuda.synchronize()
        ohp = self.ohp
        if lr is not None:
            ohp = fo.Hyper(**{**ohp.__dict__, "lr": lr})
        lam_row = []
        for i in self.check:
            self.Wo[i], d = fo.fira_step(self.Wo[i], to_np64(Gs[i]), projs[i], self.st[i], ohp,
                                         store=self.kind)
            lam_row.append(d["lam"])
            if compare:
                Wg = to_np64(self.W[i])
                self.max_w = max(self.max_w, rel_err(Wg, self.Wo[i]))
                self.max_dw = max(self.max_dw, rel_err(Wg - self.W0[i], self.Wo[i] - self.W0[i]))
        self.lams.append(lam_row)
        return lam_row

    def assert_ok(self, tol_w=None, tol_dw=None):
        tol_w = TOL_W[self.kind] if tol_w is None else tol_w
        tol_dw = TOL_DW[self.kind] if tol_dw is None else tol_dw
        assert self.f.poll() == 0
        assert math.isfinite(self.max_w) and self.max_w <= tol_w, (self.max_w, tol_w)
        assert math.isfinite(self.max_dw) and self.max_dw <= tol_dw, (self.max_dw, tol_dw)


def workload_trajectory(wl: wk.Workload, steps: int, device="cuda", gen_device="cpu",
                        check: Optional[Sequence[int]] = None, flags: int = 0,
                        refresh_at=(), refresh_iters=-1) -> Trajectory:
    """Runs `steps` steps of a named workload.  Projections come from the seeded
    random orthonormal generator unless `refresh_at` lists 0-based step counts at
    which the library's own refresh runs first (as Algorithm 1's t mod T branch)."""
    hp = fb.make_hparams(lr=wl.lr, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, alpha=wl.alpha,
                         gamma=wl.gamma, T=wl.T, flags=flags)
    n = len(wl.shapes)
    W0 = [wk.initial_weight(wl, i, gen_device) for i in range(n)]
    tr = Trajectory(wl.shapes, wl.r, wl.torch_dtype, hp, W0, device, check)
    scales = [wk.column_scale(wl, i, gen_device) for i in range(n)]
    if 0 not in refresh_at:
        for i in range(n):
            tr.f.set_projection(i, wk.random_projection(wl, i, device))
    for s in range(1, steps + 1):
        Gs = [wk.gradient(wl, i, s, gen_device, scales[i]) for i in range(n)]
        if (s - 1) in refresh_at:
            tr.f.refresh_projection([g.to(device) for g in Gs], None, seed=s, iters=refresh_iters)
        tr.step(Gs)
    return tr


def residual_jump(G: torch.Tensor, proj: torch.Tensor, mult: float = 9.0) -> torch.Tensor:
    """G + mult * (the part of G outside the projection's subspace): a jump that the
    column factors do not absorb (they scale with 1/||R||, and R is unchanged), so the
    norm of the scaled residual grows by about 1 + mult and the limiter must act."""
    G64, P64 = G.to(torch.float64), proj.to(torch.float64).cpu()
    m, n = G.shape
    resid = G64 - P64 @ (P64.T @ G64) if m <= n else G64 - (G64 @ P64) @ P64.T
    return (G64 + mult * resid).to(G.dtype)
