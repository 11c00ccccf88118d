"""fp64 CPU oracle for the Fira optimizer update (arXiv 2410.01623).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
library is checked against.  It shares no code with the CUDA path and is
imported only by tests, the smoke check and the CPU-baseline leg of the
benchmark; the product never routes through it.

Everything is numpy float64.  The steps are taken in the order and notation of
Algorithm 1 ("Fira with Adam", Appendix A.1); each function names the equation
or algorithm step it follows.  Nothing is blocked, fused or reordered.

Orientation.  Algorithm 1 is written for m <= n with a left projection
P (m x r): R = P^T G is r x n and the scaling factors are per column of G.
For m > n the footnote of Section 3.3 ("Gradient Low-Rank Projection") uses a
right projection Q (n x r): R = G Q is m x r.  Here that case is taken as the
whole algorithm applied to the transposed problem, so the factors are per row
of G.  `fira_step` handles it by literally transposing W and G, running the
m <= n code and transposing back.

Readings of the paper where it is silent or inconsistent:
  * Bias-correction exponent: Algorithm 1 starts at t = 0 and increments after
    the update, which read literally gives 0/0 on the first step.  The exponent
    used is s = t + 1, the number of Adam updates including the current one,
    as in Eq. 4's source (Adam).
  * alpha multiplies both terms, as Algorithm 1 writes
    G~ = alpha (P N + S).  `alpha_lowrank_only=True` gives the other reading,
    alpha P N + S.
  * phi uses the Algorithm-1 form with + eps in the denominator (Eq. 11 has
    none); the same eps as Adam's.
  * Limiter: the Algorithm-1 form S <- S * gamma / max(||S|| / (||S_prev|| + eps), gamma)
    (Eq. 12 is the same up to eps).  The remembered norm is the norm AFTER
    limiting, because Algorithm 1 overwrites S_t.  On a matrix's first step
    there is no previous norm and nothing is limited.  gamma = inf switches
    the limiter off.
  * Norms: Frobenius for matrices, l2 for columns.
  * A projection switch keeps M, V, the remembered norm and t (Section 4.2,
    "Loss spike analysis").
  * Ablation variants (Section 5.4 "Ablation Study", Eq. 6, 8, 9-10): `scaling`
    = "column" (Fira, Eq. 11), "matrix" (Fira-matrix: one factor
    ||N||_F / (||R||_F + eps) for the whole matrix, Eq. 9 with the same + eps),
    "none" (Fira-w.o.-scaling: the factor is 1; without the limiter this is
    GaLore-add, Eq. 8); `residual=False` drops S altogether (GaLore, Eq. 6): then
    there is no norm to limit or to remember.
  * Fira-only-scaling (appendix "Theoretical Analysis", item "Variability of Scaling
    Factor", and the only-scaling equation of the appendix on Fira versus full-rank
    Adam): W <- W - eta phi(R) G.  `only_scaling=True` takes it as Algorithm 1 with the
    scaled matrix S := G diag(k) in place of the scaled residual and without the P N
    term; alpha and the limiter act on that S exactly as they act on the residual in
    Algorithm 1 (alpha = 1 or `alpha_lowrank_only`, and gamma = inf, give the printed
    equation literally).  Column and matrix level as for `scaling`.
  * Other base optimizers (Algorithm 2 names Adam and RMSProp as examples of the
    adaptive optimizer; the appendix reports Fira + Adagrad): `psi` = "rmsprop" or
    "adagrad" replaces Eq. 2-4 by the textbook update of that optimizer on R; the
    paper gives no formulas for them.  M is then unused.
  * bf16 storage: when `store="bf16"` the new W is rounded to bfloat16
    (round to nearest, ties to even) after the update, because on that path W
    IS a bf16 tensor.  Nothing else is rounded.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np


@dataclasses.dataclass
class Hyper:
    """Inputs of Algorithm 1: eta (lr), beta1, beta2, eps, alpha, gamma."""
    lr: float = 1e-2
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    alpha: float = 0.25
    gamma: float = 1.01
    alpha_lowrank_only: bool = False
    scaling: str = "column"      # "column" | "matrix" | "none"
    psi: str = "adam"            # base optimizer psi_t: "adam" | "rmsprop" | "adagrad"
    residual: bool = True
    only_scaling: bool = False   # Fira-only-scaling: W <- W - eta phi(R) G


@dataclasses.dataclass
class State:
    """Optimizer state of one matrix (Table "Comparison": m r + 2 n r + 1 numbers,
    plus the step count).  M, V have the shape of R: r x n when m <= n, m x r
    when m > n.  prev_norm is None until the first step has stored ||S||."""
    M: np.ndarray
    V: np.ndarray
    prev_norm: Optional[float] = None
    t: int = 0

    def num_state_elements(self, proj: np.ndarray) -> int:
        return int(proj.size + self.M.size + self.V.size + 1)


def new_state(m: int, n: int, r: int) -> State:
    """M_0 = V_0 = 0, t = 0 (Algorithm 1, initialisation)."""
    shape = (r, n) if m <= n else (m, r)
    return State(M=np.zeros(shape), V=np.zeros(shape), prev_norm=None, t=0)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 to the nearest bfloat16 value (ties to even), returned as
    float64.  bfloat16 keeps 7 explicit mantissa bits, float64 has 52, so the
    low 45 bits are rounded away on the integer image of the number.  Valid for
    magnitudes in bfloat16's normal range (2^-126 .. 3.39e38) and for zero."""
    a = np.ascontiguousarray(x, dtype=np.float64)
    bits = a.view(np.uint64)
    drop = np.uint64(45)
    lsb = (bits >> drop) & np.uint64(1)
    bits = bits + (np.uint64((1 << 44) - 1) + lsb)
    bits = bits & ~np.uint64((1 << 45) - 1)
    return bits.view(np.float64).reshape(a.shape)


def adam_direction(R: np.ndarray, st: State, hp: Hyper) -> np.ndarray:
    """Eq. 2-4 applied to the low-rank gradient (Algorithm 1, the psi_t block):
    M <- b1 M + (1-b1) R;  V <- b2 V + (1-b2) R^2;
    N = sqrt(1-b2^s)/(1-b1^s) * M / (sqrt(V) + eps), element-wise, s = t+1."""
    if hp.psi == "rmsprop":     # Tieleman & Hinton: V <- b2 V + (1-b2) R^2, N = R / (sqrt V + eps)
        st.V = hp.beta2 * st.V + (1.0 - hp.beta2) * (R * R)
        return R / (np.sqrt(st.V) + hp.eps)
    if hp.psi == "adagrad":     # Duchi et al.: V <- V + R^2, N = R / (sqrt V + eps)
        st.V = st.V + R * R
        return R / (np.sqrt(st.V) + hp.eps)
    if hp.psi != "adam":
        raise ValueError(hp.psi)
    s = st.t + 1
    st.M = hp.beta1 * st.M + (1.0 - hp.beta1) * R
    st.V = hp.beta2 * st.V + (1.0 - hp.beta2) * (R * R)
    bias = math.sqrt(1.0 - hp.beta2 ** s) / (1.0 - hp.beta1 ** s)
    return bias * st.M / (np.sqrt(st.V) + hp.eps)


def column_factors(N: np.ndarray, R: np.ndarray, eps: float) -> np.ndarray:
    """Norm-based scaling, column level (Eq. 11 with Algorithm 1's + eps):
    k_i = ||N[:, i]|| / (||R[:, i]|| + eps)."""
    return np.sqrt((N * N).sum(axis=0)) / (np.sqrt((R * R).sum(axis=0)) + eps)


def matrix_factor(N: np.ndarray, R: np.ndarray, eps: float) -> float:
    """Norm-based scaling, matrix level (Eq. 9, with the + eps of Algorithm 1's
    column form): phi = ||N||_F / (||R||_F + eps)."""
    return float(np.sqrt((N * N).sum()) / (np.sqrt((R * R).sum()) + eps))


def limiter_factor(norm_S: float, prev_norm: Optional[float], hp: Hyper) -> float:
    """Norm-growth limiter (Eq. 12 in Algorithm 1's form):
    lambda = gamma / max(||S|| / (||S_prev|| + eps), gamma);  1 on the first step."""
    if prev_norm is None or math.isinf(hp.gamma):
        return 1.0
    return hp.gamma / max(norm_S / (prev_norm + hp.eps), hp.gamma)


def _step_left(W, G, P, st: State, hp: Hyper):
    """One pass of Algorithm 1's loop body for m <= n (P is m x r)."""
    R = P.T @ G                                   # low-rank gradient
    S = G - P @ R                                 # (I - P P^T) G
    N = adam_direction(R, st, hp)                 # psi_t(R_t)
    if not hp.residual:                           # GaLore (Eq. 6): W <- W - eta alpha P N
        st.t += 1
        diag = dict(k=np.zeros(G.shape[1]), lam=1.0, norm_scaled=0.0, norm_after=st.prev_norm, R=R, N=N)
        return W - hp.lr * hp.alpha * (P @ N), diag
    if hp.scaling == "column":
        k = column_factors(N, R, hp.eps)          # K
    elif hp.scaling == "matrix":
        k = np.full(G.shape[1], matrix_factor(N, R, hp.eps))
    elif hp.scaling == "none":
        k = np.ones(G.shape[1])
    else:
        raise ValueError(hp.scaling)
    if hp.only_scaling:                           # the factors act on the whole gradient
        S = G
    S = S * k[None, :]                            # S[:, i] <- k_i S[:, i]
    norm_scaled = float(np.sqrt((S * S).sum()))
    lam = limiter_factor(norm_scaled, st.prev_norm, hp)
    S = S * lam
    st.prev_norm = float(np.sqrt((S * S).sum()))  # norm after limiting
    low = np.zeros_like(G) if hp.only_scaling else P @ N
    if hp.alpha_lowrank_only:
        Gt = hp.alpha * low + S
    else:
        Gt = hp.alpha * (low + S)                 # G~ = alpha (P N + S)
    st.t += 1
    diag = dict(k=k, lam=lam, norm_scaled=norm_scaled, norm_after=st.prev_norm,
                R=R, N=N)
    return W - hp.lr * Gt, diag


def fira_step(W: np.ndarray, G: np.ndarray, proj: np.ndarray, st: State, hp: Hyper,
              store: Optional[str] = None):
    """One Fira update of one weight matrix.  proj is P (m x r) when m <= n and
    Q (n x r) when m > n.  Returns (W_new, diagnostics); st is updated in place.
    Diagnostics are in the orientation of the m <= n problem that was solved
    (for m > n: of the transposed problem)."""
    W = np.asarray(W, dtype=np.float64)
    G = np.asarray(G, dtype=np.float64)
    proj = np.asarray(proj, dtype=np.float64)
    m, n = G.shape
    if m <= n:
        Wn, diag = _step_left(W, G, proj, st, hp)
    else:
        st.M, st.V = st.M.T, st.V.T
        WnT, diag = _step_left(W.T, G.T, proj, st, hp)
        st.M, st.V = st.M.T, st.V.T
        Wn = WnT.T
    if store == "bf16":
        Wn = round_to_bf16(Wn)
    elif store == "f32":
        Wn = Wn.astype(np.float32).astype(np.float64)
    elif store is not None:
        raise ValueError(store)
    return np.ascontiguousarray(Wn), diag


def adam_dense_step(W: np.ndarray, G: np.ndarray, st: State, hp: Hyper, store: Optional[str] = None):
    """Eq. 1-4 for a parameter that is not projected (embeddings, output head, norm gains: the
    experiments follow GaLore's set-up, which leaves these to plain Adam):
    W <- W - eta psi_t(G) with the moments of Eq. 2-3 in the shape of W.  st.M, st.V have W's shape."""
    W = np.asarray(W, dtype=np.float64)
    G = np.asarray(G, dtype=np.float64)
    Wn = W - hp.lr * adam_direction(G, st, hp)
    st.t += 1
    if store == "bf16":
        Wn = round_to_bf16(Wn)
    elif store == "f32":
        Wn = Wn.astype(np.float32).astype(np.float64)
    elif store is not None:
        raise ValueError(store)
    return Wn


def refresh_projection(G: np.ndarray, r: int) -> np.ndarray:
    """Eq. 7: G = U Sigma V^T, P = [u_1 .. u_r] (m <= n); for m > n the first r
    right singular vectors (n x r).  Full SVD by the library routine."""
    G = np.asarray(G, dtype=np.float64)
    m, n = G.shape
    U, _, Vt = np.linalg.svd(G, full_matrices=False)
    return np.ascontiguousarray(U[:, :r] if m <= n else Vt[:r, :].T)


def principal_angles(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """Principal angles (radians, ascending) between the column spaces of A and
    B, both orthonormalised first.  The small angles are taken from the sines
    (singular values of (I - Qa Qa^T) Qb), which keeps precision near zero."""
    Qa, _ = np.linalg.qr(np.asarray(A, dtype=np.float64))
    Qb, _ = np.linalg.qr(np.asarray(B, dtype=np.float64))
    c = np.clip(np.linalg.svd(Qa.T @ Qb, compute_uv=False), 0.0, 1.0)
    s = np.clip(np.linalg.svd(Qb - Qa @ (Qa.T @ Qb), compute_uv=False), 0.0, 1.0)
    ang_c = np.sort(np.arccos(c))
    ang_s = np.sort(np.arcsin(s))
    return np.where(ang_c < 0.5, ang_s, ang_c)


def captured_energy(G: np.ndarray, proj: np.ndarray) -> float:
    """||P^T G||_F^2 (or ||G Q||_F^2 for m > n): the energy of G inside the
    subspace, to compare with the sum of the r largest sigma_i^2 of Eq. 7."""
    G = np.asarray(G, dtype=np.float64)
    proj = np.asarray(proj, dtype=np.float64)
    R = proj.T @ G if G.shape[0] <= G.shape[1] else G @ proj
    return float((R * R).sum())
