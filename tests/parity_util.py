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
# A Frobenius ratio over a whole matrix cannot see one wrong column, row or tile, so three local
# measures are bounded as well, each as a ratio (error / allowance) that must stay below 1; all are
# taken on the accumulated update dW = W_t - W_0 or on single elements of W.  Three effects make up the
# allowance on the bf16 path:
#   (a) arithmetic: the rank-r operand X of the back-projection (and N, R before it) is rounded to
#       bf16, which puts an error of about 2^-9 of the typical size of (Pi X) into every element of
#       W, however small the exact update of a particular column may be (so norms of columns and
#       rows of dW are floored at half their median).  Measured: 0.6 % of a column's norm (median),
#       2 % (worst column over 100 steps);
#   (b) storage: W is rounded to bf16 once per step on both sides.  After one step the two sides
#       round nearly equal numbers and differ by one spacing (ulp) at most (two across a binade
#       boundary), in a few per cent of the elements; over t steps the difference of an element
#       performs a lazy random walk, so its rms grows like sqrt(t) spacings (measured: about
#       0.3 sqrt(t)).  The spacing is taken at the largest magnitude the element has had so far.
#   (c) large entries of the rank-r operand: the rounding error of X[l][q] is proportional to
#       |X[l][q]| (and to |N|, |R|, rounded before it), not to the size of the net update.  Where the
#       projection has a column concentrated on one coordinate d (a gradient with a few dominant
#       columns gives such a basis) the terms k_l R_lq Pi_dq and k_l G_dl of the update nearly cancel,
#       so X[l][q] is many times larger than the element's update and its rounding error is no
#       longer a small share of s.  The allowance therefore carries the error model of the three
#       roundings: per step, var(dW[d][l]) = lr^2 (2^-9)^2 / 3 * sum_q Pi_dq^2 ((a N_lq)^2 +
#       (c_l R_lq)^2 + X_lq^2) with c_l = a lambda k_l, summed over the steps (independent roundings)
#       into A[d][l] from the ORACLE's N, R, k, lambda; an element may be off by ELEM_MODEL_SIGMAS
#       standard deviations sqrt(A) (the maximum of 10^7 to 10^8 samples), a column or row by
#       LINE_MODEL_SIGMAS times the root of its summed variance.  On matrices without such entries
#       this term is a few per cent of the others.
#  * col / row: ||err_col|| / (COL_ARITH ||dW_col|| + COL_WALK sqrt(t) ||ulp_col|| + the (c) term), largest over the
#    columns (rows).  A stale or misplaced column has ||err_col|| = ||dW_col||: a ratio of 5 to 30.
#  * bf16 elem: |err| / (U(t) ulp + ELEM_UPDATE_SHARE s + the (c) term) over all elements, U(t) = 2 + 1.5 sqrt(t - 1)
#    (the maximum of the walk over 10^7 elements), s the rms size of the update in the element's
#    column or row (the larger): the arithmetic error of one element is about 1 % of s, its maximum
#    over 10^7 elements about 6 %, whereas an element of a misplaced or stale tile is off by about s.
#  * fp32: no storage term; col / row relative to TOL_COL_F32 ||dW_col||; elem = the largest
#    |W_gpu - W_oracle| relative to max |W|, bounded by TOL_ELEM_F32.
COL_ARITH = 0.03
COL_WALK = 0.6
TOL_COL_F32 = 5e-4
TOL_ELEM_F32 = 1e-5
ELEM_UPDATE_SHARE = 0.1
ELEM_MODEL_SIGMAS = 6.0
LINE_MODEL_SIGMAS = 3.0
BF16_REL_VAR = (2.0 ** -9) ** 2 / 3.0


def max_ulp_bound(steps: int) -> float:
    """bf16: U(t), the ulp distance allowed to an element after `steps` steps."""
    return 2.0 + 1.5 * math.sqrt(max(steps - 1, 0))


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def rel_err(a: np.ndarray, b: np.ndarray) -> float:
    den = float(np.linalg.norm(b))
    return float(np.linalg.norm(a - b)) / (den if den > 0 else 1.0)


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    """Spacing of bfloat16 numbers (8 significant bits) at the magnitude of x."""
    e = np.floor(np.log2(np.maximum(np.abs(x), 2.0 ** -126)))
    return np.exp2(e - 7.0)


def local_errors(Wg: np.ndarray, Wo: np.ndarray, W0: np.ndarray, wmax: np.ndarray, kind: str, steps: int,
                 var: Optional[np.ndarray] = None, flip: Optional[np.ndarray] = None) -> dict:
    """Column-, row- and element-wise differences between the library's W and the oracle's, each
    divided by its allowance (see above).  wmax is the largest |W| that the oracle has held in each
    element so far; var (bf16) the accumulated variance A of the operand roundings per element; flip
    (bf16) the accumulated bound F of the changes of ill-conditioned direction elements."""
    err = Wg - Wo
    dO = Wo - W0
    e2, d2 = err * err, dO * dO
    ulp = bf16_ulp(wmax) if kind == "bf16" else None
    out, rms = {}, {}
    for name, ax in (("col", 0), ("row", 1)):
        den = np.sqrt(d2.sum(axis=ax))
        den = np.maximum(den, max(0.5 * float(np.median(den)), 1e-300))
        rms[name] = den / math.sqrt(err.shape[ax])
        if kind == "bf16":
            allow = COL_ARITH * den + COL_WALK * math.sqrt(steps) * np.sqrt((ulp * ulp).sum(axis=ax))
            if var is not None:
                allow = allow + LINE_MODEL_SIGMAS * np.sqrt(var.sum(axis=ax))
            if flip is not None:
                allow = allow + np.sqrt((flip.astype(np.float64) ** 2).sum(axis=ax))
        else:
            allow = TOL_COL_F32 * den
        out[name] = float((np.sqrt(e2.sum(axis=ax)) / allow).max())
    aerr = np.abs(err)
    if kind == "bf16":
        s = np.maximum(rms["col"][None, :], rms["row"][:, None])
        allow = max_ulp_bound(steps) * ulp + ELEM_UPDATE_SHARE * s
        if var is not None:
            allow = allow + ELEM_MODEL_SIGMAS * np.sqrt(var)
        if flip is not None:
            allow = allow + flip
        out["elem"] = float((aerr / allow).max())
        out["ulp"] = float((aerr / ulp).max())
        out["frac_off"] = float(np.count_nonzero(err) / err.size)
    else:
        out["elem"] = float(aerr.max() / max(float(np.abs(Wo).max()), 1e-300)) / TOL_ELEM_F32
    return out


# --- conditioning of Adam's direction at fp32 working precision -------------------------------------
# N = b M / (sqrt V + eps) is a steep function of R wherever sqrt V is of the order of eps: on a
# matrix's first step (M = V = 0 before it) N = R / (|R| + eps / sqrt(1 - beta2)), the sign of R
# smoothed over a width of about 3e-7.  An fp32 projection product carries an absolute error of about
# 2^-23 ||G_l|| in every element of R, so an element of R that happens to lie within that distance of
# zero gets a direction that is undetermined at working precision (anything between -1 and +1), while
# the fp64 oracle resolves it.  Such an element changes one column l of the update (N_l and k_l) and
# nothing else.  The fp32 bounds (1e-5 on W) leave no room for a single such element, so the fp32
# comparisons leave out the unprojected indices l for which the ORACLE's own numbers predict an error
# of N above N_ERR_MARK; how many were left out is bounded and what happened in them is checked for
# plausibility separately.
# The tensor-core path has the same property (bf16 operands multiply exactly, the sums are fp32; the
# measured error of its R is about 2^-22 ||G_l|| at d = 4096, taken as 2^-20 here).  Its Frobenius
# bounds are far above the effect, but one changed direction element (q, l) moves element (d, l) of W
# by lr a dN |Pi_dq|, which the element bound sees where r is small or the projection has large
# entries.  Nothing is left out of the bf16 comparisons; instead the allowances carry that term: for
# every element of N that the oracle's numbers show to be changeable (adam_direction_changes) the bound
# lr a dN |Pi_dq| is added to the allowance F[d][l] of the elements of line l, for good (W carries the
# difference forward; M and V do not: R is tiny there).  Lines are allowed the norm of their F entries.
N_ERR_MARK = {"f32": 5e-3, "bf16": 2e-2}
DOT_ERR = {"f32": 2.0 ** -23, "bf16": 2.0 ** -20}


def adam_direction_changes(R, G_l_norm, M0, V0, st_t_before: int, ohp: fo.Hyper, kind: str = "f32"):
    """The elements (q, l) of N that an error of the computed R of the size DOT_ERR ||G_l|| can change
    by more than a tenth of N_ERR_MARK, with the largest such change dN.  The change is evaluated, not
    linearised (N jumps by up to 2 where R crosses zero within that error), at the elements where the
    closeness of R to zero makes it possible at all.  R, M0, V0 are r x l (the
    oracle's orientation); M0, V0 are the moments BEFORE the step, st_t_before the steps taken before
    it.  Returns (q indices, l indices, dN)."""
    s = st_t_before + 1
    b = math.sqrt(1.0 - ohp.beta2 ** s) / (1.0 - ohp.beta1 ** s)
    err_l = DOT_ERR[kind] * G_l_norm
    thr = 0.1 * N_ERR_MARK[kind]

    def direction(Rx, M0x, V0x):
        M = ohp.beta1 * M0x + (1.0 - ohp.beta1) * Rx
        V = ohp.beta2 * V0x + (1.0 - ohp.beta2) * Rx * Rx
        return b * M / (np.sqrt(V) + ohp.eps)

    # N can be steep in R only where R itself is small (next to its own error, or next to what the
    # moments remember of earlier small values): everything else is left out before the evaluation
    cand = np.abs(R) < (512.0 * err_l)[None, :]
    qs, ls = np.nonzero(cand)
    if qs.size == 0:
        return qs, ls, np.zeros(0)
    Rc, Mc, Vc, ec = R[cand], M0[cand], V0[cand], err_l[ls]
    n0 = direction(Rc, Mc, Vc)
    dn = np.maximum(np.abs(direction(Rc + ec, Mc, Vc) - n0), np.abs(direction(Rc - ec, Mc, Vc) - n0))
    keep = dn > thr
    return qs[keep], ls[keep], dn[keep]


def adam_sensitive_indices(R, G_l_norm, M0, V0, st_t_before: int, ohp: fo.Hyper, kind: str = "f32") -> np.ndarray:
    """Boolean mask over the unprojected index l: True where some element of N can change by more than
    N_ERR_MARK (see adam_direction_changes)."""
    _, ls, dn = adam_direction_changes(R, G_l_norm, M0, V0, st_t_before, ohp, kind)
    out = np.zeros(R.shape[1], dtype=bool)
    out[np.unique(ls[dn > N_ERR_MARK[kind]])] = True
    return out


def rounding_variance(proj: np.ndarray, d: dict, ohp: fo.Hyper, left: bool) -> torch.Tensor:
    """One step's variance of the error that the bf16 roundings of N, R and X = a N - c_l R put into
    every element of W (in W's orientation, float32): lr^2 (2^-9)^2 / 3 * Pi^2 (a^2 N^2 + c^2 R^2 + X^2)
    with the oracle's N, R (r x l), k and lambda of that step.  This allowance (a bound, not an
    expected value) is formed with the tensor library, on the device when there is one: its one large
    product (d x r by r x l) would otherwise cost as much as a product of the oracle itself."""
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    N = torch.from_numpy(d["N"].astype(np.float32)).to(dev)
    R = torch.from_numpy(d["R"].astype(np.float32)).to(dev)
    a_low = float(ohp.alpha)
    if ohp.residual:
        c = torch.from_numpy(((1.0 if ohp.alpha_lowrank_only else ohp.alpha) * d["lam"] * d["k"]).astype(np.float32)).to(dev)
        cR = R * c[None, :]
    else:
        cR = torch.zeros_like(R)
    aN = a_low * N
    Y2 = aN * aN + cR * cR + (aN - cR) ** 2
    if ohp.residual and d["lam"] < 1.0:
        # the plain step forms X for lambda = 1 in the projection epilogue (one bf16 rounding) and
        # adds a_res (1 - lambda) k_l R where the limiter acted (a second one)
        X1 = aN - cR / float(d["lam"])
        Y2 = Y2 + X1 * X1
    P2 = torch.from_numpy((proj * proj).astype(np.float32)).to(dev)
    v = (P2 @ Y2) * float(ohp.lr ** 2 * BF16_REL_VAR)                      # d x l
    return v if left else v.T.contiguous()


def oracle_hyper(hp: fb.Hparams) -> fo.Hyper:
    return fo.Hyper(lr=hp.lr, beta1=hp.beta1, beta2=hp.beta2, eps=hp.eps, alpha=hp.alpha,
                    gamma=hp.gamma, alpha_lowrank_only=bool(hp.flags & fb.FLAG_ALPHA_LOWRANK_ONLY),
                    scaling=("matrix" if hp.flags & fb.FLAG_MATRIX_SCALING else
                             "none" if hp.flags & fb.FLAG_NO_SCALING else "column"),
                    residual=not (hp.flags & fb.FLAG_NO_RESIDUAL),
                    psi=("rmsprop" if hp.flags & fb.FLAG_PSI_RMSPROP else
                         "adagrad" if hp.flags & fb.FLAG_PSI_ADAGRAD else "adam"),
                    only_scaling=bool(hp.flags & fb.FLAG_ONLY_SCALING))


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
        self.local = {"col": 0.0, "row": 0.0, "elem": 0.0, "ulp": 0.0, "frac_off": 0.0}
        self.nsteps = 0
        # fp32 runs: unprojected indices whose direction was undetermined at working precision on
        # some step (see adam_sensitive_indices); sticky, since W carries the difference forward
        self.marked = {i: np.zeros(max(self.shapes[i]), dtype=bool) for i in self.check}
        self.wmax = {i: np.abs(self.W0[i]) for i in self.check}     # largest |W| seen per element (oracle)
        # bf16: accumulated variance of the operand roundings per element of W (see (c) above)
        self.var = {}                                              # (device tensors, created on the first step)
        # bf16: accumulated bound of the changes of ill-conditioned direction elements per element of W
        self.flip = {i: np.zeros(self.shapes[i], dtype=np.float32) for i in self.check} if self.kind == "bf16" else {}
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
        self.nsteps += 1
        for i in self.check:
            Wprev = self.Wo[i]
            m, n = self.shapes[i]
            left = m <= n
            track = ohp.psi == "adam" and not ohp.only_scaling
            if track:
                st = self.st[i]
                M0, V0, t0 = (st.M.copy(), st.V.copy(), st.t) if left else (st.M.T.copy(), st.V.T.copy(), st.t)
            G64 = to_np64(Gs[i])
            self.Wo[i], d = fo.fira_step(Wprev, G64, projs[i], self.st[i], ohp, store=self.kind)
            lam_row.append(d["lam"])
            self.wmax[i] = np.maximum(self.wmax[i], np.abs(self.Wo[i]))
            if track:
                gn = np.sqrt((G64 * G64).sum(axis=0 if left else 1))
                if self.kind == "f32":
                    self.marked[i] |= adam_sensitive_indices(d["R"], gn, M0, V0, t0, ohp, self.kind)
                else:
                    qs, ls, dn = adam_direction_changes(d["R"], gn, M0, V0, t0, ohp, self.kind)
                    F = self.flip[i] if left else self.flip[i].T          # d x l view
                    for q, l, x in zip(qs, ls, dn):
                        F[:, l] += np.float32(ohp.lr * ohp.alpha * x) * np.abs(projs[i][:, q]).astype(np.float32)
            if self.kind == "bf16" and not ohp.only_scaling:
                v = rounding_variance(projs[i], d, ohp, left)
                self.var[i] = v if i not in self.var else self.var[i] + v
            if compare:
                Wg = to_np64(self.W[i])
                Wo, W0, wmax, flip = self.Wo[i], self.W0[i], self.wmax[i], self.flip.get(i)
                var = self.var[i].cpu().numpy() if i in self.var else None
                if self.marked[i].any():
                    keep = ~self.marked[i]
                    self.check_marked(i, Wg, Wo, W0, left)
                    sel = (slice(None), keep) if left else (keep, slice(None))
                    Wg, Wo, W0, wmax = Wg[sel], Wo[sel], W0[sel], wmax[sel]
                    var = None if var is None else var[sel]
                    flip = None if flip is None else flip[sel]
                self.max_w = max(self.max_w, rel_err(Wg, Wo))
                self.max_dw = max(self.max_dw, rel_err(Wg - W0, Wo - W0))
                for k, v in local_errors(Wg, Wo, W0, wmax, self.kind, self.nsteps, var, flip).items():
                    self.local[k] = max(self.local[k], v)
        self.lams.append(lam_row)
        return lam_row

    def check_marked(self, i, Wg, Wo, W0, left):
        """The indices left out of the fp32 comparison are few, and what the library wrote there is an
        update of the right size and direction (a direction element flipped between -1 and +1 moves one
        column of the update by at most 2 / sqrt(r) of its norm per flipped element)."""
        mk = self.marked[i]
        assert mk.mean() <= 0.02, f"matrix {i}: {mk.sum()} of {mk.size} indices marked as sensitive"
        sel = (slice(None), mk) if left else (mk, slice(None))
        dg, do = Wg[sel] - W0[sel], Wo[sel] - W0[sel]
        ax = 0 if left else 1
        err = np.sqrt(((dg - do) ** 2).sum(axis=ax)) / np.maximum(np.sqrt((do ** 2).sum(axis=ax)), 1e-300)
        assert err.max() <= 0.5, f"matrix {i}: a sensitive index is off by {err.max():.2f} of its update"

    def summary(self) -> str:
        return (f"steps {self.nsteps} W {self.max_w:.2e} dW {self.max_dw:.2e} col {self.local['col']:.2e} "
                f"row {self.local['row']:.2e} elem {self.local['elem']:.2e} ulp {self.local['ulp']:.2f} "
                f"off {self.local['frac_off']:.3f} marked {sum(int(v.sum()) for v in self.marked.values())}")

    def assert_ok(self, tol_w=None, tol_dw=None):
        tol_w = TOL_W[self.kind] if tol_w is None else tol_w
        tol_dw = TOL_DW[self.kind] if tol_dw is None else tol_dw
        print("parity:", self.summary())
        assert self.f.poll() == 0
        assert math.isfinite(self.max_w) and self.max_w <= tol_w, (self.max_w, tol_w)
        assert math.isfinite(self.max_dw) and self.max_dw <= tol_dw, (self.max_dw, tol_dw)
        # column, row and element errors as fractions of their allowances
        assert self.local["col"] <= 1.0 and self.local["row"] <= 1.0 and self.local["elem"] <= 1.0, self.summary()


def workload_trajectory(wl: wk.Workload, steps: int, device="cuda", gen_device="cpu",
                        check: Optional[Sequence[int]] = None, flags: int = 0,
                        refresh_at=(), refresh_iters=-1, compare_steps=None) -> Trajectory:
    """Runs `steps` steps of a named workload.  Projections come from the seeded
    random orthonormal generator unless `refresh_at` lists 0-based step counts at
    which the library's own refresh runs first (as Algorithm 1's t mod T branch).
    compare_steps: the 1-based steps after which W is compared (default: every step); the
    oracle runs every step in any case, since it carries its own state."""
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
        tr.step(Gs, compare=compare_steps is None or s in compare_steps)
    return tr


def residual_jump(G: torch.Tensor, proj: torch.Tensor, mult: float = 9.0) -> torch.Tensor:
    """G + mult * (the part of G outside the projection's subspace): a jump that the
    column factors do not absorb (they scale with 1/||R||, and R is unchanged), so the
    norm of the scaled residual grows by about 1 + mult and the limiter must act."""
    G64, P64 = G.to(torch.float64), proj.to(torch.float64).cpu()
    m, n = G.shape
    resid = G64 - P64 @ (P64.T @ G64) if m <= n else G64 - (G64 @ P64) @ P64.T
    return (G64 + mult * resid).to(G.dtype)
