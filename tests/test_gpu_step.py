"""GPU parity of fira_step against the fp64 oracle (through the C ABI)."""
import math

import numpy as np
import pytest
import torch

from oracle import fira_oracle as fo
from paper_2410_01623_b200 import binding as fb
from paper_2410_01623_b200 import workloads as wk
from tests.parity_util import Trajectory, rel_err, residual_jump, to_np64, workload_trajectory

pytestmark = pytest.mark.gpu


def test_single_matrix_workload_with_spike():
    """The single 512 x 1376, r = 128 fp32 matrix: 10 steps, spike at step 6."""
    wl = wk.workload("single-60m")
    tr = workload_trajectory(wl, wl.steps)
    tr.assert_ok()
    lams = [row[0] for row in tr.lams]
    assert lams[5] < 1.0                      # the spike step is limited
    assert all(l == 1.0 for l in lams[:5])
    d = tr.f.diagnostics(0)
    assert d["t"] == wl.steps and d["engine"] == 0
    assert d["norm_prev"] == pytest.approx(tr.st[0].prev_norm, rel=1e-4)
    assert tr.f.state_elements(0) == 512 * 128 + 2 * 1376 * 128 + 1


def _random_case(shapes, r, dtype, steps, seed, hp=None, spike=None, flags=0):
    g = torch.Generator().manual_seed(seed)
    hp = hp or fb.make_hparams(lr=1e-2, alpha=0.25, gamma=1.01, flags=flags)
    W0 = [(torch.randn(m, n, generator=g) * 0.02).to(dtype) for (m, n) in shapes]
    tr = Trajectory(shapes, r, dtype, hp, W0)
    Ps = []
    for i, (m, n) in enumerate(shapes):
        q, _ = torch.linalg.qr(torch.randn(min(m, n), tr.f.ranks[i], generator=g, dtype=torch.float64))
        Ps.append(q.to(dtype))
        tr.f.set_projection(i, Ps[i].cuda())
    scales = [torch.exp(torch.randn(n, generator=g)) for (_, n) in shapes]
    for s in range(1, steps + 1):
        Gs = [(torch.randn(m, n, generator=g) * scales[i][None, :]).to(dtype)
              for i, (m, n) in enumerate(shapes)]
        if spike and s in spike:      # a jump outside the subspace, which the limiter must cut
            Gs = [residual_jump(G, Ps[i]) for i, G in enumerate(Gs)]
        tr.step(Gs)
    return tr


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_ragged_shapes_both_orientations(dtype):
    # several 64-wide tiles plus ragged tails in every extent; left, right and square
    shapes = [(150, 333), (333, 150), (130, 130), (64, 200), (7, 9), (9, 7)]
    ranks = [37, 37, 64, 64, 3, 7]
    tr = _random_case(shapes, ranks, dtype, steps=6, seed=3, spike=(4,))
    tr.assert_ok()
    assert any(l < 1.0 for row in tr.lams for l in row)


def test_full_rank_projection_has_no_residual():
    # r = d with an orthonormal basis: S = 0, the step is Adam through the projection
    tr = _random_case([(48, 80)], 48, torch.float32, steps=3, seed=5)
    tr.assert_ok()
    assert tr.f.diagnostics(0)["norm_prev"] < 1e-4


def test_alpha_lowrank_only_flag():
    tr = _random_case([(96, 160), (160, 96)], 16, torch.float32, steps=4, seed=7,
                      flags=fb.FLAG_ALPHA_LOWRANK_ONLY)
    tr.assert_ok()


@pytest.mark.parametrize("flags", [fb.FLAG_MATRIX_SCALING, fb.FLAG_NO_SCALING, fb.FLAG_NO_RESIDUAL,
                                   fb.FLAG_NO_SCALING | fb.FLAG_ALPHA_LOWRANK_ONLY])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_ablation_variants(flags, dtype):
    """Fira-matrix, Fira-w.o.-scaling and GaLore (Section 5.4, Eq. 6, 8, 9) as switches of the
    same kernels, both orientations, with a jump that the limiter must cut where there is one."""
    tr = _random_case([(150, 333), (333, 150), (64, 200)], [37, 37, 16], dtype, steps=5, seed=19,
                      spike=(4,), flags=flags)
    tr.assert_ok()
    for i in range(3):
        d = tr.f.diagnostics(i)
        if flags & fb.FLAG_NO_RESIDUAL:
            assert tr.st[i].prev_norm is None and d["lam"] == 1.0
        else:
            assert d["norm_prev"] == pytest.approx(tr.st[i].prev_norm, rel=1e-3 if dtype == torch.float32 else 2e-2)
            if flags & fb.FLAG_MATRIX_SCALING:
                assert d["k_min"] == d["k_max"]
            if flags & fb.FLAG_NO_SCALING:
                assert d["k_min"] == d["k_max"] == 1.0
    if not flags & fb.FLAG_NO_RESIDUAL:
        assert any(l < 1.0 for row in tr.lams for l in row)


@pytest.mark.parametrize("flags", [fb.FLAG_ONLY_SCALING, fb.FLAG_ONLY_SCALING | fb.FLAG_MATRIX_SCALING])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_only_scaling_variant(flags, dtype):
    """Fira-only-scaling, W <- W - eta phi(R) G, column and matrix level, both orientations: the
    factors multiply the whole gradient, there is no P N term, and the limiter acts on ||G diag k||."""
    tr = _random_case([(150, 333), (333, 150), (64, 200)], [37, 37, 16], dtype, steps=5, seed=53,
                      spike=(4,), flags=flags)
    tr.assert_ok()
    assert any(l < 1.0 for row in tr.lams for l in row)
    for i in range(3):
        d = tr.f.diagnostics(i)
        assert d["t"] == 5
        assert d["norm_prev"] == pytest.approx(tr.st[i].prev_norm, rel=1e-3 if dtype == torch.float32 else 2e-2)
        M, V, pn, t = tr.f.get_state(i)                    # the moments advance as in the ordinary step
        Mo = tr.st[i].M.T if tr.shapes[i][0] <= tr.shapes[i][1] else tr.st[i].M
        assert rel_err(to_np64(M), Mo) < 1e-4


def test_only_scaling_printed_equation_on_the_device():
    """alpha dropped from the scaled term and gamma = inf: (W_0 - W_1) / eta is G with column j
    multiplied by k_j, element by element."""
    hp = fb.make_hparams(lr=0.05, gamma=math.inf, flags=fb.FLAG_ONLY_SCALING | fb.FLAG_ALPHA_LOWRANK_ONLY)
    tr = _random_case([(96, 160)], 16, torch.float32, steps=1, seed=59, hp=hp)
    tr.assert_ok()
    assert all(l == 1.0 for row in tr.lams for l in row)
    d = tr.f.diagnostics(0)
    assert d["k_max"] > d["k_min"] > 0
    # every column of the update is a multiple of the same column of G, with a factor inside [k_min, k_max]
    upd = (tr.W0[0] - to_np64(tr.W[0])) / 0.05
    Wo_upd = (tr.W0[0] - tr.Wo[0]) / 0.05
    kcol = (upd * Wo_upd).sum(axis=0) / (Wo_upd * Wo_upd).sum(axis=0)
    np.testing.assert_allclose(kcol, 1.0, rtol=1e-5)


def test_variant_flags_that_exclude_each_other_are_rejected():
    with pytest.raises(fb.FiraError):
        fb.Fira([(64, 96)], 8, torch.float32, fb.make_hparams(flags=fb.FLAG_ONLY_SCALING | fb.FLAG_NO_RESIDUAL))
    with pytest.raises(fb.FiraError):
        fb.Fira([(64, 96)], 8, torch.float32, fb.make_hparams(flags=fb.FLAG_MATRIX_SCALING | fb.FLAG_NO_SCALING))
    with pytest.raises(fb.FiraError):
        fb.Fira([(64, 96)], 8, torch.float32, fb.make_hparams(flags=fb.FLAG_PSI_RMSPROP | fb.FLAG_PSI_ADAGRAD))


@pytest.mark.parametrize("flags", [fb.FLAG_PSI_RMSPROP, fb.FLAG_PSI_ADAGRAD, fb.FLAG_PSI_ADAGRAD | fb.FLAG_MATRIX_SCALING])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_other_base_optimizers(flags, dtype):
    """RMSProp and Adagrad as the base optimizer (Algorithm 2's "adaptive optimizer" slot): M stays
    zero, V follows the other rule, the factors and the limiter act on the new direction."""
    tr = _random_case([(150, 333), (333, 150)], 37, dtype, steps=5, seed=23, spike=(4,), flags=flags,
                      hp=fb.make_hparams(lr=1e-2, alpha=0.25, gamma=1.01, beta2=0.95, flags=flags))
    tr.assert_ok()
    for i in range(2):
        M, V, pn, t = tr.f.get_state(i)
        assert float(M.abs().max()) == 0.0
        Vo = tr.st[i].V.T if tr.shapes[i][0] <= tr.shapes[i][1] else tr.st[i].V
        assert rel_err(to_np64(V), Vo) < 1e-5
        assert pn == pytest.approx(tr.st[i].prev_norm, rel=1e-3 if dtype == torch.float32 else 2e-2)


@pytest.mark.parametrize("gamma", [math.inf, 1.0])
def test_gamma_extremes(gamma):
    hp = fb.make_hparams(gamma=gamma)
    tr = _random_case([(100, 140)], 20, torch.float32, steps=5, seed=11, hp=hp, spike=(3,))
    tr.assert_ok()
    lams = [row[0] for row in tr.lams]
    if math.isinf(gamma):
        assert all(l == 1.0 for l in lams)
    else:
        assert lams[2] < 0.5                       # the jump at step 3 is cut back


def test_zero_gradient_and_zero_columns():
    shapes = [(40, 70)]
    hp = fb.make_hparams()
    g = torch.Generator().manual_seed(1)
    W0 = [torch.randn(40, 70, generator=g) * 0.02]
    tr = Trajectory(shapes, 8, torch.float32, hp, W0)
    q, _ = torch.linalg.qr(torch.randn(40, 8, generator=g, dtype=torch.float64))
    tr.f.set_projection(0, q.float().cuda())
    G = torch.randn(40, 70, generator=g)
    G[:, 5] = 0.0
    tr.step([G])
    tr.step([torch.zeros(40, 70)])          # k = ||N|| / eps is huge, S = 0: finite result
    tr.step([G])
    tr.assert_ok()
    assert torch.isfinite(tr.W[0]).all()


def test_per_call_learning_rate_and_pointer_change():
    shapes = [(70, 90)]
    g = torch.Generator().manual_seed(2)
    W0 = [torch.randn(70, 90, generator=g) * 0.02]
    tr = Trajectory(shapes, 10, torch.float32, fb.make_hparams(lr=1e-2), W0)
    q, _ = torch.linalg.qr(torch.randn(70, 10, generator=g, dtype=torch.float64))
    tr.f.set_projection(0, q.float().cuda())
    tr.step([torch.randn(70, 90, generator=g)], lr=3e-3)
    # move W to a new allocation: the library must follow the new pointer
    tr.W = [tr.W[0].clone()]
    tr.step([torch.randn(70, 90, generator=g)], lr=5e-2)
    tr.assert_ok()


def test_checkpoint_resume_is_bitwise():
    shapes = [(96, 130), (130, 96)]
    hp = fb.make_hparams()
    g = torch.Generator().manual_seed(4)
    W0 = [torch.randn(m, n, generator=g) * 0.02 for (m, n) in shapes]
    Ps = [torch.linalg.qr(torch.randn(96, 12, generator=g, dtype=torch.float64))[0].float().cuda()
          for _ in shapes]
    Gs = [[torch.randn(m, n, generator=g).cuda() for (m, n) in shapes] for _ in range(6)]

    def run(n_first):
        f = fb.Fira(shapes, 12, torch.float32, hp)
        for i in range(2):
            f.set_projection(i, Ps[i])
        W = [w.cuda().clone() for w in W0]
        for s in range(n_first):
            f.step(W, Gs[s])
        return f, W

    f_all, W_all = run(6)
    f_a, W_a = run(3)
    saved = [f_a.get_state(i) for i in range(2)]
    projs = [f_a.get_projection(i) for i in range(2)]
    f_b = fb.Fira(shapes, 12, torch.float32, hp)
    for i in range(2):
        f_b.set_projection(i, projs[i])
        M, V, pn, t = saved[i]
        assert t == 3 and pn is not None
        f_b.set_state(i, M, V, pn, t)
    for s in range(3, 6):
        f_b.step(W_a, Gs[s])
    torch.cuda.synchronize()
    for i in range(2):
        assert torch.equal(W_a[i], W_all[i])
        Ma, Va, pa, ta = f_all.get_state(i)
        Mb, Vb, pb, tb = f_b.get_state(i)
        assert torch.equal(Ma, Mb) and torch.equal(Va, Vb) and pa == pb and ta == tb == 6


def test_moments_match_oracle_layout():
    tr = _random_case([(60, 100), (100, 60)], 9, torch.float32, steps=3, seed=13)
    for i, (m, n) in enumerate(tr.shapes):
        M, V, pn, t = tr.f.get_state(i)
        Mo = tr.st[i].M.T if m <= n else tr.st[i].M      # library layout is l x r
        Vo = tr.st[i].V.T if m <= n else tr.st[i].V
        assert rel_err(to_np64(M), Mo) < 1e-5
        assert rel_err(to_np64(V), Vo) < 1e-5
        assert pn == pytest.approx(tr.st[i].prev_norm, rel=1e-4)
        assert t == 3


def test_run_twice_is_bitwise_deterministic():
    a = _random_case([(150, 333), (333, 150)], 37, torch.bfloat16, steps=4, seed=21, spike=(3,))
    b = _random_case([(150, 333), (333, 150)], 37, torch.bfloat16, steps=4, seed=21, spike=(3,))
    for x, y in zip(a.W, b.W):
        assert torch.equal(x, y)


def test_nonfinite_gradient_is_flagged():
    f = fb.Fira([(32, 48)], 4, torch.float32, fb.make_hparams())
    W = [torch.zeros(32, 48, device="cuda")]
    G = torch.ones(32, 48, device="cuda")
    G[3, 3] = float("inf")
    f.set_projection(0, torch.eye(32, 4, device="cuda"))
    f.step(W, [G])
    assert f.poll() == 6
    assert f.poll() == 0      # cleared by the previous poll


def test_step_argument_errors():
    f = fb.Fira([(32, 48)], 4, torch.float32, fb.make_hparams())
    W = torch.zeros(32, 48, device="cuda")
    with pytest.raises(fb.FiraError) as e:
        f.step([W], [None])
    assert e.value.status == 1
    with pytest.raises(fb.FiraError):
        f.step([W], [W], lr=float("nan"))
    assert f.L.fira_get_diagnostics(f.ctx, 5, None) == 1
    assert f.diagnostics(0)["t"] == 0


def test_step_host_matches_device_step():
    shapes = [(96, 130), (130, 96)]
    hp = fb.make_hparams()
    g = torch.Generator().manual_seed(8)
    W0 = [torch.randn(m, n, generator=g) * 0.02 for (m, n) in shapes]
    Gs = [torch.randn(m, n, generator=g) for (m, n) in shapes]
    Ps = [torch.linalg.qr(torch.randn(96, 12, generator=g, dtype=torch.float64))[0].float().cuda()
          for _ in shapes]
    fa = fb.Fira(shapes, 12, torch.float32, hp)
    fh = fb.Fira(shapes, 12, torch.float32, hp)
    for i in range(2):
        fa.set_projection(i, Ps[i])
        fh.set_projection(i, Ps[i])
    Wd = [w.cuda().clone() for w in W0]
    fa.step(Wd, [x.cuda() for x in Gs])
    Wh = [w.clone().pin_memory() for w in W0]
    Gh = [x.clone().pin_memory() for x in Gs]
    staging = torch.empty(fh.staging_bytes(), dtype=torch.uint8, device="cuda")
    fh.step_host(Wh, Gh, staging)
    torch.cuda.synchronize()
    for i in range(2):
        assert torch.equal(Wh[i], Wd[i].cpu())


@pytest.mark.parametrize("dtype,shape,r,pad", [(torch.float32, (150, 333), 37, 5), (torch.float32, (333, 150), 37, 3),
                                               (torch.bfloat16, (512, 768), 128, 8), (torch.bfloat16, (768, 512), 128, 64),
                                               (torch.bfloat16, (512, 768), 128, 3), (torch.bfloat16, (300, 333), 37, 1),
                                               (torch.bfloat16, (512, 765), 128, 3), (torch.bfloat16, (768, 509), 128, 3),
                                               (torch.bfloat16, (765, 512), 128, 8)])
def test_padded_row_pitch(dtype, shape, r, pad):
    """W and G as views of wider buffers (ld = n + pad): the CUDA-core kernels, the tensor-core
    kernels reading in place (pitch and width multiples of 8 elements) and through aligned copies
    (odd pitch, or an odd width without the caller's leave to write the padding).  The padding
    columns must come back untouched."""
    m, n = shape
    ld = n + pad
    g = torch.Generator().manual_seed(m + pad)
    hp = fb.make_hparams(lr=1e-2, alpha=0.25, gamma=1.01)
    f = fb.Fira([shape], r, dtype, hp, lds=[ld])
    q, _ = torch.linalg.qr(torch.randn(min(m, n), r, generator=g, dtype=torch.float64))
    f.set_projection(0, q.to(dtype).cuda())
    P = to_np64(f.get_projection(0))
    Wbuf = torch.full((m, ld), 7.0, dtype=dtype, device="cuda")
    Gbuf = torch.full((m, ld), float("nan"), dtype=dtype, device="cuda")     # the padding is never read
    W0 = (torch.randn(m, n, generator=g) * 0.02).to(dtype)
    Wbuf[:, :n] = W0.cuda()
    st = fo.new_state(m, n, r)
    ohp = fo.Hyper(lr=hp.lr, alpha=hp.alpha, gamma=hp.gamma, eps=hp.eps)
    Wo = to_np64(W0)
    kind = "bf16" if dtype == torch.bfloat16 else "f32"
    for s_ in range(3):
        G = torch.randn(m, n, generator=g).to(dtype)
        Gbuf[:, :n] = G.cuda()
        f.step([Wbuf], [Gbuf])
        Wo, _ = fo.fira_step(Wo, to_np64(G), P, st, ohp, store=kind)
    assert f.poll() == 0
    assert rel_err(to_np64(Wbuf[:, :n]), Wo) <= (2e-2 if dtype == torch.bfloat16 else 1e-5)
    assert rel_err(to_np64(Wbuf[:, :n]) - to_np64(W0), Wo - to_np64(W0)) <= (3e-2 if dtype == torch.bfloat16 else 2e-4)
    assert (Wbuf[:, n:] == 7.0).all()



@pytest.mark.parametrize("shape,ld", [((512, 765), 776), ((768, 509), 520), ((765, 512), 512)])
def test_row_padding_writable_lets_odd_widths_run_in_place(shape, ld):
    """FIRA_FLAG_ROW_PADDING_WRITABLE: rows that start on 16-byte boundaries are worked on where they
    are even if the width is not a multiple of 8 (no staging kernels: 6 launches, not 8); the stores
    may then overwrite the padding up to the next multiple of 8 elements, and nothing beyond it.
    G's padding holds NaN: it must never enter the result."""
    m, n = shape
    g = torch.Generator().manual_seed(m + n)
    hp = fb.make_hparams(lr=1e-2, alpha=0.25, gamma=1.01, flags=fb.FLAG_ROW_PADDING_WRITABLE)
    f = fb.Fira([shape], 128, torch.bfloat16, hp, lds=[ld])
    q, _ = torch.linalg.qr(torch.randn(min(m, n), 128, generator=g, dtype=torch.float64))
    f.set_projection(0, q.to(torch.bfloat16).cuda())
    P = to_np64(f.get_projection(0))
    Wbuf = torch.full((m, ld), 7.0, dtype=torch.bfloat16, device="cuda")
    Gbuf = torch.full((m, ld), float("nan"), dtype=torch.bfloat16, device="cuda")
    W0 = (torch.randn(m, n, generator=g) * 0.02).to(torch.bfloat16)
    Wbuf[:, :n] = W0.cuda()
    st = fo.new_state(m, n, 128)
    ohp = fo.Hyper(lr=hp.lr, alpha=hp.alpha, gamma=hp.gamma, eps=hp.eps)
    Wo = to_np64(W0)
    for _ in range(3):
        G = torch.randn(m, n, generator=g).to(torch.bfloat16)
        Gbuf[:, :n] = G.cuda()
        f.step([Wbuf[:, :n]], [Gbuf[:, :n]])
        Wo, _ = fo.fira_step(Wo, to_np64(G), P, st, ohp, store="bf16")
    assert f.poll() == 0 and f.diagnostics(0)["engine"] == 1
    assert f.last_step_launches() == 6
    assert rel_err(to_np64(Wbuf[:, :n]), Wo) <= 2e-2
    assert rel_err(to_np64(Wbuf[:, :n]) - to_np64(W0), Wo - to_np64(W0)) <= 3e-2
    assert (Wbuf[:, (n + 7) // 8 * 8:] == 7.0).all()
    assert torch.isnan(Gbuf[:, n:]).all()
