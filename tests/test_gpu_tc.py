"""GPU parity of the bf16 tensor-core (tcgen05) step kernels against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import fira_oracle as fo
from paper_2410_01623_b200 import binding as fb
from paper_2410_01623_b200 import workloads as wk
from tests.parity_util import Trajectory, rel_err, residual_jump, to_np64, workload_trajectory

pytestmark = pytest.mark.gpu


def _case(shapes, r, steps, seed, spike=(), hp=None, flags=0):
    g = torch.Generator().manual_seed(seed)
    hp = hp or fb.make_hparams(lr=1e-2, alpha=0.25, gamma=1.01, flags=flags)
    W0 = [(torch.randn(m, n, generator=g) * 0.02).to(torch.bfloat16) for (m, n) in shapes]
    tr = Trajectory(shapes, r, torch.bfloat16, hp, W0)
    Ps = []
    for i, (m, n) in enumerate(shapes):
        q, _ = torch.linalg.qr(torch.randn(min(m, n), tr.f.ranks[i], generator=g, dtype=torch.float64))
        Ps.append(q.to(torch.bfloat16))
        tr.f.set_projection(i, Ps[i].cuda())
    scales = [torch.exp(torch.randn(n, generator=g)) for (_, n) in shapes]
    for s in range(1, steps + 1):
        Gs = [(torch.randn(m, n, generator=g) * scales[i][None, :]).to(torch.bfloat16)
              for i, (m, n) in enumerate(shapes)]
        if s in spike:                # a jump outside the subspace, which the limiter must cut
            Gs = [residual_jump(G, Ps[i]) for i, G in enumerate(Gs)]
        tr.step(Gs)
    return tr


@pytest.mark.parametrize("shape,r", [((512, 768), 128), ((768, 512), 128), ((256, 256), 128),
                                     ((384, 1000), 256), ((1000, 384), 256), ((512, 1376), 384)])
def test_first_step_moments_expose_the_projection_product(shape, r):
    """After one step M = (1 - beta1) R, so M checks the projection product (both operand
    layouts, ragged tile edges) on its own, and V = (1 - beta2) R^2."""
    tr = _case([shape], r, steps=1, seed=shape[0] + r)
    assert tr.f.diagnostics(0)["engine"] == 1
    M, V, pn, t = tr.f.get_state(0)
    m, n = shape
    Mo = tr.st[0].M.T if m <= n else tr.st[0].M
    Vo = tr.st[0].V.T if m <= n else tr.st[0].V
    assert rel_err(to_np64(M), Mo) < 1e-5          # bf16 inputs are exact, fp32 accumulation
    assert rel_err(to_np64(V), Vo) < 1e-5
    assert t == 1
    # ||S|| comes from the column identity ||S_l||^2 = ||G_l||^2 - ||R_l||^2
    assert pn == pytest.approx(tr.st[0].prev_norm, rel=2e-2)
    tr.assert_ok()


@pytest.mark.parametrize("shape,r", [((512, 768), 128), ((768, 512), 128), ((1024, 1280), 512), ((1280, 1024), 512)])
def test_axis_projection_pins_the_sums_of_g_squared(shape, r):
    """With coordinate axes as the projection (orthonormal and exact in bf16) the column identity
    ||S_l||^2 = ||G_l||^2 - ||R_l||^2 is exact, so the remembered norm checks the fused sums of G^2
    (every k-block, both CTAs of a pair, every r-tile's share) far below the bf16 tolerance."""
    m, n = shape
    g = torch.Generator().manual_seed(m + r)
    hp = fb.make_hparams(lr=1e-2, alpha=0.25, gamma=1.01)
    W0 = [(torch.randn(m, n, generator=g) * 0.02).to(torch.bfloat16)]
    tr = Trajectory([shape], r, torch.bfloat16, hp, W0)
    d = min(m, n)
    P = torch.zeros(d, r)
    P[torch.randperm(d, generator=g)[:r], torch.arange(r)] = 1.0
    tr.f.set_projection(0, P.to(torch.bfloat16).cuda())
    for s in range(2):
        tr.step([(torch.randn(m, n, generator=g) * torch.exp(torch.randn(n, generator=g))[None, :]).to(torch.bfloat16)])
        assert tr.f.diagnostics(0)["norm_prev"] == pytest.approx(tr.st[0].prev_norm, rel=2e-4)
    assert tr.f.diagnostics(0)["engine"] == 1
    tr.assert_ok()


def test_mixed_list_left_right_square_with_limiter():
    shapes = [(512, 1376), (1376, 512), (512, 512), (256, 2048), (640, 264)]
    tr = _case(shapes, [128, 128, 128, 256, 128], steps=6, seed=17, spike=(4,))
    assert [tr.f.diagnostics(i)["engine"] for i in range(5)] == [1, 1, 1, 1, 1]
    tr.assert_ok()
    # the jump at step 4 is cut on every matrix that has a residual (matrix 3 has r = d)
    assert all(l < 0.5 for i, l in enumerate(tr.lams[3]) if i != 3)
    for i in range(5):
        d = tr.f.diagnostics(i)
        if i != 3:
            assert d["norm_prev"] == pytest.approx(tr.st[i].prev_norm, rel=2e-2)
        assert d["t"] == 6


def test_x_formed_in_the_projection_epilogue_with_ragged_rows_and_limiter():
    """Projected extent 4096 with rank 512: two r-tiles per row of tiles, so the projection epilogues
    of two CTA pairs exchange their partial row sums before they form X, here with a ragged last
    row of tiles (4200 = 16 x 256 + 104), in both orientations, mixed in one list with a matrix
    whose X still comes from the separate pass (d = 1024, two r-tiles) and one with a single r-tile;
    a jump at step 3 makes the limiter act, which exercises the correction pass on X."""
    shapes = [(4096, 4200), (4200, 4096), (1024, 1536), (640, 512)]
    tr = _case(shapes, [512, 512, 512, 256], steps=4, seed=77, spike=(3,))
    assert [tr.f.diagnostics(i)["engine"] for i in range(4)] == [1, 1, 1, 1]
    tr.assert_ok()
    assert all(l < 0.5 for l in tr.lams[2])
    for i in range(4):
        assert tr.f.diagnostics(i)["norm_prev"] == pytest.approx(tr.st[i].prev_norm, rel=2e-2)


def test_odd_widths_run_on_tensor_cores_through_aligned_copies():
    """Rows of an odd-width bf16 matrix are not 16-byte aligned, which TMA needs: the library
    works on copies with an aligned pitch and writes W back.  Odd heights need nothing special."""
    shapes = [(512, 1365), (1365, 512), (515, 1365), (1367, 517)]
    tr = _case(shapes, 128, steps=4, seed=41, spike=(3,))
    assert [tr.f.diagnostics(i)["engine"] for i in range(4)] == [1, 1, 1, 1]
    tr.assert_ok()
    for i in range(4):
        assert tr.f.diagnostics(i)["norm_prev"] == pytest.approx(tr.st[i].prev_norm, rel=2e-2)


def test_mixed_engines_in_one_context():
    # the odd-width matrix cannot be loaded by TMA (rows not 16-byte aligned) and a rank that is
    # not a multiple of 128 does not fit the tensor-core tiles: CUDA-core kernels
    shapes = [(512, 768), (300, 333), (768, 512), (512, 512)]
    tr = _case(shapes, [128, 37, 128, 64], steps=3, seed=23)
    assert [tr.f.diagnostics(i)["engine"] for i in range(4)] == [1, 0, 1, 0]
    tr.assert_ok()


def test_tensor_core_and_cuda_core_paths_agree():
    shapes = [(512, 768), (768, 512)]
    a = _case(shapes, 128, steps=4, seed=29, spike=(3,))
    b = _case(shapes, 128, steps=4, seed=29, spike=(3,), flags=fb.FLAG_FORCE_SIMT)
    assert b.f.diagnostics(0)["engine"] == 0 and a.f.diagnostics(0)["engine"] == 1
    for x, y, w0 in zip(a.W, b.W, a.W0.values()):
        dx, dy = to_np64(x) - w0, to_np64(y) - w0
        assert rel_err(dx, dy) < 3e-2


def test_alpha_lowrank_only_and_gamma_inf_on_tensor_cores():
    hp = fb.make_hparams(gamma=float("inf"), flags=fb.FLAG_ALPHA_LOWRANK_ONLY)
    tr = _case([(512, 768), (768, 512)], 128, steps=3, seed=31, hp=hp, spike=(2,))
    tr.assert_ok()
    assert all(l == 1.0 for row in tr.lams for l in row)


@pytest.mark.parametrize("flags", [fb.FLAG_MATRIX_SCALING, fb.FLAG_NO_SCALING, fb.FLAG_NO_RESIDUAL])
def test_ablation_variants_on_tensor_cores(flags):
    """The ablation variants of Section 5.4 on the tensor-core kernels (left, right, odd width)."""
    shapes = [(512, 768), (768, 512), (512, 1365)]
    tr = _case(shapes, 128, steps=4, seed=43, spike=(3,), flags=flags)
    assert [tr.f.diagnostics(i)["engine"] for i in range(3)] == [1, 1, 1]
    tr.assert_ok()
    for i in range(3):
        d = tr.f.diagnostics(i)
        if flags & fb.FLAG_NO_RESIDUAL:
            assert tr.st[i].prev_norm is None
        else:
            assert d["norm_prev"] == pytest.approx(tr.st[i].prev_norm, rel=2e-2)
            assert d["k_min"] == d["k_max"]
    if not flags & fb.FLAG_NO_RESIDUAL:
        assert any(l < 1.0 for row in tr.lams for l in row)


@pytest.mark.parametrize("flags", [fb.FLAG_ONLY_SCALING, fb.FLAG_ONLY_SCALING | fb.FLAG_MATRIX_SCALING])
def test_only_scaling_on_tensor_cores(flags):
    """Fira-only-scaling on the tensor-core engine (left, right, an odd width that is staged): the
    projection product and its Adam epilogue run as usual, the back-projection is replaced by the
    element-wise update W <- W - eta alpha lambda k G."""
    shapes = [(512, 768), (768, 512), (512, 1365)]
    tr = _case(shapes, 128, steps=4, seed=61, spike=(3,), flags=flags)
    assert [tr.f.diagnostics(i)["engine"] for i in range(3)] == [1, 1, 1]
    tr.assert_ok()
    assert any(l < 1.0 for row in tr.lams for l in row)
    for i in range(3):
        assert tr.f.diagnostics(i)["norm_prev"] == pytest.approx(tr.st[i].prev_norm, rel=2e-2)


@pytest.mark.parametrize("shape,r", [((512, 1376), 256), ((1376, 512), 128)])
def test_low_rank_direction_alone_element_by_element(shape, r):
    """GaLore mode (no residual): W_0 - W_1 = eta alpha P N, so one step isolates N as the projection
    epilogue forms it (its square root and division are approximate instructions, rounded to bf16
    next).  Every element of W must sit within two bf16 spacings of the oracle's (one, unless a binade
    boundary lies between the two), and the update must agree column by column and row by row."""
    tr = _case([shape], r, steps=1, seed=67, flags=fb.FLAG_NO_RESIDUAL)
    assert tr.f.diagnostics(0)["engine"] == 1
    tr.assert_ok()
    assert tr.local["ulp"] <= 2.0


@pytest.mark.parametrize("flags", [fb.FLAG_PSI_RMSPROP, fb.FLAG_PSI_ADAGRAD])
def test_other_base_optimizers_on_tensor_cores(flags):
    hp = fb.make_hparams(lr=1e-2, alpha=0.25, gamma=1.01, beta2=0.95, flags=flags)
    tr = _case([(512, 768), (768, 512)], 128, steps=4, seed=47, spike=(3,), hp=hp)
    assert [tr.f.diagnostics(i)["engine"] for i in range(2)] == [1, 1]
    tr.assert_ok()
    for i in range(2):
        M, V, pn, t = tr.f.get_state(i)
        assert float(M.abs().max()) == 0.0
        Vo = tr.st[i].V.T if tr.shapes[i][0] <= tr.shapes[i][1] else tr.st[i].V
        assert rel_err(to_np64(V), Vo) < 1e-5


def test_run_twice_is_bitwise_deterministic_on_tensor_cores():
    a = _case([(512, 1376), (1376, 512)], 128, steps=3, seed=37, spike=(2,))
    b = _case([(512, 1376), (1376, 512)], 128, steps=3, seed=37, spike=(2,))
    for x, y in zip(a.W, b.W):
        assert torch.equal(x, y)
