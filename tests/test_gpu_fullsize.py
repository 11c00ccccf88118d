"""GPU parity at the full matrix sizes of the benchmarked workload (LLaMA-7B shapes,
r = 1024, bf16): one whole layer (4096 x 4096, 4096 x 11008, 11008 x 4096) in the same
launch configuration as the benchmark (persistent grids over all SMs), with one matrix
of each shape checked element by element against the fp64 oracle."""
import pytest
import torch

from paper_2410_01623_b200 import binding as fb
from paper_2410_01623_b200 import workloads as wk
from tests.parity_util import workload_trajectory

pytestmark = pytest.mark.gpu


def test_llama_7b_layer_two_steps():
    wl = wk.workload("llama-7b", layers=1)
    assert wl.shapes[0] == (4096, 4096) and wl.shapes[4] == (4096, 11008) and wl.shapes[6] == (11008, 4096)
    # two steps with seeded orthonormal projections; the right-orientation matrix is compared (the
    # 50-step run of the same layer in test_gpu_configs.py compares all three shapes)
    tr = workload_trajectory(wl, 2, gen_device="cuda", check=[6])
    assert [tr.f.diagnostics(i)["engine"] for i in range(7)] == [1] * 7
    tr.assert_ok()
    d = tr.f.diagnostics(6)
    assert d["t"] == 2
    assert d["norm_prev"] == pytest.approx(tr.st[6].prev_norm, rel=2e-2)


def test_llama_1b_layer_odd_width_on_tensor_cores():
    """2048 x 5461: rows of 10922 bytes cannot be addressed by TMA, so the library works on
    copies with an aligned pitch; every matrix of the layer runs on the tensor cores."""
    wl = wk.workload("llama-1b", layers=1)
    tr = workload_trajectory(wl, 2, gen_device="cuda", check=[0, 4, 6])
    assert [tr.f.diagnostics(i)["engine"] for i in range(7)] == [1] * 7
    tr.assert_ok()
    for i in (0, 4, 6):
        assert tr.f.diagnostics(i)["norm_prev"] == pytest.approx(tr.st[i].prev_norm, rel=2e-2)


def test_two_7b_layers_run_twice_bitwise():
    """Many tiles per CTA pair, every role of the persistent kernels re-entered hundreds of times:
    two runs of the same three steps must agree bit for bit in W, in the moments and in the
    diagnostics (which depend on the sums of G^2 taken inside the projection kernel)."""
    wl = wk.workload("llama-7b", layers=2)

    def run():
        f = fb.Fira(wl.shapes, wl.r, wl.torch_dtype, fb.make_hparams(lr=wl.lr, alpha=wl.alpha), "cuda")
        W = [wk.initial_weight(wl, i, "cuda") for i in range(len(wl.shapes))]
        P = {}
        for i, (m, n) in enumerate(wl.shapes):
            if min(m, n) not in P:
                P[min(m, n)] = wk.random_projection(wl, i, "cuda")
            f.set_projection(i, P[min(m, n)])
        for s in range(1, 4):
            f.step(W, [wk.gradient(wl, i, s, "cuda") for i in range(len(wl.shapes))])
        assert f.poll() == 0
        return W, [f.diagnostics(i) for i in range(len(wl.shapes))], [f.get_state(i)[:2] for i in (0, 4, 6, 13)]

    Wa, da, sa = run()
    Wb, db, sb = run()
    assert all(torch.equal(a, b) for a, b in zip(Wa, Wb))
    assert da == db
    assert all(torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) for a, b in zip(sa, sb))


def test_full_llama_7b_list_sampled_matrices():
    """The whole benchmarked workload (224 matrices, 51 GB on the device) in exactly the launch
    configuration that the benchmark times, one step; three matrices (first square one, a 4096 x 11008
    in the middle, the last 11008 x 4096) are checked element by element against the oracle."""
    free, _ = torch.cuda.mem_get_info()
    if free < 70 * 2 ** 30:
        pytest.skip("needs about 60 GB of free device memory")
    wl = wk.workload("llama-7b")
    assert len(wl.shapes) == 224
    tr = workload_trajectory(wl, 1, gen_device="cuda", check=[0, 116, 223])
    assert wl.shapes[116] == (4096, 11008) and wl.shapes[223] == (11008, 4096)
    tr.assert_ok()
    assert all(tr.f.diagnostics(i)["engine"] == 1 and tr.f.diagnostics(i)["t"] == 1 for i in (0, 116, 223))

