"""GPU parity at the full matrix sizes of the benchmarked workload (LLaMA-7B shapes,
r = 1024, bf16): one whole layer (4096 x 4096, 4096 x 11008, 11008 x 4096) in the same
launch configuration as the benchmark (persistent grids over all SMs), with one matrix
of each shape checked element by element against the fp64 oracle."""
import pytest
import torch

from paper_2410_01623_b200 import workloads as wk
from tests.parity_util import workload_trajectory

pytestmark = pytest.mark.gpu


def test_llama_7b_layer_two_steps():
    wl = wk.workload("llama-7b", layers=1)
    assert wl.shapes[0] == (4096, 4096) and wl.shapes[4] == (4096, 11008) and wl.shapes[6] == (11008, 4096)
    tr = workload_trajectory(wl, 2, gen_device="cuda", check=[0, 4, 6])
    assert [tr.f.diagnostics(i)["engine"] for i in range(7)] == [1] * 7
    tr.assert_ok()
    for i in (0, 4, 6):
        d = tr.f.diagnostics(i)
        assert d["t"] == 2
        assert d["norm_prev"] == pytest.approx(tr.st[i].prev_norm, rel=2e-2)


def test_llama_1b_layer_odd_width_on_tensor_cores():
    """2048 x 5461: rows of 10922 bytes cannot be addressed by TMA, so the library works on
    copies with an aligned pitch; every matrix of the layer runs on the tensor cores."""
    wl = wk.workload("llama-1b", layers=1)
    tr = workload_trajectory(wl, 2, gen_device="cuda", check=[0, 4, 6])
    assert [tr.f.diagnostics(i)["engine"] for i in range(7)] == [1] * 7
    tr.assert_ok()
    for i in (0, 4, 6):
        assert tr.f.diagnostics(i)["norm_prev"] == pytest.approx(tr.st[i].prev_norm, rel=2e-2)
