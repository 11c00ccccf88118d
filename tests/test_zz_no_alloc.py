"""fira_step_single_noalloc: the step for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is not an option: inside another
framework's memory pool, in a loop that must keep away from the driver's allocator,
or in a process whose device memory was handed out once at start.  They cannot give
fira_init() its state and scratch buffers, so this entry point keeps the step's
intermediates in a fixed array inside the library and takes only the inputs and
outputs.  Here it is called through the C ABI twice in a row and compared with
fira_step() on the same inputs; the second call finds the first call's leftovers in
the shared array and must not be disturbed by them.

This file is named so that pytest collects it last: if it fails under -x, every
other test has already run.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import fira_oracle as fo
from paper_2410_01623_b200 import binding as fb

pytestmark = pytest.mark.gpu

# same bound as the other fp32 parity tests (relative Frobenius error on W)
TOL = 1e-5


def _rel(a, b):
    return float((a.double() - b.double()).norm() / b.double().norm().clamp_min(1e-30))


def _run_both(shape, r, dtype, steps=2):
    m, n = shape
    d, l = min(m, n), max(m, n)
    lib = fb.lib()
    hp = fb.make_hparams(lr=1e-2, alpha=0.25, gamma=1.01)
    g = torch.Generator().manual_seed(m * 31 + n)
    W0 = (torch.randn(m, n, generator=g) * 0.02).to(dtype).cuda()
    P = torch.linalg.qr(torch.randn(d, r, generator=g, dtype=torch.float64))[0].to(dtype).contiguous().cuda()
    Gs = [(torch.randn(m, n, generator=g) * (3.0 if s == 1 else 1.0)).to(dtype).cuda() for s in range(steps)]

    # existing entry point (the bf16 case is forced onto the same CUDA-core kernels)
    ref = fb.Fira([shape], r, dtype, fb.make_hparams(lr=1e-2, alpha=0.25, gamma=1.01,
                                                     flags=fb.FLAG_FORCE_SIMT))
    ref.set_projection(0, P)
    W_ref = W0.clone()

    # new entry point: only inputs, outputs and the optimizer state of this matrix
    W_new = W0.clone()
    M = torch.zeros(l, r, device="cuda")
    V = torch.zeros(l, r, device="cuda")
    norm_prev = torch.full((1,), -1.0, device="cuda")
    t = torch.zeros(1, dtype=torch.int64, device="cuda")
    desc = fb.MatrixDesc(m, n, r, fb.FIRA_BF16 if dtype == torch.bfloat16 else fb.FIRA_F32, 0)
    stream = torch.cuda.current_stream().cuda_stream

    # the fp64 oracle on the same inputs: the entry point is also held to the parity bound itself
    kind = "bf16" if dtype == torch.bfloat16 else "f32"
    Wo = W0.double().cpu().numpy()
    st = fo.new_state(m, n, r)
    ohp = fo.Hyper(lr=1e-2, alpha=0.25, gamma=1.01)

    for s in range(steps):
        Wo, _ = fo.fira_step(Wo, Gs[s].double().cpu().numpy(), P.double().cpu().numpy(), st, ohp, store=kind)
        ref.step([W_ref], [Gs[s]])
        fb.check(lib.fira_step_single_noalloc(C.byref(hp), C.byref(desc), W_new.data_ptr(),
                                              Gs[s].data_ptr(), P.data_ptr(), M.data_ptr(), V.data_ptr(),
                                              norm_prev.data_ptr(), t.data_ptr(), -1.0, stream))
        torch.cuda.synchronize()
        Mr, Vr, pn, tr = ref.get_state(0)
        assert _rel(W_new, W_ref) <= TOL
        assert _rel(W_new, torch.from_numpy(Wo).cuda()) <= (TOL if kind == "f32" else 2e-2)
        assert fb.lib().fira_noalloc_poll(stream) == 0
        assert _rel(M, Mr) <= TOL and _rel(V, Vr) <= TOL
        assert int(t.item()) == tr == s + 1
        assert float(norm_prev.item()) == pytest.approx(pn, rel=1e-5)
    assert not torch.equal(W_new, W0)
    return ref


def test_two_calls_in_a_row_match_fira_step_fp32():
    """The single 512 x 1376, r = 128 matrix, two steps back to back."""
    _run_both((512, 1376), 128, torch.float32)


def test_right_projection_and_bf16_storage():
    # a smaller matrix after a larger one: the array still holds the larger call's data
    _run_both((333, 150), 37, torch.bfloat16)


def test_sizes_beyond_the_built_in_array_are_rejected():
    lib = fb.lib()
    assert lib.fira_noalloc_max_scratch_bytes() == 8 << 20
    hp = fb.make_hparams()
    desc = fb.MatrixDesc(4096, 4096, 1024, fb.FIRA_F32, 0)
    x = torch.zeros(16, device="cuda")
    st = lib.fira_step_single_noalloc(C.byref(hp), C.byref(desc), x.data_ptr(), x.data_ptr(), x.data_ptr(),
                                      x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), -1.0, None)
    assert st == 2
    msg = lib.fira_last_error().decode()
    assert "scratch" in msg and "8388608" in msg
    assert lib.fira_step_single_noalloc(C.byref(hp), C.byref(desc), None, None, None, None, None, None,
                                        None, -1.0, None) == 1


def test_unsupported_flags_are_rejected_before_anything_is_enqueued():
    """A call with a variant flag returns FIRA_ERR_UNSUPPORTED without touching the shared array or
    the caller's tensors: the next ordinary call and its result are unaffected."""
    lib = fb.lib()
    m, n, r = 64, 96, 8
    g = torch.Generator().manual_seed(3)
    W = (torch.randn(m, n, generator=g) * 0.02).cuda()
    G = torch.randn(m, n, generator=g).cuda()
    P = torch.linalg.qr(torch.randn(m, r, generator=g))[0].contiguous().cuda()
    M, V = torch.zeros(n, r, device="cuda"), torch.zeros(n, r, device="cuda")
    pn, t = torch.full((1,), -1.0, device="cuda"), torch.zeros(1, dtype=torch.int64, device="cuda")
    desc = fb.MatrixDesc(m, n, r, fb.FIRA_F32, 0)
    W_before = W.clone()
    for flag in (fb.FLAG_MATRIX_SCALING, fb.FLAG_NO_RESIDUAL, fb.FLAG_PSI_ADAGRAD, fb.FLAG_ONLY_SCALING):
        bad = fb.make_hparams(flags=flag)
        st = lib.fira_step_single_noalloc(C.byref(bad), C.byref(desc), W.data_ptr(), G.data_ptr(), P.data_ptr(),
                                          M.data_ptr(), V.data_ptr(), pn.data_ptr(), t.data_ptr(), -1.0, None)
        assert st == 3
    torch.cuda.synchronize()
    assert torch.equal(W, W_before) and int(t.item()) == 0 and float(M.abs().max()) == 0.0


def test_nonfinite_gradient_is_reported_by_the_poll():
    lib = fb.lib()
    m, n, r = 64, 96, 8
    g = torch.Generator().manual_seed(4)
    hp = fb.make_hparams()
    W = (torch.randn(m, n, generator=g) * 0.02).cuda()
    G = torch.randn(m, n, generator=g).cuda()
    G[3, 5] = float("inf")
    P = torch.linalg.qr(torch.randn(m, r, generator=g))[0].contiguous().cuda()
    M, V = torch.zeros(n, r, device="cuda"), torch.zeros(n, r, device="cuda")
    pn, t = torch.full((1,), -1.0, device="cuda"), torch.zeros(1, dtype=torch.int64, device="cuda")
    desc = fb.MatrixDesc(m, n, r, fb.FIRA_F32, 0)
    assert lib.fira_noalloc_poll(None) == 0
    fb.check(lib.fira_step_single_noalloc(C.byref(hp), C.byref(desc), W.data_ptr(), G.data_ptr(), P.data_ptr(),
                                          M.data_ptr(), V.data_ptr(), pn.data_ptr(), t.data_ptr(), -1.0, None))
    assert lib.fira_noalloc_poll(None) == 6                # FIRA_ERR_NONFINITE
    assert lib.fira_noalloc_poll(None) == 0                # cleared by the read
