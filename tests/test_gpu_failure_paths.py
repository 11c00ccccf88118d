"""Failure paths and memory bounds of the library, exercised without faulting anything.

* Every wait inside the tensor-core kernels is bounded.  The self-test entry point runs a one-block
  kernel whose wait cannot be satisfied (a barrier that nothing arrives on, no copy in flight) with a
  small limit: the wait gives up, a second waiter sees the abort flag and leaves, the kernel returns
  and the time-out reaches the host through the status word.  The context stays usable.
* Guard words: every buffer that the library writes is allocated here with a fixed byte pattern on
  both sides, every entry point is run, and the pattern must be intact afterwards.
"""
import ctypes as C

import pytest
import torch

from paper_2410_01623_b200 import binding as fb
from paper_2410_01623_b200 import workloads as wk
from tests.parity_util import Trajectory, workload_trajectory

pytestmark = pytest.mark.gpu

GUARD = 4096
PATTERN = 0xA5


def guarded(nbytes: int):
    """A device buffer of nbytes with GUARD pattern bytes on either side: (whole buffer, inner view)."""
    buf = torch.full((nbytes + 2 * GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
    return buf, buf[GUARD:GUARD + nbytes]


def guarded_like(t: torch.Tensor):
    buf, inner = guarded(t.numel() * t.element_size())
    view = inner.view(t.dtype).view(t.shape)
    view.copy_(t)
    return buf, view


def intact(buf: torch.Tensor) -> bool:
    torch.cuda.synchronize()
    return bool((buf[:GUARD] == PATTERN).all()) and bool((buf[-GUARD:] == PATTERN).all())


def test_bounded_wait_runs_out_and_is_reported():
    wl = wk.workload("llama-350m", layers=1)
    tr = workload_trajectory(wl, 1, check=[0, 6])
    f = tr.f
    assert f.poll() == 0
    f.selftest_bounded_wait(rounds=2000)
    assert f.poll() == 5                                   # FIRA_ERR_DEVICE_TIMEOUT
    assert "wait" in fb.lib().fira_last_error().decode()
    assert f.poll() == 0                                   # reported once, then cleared
    # the context steps on as before: one more step of the same trajectory, still at parity
    tr.step([wk.gradient(wl, i, 2) for i in range(len(wl.shapes))])
    tr.assert_ok()
    with pytest.raises(fb.FiraError):
        f.selftest_bounded_wait(rounds=0)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_guard_words_around_every_buffer(dtype):
    """Both engines (bf16: tensor-core kernels incl. an odd-width matrix that is staged, and a small
    matrix on the CUDA-core kernels), the refresh, the host-buffer step: the pattern around the
    state buffer, the scratch buffer, the staging buffer and every W, G stays intact."""
    shapes = [(512, 768), (768, 512), (512, 1365), (300, 333)] if dtype == torch.bfloat16 else \
             [(200, 333), (333, 200), (96, 96)]
    r = [128, 128, 128, 37] if dtype == torch.bfloat16 else [50, 50, 17]
    g = torch.Generator().manual_seed(5)
    f = fb.Fira(shapes, r, dtype, fb.make_hparams(), guard_bytes=GUARD)
    Ws = [guarded_like((torch.randn(m, n, generator=g) * 0.02).to(dtype).cuda()) for (m, n) in shapes]
    Gs = [guarded_like(torch.randn(m, n, generator=g).to(dtype).cuda()) for (m, n) in shapes]
    f.refresh_projection([v for _, v in Gs], seed=3, iters=2)
    for _ in range(3):
        f.step([v for _, v in Ws], [v for _, v in Gs])
    sbuf, staging = guarded(f.staging_bytes())
    Wh = [v.cpu().pin_memory() for _, v in Ws]
    Gh = [v.cpu().pin_memory() for _, v in Gs]
    f.step_host(Wh, Gh, staging)
    assert f.poll() == 0
    assert f.guards_intact()
    assert intact(sbuf)
    assert all(intact(b) for b, _ in Ws) and all(intact(b) for b, _ in Gs)
    if dtype == torch.bfloat16:
        assert [f.diagnostics(i)["engine"] for i in range(4)] == [1, 1, 1, 0]


def test_guard_words_dense_adam_and_no_alloc_entry_point():
    g = torch.Generator().manual_seed(6)
    hp = fb.make_hparams()
    n = 100003
    bufs = [guarded_like(t.cuda()) for t in (torch.randn(n, generator=g), torch.randn(n, generator=g),
                                            torch.zeros(n), torch.zeros(n))]
    (wb, W), (gb, G), (mb, M), (vb, V) = bufs
    fb.adam_dense(hp, [W], [G], [M], [V], 0)
    assert all(intact(b) for b, _ in bufs)
    # the step that keeps its intermediates inside the library
    m, nn, r = 150, 333, 37
    W2 = guarded_like((torch.randn(m, nn, generator=g) * 0.02).cuda())
    G2 = guarded_like(torch.randn(m, nn, generator=g).cuda())
    P2 = guarded_like(torch.linalg.qr(torch.randn(m, r, generator=g))[0].contiguous().cuda())
    M2, V2 = guarded_like(torch.zeros(nn, r).cuda()), guarded_like(torch.zeros(nn, r).cuda())
    pn = guarded_like(torch.full((4,), -1.0).cuda())
    t = guarded_like(torch.zeros(2, dtype=torch.int64).cuda())
    desc = fb.MatrixDesc(m, nn, r, fb.FIRA_F32, 0)
    for _ in range(2):
        fb.check(fb.lib().fira_step_single_noalloc(C.byref(hp), C.byref(desc), W2[1].data_ptr(), G2[1].data_ptr(),
                                                  P2[1].data_ptr(), M2[1].data_ptr(), V2[1].data_ptr(),
                                                  pn[1].data_ptr(), t[1].data_ptr(), -1.0,
                                                  torch.cuda.current_stream().cuda_stream))
    assert int(t[1][0].item()) == 2 and int(t[1][1].item()) == 0 and float(pn[1][1].item()) == -1.0
    assert all(intact(b) for b, _ in (W2, G2, P2, M2, V2, pn, t))
