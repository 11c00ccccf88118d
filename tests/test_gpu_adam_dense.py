"""GPU parity of fira_adam_dense (plain Adam for unprojected parameters, Eq. 1-4) with the oracle."""
import numpy as np
import pytest
import torch

from oracle import fira_oracle as fo
from paper_2410_01623_b200 import binding as fb
from tests.parity_util import rel_err, to_np64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 2e-6), (torch.bfloat16, 4e-3)])
def test_dense_adam_matches_oracle(dtype, tol):
    # 30 tensors (two launches of 24), sizes from 1 element over ragged tails to several blocks
    g = torch.Generator().manual_seed(3)
    sizes = [1, 3, 4, 5, 4095, 4096, 4097, 32000 * 8 + 4, 70001] + [1000 + 37 * i for i in range(21)]
    hp = fb.make_hparams(lr=1e-2, beta1=0.9, beta2=0.99, eps=1e-8)
    W = [(torch.randn(n, generator=g) * 0.05).to(dtype).cuda() for n in sizes]
    M = [torch.zeros(n, device="cuda") for n in sizes]
    V = [torch.zeros(n, device="cuda") for n in sizes]
    ohp = fo.Hyper(lr=hp.lr, beta1=hp.beta1, beta2=hp.beta2, eps=hp.eps)
    Wo = [to_np64(w) for w in W]
    st = [fo.State(M=np.zeros(n), V=np.zeros(n)) for n in sizes]
    store = "bf16" if dtype == torch.bfloat16 else "f32"
    for t in range(4):
        G = [torch.randn(n, generator=g).to(dtype) for n in sizes]
        fb.adam_dense(hp, W, [x.cuda() for x in G], M, V, t, lr=None if t < 2 else 3e-3)
        for i in range(len(sizes)):
            h = ohp if t < 2 else fo.Hyper(**{**ohp.__dict__, "lr": 3e-3})
            Wo[i] = fo.adam_dense_step(Wo[i], to_np64(G[i]), st[i], h, store=store)
    torch.cuda.synchronize()
    for i in range(len(sizes)):
        assert rel_err(to_np64(W[i]), Wo[i]) <= tol, (sizes[i], rel_err(to_np64(W[i]), Wo[i]))
        assert rel_err(to_np64(M[i]), st[i].M) <= 1e-5
        assert rel_err(to_np64(V[i]), st[i].V) <= 1e-5


def test_dense_adam_argument_errors():
    hp = fb.make_hparams()
    w = torch.zeros(8, device="cuda")
    L = fb.lib()
    import ctypes as C
    n = (C.c_int64 * 1)(0)
    assert L.fira_adam_dense(C.byref(hp), 1, fb.ptr_array([w]), fb.ptr_array([w]), fb.ptr_array([w]),
                             fb.ptr_array([w]), n, 0, 0, -1.0, None) == 1      # numel = 0
    assert L.fira_adam_dense(C.byref(hp), 0, fb.ptr_array([w]), fb.ptr_array([w]), fb.ptr_array([w]),
                             fb.ptr_array([w]), n, 0, 0, -1.0, None) == 1      # empty list
