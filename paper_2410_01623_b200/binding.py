"""ctypes binding of libfira.so: argument marshalling only.

Every entry point of include/fira.h has a function of the same name on `lib()`;
`Fira` wraps a context and takes torch tensors for device memory.  Nothing here
computes: all arithmetic runs in the library's CUDA kernels.  If the shared
library is missing, `lib()` raises; there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libfira.so")

FIRA_OK = 0
FIRA_F32, FIRA_BF16 = 0, 1
FLAG_ALPHA_LOWRANK_ONLY, FLAG_AUTO_REFRESH, FLAG_FORCE_SIMT = 1, 2, 4
FLAG_MATRIX_SCALING, FLAG_NO_SCALING, FLAG_NO_RESIDUAL = 8, 16, 32
FLAG_PSI_RMSPROP, FLAG_PSI_ADAGRAD = 64, 128
FLAG_ONLY_SCALING = 256
FLAG_ROW_PADDING_WRITABLE = 512

STATUS_NAMES = {0: "FIRA_OK", 1: "FIRA_ERR_INVALID_ARG", 2: "FIRA_ERR_WORKSPACE_TOO_SMALL",
                3: "FIRA_ERR_UNSUPPORTED", 4: "FIRA_ERR_CUDA", 5: "FIRA_ERR_DEVICE_TIMEOUT",
                6: "FIRA_ERR_NONFINITE"}


class Hparams(C.Structure):
    _fields_ = [("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float), ("lr", C.c_float),
                ("alpha", C.c_float), ("gamma", C.c_float), ("T", C.c_int32), ("flags", C.c_uint32)]


class MatrixDesc(C.Structure):
    _fields_ = [("m", C.c_int32), ("n", C.c_int32), ("r", C.c_int32), ("dtype", C.c_int32),
                ("ld", C.c_int64)]


class Diag(C.Structure):
    _fields_ = [("norm_scaled", C.c_float), ("lambda_", C.c_float), ("norm_prev", C.c_float),
                ("k_min", C.c_float), ("k_max", C.c_float), ("t", C.c_int64), ("engine", C.c_int32)]


class FiraError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


# name -> (restype, argtypes); mirrors include/fira.h one to one
SIGNATURES = {
    "fira_query_workspace": (C.c_int, [C.POINTER(Hparams), C.POINTER(MatrixDesc), C.c_int32,
                                       C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "fira_init": (C.c_int, [C.POINTER(C.c_void_p), C.POINTER(Hparams), C.POINTER(MatrixDesc), C.c_int32,
                            C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p]),
    "fira_step": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.c_float]),
    "fira_step_host": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.c_float,
                                 C.c_void_p, C.c_size_t]),
    "fira_staging_bytes": (C.c_size_t, [C.c_void_p]),
    "fira_refresh_projection": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_int32),
                                          C.c_int32, C.c_uint64, C.c_int32]),
    "fira_refresh_projection_f32": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_int32),
                                              C.c_int32, C.c_uint64, C.c_int32, C.POINTER(C.c_void_p)]),
    "fira_refresh_side_work_bytes": (C.c_size_t, [C.c_void_p]),
    "fira_refresh_projection_side": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_int32), C.c_int32,
                                               C.c_uint64, C.c_int32, C.POINTER(C.c_void_p), C.c_void_p,
                                               C.c_size_t, C.c_void_p]),
    "fira_set_projection": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p]),
    "fira_get_projection": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p]),
    "fira_get_state": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(C.c_float),
                                 C.POINTER(C.c_int64)]),
    "fira_set_state": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_float, C.c_int64]),
    "fira_state_elements": (C.c_int64, [C.c_void_p, C.c_int32]),
    "fira_get_diagnostics": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(Diag)]),
    "fira_poll": (C.c_int, [C.c_void_p]),
    "fira_selftest_bounded_wait": (C.c_int, [C.c_void_p, C.c_int32]),
    "fira_last_step_launches": (C.c_int32, [C.c_void_p]),
    "fira_enable_phase_timing": (C.c_int, [C.c_void_p, C.c_int32]),
    "fira_get_phase_times": (C.c_int, [C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_float),
                                       C.POINTER(C.c_int32)]),
    "fira_phase_name": (C.c_char_p, [C.c_void_p, C.c_int32]),
    "fira_step_single_noalloc": (C.c_int, [C.POINTER(Hparams), C.POINTER(MatrixDesc), C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_float, C.c_void_p]),
    "fira_noalloc_max_scratch_bytes": (C.c_size_t, []),
    "fira_noalloc_poll": (C.c_int, [C.c_void_p]),
    "fira_adam_dense": (C.c_int, [C.POINTER(Hparams), C.c_int32, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p),
                                  C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.POINTER(C.c_int64), C.c_int,
                                  C.c_int64, C.c_float, C.c_void_p]),
    "fira_status_string": (C.c_char_p, [C.c_int]),
    "fira_last_error": (C.c_char_p, []),
    "fira_destroy": (None, [C.c_void_p]),
}

_LIB = None


def lib() -> C.CDLL:
    """Loads libfira.so (once).  Raises if it has not been built."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2410_01623_b200.build`")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _LIB = handle
    return _LIB


def check(status: int) -> None:
    if status != FIRA_OK:
        raise FiraError(status, lib().fira_last_error().decode())


def ptr_array(tensors: Sequence[Optional[torch.Tensor]]):
    arr = (C.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = None if t is None else t.data_ptr()
    return arr


def make_hparams(lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, alpha=0.25, gamma=1.01, T=0,
                 flags=0) -> Hparams:
    return Hparams(beta1, beta2, eps, lr, alpha, gamma, T, flags)


def adam_dense(hp: Hparams, Ws: Sequence[torch.Tensor], Gs: Sequence[torch.Tensor], Ms: Sequence[torch.Tensor],
               Vs: Sequence[torch.Tensor], t: int, lr: Optional[float] = None) -> None:
    """fira_adam_dense: one plain Adam step (Eq. 1-4) of a list of unprojected tensors, in place.
    Argument marshalling only."""
    n = len(Ws)
    assert n == len(Gs) == len(Ms) == len(Vs) and n > 0
    dt = Ws[0].dtype
    for w, g, m, v in zip(Ws, Gs, Ms, Vs):
        assert w.is_cuda and w.is_contiguous() and g.is_contiguous() and m.is_contiguous() and v.is_contiguous()
        assert w.dtype == g.dtype == dt and m.dtype == v.dtype == torch.float32
        assert w.numel() == g.numel() == m.numel() == v.numel()
    numel = (C.c_int64 * n)(*[w.numel() for w in Ws])
    stream = torch.cuda.current_stream(Ws[0].device).cuda_stream
    with torch.cuda.device(Ws[0].device):
        check(lib().fira_adam_dense(C.byref(hp), n, ptr_array(Ws), ptr_array(Gs), ptr_array(Ms), ptr_array(Vs),
                                    numel, 1 if dt == torch.bfloat16 else 0, int(t),
                                    -1.0 if lr is None else float(lr), C.c_void_p(stream)))


class Fira:
    """A library context over a list of weight matrices on one CUDA device.

    shapes: (m, n) per matrix; r: rank (int or one per matrix); dtype: torch.float32
    or torch.bfloat16 (storage of W, G and the projection).  The state and scratch
    buffers are torch byte tensors owned by this object."""

    GUARD_BYTE = 0xA5

    def __init__(self, shapes: Sequence[Tuple[int, int]], r, dtype: torch.dtype, hp: Hparams,
                 device="cuda", lds: Optional[Sequence[int]] = None, guard_bytes: int = 0):
        self.L = lib()
        self.device = torch.device(device)
        if self.device.type != "cuda":
            raise ValueError("the Fira library runs on a CUDA device only")
        self.shapes = [tuple(s) for s in shapes]
        self.count = len(self.shapes)
        self.ranks = [r] * self.count if isinstance(r, int) else list(r)
        self.dtype = dtype
        self.hp = hp
        code = FIRA_BF16 if dtype == torch.bfloat16 else FIRA_F32
        self.descs = (MatrixDesc * self.count)()
        for i, (m, n) in enumerate(self.shapes):
            self.descs[i] = MatrixDesc(m, n, self.ranks[i], code, 0 if lds is None else lds[i])
        sb, wb = C.c_size_t(), C.c_size_t()
        check(self.L.fira_query_workspace(C.byref(hp), self.descs, self.count, C.byref(sb), C.byref(wb)))
        self.state_bytes, self.scratch_bytes = sb.value, wb.value
        self.ctx = None
        # guard_bytes > 0 (a multiple of 256): both buffers get that many bytes of a fixed pattern on
        # either side, which guards_intact() checks: nothing the library launches may write there
        assert guard_bytes % 256 == 0
        self.guard_bytes = guard_bytes
        with torch.cuda.device(self.device):
            self.state = torch.full((sb.value + 2 * guard_bytes,), self.GUARD_BYTE, dtype=torch.uint8,
                                    device=self.device)
            self.scratch = torch.full((wb.value + 2 * guard_bytes,), self.GUARD_BYTE, dtype=torch.uint8,
                                      device=self.device)
            self.stream = torch.cuda.current_stream(self.device)
            ctx = C.c_void_p()
            check(self.L.fira_init(C.byref(ctx), C.byref(hp), self.descs, self.count,
                                   self.state.data_ptr() + guard_bytes, sb.value,
                                   self.scratch.data_ptr() + guard_bytes, wb.value,
                                   self.stream.cuda_stream))
        self.ctx = ctx

    def guards_intact(self) -> bool:
        g = self.guard_bytes
        if g == 0:
            return True
        torch.cuda.synchronize(self.device)
        return all(bool((buf[:g] == self.GUARD_BYTE).all()) and bool((buf[-g:] == self.GUARD_BYTE).all())
                   for buf in (self.state, self.scratch))

    def close(self):
        if getattr(self, "ctx", None):
            self.L.fira_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _dl(self, idx):
        m, n = self.shapes[idx]
        return min(m, n), max(m, n)

    def step(self, Ws: Sequence[torch.Tensor], Gs: Sequence[torch.Tensor], lr: Optional[float] = None):
        assert len(Ws) == self.count and len(Gs) == self.count
        check(self.L.fira_step(self.ctx, ptr_array(Ws), ptr_array(Gs), -1.0 if lr is None else lr))

    def staging_bytes(self) -> int:
        return self.L.fira_staging_bytes(self.ctx)

    def step_host(self, Ws_host, Gs_host, staging: torch.Tensor, lr: Optional[float] = None):
        check(self.L.fira_step_host(self.ctx, ptr_array(Ws_host), ptr_array(Gs_host),
                                    -1.0 if lr is None else lr, staging.data_ptr(), staging.numel()))

    def refresh_projection(self, Gs: Sequence[Optional[torch.Tensor]],
                           which: Optional[Sequence[int]] = None, seed: int = 0, iters: int = -1,
                           basis_f32: Optional[Sequence[Optional[torch.Tensor]]] = None):
        """basis_f32: optional list (one entry per matrix, None to skip) of (d, r) float32 device
        tensors that receive the basis before it is rounded to the storage type."""
        w, nw = (None, 0) if which is None else ((C.c_int32 * len(which))(*which), len(which))
        if basis_f32 is None:
            check(self.L.fira_refresh_projection(self.ctx, ptr_array(Gs), w, nw, seed, iters))
        else:
            for i, b in enumerate(basis_f32):
                assert b is None or (b.dtype == torch.float32 and b.is_contiguous() and
                                     b.shape == (self._dl(i)[0], self.ranks[i]))
            check(self.L.fira_refresh_projection_f32(self.ctx, ptr_array(Gs), w, nw, seed, iters,
                                                     ptr_array(basis_f32)))

    def refresh_side_work_bytes(self) -> int:
        return self.L.fira_refresh_side_work_bytes(self.ctx)

    def refresh_projection_side(self, Gs: Sequence[Optional[torch.Tensor]], P_out: Sequence[Optional[torch.Tensor]],
                                work: torch.Tensor, stream: "torch.cuda.Stream",
                                which: Optional[Sequence[int]] = None, seed: int = 0, iters: int = -1):
        """The refresh on a side stream with its own work buffer; the bases go to P_out (one (d, r)
        tensor of the storage type per selected matrix) and the context is left as it is."""
        w, nw = (None, 0) if which is None else ((C.c_int32 * len(which))(*which), len(which))
        for i, p in enumerate(P_out):
            assert p is None or (p.dtype == self.dtype and p.is_contiguous() and
                                 p.shape == (self._dl(i)[0], self.ranks[i]))
        check(self.L.fira_refresh_projection_side(self.ctx, ptr_array(Gs), w, nw, seed, iters, ptr_array(P_out),
                                                  work.data_ptr(), work.numel() * work.element_size(),
                                                  stream.cuda_stream))

    def set_projection(self, idx: int, P: torch.Tensor):
        d, _ = self._dl(idx)
        assert P.shape == (d, self.ranks[idx]) and P.dtype == self.dtype and P.is_cuda
        P = P.contiguous()   # the copy below is ordered on the same stream as torch's allocator
        check(self.L.fira_set_projection(self.ctx, idx, P.data_ptr()))

    def get_projection(self, idx: int) -> torch.Tensor:
        d, _ = self._dl(idx)
        P = torch.empty(d, self.ranks[idx], dtype=self.dtype, device=self.device)
        check(self.L.fira_get_projection(self.ctx, idx, P.data_ptr()))
        return P

    def get_state(self, idx: int):
        """M, V as (l, r) float tensors (row i = column i of G for m <= n, row i of G
        otherwise), the remembered norm (None if unset) and the step count."""
        _, l = self._dl(idx)
        M = torch.empty(l, self.ranks[idx], dtype=torch.float32, device=self.device)
        V = torch.empty_like(M)
        pn, t = C.c_float(), C.c_int64()
        check(self.L.fira_get_state(self.ctx, idx, M.data_ptr(), V.data_ptr(), C.byref(pn), C.byref(t)))
        return M, V, (None if pn.value < 0 else pn.value), t.value

    def set_state(self, idx: int, M: torch.Tensor, V: torch.Tensor, prev_norm: Optional[float], t: int):
        _, l = self._dl(idx)
        assert M.shape == (l, self.ranks[idx]) and M.dtype == torch.float32 and M.is_contiguous()
        assert V.shape == M.shape and V.dtype == torch.float32 and V.is_contiguous()
        check(self.L.fira_set_state(self.ctx, idx, M.data_ptr(), V.data_ptr(),
                                    -1.0 if prev_norm is None else prev_norm, t))

    def state_elements(self, idx: int) -> int:
        return self.L.fira_state_elements(self.ctx, idx)

    def diagnostics(self, idx: int) -> dict:
        d = Diag()
        check(self.L.fira_get_diagnostics(self.ctx, idx, C.byref(d)))
        return dict(norm_scaled=d.norm_scaled, lam=d.lambda_, norm_prev=d.norm_prev, k_min=d.k_min,
                    k_max=d.k_max, t=d.t, engine=d.engine)

    def poll(self) -> int:
        return self.L.fira_poll(self.ctx)

    def selftest_bounded_wait(self, rounds: int = 1000):
        check(self.L.fira_selftest_bounded_wait(self.ctx, rounds))

    def last_step_launches(self) -> int:
        return self.L.fira_last_step_launches(self.ctx)

    def enable_phase_timing(self, enable: bool = True):
        check(self.L.fira_enable_phase_timing(self.ctx, 1 if enable else 0))

    def phase_times(self):
        """[(kernel name, mean ms per step)] over the steps recorded since enabling."""
        n, steps = C.c_int32(), C.c_int32()
        ms = (C.c_float * 16)()
        check(self.L.fira_get_phase_times(self.ctx, C.byref(n), ms, C.byref(steps)))
        return [(self.L.fira_phase_name(self.ctx, i).decode(), ms[i]) for i in range(n.value)], steps.value
