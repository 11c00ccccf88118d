"""Host-side checks that need no GPU: the library builds, loads, exports every
symbol include/fira.h declares, the binding mirrors them, and argument errors are
reported without touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2410_01623_b200 import binding as fb
from paper_2410_01623_b200 import build as fbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fbuild.build()
    return fb.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fira.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"FIRA_API\s+[\w\s\*]+?\b(fira_\w+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound(lib):
    names = declared_functions()
    assert len(names) >= 17 and "fira_step" in names and "fira_refresh_projection" in names
    for name in names:
        assert hasattr(lib, name), name
        assert name in fb.SIGNATURES, name
    assert sorted(fb.SIGNATURES) == names


def test_status_strings(lib):
    assert lib.fira_status_string(0) == b"ok"
    for code in range(1, 7):
        assert len(lib.fira_status_string(code)) > 0


def _query(lib, hp, descs):
    arr = (fb.MatrixDesc * len(descs))(*descs)
    sb, wb = C.c_size_t(), C.c_size_t()
    st = lib.fira_query_workspace(C.byref(hp), arr, len(descs), C.byref(sb), C.byref(wb))
    return st, sb.value, wb.value


def test_query_workspace_counts_the_state_of_the_comparison_table(lib):
    # state = projection d*r + M, V 2*l*r floats + scalars, each section padded to 256 B
    hp = fb.make_hparams()
    st, sb, wb = _query(lib, hp, [fb.MatrixDesc(512, 1376, 128, fb.FIRA_F32, 0)])
    assert st == 0
    exact = (512 * 128 + 2 * 1376 * 128) * 4
    assert exact <= sb <= exact + 4 * 256
    assert wb > 0
    st, sb16, _ = _query(lib, hp, [fb.MatrixDesc(1376, 512, 128, fb.FIRA_BF16, 0)])
    assert st == 0
    exact16 = 512 * 128 * 2 + 2 * 1376 * 128 * 4
    assert exact16 <= sb16 <= exact16 + 4 * 256


@pytest.mark.parametrize("bad", [
    dict(eps=0.0), dict(eps=-1.0), dict(beta1=1.0), dict(beta2=-0.1), dict(gamma=0.5),
    dict(gamma=float("nan")), dict(lr=float("inf")), dict(T=-1)])
def test_invalid_hparams_are_rejected(lib, bad):
    hp = fb.make_hparams(**bad)
    st, _, _ = _query(lib, hp, [fb.MatrixDesc(8, 8, 2, fb.FIRA_F32, 0)])
    assert st == 1
    assert len(lib.fira_last_error()) > 0


@pytest.mark.parametrize("desc", [
    fb.MatrixDesc(0, 8, 1, 0, 0), fb.MatrixDesc(8, 8, 0, 0, 0), fb.MatrixDesc(8, 16, 9, 0, 0),
    fb.MatrixDesc(8, 8, 2, 7, 0), fb.MatrixDesc(8, 8, 2, 0, 4)])
def test_invalid_matrices_are_rejected(lib, desc):
    st, _, _ = _query(lib, fb.make_hparams(), [desc])
    assert st == 1


def test_gamma_infinity_is_accepted(lib):
    st, _, _ = _query(lib, fb.make_hparams(gamma=float("inf")), [fb.MatrixDesc(8, 8, 2, 0, 0)])
    assert st == 0


def test_init_rejects_null_and_small_buffers(lib):
    hp = fb.make_hparams()
    arr = (fb.MatrixDesc * 1)(fb.MatrixDesc(8, 8, 2, 0, 0))
    ctx = C.c_void_p()
    assert lib.fira_init(C.byref(ctx), C.byref(hp), arr, 1, None, 0, None, 0, None) == 1
    assert not ctx.value
    # aligned fake addresses with sizes that are too small: rejected before any device access
    assert lib.fira_init(C.byref(ctx), C.byref(hp), arr, 1, 4096, 16, 8192, 16, None) == 2
    assert b"workspace too small" in lib.fira_last_error()
    assert lib.fira_step(None, None, None, -1.0) == 1
    assert lib.fira_state_elements(None, 0) == -1
    lib.fira_destroy(None)
