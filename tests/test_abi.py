"""The C-ABI library loads without a GPU and exports every symbol the header declares; host-side
argument validation returns the documented codes without launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def b2():
    from paper_2411_07211_b200 import build
    build.build()
    from paper_2411_07211_b200 import binding
    return binding


def test_header_symbols_exported(b2):
    header = open(os.path.join(ROOT, "include", "b2blas.h")).read()
    declared = sorted(set(re.findall(r"\b(b2_\w+)\s*\(", header)))
    assert len(declared) >= 34
    h = ctypes.CDLL(b2.LIB_PATH)
    for name in declared:
        assert hasattr(h, name), f"{name} declared in b2blas.h but not exported"
    assert set(b2.exported_symbols()) == set(declared)
    assert b2.lib().b2_version() >= 100
    assert b2.lib().b2_workspace_bytes() >= b2.lib().b2_workspace_min_bytes() > 4096
    q = b2.lib().b2_workspace_query
    assert q(1, 1, 4) >= b2.lib().b2_workspace_min_bytes() and q(-1, 1, 4) == 0 and q(1, 1, 3) == 0
    assert q(32768, 32768, 8) <= b2.lib().b2_workspace_bytes()  # the default serves the largest config
    assert q(1 << 20, 64, 8) >= ((1 << 20) + 64) * 8 and q(70000, 70000, 8) >= 70000 * 16
    assert b"ok" == b2.lib().b2_status_string(0)
    assert b"argument" in b2.lib().b2_status_string(-3)


def test_argument_validation_without_gpu(b2):
    """Invalid arguments are rejected on the host before any CUDA call."""
    h = b2.lib()
    ctx = b2.B2Ctx(None, 0x1000, 1 << 20, None, 0)  # fake, never dereferenced on these paths
    c = ctypes.byref(ctx)
    p = 0x10000  # non-null, aligned fake device pointer
    assert h.b2_saxpy(c, -1, 1.0, p, 1, p, 1) == -1
    assert h.b2_saxpy(c, 4, 1.0, None, 1, p, 1) == -3
    assert h.b2_saxpy(c, 4, 1.0, p, 0, p, 1) == -4
    assert h.b2_saxpy(c, 4, 1.0, p, 1, None, 1) == -5
    assert h.b2_saxpy(c, 4, 1.0, p, 1, p, 0) == -6
    assert h.b2_dscal(c, 4, 1.0, p + 4, 1) == -3  # misaligned for double
    assert h.b2_dscal(c, 4, 1.0, p, 0) == -4
    assert h.b2_sdot(c, 4, p, 1, p, 1, None) == -6
    assert h.b2_isamax(c, 4, p, 1, None) == -4
    assert h.b2_sgemv(c, 99, b2.NO_TRANS, 2, 2, 1.0, p, 2, p, 1, 0.0, p, 1) == -1
    assert h.b2_sgemv(c, b2.ROW_MAJOR, 5, 2, 2, 1.0, p, 2, p, 1, 0.0, p, 1) == -2
    assert h.b2_sgemv(c, b2.ROW_MAJOR, b2.NO_TRANS, -2, 2, 1.0, p, 2, p, 1, 0.0, p, 1) == -3
    assert h.b2_sgemv(c, b2.ROW_MAJOR, b2.NO_TRANS, 2, 3, 1.0, p, 2, p, 1, 0.0, p, 1) == -7  # lda < n
    assert h.b2_sgemv(c, b2.COL_MAJOR, b2.NO_TRANS, 3, 2, 1.0, p, 2, p, 1, 0.0, p, 1) == -7  # lda < m
    assert h.b2_sgemv(c, b2.ROW_MAJOR, b2.NO_TRANS, 2, 2, 1.0, p, 2, p, 0, 0.0, p, 1) == -9
    assert h.b2_sgemv(c, b2.ROW_MAJOR, b2.NO_TRANS, 2, 2, 1.0, p, 2, p, 1, 0.0, p, 0) == -12
    assert h.b2_dger(c, b2.ROW_MAJOR, 2, 2, 1.0, p, 1, p, 1, p, 1) == -10
    assert h.b2_ssymv(c, b2.ROW_MAJOR, 7, 2, 1.0, p, 2, p, 1, 0.0, p, 1) == -2
    assert h.b2_strmv(c, b2.ROW_MAJOR, b2.UPPER, b2.NO_TRANS, 0, 2, p, 2, p, 1) == -4
    assert h.b2_dtrsv(c, b2.ROW_MAJOR, b2.UPPER, b2.NO_TRANS, b2.UNIT, 2, p, 1, p, 1) == -7
    assert h.b2_dtrsv(c, b2.ROW_MAJOR, b2.UPPER, b2.NO_TRANS, b2.UNIT, 2, p, 2, p, 0) == -9
    # the routines built after the headline set
    assert h.b2_ssyr(c, 7, b2.UPPER, 2, 1.0, p, 1, p, 2) == -1
    assert h.b2_ssyr(c, b2.ROW_MAJOR, 7, 2, 1.0, p, 1, p, 2) == -2
    assert h.b2_dsyr(c, b2.ROW_MAJOR, b2.UPPER, 2, 1.0, p, 0, p, 2) == -6
    assert h.b2_dsyr(c, b2.ROW_MAJOR, b2.UPPER, 2, 1.0, p, 1, p, 1) == -8
    assert h.b2_ssyr2(c, b2.ROW_MAJOR, b2.UPPER, 2, 1.0, p, 1, None, 1, p, 2) == -7
    assert h.b2_ssyr2(c, b2.ROW_MAJOR, b2.UPPER, 2, 1.0, p, 1, p, 1, p, 1) == -10
    fpar = (ctypes.c_float * 5)(-1.0, 1.0, 0.0, 0.0, 1.0)
    bad_flag = (ctypes.c_float * 5)(3.0, 1.0, 0.0, 0.0, 1.0)
    assert h.b2_srotm(c, -1, p, 1, p, 1, ctypes.cast(fpar, ctypes.c_void_p)) == -1
    assert h.b2_srotm(c, 4, p, 1, p, 0, ctypes.cast(fpar, ctypes.c_void_p)) == -5
    assert h.b2_srotm(c, 4, p, 1, p, 1, None) == -6
    assert h.b2_srotm(c, 4, p, 1, p, 1, ctypes.cast(bad_flag, ctypes.c_void_p)) == -6
    assert h.b2_dsdot(c, 4, p, 1, p, 1, None) == -6
    assert h.b2_sdsdot(c, 4, 0.0, p, 1, p, 0, p) == -6
    assert h.b2_sdsdot(c, 4, 0.0, p, 1, p, 1, None) == -7
    # context checks come after argument checks and before any launch
    assert h.b2_saxpy(None, 4, 1.0, p, 1, p, 1) == b2.STATUS_BAD_CONTEXT
    bad = b2.B2Ctx(None, 0x1001, 1 << 20, None, 0)
    assert h.b2_saxpy(ctypes.byref(bad), 4, 1.0, p, 1, p, 1) == b2.STATUS_BAD_CONTEXT
    small = b2.B2Ctx(None, 0x1000, 16, None, 0)
    assert h.b2_saxpy(ctypes.byref(small), 4, 1.0, p, 1, p, 1) == b2.STATUS_WORKSPACE_TOO_SMALL
    # empty problems succeed without touching anything
    assert h.b2_saxpy(c, 0, 1.0, None, 1, None, 1) == 0
    assert h.b2_sgemv(c, b2.ROW_MAJOR, b2.NO_TRANS, 0, 5, 1.0, None, 5, None, 1, 0.0, None, 1) == 0
    assert h.b2_strsv(c, b2.ROW_MAJOR, b2.UPPER, b2.NO_TRANS, b2.UNIT, 0, None, 1, None, 1) == 0


def test_tuning_knobs(b2):
    old = b2.get_tuning(b2.KNOB_GER_ROWS)
    b2.set_tuning(b2.KNOB_GER_ROWS, old + 1)
    assert b2.get_tuning(b2.KNOB_GER_ROWS) == old + 1
    b2.set_tuning(b2.KNOB_GER_ROWS, old)
    with pytest.raises(ValueError):
        b2.set_tuning(99, 1)
