"""ctypes front-end of the CPU oracle (blas_oracle.c) -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the bench's CPU-baseline leg may import this module.  It
never touches the CUDA library.  Every function takes numpy arrays, works in place where
the BLAS routine does, and returns the extra "absterms" arrays the C code produces (the
per-output sum of |terms| that parity tolerances are scaled by).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libblas_oracle.so")
_SRC = [os.path.join(_HERE, "blas_oracle.c"), os.path.join(_HERE, "blas_oracle_impl.h")]

ROW_MAJOR, COL_MAJOR = 101, 102
NO_TRANS, TRANS = 111, 112
UPPER, LOWER = 121, 122
NON_UNIT, UNIT = 131, 132

_lib = None
_omp = False  # True: calls go to the OpenMP copy (the bench's all-cores baseline; timing only)
_LIB_OMP_PATH = os.path.join(_HERE, "libblas_oracle_omp.so")
_lib_omp = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, no fast-math, no FMA contraction)."""
    stale = force or not os.path.exists(_LIB_PATH) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB_PATH) for s in _SRC)
    if stale:
        tmp = _LIB_PATH + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-Wall", "-shared", "-fPIC",
             _SRC[0], "-o", tmp, "-lm"])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def build_omp(force: bool = False) -> str:
    """The same source with ORACLE_OMP defined: an OpenMP parallel-for on the outermost independent
    loop of each routine (trsv, iamax and the float-only dots stay serial).  Timing only."""
    stale = force or not os.path.exists(_LIB_OMP_PATH) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB_OMP_PATH) for s in _SRC)
    if stale:
        tmp = _LIB_OMP_PATH + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-DORACLE_OMP", "-ffp-contract=off", "-fno-fast-math", "-Wall", "-shared", "-fPIC",
             _SRC[0], "-o", tmp, "-lm"])
        os.replace(tmp, _LIB_OMP_PATH)
    return _LIB_OMP_PATH


def use_all_cores(on: bool) -> None:
    """Routes the calls of this module to the OpenMP copy (True) or back to the oracle proper."""
    global _omp
    _omp = bool(on)


def lib():
    global _lib, _lib_omp
    if _omp:
        if _lib_omp is None:
            _lib_omp = ctypes.CDLL(build_omp())
            _lib_omp.oracle_wide_bytes.restype = ctypes.c_int
        return _lib_omp
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_wide_bytes.restype = ctypes.c_int
    return _lib


_i64 = ctypes.c_int64
_int = ctypes.c_int
_vp = ctypes.c_void_p


def _prefix(dtype) -> str:
    dtype = np.dtype(dtype)
    if dtype == np.float32:
        return "s"
    if dtype == np.float64:
        return "d"
    raise TypeError(f"oracle supports float32/float64, got {dtype}")


def _scalar(dtype, v):
    return ctypes.c_float(v) if np.dtype(dtype) == np.float32 else ctypes.c_double(v)


def _ptr(a):
    if a is None:
        return _vp(0)
    assert isinstance(a, np.ndarray) and a.flags["C_CONTIGUOUS"], "oracle wants contiguous numpy"
    return _vp(a.ctypes.data)


def _call(name, dtype, *args):
    f = getattr(lib(), f"oracle_{_prefix(dtype)}{name}")
    f.restype = None
    f(*args)


def _scratch(n):
    return np.zeros(max(1, n) * lib().oracle_wide_bytes(), dtype=np.uint8)


# ------------------------------------------------------------------ level 1
def axpy(n, alpha, x, incx, y, incy):
    absterms = np.zeros(n, dtype=np.float64)
    _call("axpy", x.dtype, _i64(n), _scalar(x.dtype, alpha), _ptr(x), _i64(incx), _ptr(y),
          _i64(incy), _ptr(absterms))
    return absterms


def scal(n, alpha, x, incx):
    _call("scal", x.dtype, _i64(n), _scalar(x.dtype, alpha), _ptr(x), _i64(incx))


def copy(n, x, incx, y, incy):
    _call("copy", x.dtype, _i64(n), _ptr(x), _i64(incx), _ptr(y), _i64(incy))


def swap(n, x, incx, y, incy):
    _call("swap", x.dtype, _i64(n), _ptr(x), _i64(incx), _ptr(y), _i64(incy))


def rot(n, x, incx, y, incy, c, s):
    ax = np.zeros(n, dtype=np.float64)
    ay = np.zeros(n, dtype=np.float64)
    _call("rot", x.dtype, _i64(n), _ptr(x), _i64(incx), _ptr(y), _i64(incy),
          _scalar(x.dtype, c), _scalar(x.dtype, s), _ptr(ax), _ptr(ay))
    return ax, ay


def rotm(n, x, incx, y, incy, param):
    """param = [flag, h11, h21, h12, h22] (numpy, same dtype as x); returns absterms of x' and y'."""
    ax = np.zeros(n, dtype=np.float64)
    ay = np.zeros(n, dtype=np.float64)
    param = np.ascontiguousarray(param, dtype=x.dtype)
    assert param.shape == (5,)
    _call("rotm", x.dtype, _i64(n), _ptr(x), _i64(incx), _ptr(y), _i64(incy), _ptr(param), _ptr(ax), _ptr(ay))
    return ax, ay


def dsdot(n, x, incx, y, incy):
    """float32 inputs, double result."""
    assert x.dtype == np.float32 and y.dtype == np.float32
    res = np.zeros(1, dtype=np.float64)
    absterms = np.zeros(1, dtype=np.float64)
    f = lib().oracle_dsdot
    f.restype = None
    f(_i64(n), _ptr(x), _i64(incx), _ptr(y), _i64(incy), _ptr(res), _ptr(absterms))
    return res[0], absterms[0]


def sdsdot(n, sb, x, incx, y, incy):
    """float32 inputs, float32 result = sb + the double-accumulated dot."""
    assert x.dtype == np.float32 and y.dtype == np.float32
    res = np.zeros(1, dtype=np.float32)
    absterms = np.zeros(1, dtype=np.float64)
    f = lib().oracle_sdsdot
    f.restype = None
    f(_i64(n), ctypes.c_float(sb), _ptr(x), _i64(incx), _ptr(y), _i64(incy), _ptr(res), _ptr(absterms))
    return res[0], absterms[0]


def dot(n, x, incx, y, incy):
    res = np.zeros(1, dtype=x.dtype)
    absterms = np.zeros(1, dtype=np.float64)
    _call("dot", x.dtype, _i64(n), _ptr(x), _i64(incx), _ptr(y), _i64(incy), _ptr(res),
          _ptr(absterms))
    return res[0], absterms[0]


def asum(n, x, incx):
    res = np.zeros(1, dtype=x.dtype)
    absterms = np.zeros(1, dtype=np.float64)
    _call("asum", x.dtype, _i64(n), _ptr(x), _i64(incx), _ptr(res), _ptr(absterms))
    return res[0], absterms[0]


def nrm2(n, x, incx):
    res = np.zeros(1, dtype=x.dtype)
    absterms = np.zeros(1, dtype=np.float64)
    _call("nrm2", x.dtype, _i64(n), _ptr(x), _i64(incx), _ptr(res), _ptr(absterms))
    return res[0], absterms[0]


def iamax(n, x, incx):
    res = np.zeros(1, dtype=np.int64)
    _call("iamax", x.dtype, _i64(n), _ptr(x), _i64(incx), _ptr(res))
    return int(res[0])


# ------------------------------------------------------------------ level 2
def gemv(order, trans, m, n, alpha, a, lda, x, incx, beta, y, incy):
    leny = m if trans == NO_TRANS else n
    absterms = np.zeros(leny, dtype=np.float64)
    _call("gemv", a.dtype, _int(order), _int(trans), _i64(m), _i64(n), _scalar(a.dtype, alpha),
          _ptr(a), _i64(lda), _ptr(x), _i64(incx), _scalar(a.dtype, beta), _ptr(y), _i64(incy),
          _ptr(absterms))
    return absterms


def ger(order, m, n, alpha, x, incx, y, incy, a, lda, want_absterms=True):
    absterms = np.zeros(m * n, dtype=np.float64) if want_absterms else None
    _call("ger", a.dtype, _int(order), _i64(m), _i64(n), _scalar(a.dtype, alpha), _ptr(x),
          _i64(incx), _ptr(y), _i64(incy), _ptr(a), _i64(lda), _ptr(absterms))
    return None if absterms is None else absterms.reshape(m, n)


def syr(order, uplo, n, alpha, x, incx, a, lda, want_absterms=True):
    absterms = np.zeros(n * n, dtype=np.float64) if want_absterms else None
    _call("syr", a.dtype, _int(order), _int(uplo), _i64(n), _scalar(a.dtype, alpha), _ptr(x), _i64(incx),
          _ptr(a), _i64(lda), _ptr(absterms))
    return None if absterms is None else absterms.reshape(n, n)


def syr2(order, uplo, n, alpha, x, incx, y, incy, a, lda, want_absterms=True):
    absterms = np.zeros(n * n, dtype=np.float64) if want_absterms else None
    _call("syr2", a.dtype, _int(order), _int(uplo), _i64(n), _scalar(a.dtype, alpha), _ptr(x), _i64(incx),
          _ptr(y), _i64(incy), _ptr(a), _i64(lda), _ptr(absterms))
    return None if absterms is None else absterms.reshape(n, n)


def symv(order, uplo, n, alpha, a, lda, x, incx, beta, y, incy):
    absterms = np.zeros(n, dtype=np.float64)
    _call("symv", a.dtype, _int(order), _int(uplo), _i64(n), _scalar(a.dtype, alpha), _ptr(a),
          _i64(lda), _ptr(x), _i64(incx), _scalar(a.dtype, beta), _ptr(y), _i64(incy),
          _ptr(absterms))
    return absterms


def trmv(order, uplo, trans, diag, n, a, lda, x, incx):
    absterms = np.zeros(n, dtype=np.float64)
    scratch = _scratch(n)
    _call("trmv", a.dtype, _int(order), _int(uplo), _int(trans), _int(diag), _i64(n), _ptr(a),
          _i64(lda), _ptr(x), _i64(incx), _ptr(absterms), _ptr(scratch))
    return absterms


def trsv(order, uplo, trans, diag, n, a, lda, x, incx):
    absterms = np.zeros(n, dtype=np.float64)
    scratch = _scratch(n)
    _call("trsv", a.dtype, _int(order), _int(uplo), _int(trans), _int(diag), _i64(n), _ptr(a),
          _i64(lda), _ptr(x), _i64(incx), _ptr(absterms), _ptr(scratch))
    return absterms


def trsv_residual(order, uplo, trans, diag, n, a, lda, b, incb, xs, incx):
    resid = np.zeros(n, dtype=np.float64)
    scale = np.zeros(n, dtype=np.float64)
    _call("trsv_residual", a.dtype, _int(order), _int(uplo), _int(trans), _int(diag), _i64(n),
          _ptr(a), _i64(lda), _ptr(b), _i64(incb), _ptr(xs), _i64(incx), _ptr(resid), _ptr(scale))
    return resid, scale
