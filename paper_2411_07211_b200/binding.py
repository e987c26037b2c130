"""ctypes binding of libb2blas.so: argument marshalling only.

Every routine of ``include/b2blas.h`` is exposed twice:

* ``lib().b2_saxpy`` etc. -- the raw C symbols with their prototypes set;
* ``axpy``, ``scal``, ... -- thin wrappers that pick the s/d symbol from the tensor dtype, pass
  ``tensor.data_ptr()`` and raise :class:`B2Error` on a non-zero status.

PyTorch is used for device memory and streams only.  There is no CPU path: if the compiled
CUDA library is missing the import of the symbols fails loudly.
"""
from __future__ import annotations

import ctypes
import os

import torch

ROW_MAJOR, COL_MAJOR = 101, 102
NO_TRANS, TRANS = 111, 112
UPPER, LOWER = 121, 122
NON_UNIT, UNIT = 131, 132

STATUS_OK, STATUS_LAUNCH_FAILED, STATUS_WORKSPACE_TOO_SMALL = 0, 1, 2
STATUS_NOT_IMPLEMENTED, STATUS_TIMEOUT, STATUS_BAD_CONTEXT = 3, 4, 5
STATUS_TOO_LARGE = 6

KNOB_L1_BLOCKS_PER_SM, KNOB_GEMV_N_TILE_BYTES, KNOB_GEMV_T_ROWS, KNOB_TRI_ROWS = 0, 1, 2, 3
KNOB_GER_ROWS, KNOB_USE_PDL, KNOB_TRSV_DEBUG_SKIP, KNOB_TRI_WIDE = 4, 5, 6, 7
KNOB_TRSV_PREFETCH_BYTES = 8
KNOB_TRSV_FRONT, KNOB_TRSV_CLUSTER = 9, 10
KNOB_TRSV_PM_FROM, KNOB_TRI_TILE, KNOB_TRI_TILE_UNIT, KNOB_NARROW_BLOCK = 11, 12, 13, 14
KNOB_TRI_BULK = 15

# B2BLAS_LIB selects another build of the same library (the bounds-checking one, libb2blas_dbg.so)
LIB_PATH = os.environ.get("B2BLAS_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libb2blas.so")

_i64, _int, _vp, _f, _d = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_float, ctypes.c_double


class B2Ctx(ctypes.Structure):
    _fields_ = [("stream", _vp), ("workspace", _vp), ("workspace_bytes", ctypes.c_size_t),
                ("device_status", _vp), ("wait_limit", ctypes.c_ulonglong)]


class B2Error(RuntimeError):
    def __init__(self, name, status):
        self.status = status
        msg = lib().b2_status_string(status).decode()
        super().__init__(f"{name} returned {status}: {msg}")


def _protos():
    cp = ctypes.POINTER(B2Ctx)
    out = {}
    for p, sc in (("s", _f), ("d", _d)):
        out[f"b2_{p}axpy"] = [cp, _i64, sc, _vp, _i64, _vp, _i64]
        out[f"b2_{p}scal"] = [cp, _i64, sc, _vp, _i64]
        out[f"b2_{p}copy"] = [cp, _i64, _vp, _i64, _vp, _i64]
        out[f"b2_{p}swap"] = [cp, _i64, _vp, _i64, _vp, _i64]
        out[f"b2_{p}rot"] = [cp, _i64, _vp, _i64, _vp, _i64, sc, sc]
        out[f"b2_{p}rotm"] = [cp, _i64, _vp, _i64, _vp, _i64, _vp]
        out[f"b2_{p}dot"] = [cp, _i64, _vp, _i64, _vp, _i64, _vp]
        out[f"b2_{p}asum"] = [cp, _i64, _vp, _i64, _vp]
        out[f"b2_{p}nrm2"] = [cp, _i64, _vp, _i64, _vp]
        out[f"b2_i{p}amax"] = [cp, _i64, _vp, _i64, _vp]
        out[f"b2_{p}gemv"] = [cp, _int, _int, _i64, _i64, sc, _vp, _i64, _vp, _i64, sc, _vp, _i64]
        out[f"b2_{p}ger"] = [cp, _int, _i64, _i64, sc, _vp, _i64, _vp, _i64, _vp, _i64]
        out[f"b2_{p}symv"] = [cp, _int, _int, _i64, sc, _vp, _i64, _vp, _i64, sc, _vp, _i64]
        out[f"b2_{p}syr"] = [cp, _int, _int, _i64, sc, _vp, _i64, _vp, _i64]
        out[f"b2_{p}syr2"] = [cp, _int, _int, _i64, sc, _vp, _i64, _vp, _i64, _vp, _i64]
        out[f"b2_{p}trmv"] = [cp, _int, _int, _int, _int, _i64, _vp, _i64, _vp, _i64]
        out[f"b2_{p}trsv"] = [cp, _int, _int, _int, _int, _i64, _vp, _i64, _vp, _i64]
    out["b2_dsdot"] = [cp, _i64, _vp, _i64, _vp, _i64, _vp]
    out["b2_sdsdot"] = [cp, _i64, _f, _vp, _i64, _vp, _i64, _vp]
    out["b2_sdot_noalloc"] = [_vp, _i64, _vp, _i64, _vp, _i64, _vp]
    out["b2_workspace_reset"] = [cp]
    return out


_lib = None


def lib():
    """The loaded library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2411_07211_b200.build` "
                "(there is no CPU fallback)")
        h = ctypes.CDLL(LIB_PATH)
        for name, args in _protos().items():
            fn = getattr(h, name)
            fn.argtypes = args
            fn.restype = _int
        h.b2_workspace_min_bytes.restype = ctypes.c_size_t
        h.b2_workspace_bytes.restype = ctypes.c_size_t
        h.b2_workspace_query.restype = ctypes.c_size_t
        h.b2_workspace_query.argtypes = [_i64, _i64, ctypes.c_size_t]
        h.b2_status_string.restype = ctypes.c_char_p
        h.b2_status_string.argtypes = [_int]
        h.b2_version.restype = _int
        h.b2_launch_count.restype = ctypes.c_ulonglong
        h.b2_set_tuning.argtypes = [_int, _i64]
        h.b2_set_tuning.restype = _int
        h.b2_get_tuning.argtypes = [_int]
        h.b2_get_tuning.restype = _i64
        h.b2_debug_bounds_report.argtypes = [ctypes.POINTER(ctypes.c_ulonglong)]
        h.b2_debug_bounds_report.restype = _int
        h.b2_debug_bounds_shrink.argtypes = [_int]
        h.b2_debug_bounds_shrink.restype = _int
        _lib = h
    return _lib


def exported_symbols():
    return sorted(_protos().keys()) + ["b2_workspace_min_bytes", "b2_workspace_bytes", "b2_workspace_query", "b2_status_string",
                                       "b2_version", "b2_launch_count", "b2_set_tuning", "b2_get_tuning",
                                       "b2_debug_bounds_report", "b2_debug_bounds_shrink"]


class Context:
    """Owns the workspace and status word (torch tensors) and builds the b2_ctx per call from
    torch's current stream."""

    def __init__(self, device="cuda", workspace_bytes: int | None = None, wait_limit: int = 0):
        h = lib()
        self.device = torch.device(device)
        nbytes = int(workspace_bytes if workspace_bytes is not None else h.b2_workspace_bytes())
        self.workspace = torch.zeros(nbytes + 256, dtype=torch.uint8, device=self.device)
        off = (-self.workspace.data_ptr()) % 256
        self._ws_ptr = self.workspace.data_ptr() + off
        self._ws_bytes = nbytes
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.wait_limit = wait_limit

    def struct(self) -> B2Ctx:
        stream = torch.cuda.current_stream(self.device).cuda_stream
        return B2Ctx(stream, self._ws_ptr, self._ws_bytes, self.status.data_ptr(), self.wait_limit)

    def reset(self):
        c = self.struct()
        st = lib().b2_workspace_reset(ctypes.byref(c))
        if st:
            raise B2Error("b2_workspace_reset", st)
        self.status.zero_()

    def device_status(self) -> int:
        return int(self.status.item())


def _p(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_cuda, "b2blas routines take device tensors"
    return t.data_ptr()


def _prefix(t) -> str:
    if t.dtype == torch.float32:
        return "s"
    if t.dtype == torch.float64:
        return "d"
    raise TypeError(f"b2blas supports float32/float64, got {t.dtype}")


_recording = None  # list of (function, ctx struct, args) while prepare() runs a thunk


def _call(name, ctx: Context, *args, check=True):
    c = ctx.struct()
    fn = getattr(lib(), name)
    st = fn(ctypes.byref(c), *args)
    if _recording is not None:
        _recording.append((fn, c, args))
    if check and st != 0:
        raise B2Error(name, st)
    return st


def prepare(thunk):
    """Runs `thunk` (calls of this module) once and returns a callable that repeats exactly those
    library calls with the arguments marshalled then -- same stream, same pointers -- without the
    per-call Python work of the wrappers (about 10 us a call, more than a small kernel takes).
    For timing loops over small problems; the returned callable returns the last status."""
    global _recording
    _recording = rec = []
    try:
        thunk()
    finally:
        _recording = None
    calls = [(fn, ctypes.byref(c), args, c) for fn, c, args in rec]

    def replay():
        st = 0
        for fn, ref, args, _keep in calls:
            st = fn(ref, *args)
        return st
    return replay


# ---- level 1 ----------------------------------------------------------------------------
def axpy(ctx, n, alpha, x, incx, y, incy, check=True):
    return _call(f"b2_{_prefix(x)}axpy", ctx, n, alpha, _p(x), incx, _p(y), incy, check=check)


def scal(ctx, n, alpha, x, incx, check=True):
    return _call(f"b2_{_prefix(x)}scal", ctx, n, alpha, _p(x), incx, check=check)


def copy(ctx, n, x, incx, y, incy, check=True):
    return _call(f"b2_{_prefix(x)}copy", ctx, n, _p(x), incx, _p(y), incy, check=check)


def swap(ctx, n, x, incx, y, incy, check=True):
    return _call(f"b2_{_prefix(x)}swap", ctx, n, _p(x), incx, _p(y), incy, check=check)


def rot(ctx, n, x, incx, y, incy, c, s, check=True):
    return _call(f"b2_{_prefix(x)}rot", ctx, n, _p(x), incx, _p(y), incy, c, s, check=check)


def rotm(ctx, n, x, incx, y, incy, param, check=True):
    """param: 5 host values [flag, h11, h21, h12, h22] (any sequence); None passes a NULL pointer."""
    if param is None:
        hp = None
    else:
        ctype = ctypes.c_float if x.dtype == torch.float32 else ctypes.c_double
        hp = ctypes.cast((ctype * 5)(*[float(v) for v in param]), _vp)
    return _call(f"b2_{_prefix(x)}rotm", ctx, n, _p(x), incx, _p(y), incy, hp, check=check)


def dsdot(ctx, n, x, incx, y, incy, result, check=True):
    """float32 vectors, float64 device result."""
    return _call("b2_dsdot", ctx, n, _p(x), incx, _p(y), incy, _p(result), check=check)


def sdsdot(ctx, n, sb, x, incx, y, incy, result, check=True):
    return _call("b2_sdsdot", ctx, n, sb, _p(x), incx, _p(y), incy, _p(result), check=check)


def dot(ctx, n, x, incx, y, incy, result, check=True):
    return _call(f"b2_{_prefix(x)}dot", ctx, n, _p(x), incx, _p(y), incy, _p(result), check=check)


def asum(ctx, n, x, incx, result, check=True):
    return _call(f"b2_{_prefix(x)}asum", ctx, n, _p(x), incx, _p(result), check=check)


def nrm2(ctx, n, x, incx, result, check=True):
    return _call(f"b2_{_prefix(x)}nrm2", ctx, n, _p(x), incx, _p(result), check=check)


def iamax(ctx, n, x, incx, result, check=True):
    return _call(f"b2_i{_prefix(x)}amax", ctx, n, _p(x), incx, _p(result), check=check)


# ---- level 2 ----------------------------------------------------------------------------
def gemv(ctx, order, trans, m, n, alpha, a, lda, x, incx, beta, y, incy, check=True):
    return _call(f"b2_{_prefix(a)}gemv", ctx, order, trans, m, n, alpha, _p(a), lda, _p(x), incx, beta, _p(y),
                 incy, check=check)


def ger(ctx, order, m, n, alpha, x, incx, y, incy, a, lda, check=True):
    return _call(f"b2_{_prefix(a)}ger", ctx, order, m, n, alpha, _p(x), incx, _p(y), incy, _p(a), lda, check=check)


def syr(ctx, order, uplo, n, alpha, x, incx, a, lda, check=True):
    return _call(f"b2_{_prefix(a)}syr", ctx, order, uplo, n, alpha, _p(x), incx, _p(a), lda, check=check)


def syr2(ctx, order, uplo, n, alpha, x, incx, y, incy, a, lda, check=True):
    return _call(f"b2_{_prefix(a)}syr2", ctx, order, uplo, n, alpha, _p(x), incx, _p(y), incy, _p(a), lda,
                 check=check)


def symv(ctx, order, uplo, n, alpha, a, lda, x, incx, beta, y, incy, check=True):
    return _call(f"b2_{_prefix(a)}symv", ctx, order, uplo, n, alpha, _p(a), lda, _p(x), incx, beta, _p(y), incy,
                 check=check)


def trmv(ctx, order, uplo, trans, diag, n, a, lda, x, incx, check=True):
    return _call(f"b2_{_prefix(a)}trmv", ctx, order, uplo, trans, diag, n, _p(a), lda, _p(x), incx, check=check)


def trsv(ctx, order, uplo, trans, diag, n, a, lda, x, incx, check=True):
    return _call(f"b2_{_prefix(a)}trsv", ctx, order, uplo, trans, diag, n, _p(a), lda, _p(x), incx, check=check)


def set_tuning(knob: int, value: int):
    if lib().b2_set_tuning(knob, value) != 0:
        raise ValueError(f"unknown tuning knob {knob}")


def get_tuning(knob: int) -> int:
    return int(lib().b2_get_tuning(knob))


def debug_bounds_report():
    """(violations since the last report, first offending address, its size) of the bounds-checking
    build; None in the ordinary build."""
    out = (ctypes.c_ulonglong * 3)()
    st = lib().b2_debug_bounds_report(out)
    if st == STATUS_NOT_IMPLEMENTED:
        return None
    if st:
        raise B2Error("b2_debug_bounds_report", st)
    return int(out[0]), int(out[1]), int(out[2])


def debug_bounds_shrink(nbytes: int) -> bool:
    """Test hook of the bounds-checking build; False in the ordinary build."""
    return lib().b2_debug_bounds_shrink(int(nbytes)) == 0


def launch_count() -> int:
    return int(lib().b2_launch_count())


def sdot_noalloc(n, x, incx, y, incy, result, stream=None, check=True):
    """b2_sdot_noalloc: float dot product that needs no Context (no workspace): its scratch is a
    fixed array inside the library.  For callers that cannot get device memory when they call;
    calls must not overlap on the GPU."""
    if stream is None:
        stream = torch.cuda.current_stream(x.device).cuda_stream
    st = lib().b2_sdot_noalloc(stream, n, _p(x), incx, _p(y), incy, _p(result))
    if check and st != 0:
        raise B2Error("b2_sdot_noalloc", st)
    return st
