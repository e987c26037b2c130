"""GPU parity of gemv / ger / symv / trmv / trsv against the CPU oracle, through the C ABI."""
import itertools

import numpy as np
import pytest
import torch

from oracle import blas_oracle as orc
from paper_2411_07211_b200 import synth
from tests.gpu_util import TOL, Guarded, assert_close, assert_same_gaps, pick, place

pytestmark = pytest.mark.gpu

DTYPES = [np.float32, np.float64]
ORDERS = [orc.ROW_MAJOR, orc.COL_MAJOR]
UPLOS = [orc.UPPER, orc.LOWER]
TRANSES = [orc.NO_TRANS, orc.TRANS]
DIAGS = [orc.NON_UNIT, orc.UNIT]


@pytest.fixture(scope="module")
def b2():
    from paper_2411_07211_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(b2):
    c = b2.Context()
    c.reset()
    return c


def matbuf(seed, major, minor, lda, dtype):
    """major x lda buffer, pad columns NaN."""
    buf = synth.vector_np(seed, 7, major * lda, dtype).reshape(major, lda)
    buf[:, minor:] = np.nan
    return buf.ravel()


GEMV_SHAPES = [(1, 1), (3, 5), (17, 33), (64, 64), (100, 700), (700, 100), (257, 1031), (1500, 40), (40, 3000),
               (2049, 513), (130, 2100), (4100, 24),
               # narrow shapes of the paper's skinny study (Section 6.2.2): N = 40, N <= 88 / 44, M a power of 2 or 3
               (2187, 40), (2187, 44), (4096, 88), (88, 4096), (44, 2187), (6561, 8)]


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("order", ORDERS)
@pytest.mark.parametrize("trans", TRANSES)
@pytest.mark.parametrize("m,n", GEMV_SHAPES)
def test_gemv(b2, ctx, dtype, order, trans, m, n):
    minor, major = (n, m) if order == orc.ROW_MAJOR else (m, n)
    lenx, leny = (n, m) if trans == orc.NO_TRANS else (m, n)
    cases = [(0, 0, 1, 1, 0.5), (0, 0, 1, 1, 0.0), (1, 0, 2, 2, 0.5), (4, 1, -1, 3, 0.0), (3, 0, 1, -2, 0.5),
             (0, 0, -2, 3, 0.5)]  # unpadded with strided vectors: the narrow-matrix kernels see every increment
    for pad, offset, incx, incy, beta in cases:
        lda = minor + pad
        a = matbuf(m * 31 + n, major, minor, lda, dtype)
        x = synth.vector_np(1, m + n, lenx, dtype)
        y = synth.vector_np(2, m + n, leny, dtype) if beta != 0 else np.full(leny, np.nan, dtype=dtype)
        hx, hy = place(x, incx), place(y, incy)
        ga, gx, gy = Guarded(a, offset), Guarded(hx), Guarded(hy)
        b2.gemv(ctx, order, trans, m, n, 1.25, ga.t, lda, gx.t, incx, beta, gy.t, incy)
        oy = hy.copy()
        absterms = orc.gemv(order, trans, m, n, dtype(1.25), a, lda, hx, incx, dtype(beta), oy, incy)
        ry = gy.host()
        assert_close(pick(ry, leny, incy), pick(oy, leny, incy), absterms, dtype, f"gemv pad={pad} off={offset}")
        assert_same_gaps(ry, hy, leny, incy)
        assert np.array_equal(ga.host(), a, equal_nan=True) and np.array_equal(gx.host(), hx, equal_nan=True)
        ga.check_guards(), gx.check_guards(), gy.check_guards()
    # alpha == 0: y <- beta*y, A and x may hold anything
    lda = minor
    y = synth.vector_np(2, 5, leny, dtype)
    gy = Guarded(y)
    junk = Guarded(np.full(major * lda, np.nan, dtype=dtype))
    jx = Guarded(np.full(lenx, np.nan, dtype=dtype))
    b2.gemv(ctx, order, trans, m, n, 0.0, junk.t, lda, jx.t, 1, 0.5, gy.t, 1)
    assert np.array_equal(gy.host(), dtype(0.5) * y)
    b2.gemv(ctx, order, trans, m, n, 0.0, junk.t, lda, jx.t, 1, 0.0, gy.t, 1)
    assert np.array_equal(gy.host(), np.zeros(leny, dtype=dtype))


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("order", ORDERS)
@pytest.mark.parametrize("m,n", GEMV_SHAPES)
def test_ger(b2, ctx, dtype, order, m, n):
    minor, major = (n, m) if order == orc.ROW_MAJOR else (m, n)
    for pad, offset, incx, incy in [(0, 0, 1, 1), (1, 0, 2, 2), (4, 1, -1, 3), (2, 0, 1, -2), (0, 0, -1, 2)]:
        lda = minor + pad
        a = matbuf(m * 17 + n, major, minor, lda, dtype)
        x = synth.vector_np(3, m + n, m, dtype)
        y = synth.vector_np(4, m + n, n, dtype)
        hx, hy = place(x, incx), place(y, incy)
        ga, gx, gy = Guarded(a, offset), Guarded(hx), Guarded(hy)
        b2.ger(ctx, order, m, n, 1.25, gx.t, incx, gy.t, incy, ga.t, lda)
        oa = a.copy()
        absterms = orc.ger(order, m, n, dtype(1.25), hx, incx, hy, incy, oa, lda)
        ra = ga.host()
        view = (lambda b: b.reshape(major, lda)[:, :minor]) if True else None
        got, want = view(ra), view(oa)
        if order == orc.COL_MAJOR:
            got, want = got.T, want.T
        assert_close(got, want, absterms, dtype, f"ger pad={pad} off={offset}")
        assert_same_gaps(ra, a)
        ga.check_guards()
        assert np.array_equal(gx.host(), hx, equal_nan=True) and np.array_equal(gy.host(), hy, equal_nan=True)
    ga = Guarded(a)
    b2.ger(ctx, order, m, n, 0.0, gx.t, incx, gy.t, incy, ga.t, lda)
    assert np.array_equal(ga.host(), a, equal_nan=True)


def tri_buf(seed, n, lda, dtype, order, uplo, diag):
    """Conditioned triangular matrix; everything the routine must not use is NaN."""
    buf = synth.matrix_np(seed, 30 + n, n, n, lda, dtype, tri_n=n)
    p, q = np.indices((n, lda))
    r, c = (p, q) if order == orc.ROW_MAJOR else (q, p)
    inside = (r <= c) if uplo == orc.UPPER else (r >= c)
    bad = ~inside | (q >= n)
    if diag == orc.UNIT:
        bad |= (r == c)
    buf[bad] = np.nan
    return buf.ravel()


TRI_SIZES = [1, 2, 5, 31, 64, 65, 127, 128, 129, 200, 513, 1100]
TRI_CASES = [(0, 0, 1), (1, 0, 2), (4, 1, -1), (0, 0, 2)]  # pad, offset, inc


@pytest.fixture(params=[0, 2], ids=["general-kernel", "ring-kernel"])
def symv_kernel(request, b2):
    """symv picks its kernel by the size of the triangle; both are run on every test size."""
    old = b2.get_tuning(b2.KNOB_TRI_TILE)
    b2.set_tuning(b2.KNOB_TRI_TILE, request.param)
    yield request.param
    b2.set_tuning(b2.KNOB_TRI_TILE, old)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("order", ORDERS)
@pytest.mark.parametrize("uplo", UPLOS)
@pytest.mark.parametrize("n", TRI_SIZES)
def test_symv(b2, ctx, dtype, order, uplo, n, symv_kernel):
    for (pad, offset, inc), beta in zip(TRI_CASES, [0.5, 0.0, 0.5, 0.0]):
        lda = n + pad
        a = tri_buf(9, n, lda, dtype, order, uplo, orc.NON_UNIT)
        x = synth.vector_np(5, n, n, dtype)
        y = synth.vector_np(6, n, n, dtype) if beta != 0 else np.full(n, np.nan, dtype=dtype)
        hx, hy = place(x, inc), place(y, -inc)
        ga, gx, gy = Guarded(a, offset), Guarded(hx), Guarded(hy)
        b2.symv(ctx, order, uplo, n, 1.25, ga.t, lda, gx.t, inc, beta, gy.t, -inc)
        oy = hy.copy()
        absterms = orc.symv(order, uplo, n, dtype(1.25), a, lda, hx, inc, dtype(beta), oy, -inc)
        ry = gy.host()
        assert_close(pick(ry, n, -inc), pick(oy, n, -inc), absterms, dtype, f"symv pad={pad}")
        assert_same_gaps(ry, hy, n, -inc)
        ga.check_guards(), gy.check_guards()


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("order", ORDERS)
@pytest.mark.parametrize("uplo", UPLOS)
@pytest.mark.parametrize("trans", TRANSES)
@pytest.mark.parametrize("diag", DIAGS)
@pytest.mark.parametrize("n", TRI_SIZES)
def test_trmv_trsv(b2, ctx, dtype, order, uplo, trans, diag, n):
    for pad, offset, inc in TRI_CASES:
        lda = n + pad
        a = tri_buf(12, n, lda, dtype, order, uplo, diag)
        x = synth.vector_np(7, n, n, dtype)
        hx = place(x, inc)
        ga, gx = Guarded(a, offset), Guarded(hx)
        b2.trmv(ctx, order, uplo, trans, diag, n, ga.t, lda, gx.t, inc)
        ox = hx.copy()
        absterms = orc.trmv(order, uplo, trans, diag, n, a, lda, ox, inc)
        rx = gx.host()
        assert_close(pick(rx, n, inc), pick(ox, n, inc), absterms, dtype, f"trmv pad={pad}")
        assert_same_gaps(rx, hx, n, inc)
        ga.check_guards(), gx.check_guards()
        # trsv: residual of the GPU solution, then forward error against the oracle's solution
        gx = Guarded(hx)
        b2.trsv(ctx, order, uplo, trans, diag, n, ga.t, lda, gx.t, inc)
        assert ctx.device_status() == 0
        rx = gx.host()
        assert_same_gaps(rx, hx, n, inc)
        gx.check_guards()
        resid, scale = orc.trsv_residual(order, uplo, trans, diag, n, a, lda, hx, inc, rx, inc)
        tol = TOL[np.dtype(dtype)]
        assert np.all(resid <= tol * scale), f"trsv residual pad={pad}: worst {np.max(resid / scale):.3e}"
        ox = hx.copy()
        absterms = orc.trsv(order, uplo, trans, diag, n, a, lda, ox, inc)
        assert_close(pick(rx, n, inc), pick(ox, n, inc), 8 * absterms, dtype, "trsv forward")  # |a_ii| >= 1
        assert np.array_equal(ga.host(), a, equal_nan=True)


def test_trsv_bounded_wait_reports_timeout(b2):
    """Host-injected failure: one block of the solve order never publishes (a test hook in the
    library), so its dependants' waits run out.  They must return a status, not hang."""
    ctx = b2.Context(wait_limit=2000)
    ctx.reset()
    n = 128 * 6
    a = Guarded(tri_buf(3, n, n, np.float32, orc.ROW_MAJOR, orc.LOWER, orc.NON_UNIT))
    x = Guarded(synth.vector_np(1, 1, n, np.float32))
    b2.set_tuning(b2.KNOB_TRSV_DEBUG_SKIP, 2)
    try:
        b2.trsv(ctx, orc.ROW_MAJOR, orc.LOWER, orc.NO_TRANS, orc.NON_UNIT, n, a.t, n, x.t, 1)
        torch.cuda.synchronize()
        assert ctx.device_status() == b2.STATUS_TIMEOUT
    finally:
        b2.set_tuning(b2.KNOB_TRSV_DEBUG_SKIP, -1)
    # a timed-out call leaves the control block dirty: without a reset the next call must say so
    # (and leave x as it was) instead of returning an unsolved vector with status 0
    ctx.status.zero_()
    x = Guarded(synth.vector_np(1, 1, n, np.float32))
    b2.trsv(ctx, orc.ROW_MAJOR, orc.LOWER, orc.NO_TRANS, orc.NON_UNIT, n, a.t, n, x.t, 1)
    torch.cuda.synchronize()
    assert ctx.device_status() == b2.STATUS_TIMEOUT
    assert np.array_equal(x.host(), synth.vector_np(1, 1, n, np.float32))
    ctx.reset()
    x = Guarded(synth.vector_np(1, 1, n, np.float32))
    b2.trsv(ctx, orc.ROW_MAJOR, orc.LOWER, orc.NO_TRANS, orc.NON_UNIT, n, a.t, n, x.t, 1)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    resid, scale = orc.trsv_residual(orc.ROW_MAJOR, orc.LOWER, orc.NO_TRANS, orc.NON_UNIT, n, a.host(), n,
                                     synth.vector_np(1, 1, n, np.float32), 1, x.host(), 1)
    assert np.all(resid <= 2e-6 * scale)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("front,cluster,pm_from", [(0, 0, 16), (2, 0, 0), (2, 0, 5), (2, 2, 0), (2, 2, 3)])
def test_trsv_every_kernel_choice(b2, ctx, dtype, front, cluster, pm_from):
    """trsv has three code paths (block-row kernel; sub-block kernel block by block; sub-block
    kernel in clusters), and the sub-block kernel premultiplies the last tile of a block row from
    a given row on.  The defaults pick one per precision and view; here each is forced for every
    view, on sizes with a ragged last block and more block rows than one cluster holds, with the
    premultiplied tile starting at the first row and inside the matrix."""
    old = (b2.get_tuning(b2.KNOB_TRSV_FRONT), b2.get_tuning(b2.KNOB_TRSV_CLUSTER), b2.get_tuning(b2.KNOB_TRSV_PM_FROM))
    b2.set_tuning(b2.KNOB_TRSV_FRONT, front)
    b2.set_tuning(b2.KNOB_TRSV_CLUSTER, cluster)
    b2.set_tuning(b2.KNOB_TRSV_PM_FROM, pm_from)
    try:
        tol = TOL[np.dtype(dtype)]
        for n in (130, 1100, 2052):
            for uplo, trans, diag in itertools.product(UPLOS, TRANSES, DIAGS):
                a = tri_buf(21, n, n, dtype, orc.ROW_MAJOR, uplo, diag)
                hx = synth.vector_np(9, n, n, dtype)
                ga, gx = Guarded(a), Guarded(hx)
                b2.trsv(ctx, orc.ROW_MAJOR, uplo, trans, diag, n, ga.t, n, gx.t, 1)
                assert ctx.device_status() == 0
                rx = gx.host()
                gx.check_guards()
                resid, scale = orc.trsv_residual(orc.ROW_MAJOR, uplo, trans, diag, n, a, n, hx, 1, rx, 1)
                assert np.all(resid <= tol * scale), f"n={n} {uplo} {trans} {diag}: worst {np.max(resid / scale):.3e}"
    finally:
        b2.set_tuning(b2.KNOB_TRSV_FRONT, old[0])
        b2.set_tuning(b2.KNOB_TRSV_CLUSTER, old[1])
        b2.set_tuning(b2.KNOB_TRSV_PM_FROM, old[2])


@pytest.mark.parametrize("dtype", DTYPES)
def test_small_integer_level2_is_bit_exact(b2, ctx, dtype):
    rng = np.random.default_rng(2)
    m, n = 300, 1100
    a = rng.integers(-2, 3, size=(m, n)).astype(dtype)
    x = rng.integers(-2, 3, size=n).astype(dtype)
    xm = rng.integers(-2, 3, size=m).astype(dtype)
    ga, gx, gxm = Guarded(a.ravel()), Guarded(x), Guarded(xm)
    gy = Guarded(np.zeros(m, dtype=dtype))
    b2.gemv(ctx, orc.ROW_MAJOR, orc.NO_TRANS, m, n, 2.0, ga.t, n, gx.t, 1, 0.0, gy.t, 1)
    assert np.array_equal(gy.host(), 2 * (a.astype(np.int64) @ x.astype(np.int64)).astype(dtype))
    gy = Guarded(np.zeros(n, dtype=dtype))
    b2.gemv(ctx, orc.ROW_MAJOR, orc.TRANS, m, n, 2.0, ga.t, n, gxm.t, 1, 0.0, gy.t, 1)
    assert np.array_equal(gy.host(), 2 * (a.astype(np.int64).T @ xm.astype(np.int64)).astype(dtype))
    k = 700
    t = rng.integers(-2, 3, size=(k, k)).astype(dtype)
    v = rng.integers(-2, 3, size=k).astype(dtype)
    gt = Guarded(t.ravel())
    for uplo, tri in [(orc.UPPER, np.triu(t)), (orc.LOWER, np.tril(t))]:
        for trans, diag in itertools.product(TRANSES, DIAGS):
            tt = tri.astype(np.int64)
            if diag == orc.UNIT:
                np.fill_diagonal(tt, 1)
            gv = Guarded(v)
            b2.trmv(ctx, orc.ROW_MAJOR, uplo, trans, diag, k, gt.t, k, gv.t, 1)
            assert np.array_equal(gv.host(), ((tt.T if trans == orc.TRANS else tt) @ v.astype(np.int64)).astype(dtype))
        symm = (tri + tri.T - np.diag(np.diag(t))).astype(np.int64)
        gv, gy = Guarded(v), Guarded(v.copy())
        b2.symv(ctx, orc.ROW_MAJOR, uplo, k, 1.0, gt.t, k, gv.t, 1, -1.0, gy.t, 1)
        assert np.array_equal(gy.host(), (symm @ v.astype(np.int64) - v.astype(np.int64)).astype(dtype))


@pytest.mark.parametrize("dtype", DTYPES)
def test_level2_determinism(b2, ctx, dtype):
    n = 900
    a = Guarded(synth.vector_np(1, 1, n * n, dtype))
    x = synth.vector_np(1, 2, n, dtype)
    outs = []
    for _ in range(3):
        gx, gy = Guarded(x), Guarded(np.zeros(n, dtype=dtype))
        b2.gemv(ctx, orc.ROW_MAJOR, orc.TRANS, n, n, 1.0, a.t, n, gx.t, 1, 0.0, gy.t, 1)
        b2.symv(ctx, orc.ROW_MAJOR, orc.UPPER, n, 1.0, a.t, n, gx.t, 1, 1.0, gy.t, 1)
        b2.trmv(ctx, orc.ROW_MAJOR, orc.LOWER, orc.TRANS, orc.NON_UNIT, n, a.t, n, gy.t, 1)
        outs.append(gy.host().copy())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])


@pytest.mark.parametrize("dtype", DTYPES)
def test_workspace_query_is_enough(b2, dtype):
    """A workspace of exactly b2_workspace_query(m, n, s) bytes serves every level-2 routine on an
    m x n problem (the recommended default is only a default): a matrix of a few very long rows,
    where the column splits of the row-dot kind must all be merged, and a triangular one."""
    s = np.dtype(dtype).itemsize
    tol = TOL[np.dtype(dtype)]
    m, n = 6, 300000
    small = b2.Context(workspace_bytes=b2.lib().b2_workspace_query(m, n, s))
    small.reset()
    a = synth.vector_np(41, 1, m * n, dtype)
    ga = Guarded(a)
    for trans in TRANSES:
        lenx, leny = (n, m) if trans == orc.NO_TRANS else (m, n)
        x, y = synth.vector_np(41, 2, lenx, dtype), synth.vector_np(41, 3, leny, dtype)
        gx, gy = Guarded(x), Guarded(y)
        b2.gemv(small, orc.ROW_MAJOR, trans, m, n, 1.25, ga.t, n, gx.t, 1, 0.5, gy.t, 1)
        oy = y.copy()
        absterms = orc.gemv(orc.ROW_MAJOR, trans, m, n, dtype(1.25), a, n, x, 1, dtype(0.5), oy, 1)
        assert_close(gy.host(), oy, absterms, dtype, f"gemv trans={trans} on the queried workspace")
        gy.check_guards()
    k = 2100
    tri = Guarded(synth.matrix_np(41, 4, k, k, k, dtype, tri_n=k).ravel())
    small = b2.Context(workspace_bytes=b2.lib().b2_workspace_query(k, k, s))
    small.reset()
    v = synth.vector_np(41, 5, k, dtype)
    gv, gy = Guarded(v), Guarded(v.copy())
    b2.symv(small, orc.ROW_MAJOR, orc.LOWER, k, 1.25, tri.t, k, gv.t, 1, 0.5, gy.t, 1)
    oy = v.copy()
    absterms = orc.symv(orc.ROW_MAJOR, orc.LOWER, k, dtype(1.25), tri.host(), k, v, 1, dtype(0.5), oy, 1)
    assert_close(gy.host(), oy, absterms, dtype, "symv on the queried workspace")
    for trans in TRANSES:
        gx = Guarded(v)
        b2.trmv(small, orc.ROW_MAJOR, orc.UPPER, trans, orc.NON_UNIT, k, tri.t, k, gx.t, 1)
        ox = v.copy()
        absterms = orc.trmv(orc.ROW_MAJOR, orc.UPPER, trans, orc.NON_UNIT, k, tri.host(), k, ox, 1)
        assert_close(gx.host(), ox, absterms, dtype, "trmv on the queried workspace")
        gx = Guarded(v)
        b2.trsv(small, orc.ROW_MAJOR, orc.UPPER, trans, orc.NON_UNIT, k, tri.t, k, gx.t, 1)
        assert small.device_status() == 0
        resid, scale = orc.trsv_residual(orc.ROW_MAJOR, orc.UPPER, trans, orc.NON_UNIT, k, tri.host(), k, v, 1,
                                         gx.host(), 1)
        assert np.all(resid <= tol * scale), "trsv on the queried workspace"


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("c", [2.0, 8.0])
def test_trsv_moderately_conditioned(b2, ctx, dtype, c):
    """Matrices that are NOT diagonally dominant: unit diagonal, off-diagonal uniform[-1, 1] * c / sqrt(n)
    (at c = 8 the solution grows to about 3e4 from a right-hand side in [-1, 1]).  The kernels apply
    explicit inverses of the 128 x 128 / 64 x 64 diagonal blocks, whose error grows with the blocks'
    condition number; the row-wise residual of the device solution must still meet the bound."""
    n = 1100
    tol = TOL[np.dtype(dtype)]
    u = synth.vector_np(5, n, n * n, np.float64).reshape(n, n)
    a = (u * c / np.sqrt(n)).astype(dtype)
    np.fill_diagonal(a, 1.0)
    b = synth.vector_np(5, 1, n, dtype)
    ga = Guarded(a.ravel())
    for uplo, trans, diag in ((orc.LOWER, orc.NO_TRANS, orc.UNIT), (orc.UPPER, orc.TRANS, orc.NON_UNIT),
                              (orc.UPPER, orc.NO_TRANS, orc.UNIT), (orc.LOWER, orc.TRANS, orc.NON_UNIT)):
        gx = Guarded(b)
        b2.trsv(ctx, orc.ROW_MAJOR, uplo, trans, diag, n, ga.t, n, gx.t, 1)
        assert ctx.device_status() == 0
        resid, scale = orc.trsv_residual(orc.ROW_MAJOR, uplo, trans, diag, n, a.ravel(), n, b, 1, gx.host(), 1)
        assert np.all(resid <= tol * scale), f"c={c} {uplo} {trans} {diag}: worst {np.max(resid / scale) / tol:.3f} of the bound"


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("unit", [1, 2, 4])
def test_symv_trmv_every_unit_length(b2, ctx, dtype, unit):
    """The tile kernel of symv / trmv cuts block rows (columns) into units of 1, 2 or 4 tiles,
    chosen by the matrix size; here each length is forced on sizes small enough for the full oracle
    and large enough to have rows of several units, a ragged edge, units of a single tile next to
    full ones, and several units per block (more units than SMs)."""
    old = b2.get_tuning(b2.KNOB_TRI_TILE_UNIT), b2.get_tuning(b2.KNOB_TRI_TILE)
    b2.set_tuning(b2.KNOB_TRI_TILE_UNIT, unit)
    b2.set_tuning(b2.KNOB_TRI_TILE, 2)  # every trmv through the tile kernel too
    try:
        for n in (700, 2443, 1280, 2560):  # (the last two: every tile full)
            a = synth.matrix_np(17, 3, n, n, n, dtype, tri_n=n).ravel()
            x, y = synth.vector_np(17, 4, n, dtype), synth.vector_np(17, 5, n, dtype)
            ga = Guarded(a)
            for uplo in UPLOS:
                gx, gy = Guarded(x), Guarded(y)
                b2.symv(ctx, orc.ROW_MAJOR, uplo, n, 1.25, ga.t, n, gx.t, 1, 0.5, gy.t, 1)
                oy = y.copy()
                absterms = orc.symv(orc.ROW_MAJOR, uplo, n, dtype(1.25), a, n, x, 1, dtype(0.5), oy, 1)
                assert_close(gy.host(), oy, absterms, dtype, f"symv n={n} uplo={uplo} unit={unit}")
                for trans, diag in itertools.product(TRANSES, DIAGS):
                    gx = Guarded(x)
                    b2.trmv(ctx, orc.ROW_MAJOR, uplo, trans, diag, n, ga.t, n, gx.t, 1)
                    ox = x.copy()
                    absterms = orc.trmv(orc.ROW_MAJOR, uplo, trans, diag, n, a, n, ox, 1)
                    assert_close(gx.host(), ox, absterms, dtype, f"trmv n={n} {uplo} {trans} {diag} unit={unit}")
    finally:
        b2.set_tuning(b2.KNOB_TRI_TILE_UNIT, old[0])
        b2.set_tuning(b2.KNOB_TRI_TILE, old[1])


@pytest.mark.parametrize("dtype", DTYPES)
def test_tile_kernel_tma_delivery(b2, ctx, dtype):
    """The ring kernel with its tiles delivered by one tiled TMA copy each (tensor map over the
    matrix, zero fill outside it, a shared-memory barrier per ring slot with bounded waits): symv
    and every trmv on sizes with ragged edges, with only full tiles, and with more units than SMs;
    the device status must stay clean (a barrier wait that ran out would set it)."""
    old = b2.get_tuning(b2.KNOB_TRI_TILE), b2.get_tuning(b2.KNOB_TRI_BULK)
    b2.set_tuning(b2.KNOB_TRI_TILE, 2)
    b2.set_tuning(b2.KNOB_TRI_BULK, 1)
    try:
        for n, pad in ((130, 0), (700, 4), (1280, 0), (2443, 0), (2560, 8)):
            lda = n + pad
            a = synth.matrix_np(19, 3, n, lda, lda, dtype, tri_n=n).ravel()
            x, y = synth.vector_np(19, 4, n, dtype), synth.vector_np(19, 5, n, dtype)
            ga = Guarded(a)
            for uplo in UPLOS:
                gx, gy = Guarded(x), Guarded(y)
                b2.symv(ctx, orc.ROW_MAJOR, uplo, n, 1.25, ga.t, lda, gx.t, 1, 0.5, gy.t, 1)
                oy = y.copy()
                absterms = orc.symv(orc.ROW_MAJOR, uplo, n, dtype(1.25), a, lda, x, 1, dtype(0.5), oy, 1)
                assert_close(gy.host(), oy, absterms, dtype, f"symv n={n} uplo={uplo}")
                for trans, diag in itertools.product(TRANSES, DIAGS):
                    gx = Guarded(x)
                    b2.trmv(ctx, orc.ROW_MAJOR, uplo, trans, diag, n, ga.t, lda, gx.t, 1)
                    ox = x.copy()
                    absterms = orc.trmv(orc.ROW_MAJOR, uplo, trans, diag, n, a, lda, ox, 1)
                    assert_close(gx.host(), ox, absterms, dtype, f"trmv n={n} {uplo} {trans} {diag}")
            assert ctx.device_status() == 0
            ga.check_guards()
    finally:
        b2.set_tuning(b2.KNOB_TRI_TILE, old[0])
        b2.set_tuning(b2.KNOB_TRI_BULK, old[1])


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("order", ORDERS)
def test_trmv_tile_kernel_forced(b2, ctx, dtype, order):
    """trmv through the shared-memory-ring tile kernel for every option combination (by default
    only the cases where it is the faster one take it): padded leading dimension, strided and
    reversed x, guard bands, the unreferenced triangle and a unit diagonal NaN-poisoned."""
    old = b2.get_tuning(b2.KNOB_TRI_TILE)
    b2.set_tuning(b2.KNOB_TRI_TILE, 2)
    try:
        for n, (pad, inc) in itertools.product((129, 700), ((0, 1), (4, 2), (8, -1))):
            lda = n + pad
            for uplo, trans, diag in itertools.product(UPLOS, TRANSES, DIAGS):
                a = tri_buf(12, n, lda, dtype, order, uplo, diag)
                x = synth.vector_np(7, n, n, dtype)
                hx = place(x, inc)
                ga, gx = Guarded(a), Guarded(hx)
                b2.trmv(ctx, order, uplo, trans, diag, n, ga.t, lda, gx.t, inc)
                ox = hx.copy()
                absterms = orc.trmv(order, uplo, trans, diag, n, a, lda, ox, inc)
                rx = gx.host()
                assert_close(pick(rx, n, inc), pick(ox, n, inc), absterms, dtype, f"trmv n={n} pad={pad} inc={inc}")
                assert_same_gaps(rx, hx, n, inc)
                ga.check_guards(), gx.check_guards()
    finally:
        b2.set_tuning(b2.KNOB_TRI_TILE, old)
