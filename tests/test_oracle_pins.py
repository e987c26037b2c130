"""Pins the CPU oracle to things other than itself: closed forms, exact rational brute force
on n <= 8 for every option combination, exact integer arithmetic, and algebraic invariants.

The paper prints no worked numeric example for any BLAS routine (its object code for axpy,
Figure 4a, and gemv, Section 2 / Figure 7, fixes only the definitions), so the pins are
mathematical.  The brute-force evaluation here is structured differently from the oracle:
op(A) is materialised as a dense matrix of exact rationals (explicit zeros and ones), then
multiplied / solved with a generic routine, and the exact result is rounded once.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest

from oracle import blas_oracle as orc
from paper_2411_07211_b200 import synth

DTYPES = [np.float32, np.float64]
ORDERS = [orc.ROW_MAJOR, orc.COL_MAJOR]
UPLOS = [orc.UPPER, orc.LOWER]
TRANSES = [orc.NO_TRANS, orc.TRANS]
DIAGS = [orc.NON_UNIT, orc.UNIT]


# ----------------------------------------------------------------- helpers
def strided(vals, inc, fill=np.nan):
    """Place logical vector `vals` in a buffer with BLAS increment `inc` (gaps = fill)."""
    vals = np.asarray(vals)
    n = len(vals)
    buf = np.full(max(1, 1 + (n - 1) * abs(inc)) if n else 1, fill, dtype=vals.dtype)
    for i in range(n):
        buf[i * inc if inc > 0 else (i - (n - 1)) * inc] = vals[i]
    return buf


def logical(buf, n, inc):
    return np.array([buf[i * inc if inc > 0 else (i - (n - 1)) * inc] for i in range(n)],
                    dtype=buf.dtype)


def frac_round(fr, dtype):
    """Exact rational -> nearest value of dtype (float(Fraction) is correctly rounded)."""
    return dtype(float(fr))


def assert_within_ulp(got, exact_fracs, dtype, ulps=1):
    got = np.atleast_1d(got)
    for g, fr in zip(got, exact_fracs):
        ref = frac_round(fr, dtype)
        tol = ulps * float(np.spacing(np.abs(ref) if ref != 0 else dtype(0)))
        assert abs(float(g) - float(fr)) <= tol + 1e-300, (g, float(fr), tol)


def dense_full(order, rows, cols, a, lda):
    """Stored array -> dense list-of-lists of Fractions, A[i][j]."""
    out = [[None] * cols for _ in range(rows)]
    for i in range(rows):
        for j in range(cols):
            v = a[i * lda + j] if order == orc.ROW_MAJOR else a[j * lda + i]
            out[i][j] = v
    return out


def dense_tri_op(order, uplo, trans, diag, n, a, lda):
    """Dense op(A) as Fractions for a triangular A, with explicit zeros / unit diagonal."""
    full = dense_full(order, n, n, a, lda)
    tri = [[Fraction(0)] * n for _ in range(n)]
    for i in range(n):
        for j in range(n):
            inside = (i <= j) if uplo == orc.UPPER else (i >= j)
            if not inside:
                continue
            if i == j and diag == orc.UNIT:
                tri[i][j] = Fraction(1)
            else:
                tri[i][j] = Fraction(float(full[i][j]))
    if trans == orc.TRANS:
        tri = [[tri[j][i] for j in range(n)] for i in range(n)]
    return tri


def matvec(mat, vec):
    return [sum((mij * vj for mij, vj in zip(row, vec)), Fraction(0)) for row in mat]


def gauss_solve(mat, rhs):
    """Generic Gauss-Jordan elimination with partial (first non-zero) pivoting, exact."""
    n = len(rhs)
    m = [list(row) + [rhs[i]] for i, row in enumerate(mat)]
    for col in range(n):
        piv = next(r for r in range(col, n) if m[r][col] != 0)
        m[col], m[piv] = m[piv], m[col]
        inv = 1 / m[col][col]
        m[col] = [v * inv for v in m[col]]
        for r in range(n):
            if r != col and m[r][col] != 0:
                f = m[r][col]
                m[r] = [a - f * b for a, b in zip(m[r], m[col])]
    return [m[i][n] for i in range(n)]


def fr(v):
    return [Fraction(float(t)) for t in v]


def rand(seed, stream, n, dtype):
    return synth.vector_np(seed, stream, n, dtype)


# ----------------------------------------------------------------- closed forms
@pytest.mark.parametrize("dtype", DTYPES)
def test_closed_forms_reductions(dtype):
    for n in [1, 4, 16, 64, 1024]:
        ones = np.ones(n, dtype=dtype)
        assert orc.dot(n, ones, 1, ones, 1)[0] == n
        assert orc.asum(n, -ones, 1)[0] == n
        assert orc.nrm2(n, ones, 1)[0] == dtype(np.sqrt(n))  # exact for n a power of 4
    n = 100
    ramp = np.arange(1, n + 1, dtype=dtype)
    assert orc.asum(n, ramp, 1)[0] == n * (n + 1) // 2
    assert orc.dot(n, ramp, 1, np.ones(n, dtype=dtype), 1)[0] == n * (n + 1) // 2
    assert orc.dot(n, ramp, 1, ramp, 1)[0] == n * (n + 1) * (2 * n + 1) // 6
    assert orc.nrm2(2, np.array([3, -4], dtype=dtype), 1)[0] == 5
    assert orc.nrm2(n, ramp, 1)[0] == dtype(np.sqrt(n * (n + 1) * (2 * n + 1) / 6))
    # empty reductions
    e = np.zeros(1, dtype=dtype)
    assert orc.dot(0, e, 1, e, 1)[0] == 0 and orc.asum(0, e, 1)[0] == 0
    assert orc.nrm2(0, e, 1)[0] == 0 and orc.iamax(0, e, 1) == 0


@pytest.mark.parametrize("dtype", DTYPES)
def test_iamax_first_max_rule(dtype):
    n = 50
    x = rand(1, 1, n, dtype)
    for planted in [(0,), (n - 1,), (7, 8), (3, 30, 49), (49, 3)]:
        v = x.copy()
        for k, p in enumerate(planted):
            v[p] = 1.5 if k % 2 == 0 else -1.5  # equal magnitude, mixed sign
        assert orc.iamax(n, v, 1) == min(planted)
    assert orc.iamax(n, x, 1) == int(np.argmax(np.abs(x)))
    # strided and reversed walks: index is the LOGICAL index
    v = x.copy()
    v[5] = 2.0
    assert orc.iamax(n, strided(v, 3), 3) == 5
    assert orc.iamax(n, strided(v, -2), -2) == 5
    assert orc.iamax(3, np.zeros(3, dtype=dtype), 1) == 0  # all equal -> first


@pytest.mark.parametrize("dtype", DTYPES)
def test_closed_forms_level2(dtype):
    n = 6
    x = rand(2, 1, n, dtype)
    ident = np.eye(n, dtype=dtype).ravel()
    ones = np.ones(n * n, dtype=dtype)
    # A = I: gemv / symv return alpha*x (+ beta*y); power-of-two scalars keep it exact
    for order in ORDERS:
        y = np.zeros(n, dtype=dtype)
        orc.gemv(order, orc.NO_TRANS, n, n, 2.0, ident, n, x, 1, 0.0, y, 1)
        assert np.array_equal(y, 2 * x)
        for uplo in UPLOS:
            y = x.copy()
            orc.symv(order, uplo, n, 0.5, ident, n, x, 1, 4.0, y, 1)
            assert np.array_equal(y, dtype(0.5) * x + dtype(4.0) * x)
            for trans, diag in itertools.product(TRANSES, DIAGS):
                z = x.copy()
                orc.trmv(order, uplo, trans, diag, n, ident, n, z, 1)
                assert np.array_equal(z, x)
                z = x.copy()
                orc.trsv(order, uplo, trans, diag, n, ident, n, z, 1)
                assert np.array_equal(z, x)
    # A = all ones: every gemv output is alpha * sum(x)
    xi = np.arange(1, n + 1, dtype=dtype)
    y = np.zeros(n, dtype=dtype)
    orc.gemv(orc.ROW_MAJOR, orc.NO_TRANS, n, n, 1.0, ones, n, xi, 1, 0.0, y, 1)
    assert np.array_equal(y, np.full(n, 21, dtype=dtype))
    # ger from A = 0 gives the outer product (exact for small integers)
    a = np.zeros(12, dtype=dtype)
    orc.ger(orc.ROW_MAJOR, 3, 4, 2.0, np.array([1, 2, 3], dtype=dtype), 1,
            np.array([1, -1, 2, 5], dtype=dtype), 1, a, 4)
    assert np.array_equal(a.reshape(3, 4), 2 * np.outer([1, 2, 3], [1, -1, 2, 5]))
    # bidiagonal lower system with a telescoping solution: x_i - x_{i-1} = 1  =>  x_i = i+1
    l = (np.eye(n) - np.eye(n, k=-1)).astype(dtype).ravel()
    b = np.ones(n, dtype=dtype)
    orc.trsv(orc.ROW_MAJOR, orc.LOWER, orc.NO_TRANS, orc.NON_UNIT, n, l, n, b, 1)
    assert np.array_equal(b, np.arange(1, n + 1, dtype=dtype))


# ----------------------------------------------------------------- exact brute force, level 1
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", [1, 2, 3, 5, 8])
@pytest.mark.parametrize("incx,incy", [(1, 1), (2, 1), (1, 2), (-1, 1), (2, -3), (-2, -1)])
def test_level1_bruteforce(dtype, n, incx, incy):
    x = rand(3, 10 + n, n, dtype)
    y = rand(3, 20 + n, n, dtype)
    fx, fy = fr(x), fr(y)
    alpha, c, s = dtype(1.5), dtype(0.6), dtype(0.8)
    fa, fc, fs = Fraction(float(alpha)), Fraction(float(c)), Fraction(float(s))

    bx, by = strided(x, incx), strided(y, incy)
    absterms = orc.axpy(n, alpha, bx, incx, by, incy)
    assert_within_ulp(logical(by, n, incy), [fa * a + b for a, b in zip(fx, fy)], dtype)
    assert np.allclose(absterms, [float(abs(fa * a) + abs(b)) for a, b in zip(fx, fy)], rtol=1e-12)
    assert np.array_equal(bx, strided(x, incx), equal_nan=True)  # x and gaps untouched
    assert np.isnan(by).sum() == np.isnan(strided(y, incy)).sum()

    bx = strided(x, incx)
    orc.scal(n, dtype(-0.75), bx, incx)
    assert np.array_equal(logical(bx, n, incx), dtype(-0.75) * x)  # one multiply in T

    bx, by = strided(x, incx), strided(y, incy)
    orc.copy(n, bx, incx, by, incy)
    assert np.array_equal(logical(by, n, incy), x)
    assert np.isnan(by).sum() == np.isnan(strided(y, incy)).sum()

    bx, by = strided(x, incx), strided(y, incy)
    orc.swap(n, bx, incx, by, incy)
    assert np.array_equal(logical(bx, n, incx), y) and np.array_equal(logical(by, n, incy), x)

    bx, by = strided(x, incx), strided(y, incy)
    ax, ay = orc.rot(n, bx, incx, by, incy, c, s)
    assert_within_ulp(logical(bx, n, incx), [fc * a + fs * b for a, b in zip(fx, fy)], dtype)
    assert_within_ulp(logical(by, n, incy), [fc * b - fs * a for a, b in zip(fx, fy)], dtype)
    assert np.allclose(ax, [float(abs(fc * a) + abs(fs * b)) for a, b in zip(fx, fy)], rtol=1e-12)
    assert np.allclose(ay, [float(abs(fc * b) + abs(fs * a)) for a, b in zip(fx, fy)], rtol=1e-12)

    bx, by = strided(x, incx), strided(y, incy)
    d, dabs = orc.dot(n, bx, incx, by, incy)
    assert_within_ulp(d, [sum(a * b for a, b in zip(fx, fy))], dtype)
    assert np.isclose(dabs, float(sum(abs(a * b) for a, b in zip(fx, fy))), rtol=1e-12)
    assert_within_ulp(orc.asum(n, bx, incx)[0], [sum(abs(a) for a in fx)], dtype)
    nr, nabs = orc.nrm2(n, bx, incx)
    ss = sum(a * a for a in fx)
    assert np.isclose(nabs, float(ss), rtol=1e-12)
    assert abs(float(nr) ** 2 - float(ss)) <= 4 * float(np.finfo(dtype).eps) * float(ss)
    assert orc.iamax(n, bx, incx) == int(np.argmax(np.abs(x)))


# ----------------------------------------------------------------- exact brute force, level 2
def _matbuf(seed, stream, rows, cols, lda, dtype, order):
    """Stored buffer for a rows x cols matrix; pad columns (lda > minor dim) are NaN."""
    major, minor = (rows, cols) if order == orc.ROW_MAJOR else (cols, rows)
    buf = synth.vector_np(seed, stream, major * lda, dtype).reshape(major, lda)
    buf[:, minor:] = np.nan
    return buf.ravel()


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("order", ORDERS)
@pytest.mark.parametrize("m,n,pad", [(1, 1, 0), (3, 5, 0), (5, 3, 2), (8, 8, 1), (2, 7, 3)])
def test_gemv_ger_bruteforce(dtype, order, m, n, pad):
    minor = n if order == orc.ROW_MAJOR else m
    lda = minor + pad
    a = _matbuf(4, m * 10 + n, m, n, lda, dtype, order)
    dense = [[Fraction(float(v)) for v in row] for row in dense_full(order, m, n, a, lda)]
    alpha, beta = dtype(1.25), dtype(0.5)
    fa, fb = Fraction(float(alpha)), Fraction(float(beta))
    for trans, (incx, incy) in itertools.product(TRANSES, [(1, 1), (2, 1), (1, 2), (-1, -2)]):
        lenx, leny = (n, m) if trans == orc.NO_TRANS else (m, n)
        x, y = rand(5, lenx, lenx, dtype), rand(6, leny, leny, dtype)
        op = dense if trans == orc.NO_TRANS else [[dense[i][j] for i in range(m)] for j in range(n)]
        for b, fbeta in [(beta, fb), (dtype(0), Fraction(0))]:
            by = strided(y if b != 0 else np.full(leny, np.nan, dtype=dtype), incy)
            absterms = orc.gemv(order, trans, m, n, alpha, a, lda, strided(x, incx), incx, b, by, incy)
            exact = [fa * v + (fbeta * w if b != 0 else 0) for v, w in zip(matvec(op, fr(x)), fr(y))]
            assert_within_ulp(logical(by, leny, incy), exact, dtype)
            # the tolerance scale itself: sum of |alpha*a*x| over the row plus |beta*y|, exactly
            want_abs = [float(sum((abs(fa * a_ * x_) for a_, x_ in zip(row, fr(x))), Fraction(0))
                              + (abs(fbeta * w) if b != 0 else 0)) for row, w in zip(op, fr(y))]
            assert np.allclose(absterms, want_abs, rtol=1e-12, atol=0)
        # alpha == 0 => y = beta*y exactly, A and x never matter
        by = strided(y, incy)
        orc.gemv(order, trans, m, n, dtype(0), np.full_like(a, np.nan), lda,
                 np.full_like(strided(x, incx), np.nan), incx, beta, by, incy)
        assert np.array_equal(logical(by, leny, incy), beta * y)
    for incx, incy in [(1, 1), (2, 3), (-1, 1)]:
        x, y = rand(7, m, m, dtype), rand(8, n, n, dtype)
        a2 = a.copy()
        absterms = orc.ger(order, m, n, alpha, strided(x, incx), incx, strided(y, incy), incy, a2, lda)
        got = dense_full(order, m, n, a2, lda)
        for i in range(m):
            exact = [fa * Fraction(float(x[i])) * Fraction(float(y[j])) + dense[i][j] for j in range(n)]
            assert_within_ulp(np.array(got[i], dtype=dtype), exact, dtype)
            want_abs = [float(abs(fa * Fraction(float(x[i])) * Fraction(float(y[j]))) + abs(dense[i][j]))
                        for j in range(n)]
            assert np.allclose(absterms[i], want_abs, rtol=1e-12)
        assert np.isnan(a2).sum() == np.isnan(a).sum()  # pad untouched
        a3 = a.copy()
        orc.ger(order, m, n, dtype(0), strided(x, incx), incx, strided(y, incy), incy, a3, lda)
        assert np.array_equal(a3, a, equal_nan=True)


def _tri_buf(seed, n, lda, dtype, order, uplo, diag, poison=True):
    """Well-conditioned triangular matrix; the unreferenced triangle, the pad columns and (for
    unit diag) the diagonal are NaN-poisoned: the oracle must never read them."""
    buf = synth.matrix_np(seed, 30 + n, n, n, lda, dtype, tri_n=n)
    r, c = np.indices((n, lda))
    if order == orc.COL_MAJOR:
        r, c = c, r  # buffer position (p, q) holds A(q, p)
    inside = (r <= c) if uplo == orc.UPPER else (r >= c)
    bad = ~inside | (np.indices((n, lda))[1] >= n)
    if diag == orc.UNIT:
        bad |= (r == c)
    if poison:
        buf[bad] = np.nan
    return buf.ravel()


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("order", ORDERS)
@pytest.mark.parametrize("uplo", UPLOS)
@pytest.mark.parametrize("n,pad", [(1, 0), (2, 1), (5, 0), (8, 3)])
def test_symv_bruteforce(dtype, order, uplo, n, pad):
    lda = n + pad
    a = _tri_buf(9, n, lda, dtype, order, uplo, orc.NON_UNIT)
    stored = dense_full(order, n, n, a, lda)
    sym = [[None] * n for _ in range(n)]
    for i in range(n):
        for j in range(n):
            inside = (i <= j) if uplo == orc.UPPER else (i >= j)
            sym[i][j] = Fraction(float(stored[i][j] if inside else stored[j][i]))
    alpha, beta = dtype(1.25), dtype(0.5)
    for incx, incy in [(1, 1), (2, 1), (-1, 2)]:
        x, y = rand(10, n, n, dtype), rand(11, n, n, dtype)
        by = strided(y, incy)
        absterms = orc.symv(order, uplo, n, alpha, a, lda, strided(x, incx), incx, beta, by, incy)
        exact = [Fraction(float(alpha)) * v + Fraction(float(beta)) * w
                 for v, w in zip(matvec(sym, fr(x)), fr(y))]
        assert_within_ulp(logical(by, n, incy), exact, dtype)
        want_abs = [float(sum((abs(Fraction(float(alpha)) * a_ * x_) for a_, x_ in zip(row, fr(x))), Fraction(0))
                          + abs(Fraction(float(beta)) * w)) for row, w in zip(sym, fr(y))]
        assert np.allclose(absterms, want_abs, rtol=1e-12, atol=0)
        # symv == gemv on the explicitly symmetrised dense matrix (same oracle arithmetic)
        full = np.array([[float(v) for v in row] for row in sym], dtype=dtype).ravel()
        by2 = strided(y, incy)
        orc.gemv(orc.ROW_MAJOR, orc.NO_TRANS, n, n, alpha, full, n, strided(x, incx), incx, beta, by2, incy)
        assert np.array_equal(by, by2, equal_nan=True)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("order", ORDERS)
@pytest.mark.parametrize("uplo", UPLOS)
@pytest.mark.parametrize("trans", TRANSES)
@pytest.mark.parametrize("diag", DIAGS)
@pytest.mark.parametrize("n,pad", [(1, 0), (3, 1), (8, 0)])
def test_trmv_trsv_bruteforce(dtype, order, uplo, trans, diag, n, pad):
    lda = n + pad
    a = _tri_buf(12, n, lda, dtype, order, uplo, diag)
    op = dense_tri_op(order, uplo, trans, diag, n, a, lda)
    eps = float(np.finfo(dtype).eps)
    for incx in [1, 2, -1]:
        x = rand(13, n, n, dtype)
        bx = strided(x, incx)
        absterms = orc.trmv(order, uplo, trans, diag, n, a, lda, bx, incx)
        assert_within_ulp(logical(bx, n, incx), matvec(op, fr(x)), dtype)
        want_abs = [float(sum((abs(e * v) for e, v in zip(row, fr(x))), Fraction(0))) for row in op]
        assert np.allclose(absterms, want_abs, rtol=1e-12, atol=0)
        # trsv against exact Gauss-Jordan elimination of the dense op(A)
        bx = strided(x, incx)
        absterms = orc.trsv(order, uplo, trans, diag, n, a, lda, bx, incx)
        exact = gauss_solve(op, fr(x))
        got = logical(bx, n, incx)
        for g, e in zip(got, exact):
            assert abs(float(g) - float(e)) <= 4 * eps * max(abs(float(e)), 1e-30) + 0, (g, float(e))
        # row balance |b_i| + sum over the OFF-diagonal entries of |op(A)_ij x_j|, with the exact
        # solution (the oracle's own wide solution differs from it far below 1e-12 here)
        want_abs = [float(abs(b) + sum((abs(op[i][j] * exact[j]) for j in range(n) if j != i), Fraction(0)))
                    for i, b in enumerate(fr(x))]
        assert np.allclose(absterms, want_abs, rtol=1e-12, atol=0)
        # residual helper agrees with an exact evaluation
        resid, scale = orc.trsv_residual(order, uplo, trans, diag, n, a, lda, strided(x, incx), incx,
                                         bx, incx)
        ex_res = [abs(b - v) for b, v in zip(fr(x), matvec(op, fr(got)))]
        weps = 2.0 ** -52 if dtype == np.float32 else 2.0 ** -63  # rounding unit of W
        assert np.all(np.abs(resid - np.array([float(v) for v in ex_res])) <= 8 * weps * scale)
        # scale_i = |b_i| + sum_j |op(A)_ij xs_j| over the whole row (diagonal included), exactly
        want_scale = [float(abs(b) + sum((abs(e * v) for e, v in zip(row, fr(got))), Fraction(0)))
                      for b, row in zip(fr(x), op)]
        assert np.allclose(scale, want_scale, rtol=1e-12, atol=0)
        assert np.all(resid <= 2 * eps * scale)
        # trsv(trmv(x)) recovers x
        bx = strided(x, incx)
        orc.trmv(order, uplo, trans, diag, n, a, lda, bx, incx)
        orc.trsv(order, uplo, trans, diag, n, a, lda, bx, incx)
        assert np.allclose(logical(bx, n, incx), x, rtol=0, atol=32 * eps)


# ----------------------------------------------------------------- exact integer arithmetic
@pytest.mark.parametrize("dtype", DTYPES)
def test_small_integer_inputs_are_exact(dtype):
    rng = np.random.default_rng(0)
    m, n = 37, 53
    a = rng.integers(-2, 3, size=(m, n))
    x = rng.integers(-2, 3, size=n)
    xm = rng.integers(-2, 3, size=m)
    y = rng.integers(-2, 3, size=m)
    yn = rng.integers(-2, 3, size=n)
    af = a.astype(dtype).ravel()
    out = y.astype(dtype)
    orc.gemv(orc.ROW_MAJOR, orc.NO_TRANS, m, n, 2.0, af, n, x.astype(dtype), 1, 3.0, out, 1)
    assert np.array_equal(out, (2 * a @ x + 3 * y).astype(dtype))
    out = yn.astype(dtype)
    orc.gemv(orc.ROW_MAJOR, orc.TRANS, m, n, 2.0, af, n, xm.astype(dtype), 1, 3.0, out, 1)
    assert np.array_equal(out, (2 * a.T @ xm + 3 * yn).astype(dtype))
    # column-major call on the same buffer sees the transposed matrix
    out = yn.astype(dtype)
    orc.gemv(orc.COL_MAJOR, orc.NO_TRANS, n, m, 2.0, af, n, xm.astype(dtype), 1, 3.0, out, 1)
    assert np.array_equal(out, (2 * a.T @ xm + 3 * yn).astype(dtype))
    a2 = af.copy()
    orc.ger(orc.ROW_MAJOR, m, n, -2.0, xm.astype(dtype), 1, x.astype(dtype), 1, a2, n)
    assert np.array_equal(a2.reshape(m, n), (a - 2 * np.outer(xm, x)).astype(dtype))
    xi = rng.integers(-2, 3, size=1000)
    yi = rng.integers(-2, 3, size=1000)
    assert orc.dot(1000, xi.astype(dtype), 1, yi.astype(dtype), 1)[0] == int(xi @ yi)
    assert orc.asum(1000, xi.astype(dtype), 1)[0] == int(np.abs(xi).sum())
    # triangular / symmetric with integers
    k = 41
    t = rng.integers(-2, 3, size=(k, k))
    v = rng.integers(-2, 3, size=k)
    for uplo, tri in [(orc.UPPER, np.triu(t)), (orc.LOWER, np.tril(t))]:
        for trans in TRANSES:
            for diag in DIAGS:
                tt = tri.copy()
                if diag == orc.UNIT:
                    np.fill_diagonal(tt, 1)
                op = tt.T if trans == orc.TRANS else tt
                z = v.astype(dtype)
                orc.trmv(orc.ROW_MAJOR, uplo, trans, diag, k, t.astype(dtype).ravel(), k, z, 1)
                assert np.array_equal(z, (op @ v).astype(dtype))
        symm = tri + tri.T - np.diag(np.diag(t))
        z = v.astype(dtype)
        orc.symv(orc.ROW_MAJOR, uplo, k, 1.0, t.astype(dtype).ravel(), k, v.astype(dtype), 1, -1.0, z, 1)
        assert np.array_equal(z, (symm @ v - v).astype(dtype))


# ----------------------------------------------------------------- invariants
@pytest.mark.parametrize("dtype", DTYPES)
def test_invariants(dtype):
    n = 300
    eps = float(np.finfo(dtype).eps)
    x, y = rand(20, 1, n, dtype), rand(20, 2, n, dtype)
    # alpha = 0 leaves y unchanged, bit for bit, even with NaN in x
    y2 = y.copy()
    orc.axpy(n, dtype(0), np.full(n, np.nan, dtype=dtype), 1, y2, 1)
    assert np.array_equal(y2, y)
    # rot preserves sum x^2 + y^2 when c^2 + s^2 = 1; identity and quarter-turn special cases
    x2, y2 = x.copy(), y.copy()
    orc.rot(n, x2, 1, y2, 1, dtype(0.6), dtype(0.8))
    before = np.sum(x.astype(np.float64) ** 2 + y.astype(np.float64) ** 2)
    after = np.sum(x2.astype(np.float64) ** 2 + y2.astype(np.float64) ** 2)
    assert abs(before - after) <= 8 * eps * before
    x2, y2 = x.copy(), y.copy()
    orc.rot(n, x2, 1, y2, 1, dtype(1), dtype(0))
    assert np.array_equal(x2, x) and np.array_equal(y2, y)
    orc.rot(n, x2, 1, y2, 1, dtype(0), dtype(1))
    assert np.array_equal(x2, y) and np.array_equal(y2, -x)
    # swap o swap = identity; copy then dot(x,x) = nrm2^2
    x2, y2 = x.copy(), y.copy()
    orc.swap(n, x2, 1, y2, 1)
    orc.swap(n, x2, 1, y2, 1)
    assert np.array_equal(x2, x) and np.array_equal(y2, y)
    orc.copy(n, x, 1, y2, 1)
    d = float(orc.dot(n, x, 1, y2, 1)[0])
    assert abs(d - float(orc.nrm2(n, x, 1)[0]) ** 2) <= 4 * eps * d
    # strided call == unit-stride call on the gathered vector
    assert orc.dot(n, strided(x, 2), 2, strided(y, -3), -3) == orc.dot(n, x, 1, y, 1)
    # gemv-T(A) == gemv-N(A^T stored explicitly); col-major == row-major on transposed storage
    m, k = 23, 31
    a = rand(21, 1, m * k, dtype).reshape(m, k)
    xm, yk = rand(21, 2, m, dtype), rand(21, 3, k, dtype)
    o1, o2, o3 = yk.copy(), yk.copy(), yk.copy()
    orc.gemv(orc.ROW_MAJOR, orc.TRANS, m, k, 1.25, a.ravel(), k, xm, 1, 0.5, o1, 1)
    orc.gemv(orc.ROW_MAJOR, orc.NO_TRANS, k, m, 1.25, np.ascontiguousarray(a.T).ravel(), m, xm, 1, 0.5, o2, 1)
    orc.gemv(orc.COL_MAJOR, orc.TRANS, m, k, 1.25, np.ascontiguousarray(a.T).ravel(), m, xm, 1, 0.5, o3, 1)
    assert np.array_equal(o1, o2) and np.array_equal(o1, o3)
    ref = 1.25 * (a.astype(np.float64).T @ xm.astype(np.float64)) + 0.5 * yk
    assert np.allclose(o1, ref, rtol=0, atol=64 * eps)


def test_golden_sdot_config1():
    """Stored value written by tests/golden/make_golden.py (oracle + generator only)."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "sdot_n1048576_seed0.txt")
    fields = dict(line.split("=") for line in open(path).read().split() if "=" in line)
    n = int(fields["n"])
    x = synth.vector_np(0, 0, n, np.float32)
    y = synth.vector_np(0, 1, n, np.float32)
    res, absterms = orc.dot(n, x, 1, y, 1)
    assert float(res).hex() == fields["result_hex"]
    # independent evaluation: numpy pairwise float64 sum of exact float64 products
    ref = np.sum(x.astype(np.float64) * y.astype(np.float64))
    assert abs(float(res) - ref) <= 2.0 ** -24 * abs(ref) + 1e-9 * absterms


# ----------------------------------------------------------------- syr / syr2 (the "next" rows)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("order", ORDERS)
@pytest.mark.parametrize("uplo", UPLOS)
@pytest.mark.parametrize("n,pad", [(1, 0), (2, 1), (5, 0), (8, 3)])
def test_syr_syr2_bruteforce(dtype, order, uplo, n, pad):
    """Exact rational evaluation of the definition on the stored triangle; the other triangle,
    the pad columns and the strided gaps are NaN and must stay untouched / unread."""
    lda = n + pad
    a = _tri_buf(11, n, lda, dtype, order, uplo, orc.NON_UNIT)
    dense = dense_full(order, n, n, a, lda)
    alpha = dtype(1.25)
    fa = Fraction(float(alpha))
    for incx, incy in [(1, 1), (2, 3), (-1, 2)]:
        x, y = rand(3, n, n, dtype), rand(4, n + 1, n, dtype)
        fx, fy = fr(x), fr(y)
        for two in (False, True):
            a2 = a.copy()
            if two:
                absterms = orc.syr2(order, uplo, n, alpha, strided(x, incx), incx, strided(y, incy), incy, a2, lda)
            else:
                absterms = orc.syr(order, uplo, n, alpha, strided(x, incx), incx, a2, lda)
            got = dense_full(order, n, n, a2, lda)
            for i in range(n):
                for j in range(n):
                    inside = (i <= j) if uplo == orc.UPPER else (i >= j)
                    if not inside:
                        assert np.isnan(got[i][j])  # never written
                        continue
                    upd = fa * (fx[i] * fy[j] + fy[i] * fx[j]) if two else fa * fx[i] * fx[j]
                    assert_within_ulp(np.array([got[i][j]], dtype=dtype), [upd + Fraction(float(dense[i][j]))], dtype)
                    terms = ([abs(fa * fx[i] * fy[j]), abs(fa * fy[i] * fx[j])] if two else [abs(fa * fx[i] * fx[j])])
                    want_abs = float(sum(terms) + abs(Fraction(float(dense[i][j]))))
                    assert np.isclose(absterms[i, j], want_abs, rtol=1e-12)
            assert np.isnan(a2).sum() == np.isnan(a).sum()
            a3 = a.copy()  # alpha == 0: untouched, vectors never matter
            nanx = np.full_like(strided(x, incx), np.nan)
            if two:
                orc.syr2(order, uplo, n, dtype(0), nanx, incx, np.full_like(strided(y, incy), np.nan), incy, a3, lda)
            else:
                orc.syr(order, uplo, n, dtype(0), nanx, incx, a3, lda)
            assert np.array_equal(a3, a, equal_nan=True)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("uplo", UPLOS)
def test_syr_invariants(dtype, uplo):
    """syr equals ger(x, x) on the triangle; syr2(x, x) with alpha equals syr with 2*alpha (exact:
    a power of two); row-major upper equals column-major lower on the same buffer; from A = 0
    the result is alpha*x_i*x_j."""
    n = 37
    x, y = rand(5, n, n, dtype), rand(6, n, n, dtype)
    full = synth.matrix_np(9, 2, n, n, n, dtype).ravel()
    alpha = dtype(0.75)
    g = full.copy()
    orc.ger(orc.ROW_MAJOR, n, n, alpha, x, 1, x, 1, g, n, want_absterms=False)
    s1 = full.copy()
    orc.syr(orc.ROW_MAJOR, uplo, n, alpha, x, 1, s1, n, want_absterms=False)
    r, c = np.indices((n, n))
    inside = ((r <= c) if uplo == orc.UPPER else (r >= c)).ravel()
    assert np.array_equal(s1[inside], g[inside]) and np.array_equal(s1[~inside], full[~inside])
    s2 = full.copy()
    orc.syr2(orc.ROW_MAJOR, uplo, n, alpha, x, 1, x, 1, s2, n, want_absterms=False)
    s3 = full.copy()
    orc.syr(orc.ROW_MAJOR, uplo, n, dtype(2) * alpha, x, 1, s3, n, want_absterms=False)
    tol = 4 * np.finfo(dtype).eps
    assert np.all(np.abs(s2 - s3) <= tol * (np.abs(s3) + 1))
    other = orc.LOWER if uplo == orc.UPPER else orc.UPPER
    s4 = full.copy()
    orc.syr2(orc.COL_MAJOR, other, n, alpha, x, 1, y, 1, s4, n, want_absterms=False)
    s5 = full.copy()
    orc.syr2(orc.ROW_MAJOR, uplo, n, alpha, x, 1, y, 1, s5, n, want_absterms=False)
    assert np.array_equal(s4, s5)
    z = np.zeros(n * n, dtype=dtype)
    orc.syr(orc.ROW_MAJOR, uplo, n, alpha, x, 1, z, n, want_absterms=False)
    want = (np.longdouble(alpha) * np.outer(x.astype(np.longdouble), x.astype(np.longdouble))).ravel()
    err = np.abs(z.astype(np.longdouble) - want)[inside]
    assert np.all(err <= np.spacing(np.abs(z[inside])).astype(np.longdouble)) and np.all(z[~inside] == 0)


# ----------------------------------------------------------------- rotm / dsdot / sdsdot (the "next" rows)
def _h_of(flag, h11, h21, h12, h22):
    """The 2x2 matrix the flag selects, as exact rationals (BLAS definition of rotm)."""
    one = Fraction(1)
    f = lambda v: Fraction(float(v))
    if flag == -1:
        return f(h11), f(h12), f(h21), f(h22)
    if flag == 0:
        return one, f(h12), f(h21), one
    if flag == 1:
        return f(h11), one, -one, f(h22)
    return one, Fraction(0), Fraction(0), one


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("flag", [-2, -1, 0, 1])
@pytest.mark.parametrize("n", [1, 3, 8])
@pytest.mark.parametrize("incx,incy", [(1, 1), (2, -1), (-3, 2)])
def test_rotm_bruteforce(dtype, flag, n, incx, incy):
    x, y = rand(5, 30 + n, n, dtype), rand(5, 40 + n, n, dtype)
    fx, fy = fr(x), fr(y)
    h11, h21, h12, h22 = dtype(0.75), dtype(-1.3), dtype(0.4), dtype(1.7)
    a11, a12, a21, a22 = _h_of(flag, h11, h21, h12, h22)
    # the entries the flag implies must not be read: poison them
    param = np.array([flag, h11, h21, h12, h22], dtype=dtype)
    if flag == 0:
        param[1] = param[4] = np.nan
    if flag == 1:
        param[2] = param[3] = np.nan
    if flag == -2:
        param[1:] = np.nan
    bx, by = strided(x, incx), strided(y, incy)
    ax, ay = orc.rotm(n, bx, incx, by, incy, param)
    if flag == -2:  # identity: bit-for-bit untouched
        assert np.array_equal(bx, strided(x, incx), equal_nan=True)
        assert np.array_equal(by, strided(y, incy), equal_nan=True)
        return
    assert_within_ulp(logical(bx, n, incx), [a11 * a + a12 * b for a, b in zip(fx, fy)], dtype)
    assert_within_ulp(logical(by, n, incy), [a21 * a + a22 * b for a, b in zip(fx, fy)], dtype)
    assert np.allclose(ax, [float(abs(a11 * a) + abs(a12 * b)) for a, b in zip(fx, fy)], rtol=1e-12)
    assert np.allclose(ay, [float(abs(a21 * a) + abs(a22 * b)) for a, b in zip(fx, fy)], rtol=1e-12)
    assert np.isnan(bx).sum() == np.isnan(strided(x, incx)).sum()  # gaps untouched
    assert np.isnan(by).sum() == np.isnan(strided(y, incy)).sum()


@pytest.mark.parametrize("dtype", DTYPES)
def test_rotm_reduces_to_rot_and_to_explicit_h(dtype):
    """flag -1 with H = [c s; -s c] is the plain rotation (pinned above) bit for bit; flags 0 and 1
    equal flag -1 with the implied entries written out; two rotm's compose like the matrix product
    on exactly representable data."""
    n = 37
    x, y = rand(6, 1, n, dtype), rand(6, 2, n, dtype)
    c, s = dtype(0.6), dtype(0.8)
    x1, y1, x2, y2 = x.copy(), y.copy(), x.copy(), y.copy()
    orc.rot(n, x1, 1, y1, 1, c, s)
    orc.rotm(n, x2, 1, y2, 1, np.array([-1, c, -s, s, c], dtype=dtype))
    assert np.array_equal(x1, x2) and np.array_equal(y1, y2)
    h11, h21, h12, h22 = dtype(0.5), dtype(-0.25), dtype(1.5), dtype(2.0)
    for flag, full in ((0, [-1, 1, h21, h12, 1]), (1, [-1, h11, -1, 1, h22])):
        x1, y1, x2, y2 = x.copy(), y.copy(), x.copy(), y.copy()
        orc.rotm(n, x1, 1, y1, 1, np.array([flag, h11, h21, h12, h22], dtype=dtype))
        orc.rotm(n, x2, 1, y2, 1, np.array(full, dtype=dtype))
        assert np.array_equal(x1, x2) and np.array_equal(y1, y2)
    # exact data (small integers, dyadic H): H2 (H1 v) == (H2 H1) v with no rounding anywhere
    xi = np.arange(-18, 19, dtype=dtype)
    yi = np.arange(37, 0, -1, dtype=dtype)
    h1 = np.array([[0.5, 1.5], [-0.25, 2.0]])
    h2 = np.array([[2.0, -0.5], [0.75, 1.0]])
    xa, ya = xi.copy(), yi.copy()
    orc.rotm(n, xa, 1, ya, 1, np.array([-1, h1[0, 0], h1[1, 0], h1[0, 1], h1[1, 1]], dtype=dtype))
    orc.rotm(n, xa, 1, ya, 1, np.array([-1, h2[0, 0], h2[1, 0], h2[0, 1], h2[1, 1]], dtype=dtype))
    h = h2 @ h1
    assert np.array_equal(xa, (h[0, 0] * xi + h[0, 1] * yi).astype(dtype))
    assert np.array_equal(ya, (h[1, 0] * xi + h[1, 1] * yi).astype(dtype))


@pytest.mark.parametrize("n", [0, 1, 2, 5, 8])
@pytest.mark.parametrize("incx,incy", [(1, 1), (2, 1), (-1, 3), (-2, -1)])
def test_dsdot_sdsdot_bruteforce(n, incx, incy):
    x, y = rand(7, 50 + n, n, np.float32), rand(7, 60 + n, n, np.float32)
    fx, fy = fr(x), fr(y)
    exact = sum((a * b for a, b in zip(fx, fy)), Fraction(0))
    bx, by = strided(x, incx), strided(y, incy)
    d, dabs = orc.dsdot(n, bx, incx, by, incy)
    assert isinstance(d, np.float64)
    assert_within_ulp(d, [exact], np.float64)
    assert np.isclose(dabs, float(sum((abs(a * b) for a, b in zip(fx, fy)), Fraction(0))), rtol=1e-12)
    sb = np.float32(-0.3125)
    r, rabs = orc.sdsdot(n, sb, bx, incx, by, incy)
    assert isinstance(r, np.float32)
    assert_within_ulp(r, [exact + Fraction(float(sb))], np.float32)
    assert np.isclose(rabs, dabs + abs(float(sb)), rtol=1e-12)


def test_dsdot_keeps_what_float_accumulation_loses():
    """Cancellation that a float accumulator cannot survive: 2^30*1 + 1*1 - 2^30*1 is exactly 1;
    in float 2^30 + 1 rounds to 2^30 and the sum would be 0.  Also: dsdot equals the double dot
    product of the widened inputs (products of floats are exact in double)."""
    x = np.array([2.0 ** 30, 1.0, -(2.0 ** 30)], dtype=np.float32)
    y = np.ones(3, dtype=np.float32)
    assert np.float32(np.float32(2.0 ** 30) + np.float32(1.0)) == np.float32(2.0 ** 30)
    assert orc.dsdot(3, x, 1, y, 1)[0] == 1.0
    assert orc.sdsdot(3, np.float32(0.5), x, 1, y, 1)[0] == np.float32(1.5)
    # a sum whose exact value needs more than 24 bits: 2^24 + 1 is not a float, but is a double
    x = np.array([2.0 ** 12, 1.0], dtype=np.float32)
    y = np.array([2.0 ** 12, 1.0], dtype=np.float32)
    assert orc.dsdot(2, x, 1, y, 1)[0] == 2.0 ** 24 + 1
    assert orc.sdsdot(2, np.float32(0), x, 1, y, 1)[0] == np.float32(2.0 ** 24)  # ties-to-even
    n = 1000
    x, y = rand(8, 1, n, np.float32), rand(8, 2, n, np.float32)
    wide = orc.dot(n, x.astype(np.float64), 1, y.astype(np.float64), 1)[0]
    assert orc.dsdot(n, x, 1, y, 1)[0] == wide
    assert abs(wide - np.dot(x.astype(np.float64), y.astype(np.float64))) <= 1e-13 * float(np.sum(np.abs(x * y)))
