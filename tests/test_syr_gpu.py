"""GPU parity of syr / syr2 (symmetric rank-1 / rank-2 updates) against the CPU oracle, through
the C ABI.  Each updated element is a two- or three-term sum: |gpu - oracle| <= tol * sum|terms|
(2e-6 float, 4e-15 double), the bound used for ger.  The unreferenced triangle, the pad columns
and the gaps of strided vectors are NaN: they must be neither used nor changed."""
import itertools

import numpy as np
import pytest

from oracle import blas_oracle as orc
from paper_2411_07211_b200 import synth
from tests.gpu_util import TOL, Guarded, place
from tests.test_level2_gpu import tri_buf

pytestmark = pytest.mark.gpu

DTYPES = [np.float32, np.float64]
ORDERS = [orc.ROW_MAJOR, orc.COL_MAJOR]
UPLOS = [orc.UPPER, orc.LOWER]
SIZES = [1, 2, 5, 31, 64, 65, 127, 257, 300, 1100, 1537]


@pytest.fixture(scope="module")
def b2():
    from paper_2411_07211_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(b2):
    c = b2.Context()
    c.reset()
    return c


CASES = [(0, 0, 1, 1), (1, 0, 2, 2), (4, 1, -1, 3), (2, 0, 1, -2)]  # pad, offset, incx, incy


def _check(ra, oa, a, absterms, n, lda, order, uplo, dtype, what):
    got, want, before = (b.reshape(n, lda)[:, :n] for b in (ra, oa, a))
    p, q = np.indices((n, n))
    r, c = (p, q) if order == orc.ROW_MAJOR else (q, p)
    inside = (r <= c) if uplo == orc.UPPER else (r >= c)
    terms = absterms if order == orc.ROW_MAJOR else absterms.T  # absterms is indexed (i, j)
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    bound = TOL[np.dtype(dtype)] * terms
    assert np.all(err[inside] <= bound[inside]), f"{what}: worst {np.max(err[inside] / np.maximum(bound[inside], 1e-300)):.3e}"
    # everything else is bit-for-bit what it was (NaN poison included)
    assert np.array_equal(ra.reshape(n, lda)[:, :n][~inside], before[~inside], equal_nan=True)
    assert np.array_equal(ra.reshape(n, lda)[:, n:], a.reshape(n, lda)[:, n:], equal_nan=True)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("order", ORDERS)
@pytest.mark.parametrize("uplo", UPLOS)
@pytest.mark.parametrize("n", SIZES)
def test_syr_syr2(b2, ctx, dtype, order, uplo, n):
    for pad, offset, incx, incy in CASES:
        lda = n + pad
        a = tri_buf(15, n, lda, dtype, order, uplo, orc.NON_UNIT)
        x = synth.vector_np(3, n, n, dtype)
        y = synth.vector_np(4, n + 1, n, dtype)
        hx, hy = place(x, incx), place(y, incy)
        for two in (False, True):
            ga, gx, gy = Guarded(a, offset), Guarded(hx), Guarded(hy)
            oa = a.copy()
            if two:
                b2.syr2(ctx, order, uplo, n, 1.25, gx.t, incx, gy.t, incy, ga.t, lda)
                absterms = orc.syr2(order, uplo, n, dtype(1.25), hx, incx, hy, incy, oa, lda)
            else:
                b2.syr(ctx, order, uplo, n, 1.25, gx.t, incx, ga.t, lda)
                absterms = orc.syr(order, uplo, n, dtype(1.25), hx, incx, oa, lda)
            _check(ga.host(), oa, a, absterms, n, lda, order, uplo, dtype, f"syr{'2' if two else ''} n={n} pad={pad}")
            ga.check_guards()
            assert np.array_equal(gx.host(), hx, equal_nan=True) and np.array_equal(gy.host(), hy, equal_nan=True)
    # alpha == 0: nothing is touched
    ga = Guarded(a)
    b2.syr(ctx, order, uplo, n, 0.0, gx.t, incx, ga.t, lda)
    b2.syr2(ctx, order, uplo, n, 0.0, gx.t, incx, gy.t, incy, ga.t, lda)
    assert np.array_equal(ga.host(), a, equal_nan=True)


@pytest.mark.parametrize("dtype", DTYPES)
def test_syr_small_integers_bit_exact(b2, ctx, dtype):
    """Integer-valued inputs make every update exact: GPU == oracle bit for bit, whatever the
    order of the two multiplications."""
    rng = np.random.default_rng(5)
    n = 777
    a = rng.integers(-3, 4, size=(n, n)).astype(dtype).ravel()
    x = rng.integers(-2, 3, size=n).astype(dtype)
    y = rng.integers(-2, 3, size=n).astype(dtype)
    for order, uplo in itertools.product(ORDERS, UPLOS):
        ga, gx, gy = Guarded(a), Guarded(x), Guarded(y)
        oa = a.copy()
        b2.syr(ctx, order, uplo, n, 2.0, gx.t, 1, ga.t, n)
        b2.syr2(ctx, order, uplo, n, -1.0, gx.t, 1, gy.t, 1, ga.t, n)
        orc.syr(order, uplo, n, dtype(2), x, 1, oa, n, want_absterms=False)
        orc.syr2(order, uplo, n, dtype(-1), x, 1, y, 1, oa, n, want_absterms=False)
        assert np.array_equal(ga.host(), oa)


def test_syr_argument_errors(b2, ctx):
    import torch
    a = torch.zeros(16, device="cuda")
    x = torch.zeros(4, device="cuda")
    assert b2.syr(ctx, 7, orc.UPPER, 4, 1.0, x, 1, a, 4, check=False) == -1
    assert b2.syr(ctx, orc.ROW_MAJOR, 7, 4, 1.0, x, 1, a, 4, check=False) == -2
    assert b2.syr(ctx, orc.ROW_MAJOR, orc.UPPER, -1, 1.0, x, 1, a, 4, check=False) == -3
    assert b2.syr(ctx, orc.ROW_MAJOR, orc.UPPER, 4, 1.0, x, 0, a, 4, check=False) == -6
    assert b2.syr(ctx, orc.ROW_MAJOR, orc.UPPER, 4, 1.0, x, 1, a, 3, check=False) == -8
    assert b2.syr2(ctx, orc.ROW_MAJOR, orc.UPPER, 4, 1.0, x, 1, x, 0, a, 4, check=False) == -8
    assert b2.syr2(ctx, orc.ROW_MAJOR, orc.UPPER, 4, 1.0, x, 1, x, 1, a, 3, check=False) == -10
    assert b2.syr(ctx, orc.ROW_MAJOR, orc.UPPER, 0, 1.0, x, 1, a, 1, check=False) == 0
