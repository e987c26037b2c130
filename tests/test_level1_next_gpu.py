"""GPU parity of rotm, dsdot and sdsdot against the CPU oracle, through the C ABI.

rotm: each output is a two-term sum, |gpu - oracle| <= tol * (|term1| + |term2|) with the tol of
rot (2e-6 float, 4e-15 double).  dsdot: the products are exact in double, only the order of the
double additions differs: 4e-15 * sum|x_i y_i|.  sdsdot: one float rounding of sb + that sum:
2e-6 * (|sb| + sum|x_i y_i|).  Gaps of strided vectors and guard bands are NaN and must stay."""
import numpy as np
import pytest
import torch

from oracle import blas_oracle as orc
from paper_2411_07211_b200 import synth
from tests.gpu_util import Guarded, assert_close, assert_same_gaps, pick, place

pytestmark = pytest.mark.gpu

DTYPES = [np.float32, np.float64]
SIZES = [0, 1, 2, 3, 7, 8, 31, 33, 127, 129, 1023, 1025, 4099, 70001, 300007]
INCS = [(1, 1), (2, 2), (1, 2), (-1, 1), (3, -2)]
H = (0.75, -1.3, 0.4, 1.7)  # h11, h21, h12, h22


@pytest.fixture(scope="module")
def b2():
    from paper_2411_07211_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(b2):
    c = b2.Context()
    c.reset()
    return c


def _param(flag, poison):
    """[flag, h11, h21, h12, h22]; entries the flag implies are NaN when poison is set."""
    p = [float(flag), *H]
    if poison:
        if flag == 0:
            p[1] = p[4] = float("nan")
        elif flag == 1:
            p[2] = p[3] = float("nan")
        elif flag == -2:
            p[1:] = [float("nan")] * 4
    return p


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("incx,incy", INCS)
@pytest.mark.parametrize("offset", [0, 1])
def test_rotm(b2, ctx, dtype, n, incx, incy, offset):
    x, y = synth.vector_np(300 + n, 1, n, dtype), synth.vector_np(300 + n, 2, n, dtype)
    hx, hy = place(x, incx), place(y, incy)
    for flag in (-1, 0, 1, -2):
        gx, gy = Guarded(hx, offset), Guarded(hy, offset)
        b2.rotm(ctx, n, gx.t, incx, gy.t, incy, _param(flag, True))
        ox, oy = hx.copy(), hy.copy()
        ax, ay = orc.rotm(n, ox, incx, oy, incy, np.array(_param(flag, False), dtype=dtype))
        rx, ry = gx.host(), gy.host()
        if flag == -2:
            assert np.array_equal(rx, hx, equal_nan=True) and np.array_equal(ry, hy, equal_nan=True)
        else:
            assert_close(pick(rx, n, incx), pick(ox, n, incx), ax, dtype, f"rotm flag {flag} x")
            assert_close(pick(ry, n, incy), pick(oy, n, incy), ay, dtype, f"rotm flag {flag} y")
            assert_same_gaps(rx, hx, n, incx), assert_same_gaps(ry, hy, n, incy)
        gx.check_guards(), gy.check_guards()


@pytest.mark.parametrize("dtype", DTYPES)
def test_rotm_exact_data_bit_exact(b2, ctx, dtype):
    """Small integers and a dyadic H: every product and sum is exact, so GPU == oracle bit for bit."""
    n = 100003
    rng = np.random.default_rng(11)
    x = rng.integers(-64, 65, size=n).astype(dtype)
    y = rng.integers(-64, 65, size=n).astype(dtype)
    for flag in (-1, 0, 1):
        param = [flag, 0.5, -0.25, 1.5, 2.0]
        gx, gy = Guarded(x), Guarded(y)
        b2.rotm(ctx, n, gx.t, 1, gy.t, 1, param)
        ox, oy = x.copy(), y.copy()
        orc.rotm(n, ox, 1, oy, 1, np.array(param, dtype=dtype))
        assert np.array_equal(gx.host(), ox) and np.array_equal(gy.host(), oy)


@pytest.mark.parametrize("n", SIZES + [1 << 20, (1 << 22) + 5])
@pytest.mark.parametrize("incx,incy", INCS)
@pytest.mark.parametrize("offset", [0, 1])
def test_dsdot_sdsdot(b2, ctx, n, incx, incy, offset):
    if n > 400000 and (abs(incx) > 2 or abs(incy) > 2):
        pytest.skip("large strided spans are covered at inc=2")
    x, y = synth.vector_np(400 + n % 1000, 1, n, np.float32), synth.vector_np(400 + n % 1000, 2, n, np.float32)
    hx, hy = place(x, incx), place(y, incy)
    gx, gy = Guarded(hx, offset), Guarded(hy, offset)
    dres = torch.full((2,), float("nan"), dtype=torch.float64, device="cuda")
    sres = torch.full((2,), float("nan"), dtype=torch.float32, device="cuda")
    sb = np.float32(-0.3125)
    b2.dsdot(ctx, n, gx.t, incx, gy.t, incy, dres[0:1])
    b2.sdsdot(ctx, n, float(sb), gx.t, incx, gy.t, incy, sres[0:1])
    d, dabs = orc.dsdot(n, hx, incx, hy, incy)
    r, rabs = orc.sdsdot(n, sb, hx, incx, hy, incy)
    gd, gs = dres.cpu().numpy(), sres.cpu().numpy()
    assert_close(gd[0], d, dabs, np.float64, "dsdot")
    assert_close(gs[0], r, rabs, np.float32, "sdsdot")
    assert np.isnan(gd[1]) and np.isnan(gs[1])  # neighbours of the result words untouched
    assert np.array_equal(gx.host(), hx, equal_nan=True) and np.array_equal(gy.host(), hy, equal_nan=True)
    gx.check_guards(), gy.check_guards()
    # deterministic: the same bits again
    d2 = torch.zeros(1, dtype=torch.float64, device="cuda")
    b2.dsdot(ctx, n, gx.t, incx, gy.t, incy, d2)
    assert d2.cpu().numpy().view(np.uint64)[0] == gd[:1].view(np.uint64)[0]


def test_dsdot_cancellation_a_float_accumulator_loses(b2, ctx):
    """2^30 + (many ones) - 2^30: exact in double, lost entirely by float accumulation."""
    n = 4099
    x = np.ones(n, dtype=np.float32)
    x[0], x[-1] = 2.0 ** 30, -(2.0 ** 30)
    y = np.ones(n, dtype=np.float32)
    gx, gy = Guarded(x), Guarded(y)
    dres = torch.zeros(1, dtype=torch.float64, device="cuda")
    sres = torch.zeros(1, dtype=torch.float32, device="cuda")
    b2.dsdot(ctx, n, gx.t, 1, gy.t, 1, dres)
    b2.sdsdot(ctx, n, 0.5, gx.t, 1, gy.t, 1, sres)
    assert dres.item() == float(n - 2) == orc.dsdot(n, x, 1, y, 1)[0]
    assert sres.item() == float(n - 2) + 0.5 == float(orc.sdsdot(n, np.float32(0.5), x, 1, y, 1)[0])


def test_argument_errors(b2, ctx):
    x = torch.zeros(8, device="cuda")
    d = torch.zeros(1, dtype=torch.float64, device="cuda")
    s = torch.zeros(1, device="cuda")
    p = [-1.0, 1.0, 0.0, 0.0, 1.0]
    assert b2.rotm(ctx, -1, x, 1, x, 1, p, check=False) == -1
    assert b2.rotm(ctx, 4, x, 0, x, 1, p, check=False) == -3
    assert b2.rotm(ctx, 4, x, 1, x, 0, p, check=False) == -5
    assert b2.rotm(ctx, 4, x, 1, x, 1, None, check=False) == -6
    assert b2.rotm(ctx, 4, x, 1, x, 1, [3.0, 0, 0, 0, 0], check=False) == -6
    assert b2.dsdot(ctx, -1, x, 1, x, 1, d, check=False) == -1
    assert b2.dsdot(ctx, 4, x, 1, x, 0, d, check=False) == -5
    assert b2.dsdot(ctx, 4, x, 1, x, 1, None, check=False) == -6
    assert b2.sdsdot(ctx, 4, 0.0, x, 0, x, 1, s, check=False) == -4
    assert b2.sdsdot(ctx, 4, 0.0, x, 1, x, 0, s, check=False) == -6
    assert b2.sdsdot(ctx, 4, 0.0, x, 1, x, 1, None, check=False) == -7
    # n == 0: dsdot writes 0, sdsdot writes sb
    d.fill_(7.0), s.fill_(7.0)
    b2.dsdot(ctx, 0, x, 1, x, 1, d)
    b2.sdsdot(ctx, 0, 1.25, x, 1, x, 1, s)
    assert d.item() == 0.0 and s.item() == 1.25
