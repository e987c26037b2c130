"""Parity of the rows built after the headline set at the sizes the bench's next-rows leg times:
syr / syr2 on sampled row segments (each computed by the oracle as a tiny problem of its own),
rotm on sampled elements, dsdot / sdsdot against the full oracle sum."""
import numpy as np
import pytest
import torch

from oracle import blas_oracle as orc
from paper_2411_07211_b200 import synth
from tests.gpu_util import assert_close

pytestmark = pytest.mark.gpu

TD = {np.float32: torch.float32, np.float64: torch.float64}


@pytest.fixture(scope="module")
def b2():
    from paper_2411_07211_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(b2):
    c = b2.Context()
    c.reset()
    return c


def dvec(seed, stream, n, dtype, inc):
    v = synth.vector_torch(seed, stream, n, TD[dtype], "cuda")
    if inc == 1:
        return v
    buf = torch.full(((n - 1) * inc + 1,), float("nan"), dtype=TD[dtype], device="cuda")
    buf[::inc] = v
    return buf


@pytest.mark.parametrize("dtype,n", [(np.float32, 8192), (np.float64, 5760)])
@pytest.mark.parametrize("uplo", [orc.UPPER, orc.LOWER])
@pytest.mark.parametrize("inc", [1, 2])
def test_syr_syr2_bench_size(b2, ctx, dtype, n, uplo, inc):
    seed, w = 41, 48
    a0 = synth.matrix_torch(seed, 1, n, n, n, TD[dtype], "cuda")
    hx, hy = synth.vector_np(seed, 2, n, dtype), synth.vector_np(seed, 3, n, dtype)
    dx, dy = dvec(seed, 2, n, dtype, inc), dvec(seed, 3, n, dtype, inc)
    rng = np.random.default_rng(n + uplo + inc)
    rows = np.unique(np.concatenate([[0, 1, 15, 16, 17, 511, 512, n // 2, n - 2, n - 1], rng.integers(0, n, size=40)]))
    for two in (False, True):
        a = a0.clone()
        if two:
            b2.syr2(ctx, orc.ROW_MAJOR, uplo, n, 1.25, dx, inc, dy, inc, a, n)
        else:
            b2.syr(ctx, orc.ROW_MAJOR, uplo, n, 1.25, dx, inc, a, n)
        for i in rows:
            i = int(i)
            # a segment of row i inside the stored triangle, ending (upper: starting) at the diagonal
            # for every other row so that diagonal tiles are sampled too
            if uplo == orc.UPPER:
                c0 = i if i % 2 == 0 else int(rng.integers(i, n))
                c1 = min(n, c0 + w)
            else:
                c1 = i + 1 if i % 2 == 0 else int(rng.integers(0, i + 1)) + 1
                c0 = max(0, c1 - w)
            cols = np.arange(c0, c1)
            k = len(cols)
            seg = synth.matrix_entries_np(seed, 1, i, cols, n, dtype)
            # tiny problem: index 0 is row i, indices 1..k are the columns; its row 0 (upper) is the segment
            t = np.zeros((k + 1, k + 1), dtype=dtype)
            t[0, 1:] = seg
            tx = np.concatenate([hx[i:i + 1], hx[cols]])
            ty = np.concatenate([hy[i:i + 1], hy[cols]])
            tb = t.ravel().copy()
            if two:
                at = orc.syr2(orc.ROW_MAJOR, orc.UPPER, k + 1, dtype(1.25), tx, 1, ty, 1, tb, k + 1)
            else:
                at = orc.syr(orc.ROW_MAJOR, orc.UPPER, k + 1, dtype(1.25), tx, 1, tb, k + 1)
            want = tb.reshape(k + 1, k + 1)[0, 1:]
            # the diagonal element (i, i) appears in the tiny problem as (0, j) with x_j = x_i: the same terms
            assert_close(a[i, c0:c1].cpu().numpy(), want, at.reshape(k + 1, k + 1)[0, 1:], dtype,
                         f"syr{'2' if two else ''} row {i} cols {c0}:{c1}")
            # the other triangle of this row is untouched, bit for bit
            if uplo == orc.UPPER and i > 0:
                o0, o1 = max(0, i - w), i
            elif uplo == orc.LOWER and i < n - 1:
                o0, o1 = i + 1, min(n, i + 1 + w)
            else:
                continue
            assert torch.equal(a[i, o0:o1], a0[i, o0:o1])
    del a, a0
    torch.cuda.empty_cache()


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("inc", [1, 2])
def test_rotm_bench_size(b2, ctx, dtype, inc):
    n = (1 << 25 if dtype == np.float32 else 1 << 24) // inc
    hx, hy = synth.vector_np(43, 0, n, dtype), synth.vector_np(43, 1, n, dtype)
    rng = np.random.default_rng(5)
    idx = np.unique(np.concatenate([[0, 1, 2, 3, n - 1, n - 2, n // 2], rng.integers(0, n, size=3000)]))
    tidx = torch.from_numpy(idx * inc).cuda()
    for param in ([-1.0, 0.6, -0.8, 0.8, 0.6], [0.0, 9.0, -0.3, 0.7, 9.0], [1.0, 0.4, 9.0, 9.0, -1.1]):
        dx, dy = dvec(43, 0, n, dtype, inc), dvec(43, 1, n, dtype, inc)
        b2.rotm(ctx, n, dx, inc, dy, inc, param)
        ox, oy = hx[idx].copy(), hy[idx].copy()
        ax, ay = orc.rotm(len(idx), ox, 1, oy, 1, np.array(param, dtype=dtype))
        assert_close(dx[tidx].cpu().numpy(), ox, ax, dtype, f"rotm x flag {param[0]}")
        assert_close(dy[tidx].cpu().numpy(), oy, ay, dtype, f"rotm y flag {param[0]}")
        if inc == 2:
            assert bool(torch.isnan(dx[1::2]).all()) and bool(torch.isnan(dy[1::2]).all())


@pytest.mark.parametrize("inc", [1, 2])
def test_dsdot_sdsdot_bench_size(b2, ctx, inc):
    n = (1 << 25) // inc
    hx, hy = synth.vector_np(44, 0, n, np.float32), synth.vector_np(44, 1, n, np.float32)
    dx, dy = dvec(44, 0, n, np.float32, inc), dvec(44, 1, n, np.float32, inc)
    dres = torch.zeros(1, dtype=torch.float64, device="cuda")
    sres = torch.zeros(1, dtype=torch.float32, device="cuda")
    b2.dsdot(ctx, n, dx, inc, dy, inc, dres)
    b2.sdsdot(ctx, n, -0.3125, dx, inc, dy, inc, sres)
    d, dabs = orc.dsdot(n, hx, 1, hy, 1)
    r, rabs = orc.sdsdot(n, np.float32(-0.3125), hx, 1, hy, 1)
    assert_close(dres.item(), d, dabs, np.float64, "dsdot")
    assert_close(sres.item(), r, rabs, np.float32, "sdsdot")
