"""Level-2 parity at the sizes the configs name (and the bench times), on sampled outputs.

The matrices are generated on the device by the counter-based generator; for each sampled output
the host regenerates just the row / column of the matrix it depends on and the CPU oracle
computes that one output (a 1 x n gemv or a dot product in wide accumulation).
"""
import numpy as np
import pytest
import torch

from oracle import blas_oracle as orc
from paper_2411_07211_b200 import synth
from tests.gpu_util import TOL, assert_close

pytestmark = pytest.mark.gpu

TD = {np.float32: torch.float32, np.float64: torch.float64}
NS = 48  # sampled outputs per case


@pytest.fixture(scope="module")
def b2():
    from paper_2411_07211_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(b2):
    c = b2.Context()
    c.reset()
    return c


def sample(n, seed):
    rng = np.random.default_rng(seed)
    fixed = [0, 1, n // 2, n - 2, n - 1, 63, 64, 127, 128]
    return np.unique(np.clip(np.concatenate([fixed, rng.integers(0, n, size=NS)]), 0, n - 1))


def dvec(seed, stream, n, dtype, inc=1):
    v = synth.vector_torch(seed, stream, n, TD[dtype], "cuda")
    if inc == 1:
        return v
    buf = torch.full(((n - 1) * inc + 1,), float("nan"), dtype=TD[dtype], device="cuda")
    buf[::inc] = v
    return buf


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("m,n", [(4096, 4096), (8192, 8192), (5760, 5760), (16384, 16384), (1 << 20, 64), (64, 1 << 20),
                                 # the narrow shapes the bench's next-rows leg times (flat-stream kernels)
                                 (1 << 20, 40), (1 << 20, 88), (1 << 20, 44), (3 ** 13, 40), (3 ** 13, 24)])
def test_gemv_ger_config_sizes(b2, ctx, dtype, m, n):
    seed = 31
    a = synth.matrix_torch(seed, 1, m, n, n, TD[dtype], "cuda")
    hx_n, hx_m = synth.vector_np(seed, 2, n, dtype), synth.vector_np(seed, 3, m, dtype)
    hy_m, hy_n = synth.vector_np(seed, 4, m, dtype), synth.vector_np(seed, 5, n, dtype)
    for inc, beta in ((1, 0.5), (2, 0.0)):
        # gemv N: sampled rows
        y = dvec(seed, 4, m, dtype, inc)
        b2.gemv(ctx, orc.ROW_MAJOR, orc.NO_TRANS, m, n, 1.25, a, n, dvec(seed, 2, n, dtype, inc), inc, beta, y, inc)
        rows = sample(m, 1)
        got = y[torch.from_numpy(rows * inc).cuda()].cpu().numpy()
        for r, g in zip(rows, got):
            row = synth.matrix_entries_np(seed, 1, r, np.arange(n), n, dtype)
            out = hy_m[r:r + 1].copy()
            absterms = orc.gemv(orc.ROW_MAJOR, orc.NO_TRANS, 1, n, dtype(1.25), row, n, hx_n, 1, dtype(beta), out, 1)
            assert_close(g, out[0], absterms[0], dtype, f"gemv-N row {r} inc {inc}")
        # gemv T: sampled columns
        y = dvec(seed, 5, n, dtype, inc)
        b2.gemv(ctx, orc.ROW_MAJOR, orc.TRANS, m, n, 1.25, a, n, dvec(seed, 3, m, dtype, inc), inc, beta, y, inc)
        cols = sample(n, 2)
        got = y[torch.from_numpy(cols * inc).cuda()].cpu().numpy()
        for c, g in zip(cols, got):
            col = synth.matrix_entries_np(seed, 1, np.arange(m), c, n, dtype)
            out = hy_n[c:c + 1].copy()
            absterms = orc.gemv(orc.ROW_MAJOR, orc.TRANS, m, 1, dtype(1.25), col, 1, hx_m, 1, dtype(beta), out, 1)
            assert_close(g, out[0], absterms[0], dtype, f"gemv-T col {c} inc {inc}")
    # ger: sampled row segments
    a2 = a.clone()
    b2.ger(ctx, orc.ROW_MAJOR, m, n, 1.25, dvec(seed, 3, m, dtype), 1, dvec(seed, 2, n, dtype), 1, a2, n)
    for r in sample(m, 3)[:12]:
        c0 = int(min(max(0, (r * 7919) % n - 32), max(0, n - 64)))
        w = min(64, n - c0)
        seg = synth.matrix_entries_np(seed, 1, r, np.arange(c0, c0 + w), n, dtype)
        absterms = orc.ger(orc.ROW_MAJOR, 1, w, dtype(1.25), hx_m[r:r + 1], 1, hx_n[c0:c0 + w], 1, seg, w)
        assert_close(a2[r, c0:c0 + w].cpu().numpy(), seg, absterms[0], dtype, f"ger row {r}")
    del a, a2
    torch.cuda.empty_cache()


def op_row(seed, stream, n, dtype, uplo, trans, diag, i, symmetric=False):
    """Row i of op(A) (or of the symmetric matrix) as a dense host vector, from the generator."""
    j = np.arange(n)
    upper = uplo == orc.UPPER
    if symmetric:
        r = np.where((j >= i) == upper, i, j)  # stored position (r, c) of element (i, j)
        c = np.where((j >= i) == upper, j, i)
        r, c = np.where(j == i, i, r), np.where(j == i, i, c)
        return synth.matrix_entries_np(seed, stream, r, c, n, dtype, tri_n=n)
    # op(A)_ij = A_ij (N) or A_ji (T); zero outside the stored triangle
    r, c = (np.full(n, i), j) if trans == orc.NO_TRANS else (j, np.full(n, i))
    inside = (r <= c) if upper else (r >= c)
    row = synth.matrix_entries_np(seed, stream, r, c, n, dtype, tri_n=n)
    row = np.where(inside, row, 0).astype(dtype)
    if diag == orc.UNIT:
        row[i] = 1
    return row


@pytest.mark.parametrize("dtype,n", [(np.float32, 1024), (np.float32, 8192), (np.float32, 11520), (np.float32, 32768),
                                     (np.float64, 8192), (np.float64, 32768)])
def test_triangular_config_sizes(b2, ctx, dtype, n):
    seed, stream = 37, 6
    a = synth.matrix_torch(seed, stream, n, n, n, TD[dtype], "cuda", tri_n=n)
    hx, hy = synth.vector_np(seed, 7, n, dtype), synth.vector_np(seed, 8, n, dtype)
    tol = TOL[np.dtype(dtype)]
    rows = sample(n, n)
    tidx = torch.from_numpy(rows).cuda()
    for uplo in (orc.UPPER, orc.LOWER):
        gots = []
        for kernel in (0, 2):  # the general tile kernel, then the one with the shared-memory ring
            old = b2.get_tuning(b2.KNOB_TRI_TILE)
            b2.set_tuning(b2.KNOB_TRI_TILE, kernel)
            try:
                y = dvec(seed, 8, n, dtype)
                b2.symv(ctx, orc.ROW_MAJOR, uplo, n, 1.25, a, n, dvec(seed, 7, n, dtype), 1, 0.5, y, 1)
                gots.append(y[tidx].cpu().numpy())
            finally:
                b2.set_tuning(b2.KNOB_TRI_TILE, old)
        for k, i in enumerate(rows):
            row = op_row(seed, stream, n, dtype, uplo, orc.NO_TRANS, orc.NON_UNIT, i, symmetric=True)
            out = hy[i:i + 1].copy()
            absterms = orc.gemv(orc.ROW_MAJOR, orc.NO_TRANS, 1, n, dtype(1.25), row, n, hx, 1, dtype(0.5), out, 1)
            for kernel, got in zip(("general", "ring"), gots):
                assert_close(got[k], out[0], absterms[0], dtype, f"symv ({kernel} kernel) uplo {uplo} row {i}")
        for trans in (orc.NO_TRANS, orc.TRANS):
            for diag in (orc.NON_UNIT, orc.UNIT):
                x = dvec(seed, 7, n, dtype)
                b2.trmv(ctx, orc.ROW_MAJOR, uplo, trans, diag, n, a, n, x, 1)
                got = x[tidx].cpu().numpy()
                xs = dvec(seed, 7, n, dtype)
                b2.trsv(ctx, orc.ROW_MAJOR, uplo, trans, diag, n, a, n, xs, 1)
                assert ctx.device_status() == 0
                hxs = xs.cpu().numpy()
                for i, g in zip(rows, got):
                    row = op_row(seed, stream, n, dtype, uplo, trans, diag, i)
                    val, absterms = orc.dot(n, row, 1, hx, 1)
                    assert_close(g, val, absterms, dtype, f"trmv {uplo} {trans} {diag} row {i}")
                    # row-wise residual of the device solution of op(A) x = b
                    ax, aabs = orc.dot(n, row, 1, hxs, 1)
                    resid = abs(float(hx[i]) - float(ax))
                    scale = abs(float(hx[i])) + aabs
                    slack = float(np.finfo(dtype).eps) * abs(float(ax))  # the dot itself is rounded to T
                    assert resid <= tol * scale + slack, f"trsv {uplo} {trans} {diag} row {i}: {resid:.3e} > {tol * scale:.3e}"
    del a
    torch.cuda.empty_cache()


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("m,n", [(1 << 20, 40), (3 ** 13, 40), (3 ** 13, 24), (1 << 20, 88)])
def test_gemv_ger_column_major_narrow(b2, ctx, dtype, m, n):
    """The narrow shapes of the paper's skinny study (Section 6.2.2) in COLUMN-major storage, at the
    sizes the bench's next-rows leg times: the buffer holds n columns of m elements (lda = m), so the
    kernels see the transposed, very wide row-major problem; an odd m (3^13) puts every second
    column off the 16-byte boundary."""
    if dtype == np.float64 and n == 88:
        n = 44
    seed = 43
    buf = synth.matrix_torch(seed, 1, n, m, m, TD[dtype], "cuda")  # buf[j, i] = A(i, j)
    hx_n, hx_m = synth.vector_np(seed, 2, n, dtype), synth.vector_np(seed, 3, m, dtype)
    hy_m, hy_n = synth.vector_np(seed, 4, m, dtype), synth.vector_np(seed, 5, n, dtype)
    y = dvec(seed, 4, m, dtype)
    b2.gemv(ctx, orc.COL_MAJOR, orc.NO_TRANS, m, n, 1.25, buf, m, dvec(seed, 2, n, dtype), 1, 0.5, y, 1)
    rows = sample(m, 5)
    got = y[torch.from_numpy(rows).cuda()].cpu().numpy()
    for r, g in zip(rows, got):
        row = synth.matrix_entries_np(seed, 1, np.arange(n), r, m, dtype)  # A(r, :) = buf[:, r]
        out = hy_m[r:r + 1].copy()
        absterms = orc.gemv(orc.ROW_MAJOR, orc.NO_TRANS, 1, n, dtype(1.25), row, n, hx_n, 1, dtype(0.5), out, 1)
        assert_close(g, out[0], absterms[0], dtype, f"column-major gemv-N row {r}")
    y = dvec(seed, 5, n, dtype)
    b2.gemv(ctx, orc.COL_MAJOR, orc.TRANS, m, n, 1.25, buf, m, dvec(seed, 3, m, dtype), 1, 0.5, y, 1)
    got = y.cpu().numpy()
    for c in range(n):  # every output: a dot product over one stored row of the buffer
        col = synth.matrix_entries_np(seed, 1, c, np.arange(m), m, dtype)
        out = hy_n[c:c + 1].copy()
        absterms = orc.gemv(orc.ROW_MAJOR, orc.TRANS, m, 1, dtype(1.25), col, 1, hx_m, 1, dtype(0.5), out, 1)
        assert_close(got[c], out[0], absterms[0], dtype, f"column-major gemv-T column {c}")
    b2.ger(ctx, orc.COL_MAJOR, m, n, 1.25, dvec(seed, 3, m, dtype), 1, dvec(seed, 2, n, dtype), 1, buf, m)
    for r in sample(m, 6)[:16]:
        seg = synth.matrix_entries_np(seed, 1, np.arange(n), r, m, dtype)  # A(r, 0 .. n-1)
        absterms = orc.ger(orc.ROW_MAJOR, 1, n, dtype(1.25), hx_m[r:r + 1], 1, hx_n, 1, seg, n)
        assert_close(buf[:, r].cpu().numpy(), seg, absterms[0], dtype, f"column-major ger row {r}")
    del buf
    torch.cuda.empty_cache()
