"""GPU parity of the level-1 family against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import blas_oracle as orc
from paper_2411_07211_b200 import synth
from tests.gpu_util import Guarded, assert_close, assert_same_gaps, pick, place

pytestmark = pytest.mark.gpu

DTYPES = [np.float32, np.float64]
SIZES = [0, 1, 2, 3, 5, 7, 8, 31, 32, 33, 127, 128, 129, 1023, 1025, 4099, 70001, 300007]
INCS = [(1, 1), (2, 2), (1, 2), (-1, 1), (3, -2)]


@pytest.fixture(scope="module")
def b2():
    from paper_2411_07211_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(b2):
    c = b2.Context()
    c.reset()
    return c


def _vecs(n, dtype, seed):
    return synth.vector_np(seed, 1, n, dtype), synth.vector_np(seed, 2, n, dtype)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("incx,incy", INCS)
@pytest.mark.parametrize("offset", [0, 1])
def test_map_routines(b2, ctx, dtype, n, incx, incy, offset):
    x, y = _vecs(n, dtype, 100 + n)
    hx, hy = place(x, incx), place(y, incy)

    def fresh():
        return Guarded(hx, offset), Guarded(hy, offset)

    # axpy
    gx, gy = fresh()
    b2.axpy(ctx, n, 1.5, gx.t, incx, gy.t, incy)
    ox, oy = hx.copy(), hy.copy()
    absterms = orc.axpy(n, dtype(1.5), ox, incx, oy, incy)
    ry = gy.host()
    assert_close(pick(ry, n, incy), pick(oy, n, incy), absterms, dtype, "axpy")
    assert_same_gaps(ry, hy, n, incy)
    assert np.array_equal(gx.host(), hx, equal_nan=True)
    gx.check_guards(), gy.check_guards()
    # axpy alpha = 0: y untouched bit for bit
    gx, gy = fresh()
    b2.axpy(ctx, n, 0.0, gx.t, incx, gy.t, incy)
    assert np.array_equal(gy.host(), hy, equal_nan=True)
    # scal: bit-exact
    gx, _ = fresh()
    b2.scal(ctx, n, -0.75, gx.t, incx)
    ox = hx.copy()
    orc.scal(n, dtype(-0.75), ox, incx)
    assert np.array_equal(gx.host(), ox, equal_nan=True)
    gx.check_guards()
    # copy: bit-exact
    gx, gy = fresh()
    b2.copy(ctx, n, gx.t, incx, gy.t, incy)
    ox, oy = hx.copy(), hy.copy()
    orc.copy(n, ox, incx, oy, incy)
    assert np.array_equal(gy.host(), oy, equal_nan=True) and np.array_equal(gx.host(), hx, equal_nan=True)
    gx.check_guards(), gy.check_guards()
    # swap: bit-exact
    gx, gy = fresh()
    b2.swap(ctx, n, gx.t, incx, gy.t, incy)
    ox, oy = hx.copy(), hy.copy()
    orc.swap(n, ox, incx, oy, incy)
    assert np.array_equal(gx.host(), ox, equal_nan=True) and np.array_equal(gy.host(), oy, equal_nan=True)
    gx.check_guards(), gy.check_guards()
    # rot
    gx, gy = fresh()
    b2.rot(ctx, n, gx.t, incx, gy.t, incy, 0.6, 0.8)
    ox, oy = hx.copy(), hy.copy()
    ax, ay = orc.rot(n, ox, incx, oy, incy, dtype(0.6), dtype(0.8))
    rx, ry = gx.host(), gy.host()
    assert_close(pick(rx, n, incx), pick(ox, n, incx), ax, dtype, "rot x")
    assert_close(pick(ry, n, incy), pick(oy, n, incy), ay, dtype, "rot y")
    assert_same_gaps(rx, hx, n, incx), assert_same_gaps(ry, hy, n, incy)
    gx.check_guards(), gy.check_guards()


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", SIZES + [1 << 20, (1 << 22) + 5])
@pytest.mark.parametrize("incx,incy", INCS)
@pytest.mark.parametrize("offset", [0, 1])
def test_reductions(b2, ctx, dtype, n, incx, incy, offset):
    if n > 400000 and (abs(incx) > 2 or abs(incy) > 2):
        pytest.skip("large strided spans are covered at inc=2")
    x, y = _vecs(n, dtype, 200 + n % 1000)
    hx, hy = place(x, incx), place(y, incy)
    gx, gy = Guarded(hx, offset), Guarded(hy, offset)
    tdt = torch.float32 if dtype == np.float32 else torch.float64
    res = torch.full((4,), float("nan"), dtype=tdt, device="cuda")
    ires = torch.full((1,), -7, dtype=torch.int64, device="cuda")
    b2.dot(ctx, n, gx.t, incx, gy.t, incy, res[0:1])
    b2.asum(ctx, n, gx.t, incx, res[1:2])
    b2.nrm2(ctx, n, gx.t, incx, res[2:3])
    b2.iamax(ctx, n, gx.t, incx, ires)
    got = res.cpu().numpy()
    d, dabs = orc.dot(n, hx, incx, hy, incy)
    assert_close(got[0], d, dabs, dtype, "dot")
    a, aabs = orc.asum(n, hx, incx)
    assert_close(got[1], a, aabs, dtype, "asum")
    nr, _ = orc.nrm2(n, hx, incx)
    assert_close(got[2], nr, abs(float(nr)), dtype, "nrm2")
    assert int(ires.item()) == orc.iamax(n, hx, incx)
    assert np.isnan(got[3])  # neighbour of the result words untouched
    assert np.array_equal(gx.host(), hx, equal_nan=True) and np.array_equal(gy.host(), hy, equal_nan=True)
    # determinism: a second and third call give the same bits
    for _ in range(2):
        res2 = torch.zeros(3, dtype=tdt, device="cuda")
        b2.dot(ctx, n, gx.t, incx, gy.t, incy, res2[0:1])
        b2.asum(ctx, n, gx.t, incx, res2[1:2])
        b2.nrm2(ctx, n, gx.t, incx, res2[2:3])
        assert np.array_equal(res2.cpu().numpy().view(np.uint8), got[:3].view(np.uint8))


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", [1, 33, 1025, 70001, (1 << 21) + 3])
@pytest.mark.parametrize("inc", [1, 2, -1])
def test_iamax_planted_ties(b2, ctx, dtype, n, inc):
    base = synth.vector_np(5, 9, n, dtype)
    rng = np.random.default_rng(n)
    plants = [
        [0], [n - 1], [n // 2, n // 2 + 1], [3 % n, (4 * 256 * 8 + 3) % n, n - 1],
        sorted(set(rng.integers(0, n, size=4).tolist())),
        [(n // 3 // 4) * 4 + 3 if n > 8 else 0, min(n - 1, (n // 3 // 4) * 4 + 4)],  # straddle a 16-byte pack
    ]
    ires = torch.zeros(1, dtype=torch.int64, device="cuda")
    for planted in plants:
        planted = sorted({min(max(q, 0), n - 1) for q in planted})
        v = base.copy()
        for k, p in enumerate(planted):
            v[p] = 1.5 if k % 2 == 0 else -1.5
        g = Guarded(place(v, inc))
        b2.iamax(ctx, n, g.t, inc, ires)
        assert int(ires.item()) == min(planted) == orc.iamax(n, place(v, inc), inc)
    g = Guarded(place(base, inc))
    b2.iamax(ctx, n, g.t, inc, ires)
    assert int(ires.item()) == orc.iamax(n, place(base, inc), inc)
    z = Guarded(np.zeros(n, dtype=dtype))
    b2.iamax(ctx, n, z.t, 1, ires)
    assert int(ires.item()) == 0


@pytest.mark.parametrize("dtype", DTYPES)
def test_small_integer_reductions_are_bit_exact(b2, ctx, dtype):
    """Integer-valued inputs make every partial sum exact, so any summation order must give the
    oracle's bits: catches indexing mistakes that a tolerance would hide."""
    rng = np.random.default_rng(1)
    tdt = torch.float32 if dtype == np.float32 else torch.float64
    for n in [1000, 65537, 1 << 20]:
        x = rng.integers(-2, 3, size=n).astype(dtype)
        y = rng.integers(-2, 3, size=n).astype(dtype)
        gx, gy = Guarded(x), Guarded(y)
        res = torch.zeros(2, dtype=tdt, device="cuda")
        b2.dot(ctx, n, gx.t, 1, gy.t, 1, res[0:1])
        b2.asum(ctx, n, gx.t, 1, res[1:2])
        got = res.cpu().numpy()
        assert got[0] == orc.dot(n, x, 1, y, 1)[0] == float(np.dot(x.astype(np.int64), y.astype(np.int64)))
        assert got[1] == orc.asum(n, x, 1)[0] == float(np.abs(x).sum())


def test_sdot_config1_matches_golden(b2, ctx):
    """n = 1,048,576 f32, seed 0: the device generator feeds the kernel, the stored oracle value
    (tests/golden) is the reference."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "sdot_n1048576_seed0.txt")
    fields = dict(line.split("=") for line in open(path).read().split() if "=" in line)
    n = int(fields["n"])
    x = synth.vector_torch(0, 0, n, torch.float32, "cuda")
    y = synth.vector_torch(0, 1, n, torch.float32, "cuda")
    assert np.array_equal(x[:1000].cpu().numpy(), synth.vector_np(0, 0, 1000, np.float32))
    res = torch.zeros(1, dtype=torch.float32, device="cuda")
    b2.dot(ctx, n, x, 1, y, 1, res)
    want = float.fromhex(fields["result_hex"])
    absterms = float(fields["absterms"].replace("np.float64(", "").rstrip(")"))
    assert abs(float(res.item()) - want) <= 2e-6 * absterms


@pytest.mark.parametrize("dtype,tdt", [(np.float32, torch.float32), (np.float64, torch.float64)])
@pytest.mark.parametrize("inc", [1, 2])
def test_bench_sizes(b2, ctx, dtype, tdt, inc):
    """The sizes the bench times (256 MiB spans): reductions against the full oracle, map
    routines on sampled elements computed one by one."""
    n2 = (1 << 25 if dtype == np.float32 else 1 << 24) // inc  # two-vector routines
    n1 = 2 * n2                                                 # one-vector routines
    hx = synth.vector_np(11, 0, n1, dtype)
    hy = synth.vector_np(11, 1, n2, dtype)
    dx = torch.full((span_t(n1, inc),), float("nan"), dtype=tdt, device="cuda")
    dy = torch.full((span_t(n2, inc),), float("nan"), dtype=tdt, device="cuda")
    dx[::inc] = synth.vector_torch(11, 0, n1, tdt, "cuda")
    dy[::inc] = synth.vector_torch(11, 1, n2, tdt, "cuda")
    res = torch.zeros(3, dtype=tdt, device="cuda")
    ires = torch.zeros(1, dtype=torch.int64, device="cuda")
    b2.dot(ctx, n2, dx, inc, dy, inc, res[0:1])
    b2.asum(ctx, n1, dx, inc, res[1:2])
    b2.nrm2(ctx, n1, dx, inc, res[2:3])
    b2.iamax(ctx, n1, dx, inc, ires)
    got = res.cpu().numpy()
    d, dabs = orc.dot(n2, hx[:n2], 1, hy, 1)
    assert_close(got[0], d, dabs, dtype, "dot")
    a, aabs = orc.asum(n1, hx, 1)
    assert_close(got[1], a, aabs, dtype, "asum")
    nr, _ = orc.nrm2(n1, hx, 1)
    assert_close(got[2], nr, abs(float(nr)), dtype, "nrm2")
    assert int(ires.item()) == orc.iamax(n1, hx, 1)
    # planted ties at the far ends and across a block boundary
    for p in ([n1 - 1, 5], [n1 // 2, n1 // 2 + 4096 * 5]):
        dx2 = dx.clone()
        for q in p:
            dx2[q * inc] = -1.5
        b2.iamax(ctx, n1, dx2, inc, ires)
        assert int(ires.item()) == min(p)
    # map routines on sampled elements
    rng = np.random.default_rng(3)
    idx = np.unique(np.concatenate([[0, 1, 2, 3, n2 - 1, n2 - 2, n2 // 2], rng.integers(0, n2, size=2000)]))
    sx, sy = hx[idx].copy(), hy[idx].copy()
    tidx = torch.from_numpy(idx * inc).cuda()
    y2 = dy.clone()
    b2.axpy(ctx, n2, 1.5, dx, inc, y2, inc)
    oy = sy.copy()
    absterms = orc.axpy(len(idx), dtype(1.5), sx, 1, oy, 1)
    assert_close(y2[tidx].cpu().numpy(), oy, absterms, dtype, "axpy")
    x2, y2 = dx.clone(), dy.clone()
    b2.rot(ctx, n2, x2, inc, y2, inc, 0.6, 0.8)
    ox, oy = sx.copy(), sy.copy()
    ax, ay = orc.rot(len(idx), ox, 1, oy, 1, dtype(0.6), dtype(0.8))
    assert_close(x2[tidx].cpu().numpy(), ox, ax, dtype, "rot x")
    assert_close(y2[tidx].cpu().numpy(), oy, ay, dtype, "rot y")
    assert torch.equal(x2[n2 * inc:], dx[n2 * inc:]) or inc == 2  # beyond n2 untouched
    x2 = dx.clone()
    b2.scal(ctx, n1, -0.75, x2, inc)
    assert torch.equal(x2[::inc], dx[::inc] * -0.75)  # a lone multiply is exact to compare
    if inc == 2:
        assert bool(torch.isnan(x2[1::2]).all())
    y2 = torch.zeros_like(dy)
    b2.copy(ctx, n2, dx, inc, y2, inc)
    assert torch.equal(y2[::inc], dx[:n2 * inc:inc])
    x2, y2 = dx.clone(), dy.clone()
    b2.swap(ctx, n2, x2, inc, y2, inc)
    assert torch.equal(y2[::inc], dx[:n2 * inc:inc]) and torch.equal(x2[:n2 * inc:inc], dy[::inc])


def span_t(n, inc):
    return 1 + (n - 1) * inc


def test_level1_n_2_28(b2, ctx):
    """The largest level-1 size of the size sweep, n = 2^28 (1 GiB per float vector: offsets and
    chunk counts beyond 2^32 bytes): reductions against the full oracle, map routines on sampled
    elements, a planted maximum in the last chunk."""
    n, dtype, tdt = 1 << 28, np.float32, torch.float32
    hx, hy = synth.vector_np(13, 0, n, dtype), synth.vector_np(13, 1, n, dtype)
    dx, dy = synth.vector_torch(13, 0, n, tdt, "cuda"), synth.vector_torch(13, 1, n, tdt, "cuda")
    res = torch.zeros(3, dtype=tdt, device="cuda")
    ires = torch.zeros(1, dtype=torch.int64, device="cuda")
    b2.dot(ctx, n, dx, 1, dy, 1, res[0:1])
    b2.asum(ctx, n, dx, 1, res[1:2])
    b2.nrm2(ctx, n, dx, 1, res[2:3])
    b2.iamax(ctx, n, dx, 1, ires)
    got = res.cpu().numpy()
    d, dabs = orc.dot(n, hx, 1, hy, 1)
    assert_close(got[0], d, dabs, dtype, "dot")
    a, aabs = orc.asum(n, hx, 1)
    assert_close(got[1], a, aabs, dtype, "asum")
    nr, _ = orc.nrm2(n, hx, 1)
    assert_close(got[2], nr, abs(float(nr)), dtype, "nrm2")
    assert int(ires.item()) == orc.iamax(n, hx, 1)
    dx2 = dx.clone()
    dx2[n - 3] = 1.5
    dx2[n - 1] = -1.5
    b2.iamax(ctx, n, dx2, 1, ires)
    assert int(ires.item()) == n - 3
    del dx2
    rng = np.random.default_rng(4)
    idx = np.unique(np.concatenate([[0, 1, n - 1, n - 2, n // 2, (1 << 27) + 1], rng.integers(0, n, size=4000)]))
    tidx = torch.from_numpy(idx).cuda()
    sx, sy = hx[idx].copy(), hy[idx].copy()
    y2 = dy.clone()
    b2.axpy(ctx, n, 1.5, dx, 1, y2, 1)
    oy = sy.copy()
    absterms = orc.axpy(len(idx), dtype(1.5), sx, 1, oy, 1)
    assert_close(y2[tidx].cpu().numpy(), oy, absterms, dtype, "axpy")
    del y2
    x3, y3 = dx.clone(), dy.clone()
    b2.rot(ctx, n, x3, 1, y3, 1, 0.6, 0.8)
    ox, oy = sx.copy(), sy.copy()
    ax, ay = orc.rot(len(idx), ox, 1, oy, 1, dtype(0.6), dtype(0.8))
    assert_close(x3[tidx].cpu().numpy(), ox, ax, dtype, "rot x")
    assert_close(y3[tidx].cpu().numpy(), oy, ay, dtype, "rot y")
    b2.swap(ctx, n, x3, 1, y3, 1)
    b2.scal(ctx, n, -0.75, y3, 1)
    assert_close(y3[tidx].cpu().numpy(), dtype(-0.75) * ox, ax, dtype, "swap + scal")  # 0.75 x the rot bound + one rounding
    b2.copy(ctx, n, dx, 1, x3, 1)
    assert torch.equal(x3, dx)


def test_prepare_replays_the_recorded_calls(b2, ctx):
    """binding.prepare marshals the calls of a thunk once; every replay must launch exactly those
    calls again (same pointers, same scalars): axpy twice and a dot, checked against the oracle
    after the recording run and after two replays."""
    n = 70001
    x = synth.vector_np(21, 1, n, np.float32)
    y = synth.vector_np(21, 2, n, np.float32)
    gx, gy = Guarded(x), Guarded(y)
    res = torch.zeros(1, dtype=torch.float32, device="cuda")

    def thunk():
        b2.axpy(ctx, n, 0.5, gx.t, 1, gy.t, 1)
        b2.axpy(ctx, n, -0.25, gx.t, 1, gy.t, 1)
        b2.dot(ctx, n, gx.t, 1, gy.t, 1, res)

    run = b2.prepare(thunk)  # runs the thunk once
    oy = y.copy()
    yabs = np.zeros(n)
    launches = b2.launch_count()
    for rounds in range(3):
        if rounds:
            assert run() == 0
        a1 = orc.axpy(n, np.float32(0.5), x, 1, oy, 1)
        a2 = orc.axpy(n, np.float32(-0.25), x, 1, oy, 1)
        yabs = yabs + a1 + a2  # the error bound grows with every update of y
        assert_close(gy.host(), oy, yabs, np.float32, f"axpy after {rounds} replays")
        want, absterms = orc.dot(n, x, 1, oy, 1)
        assert_close(res.cpu().numpy()[0], want, absterms, np.float32, f"dot after {rounds} replays")
    assert b2.launch_count() - launches == 6  # two replays of three calls
    gx.check_guards(), gy.check_guards()
