"""b2_sdot_noalloc: the dot product for callers that cannot allocate device memory.

Some users of the library run where no device memory can be had at call time: inside a host
application whose own allocator has taken the whole GPU heap, or in a loop that must never
block on cudaMalloc.  For them the library keeps the reduction's scratch in a fixed array of
its own.  This test calls that entry point through the C ABI twice in a row (the second call
finds the first call's leftovers in the shared array) and compares each result with the CPU
oracle's dot product and with the ordinary b2_sdot on the same inputs, under the tolerance of
the other reduction tests (2e-6 x the oracle's sum of |x_i y_i|).
Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import blas_oracle as orc
from paper_2411_07211_b200 import synth

pytestmark = pytest.mark.gpu


def test_sdot_noalloc_matches_sdot_twice_in_a_row():
    from paper_2411_07211_b200 import binding as b2

    ctx = b2.Context()
    ctx.reset()
    cases = [((1 << 22) + 3, 1, 1, 0), (70001, 2, -3, 0), (1 << 20, 1, 1, 1), (5, 1, 1, 0)]
    for call, (n, incx, incy, offset) in enumerate(cases):
        lx, ly = (n - 1) * abs(incx) + 1, (n - 1) * abs(incy) + 1
        x = synth.vector_torch(21, 2 * call, lx + offset, torch.float32, "cuda")[offset:]
        y = synth.vector_torch(21, 2 * call + 1, ly + offset, torch.float32, "cuda")[offset:]
        want = torch.zeros(1, dtype=torch.float32, device="cuda")
        got = torch.full((2,), float("nan"), dtype=torch.float32, device="cuda")
        b2.dot(ctx, n, x, incx, y, incy, want)
        b2.sdot_noalloc(n, x, incx, y, incy, got[0:1])
        ref, absterms = orc.dot(n, np.ascontiguousarray(x.cpu().numpy()), incx,
                                np.ascontiguousarray(y.cpu().numpy()), incy)
        g = got.cpu().numpy()
        assert abs(float(g[0]) - float(ref)) <= 2e-6 * absterms, (call, g[0], ref)
        assert abs(float(g[0]) - float(want.item())) <= 2e-6 * absterms, (call, g[0], want.item())
        assert np.isnan(g[1])  # the word after the result is not touched


def test_sdot_noalloc_limits_and_empty():
    from paper_2411_07211_b200 import binding as b2

    x = torch.ones(8, dtype=torch.float32, device="cuda")
    res = torch.full((1,), 7.0, dtype=torch.float32, device="cuda")
    assert b2.sdot_noalloc((1 << 30) + 1, x, 1, x, 1, res, check=False) == b2.STATUS_TOO_LARGE
    assert b2.sdot_noalloc(8, x, 0, x, 1, res, check=False) == -3
    assert float(res.item()) == 7.0  # rejected calls launch nothing
    b2.sdot_noalloc(0, x, 1, x, 1, res)
    assert float(res.item()) == 0.0
    b2.sdot_noalloc(8, x, 1, x, 1, res)
    assert float(res.item()) == 8.0
