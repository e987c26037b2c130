"""The parity suite at small sizes once more, under the bounds-checking build of the library.

That build (libb2blas_dbg.so, -DB2_DEBUG_BOUNDS) tests every address a kernel touches against the
extents of the call's arguments; an access outside them is skipped and counted -- nothing traps.
It stands in for a memory checker.  The suite runs in a child process with B2BLAS_LIB pointing at
the build; the child's session ends by reading the checker's report and fails on any violation.
A second child checks the checker itself through its test hook, which shrinks every extent so
that accesses which really are in bounds get reported (nothing out of bounds is ever touched).
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _env():
    from paper_2411_07211_b200 import build
    path = build.DEBUG_LIB_PATH
    if not os.path.exists(path):
        build.build(debug_bounds=True)
    env = dict(os.environ)
    env["B2BLAS_LIB"] = path
    return env


def test_small_size_suite_is_clean_under_the_bounds_checker():
    env = _env()
    env["B2_EXPECT_CLEAN_BOUNDS"] = "1"
    files = ["tests/test_level1_gpu.py", "tests/test_level1_next_gpu.py", "tests/test_level2_gpu.py",
             "tests/test_syr_gpu.py"]
    skip = "not bench_sizes and not 2_28 and not timeout and not golden and not workspace_query"
    res = subprocess.run([sys.executable, "-m", "pytest", *files, "-m", "gpu", "-q", "-x", "-k", skip,
                          "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = "\n".join(res.stdout.splitlines()[-15:])
    assert res.returncode == 0 and "bounds check: clean" in res.stdout, tail + res.stderr[-2000:]


def test_the_checker_reports_what_it_should():
    code = r"""
import torch
from paper_2411_07211_b200 import binding as b2
assert b2.debug_bounds_report() is not None, "not the bounds-checking build"
ctx = b2.Context(); ctx.reset()
n = 1000
x = torch.ones(n, device="cuda"); y = torch.ones(n, device="cuda")
b2.axpy(ctx, n, 2.0, x, 1, y, 1)
assert b2.debug_bounds_report()[0] == 0 and float(y.sum()) == 3.0 * n
b2.debug_bounds_shrink(8)          # the last two floats of every extent now count as outside
b2.axpy(ctx, n, 2.0, x, 1, y, 1)
cnt, addr, size = b2.debug_bounds_report()
assert cnt > 0 and (x.data_ptr() + 4 * n - 16 <= addr < x.data_ptr() + 4 * n or y.data_ptr() + 4 * n - 16 <= addr < y.data_ptr() + 4 * n), (cnt, hex(addr))
assert float(y[: n - 4].sum()) == 5.0 * (n - 4) and float(y[n - 2:].sum()) == 6.0   # the skipped elements kept their values
b2.debug_bounds_shrink(0)
a = torch.ones(300 * 300, device="cuda"); v = torch.ones(300, device="cuda"); w = torch.zeros(300, device="cuda")
b2.gemv(ctx, b2.ROW_MAJOR, b2.TRANS, 300, 300, 1.0, a, 300, v, 1, 0.0, w, 1)
b2.trsv(ctx, b2.ROW_MAJOR, b2.LOWER, b2.NO_TRANS, b2.UNIT, 300, torch.eye(300, device="cuda").reshape(-1).contiguous(), 300, v, 1)
assert b2.debug_bounds_report()[0] == 0 and float(w.sum()) == 300.0 * 300
print("checker ok")
"""
    res = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=_env(), capture_output=True, text=True, timeout=600)
    assert res.returncode == 0 and "checker ok" in res.stdout, res.stdout[-1500:] + res.stderr[-1500:]
