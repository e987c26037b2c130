"""Helpers of the GPU parity tests: guarded device buffers, strided placement, tolerances."""
import numpy as np
import torch

from oracle import blas_oracle as orc

TOL = {np.dtype(np.float32): 2e-6, np.dtype(np.float64): 4e-15}
GUARD = 8  # NaN elements before and after every buffer


def span(n, inc):
    return 1 + (n - 1) * abs(inc) if n > 0 else 1


def place(vals, inc):
    """Logical vector -> host buffer with increment inc; gaps are NaN."""
    vals = np.asarray(vals)
    n = len(vals)
    buf = np.full(span(n, inc), np.nan, dtype=vals.dtype)
    if n:
        idx = np.arange(n) * inc if inc > 0 else (np.arange(n) - (n - 1)) * inc
        buf[idx] = vals
    return buf


def pick(buf, n, inc):
    idx = np.arange(n) * inc if inc > 0 else (np.arange(n) - (n - 1)) * inc
    return buf[idx] if n else buf[:0]


class Guarded:
    """Device copy of a host buffer with NaN guard bands and an optional element offset that
    breaks 16-byte alignment; `check_guards` verifies nothing outside the buffer changed."""

    def __init__(self, host, offset=0):
        self.n = host.size
        self.offset = offset
        full = np.full(self.n + 2 * GUARD + offset, np.nan, dtype=host.dtype)
        full[GUARD + offset:GUARD + offset + self.n] = host.ravel()
        self.full_host = full
        self.full = torch.from_numpy(full).cuda()
        self.t = self.full[GUARD + offset:GUARD + offset + self.n]

    def host(self):
        return self.t.cpu().numpy()

    def check_guards(self):
        after = self.full.cpu().numpy()
        lo = GUARD + self.offset
        assert np.array_equal(after[:lo], self.full_host[:lo], equal_nan=True), "front guard modified"
        assert np.array_equal(after[lo + self.n:], self.full_host[lo + self.n:], equal_nan=True), "back guard modified"


def assert_close(got, want, absterms, dtype, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    bound = TOL[np.dtype(dtype)] * np.asarray(absterms, dtype=np.float64)
    err = np.abs(got - want)
    bad = ~(err <= bound)
    if np.any(bad):
        k = int(np.argmax(np.where(bad, err - bound, -np.inf)))
        raise AssertionError(f"{what}: {bad.sum()} outputs out of bound; worst at {k}: got {got.flat[k]!r} "
                             f"want {want.flat[k]!r} err {err.flat[k]:.3e} bound {bound.flat[k]:.3e}")


def assert_same_gaps(after, before, n=None, inc=None):
    """Positions that are not logical elements (stride gaps, pad columns) must still be NaN.
    With (n, inc) the gap positions come from the vector geometry; otherwise from `before`."""
    if n is not None:
        mask = np.ones(after.shape, dtype=bool)
        if n:
            idx = np.arange(n) * inc if inc > 0 else (np.arange(n) - (n - 1)) * inc
            mask[idx] = False
        else:
            mask[:] = False
    else:
        mask = np.isnan(before)
    assert np.all(np.isnan(after[mask])), "gap elements modified"
