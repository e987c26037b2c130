"""Seeded synthetic inputs, shared by the tests, the bench and the CPU oracle's callers.

This module holds none of the BLAS arithmetic.  It is a counter-based generator: element
``i`` of stream ``(seed, stream)`` is a pure function of ``(seed, stream, i)``, so any slice,
row, column or scattered sample of a huge buffer can be produced on the host without
materialising the buffer, while the identical bits are produced on the device for the
kernels.  Two back-ends compute the same integers:

* numpy (uint64 arithmetic) for host arrays, and
* torch (int64 arithmetic, masked to 32 bits after every multiply) for device tensors.

Hash: the 32-bit integer finaliser "lowbias32" (xorshift 16, multiply 0x7feb352d, xorshift 15,
multiply 0x846ca68b, xorshift 16), applied to ``index ^ key``.  float32 values use the top
24 bits, ``k * 2**-23 - 1``; float64 values use 52 bits from two hashes, ``k * 2**-51 - 1``.
Both are exactly representable, uniform on [-1, 1).
"""
from __future__ import annotations

import numpy as np

_M32 = 0xFFFFFFFF
_C1 = 0x7FEB352D
_C2 = 0x846CA68B
_GOLD = 0x9E3779B9


def _mix32_int(h: int) -> int:
    h &= _M32
    h ^= h >> 16
    h = (h * _C1) & _M32
    h ^= h >> 15
    h = (h * _C2) & _M32
    h ^= h >> 16
    return h


def stream_keys(seed: int, stream: int) -> tuple[int, int]:
    """Two 32-bit keys for (seed, stream); plain Python integers."""
    k1 = _mix32_int((seed * _GOLD + 0x85EBCA6B) ^ _mix32_int(stream + 0x1234567))
    k2 = _mix32_int(k1 + _GOLD)
    return k1, k2


def _mix32(h, xp_and):
    # h holds values < 2**32 in a 64-bit integer container (uint64 numpy / int64 torch).
    h = h ^ (h >> 16)
    h = xp_and(h * _C1)
    h = h ^ (h >> 15)
    h = xp_and(h * _C2)
    h = h ^ (h >> 16)
    return h


def _np_and(v):
    return v & np.uint64(_M32)


def uniform_np(seed: int, stream: int, idx, dtype) -> np.ndarray:
    """Values of stream (seed, stream) at integer indices ``idx`` (any shape, < 2**32)."""
    dtype = np.dtype(dtype)
    k1, k2 = stream_keys(seed, stream)
    i = np.asarray(idx).astype(np.uint64)
    with np.errstate(over="ignore"):
        h1 = _mix32(_np_and(i ^ np.uint64(k1)), _np_and)
        if dtype == np.float32:
            k = (h1 >> np.uint64(8)).astype(np.float64)
            return (k * 2.0 ** -23 - 1.0).astype(np.float32)
        if dtype == np.float64:
            h2 = _mix32(_np_and(i ^ np.uint64(k2)), _np_and)
            k = ((h1 << np.uint64(20)) | (h2 >> np.uint64(12))).astype(np.float64)
            return k * 2.0 ** -51 - 1.0
    raise TypeError(dtype)


def vector_np(seed: int, stream: int, n: int, dtype, start: int = 0) -> np.ndarray:
    return uniform_np(seed, stream, np.arange(start, start + n, dtype=np.uint64), dtype)


def uniform_torch(seed: int, stream: int, idx, dtype):
    """Same values as :func:`uniform_np`, computed with torch ops on ``idx``'s device.

    ``idx`` is an int64 tensor of indices (< 2**32)."""
    import torch

    k1, k2 = stream_keys(seed, stream)

    def t_and(v):
        return v & _M32

    i = idx.to(torch.int64)
    h1 = _mix32(t_and(i ^ k1), t_and)
    if dtype == torch.float32:
        k = (h1 >> 8).to(torch.float64)
        return (k * 2.0 ** -23 - 1.0).to(torch.float32)
    if dtype == torch.float64:
        h2 = _mix32(t_and(i ^ k2), t_and)
        k = ((h1 << 20) | (h2 >> 12)).to(torch.float64)
        return k * 2.0 ** -51 - 1.0
    raise TypeError(dtype)


def vector_torch(seed: int, stream: int, n: int, dtype, device, start: int = 0, chunk: int = 1 << 24):
    """Device vector of n values, generated in bounded chunks."""
    import torch

    out = torch.empty(n, dtype=dtype, device=device)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        idx = torch.arange(start + s, start + e, dtype=torch.int64, device=device)
        out[s:e] = uniform_torch(seed, stream, idx, dtype)
    return out


# ---------------------------------------------------------------- matrices
# A matrix buffer of `rows` x `lda` elements is the stream indexed by its flat offset
# r*lda + c.  "Triangular-conditioned" matrices rescale that stream: off-diagonal entries are
# u/n in [-1/n, 1/n), diagonal entries are 1 + (u+1)/2 in [1, 2), so that triangular solves
# stay well conditioned.


def _tri_condition(u64, r, c, n, xp_where):
    return xp_where(r == c, 1.0 + (u64 + 1.0) * 0.5, u64 / float(n))


def matrix_entries_np(seed, stream, r, c, lda, dtype, tri_n: int | None = None) -> np.ndarray:
    """Entries at (r, c) (broadcastable integer arrays) of the matrix stream."""
    r = np.asarray(r, dtype=np.int64)
    c = np.asarray(c, dtype=np.int64)
    u = uniform_np(seed, stream, r * lda + c, dtype)
    if tri_n is None:
        return u
    r, c = np.broadcast_arrays(r, c)
    return _tri_condition(u.astype(np.float64), r, c, tri_n, np.where).astype(dtype)


def matrix_np(seed, stream, rows, cols, lda, dtype, tri_n: int | None = None) -> np.ndarray:
    """Host matrix buffer, shape (rows, lda); only the first `cols` columns are meaningful
    but all lda columns are generated so the buffer equals the device one bit for bit."""
    del cols
    r = np.arange(rows, dtype=np.int64)[:, None]
    c = np.arange(lda, dtype=np.int64)[None, :]
    return np.ascontiguousarray(matrix_entries_np(seed, stream, r, c, lda, dtype, tri_n))


def matrix_torch(seed, stream, rows, cols, lda, dtype, device, tri_n: int | None = None,
                 chunk_rows: int | None = None):
    """Device matrix buffer, shape (rows, lda), bit-identical to :func:`matrix_np`."""
    import torch

    del cols
    out = torch.empty((rows, lda), dtype=dtype, device=device)
    if chunk_rows is None:
        chunk_rows = max(1, (1 << 24) // max(1, lda))
    c = torch.arange(lda, dtype=torch.int64, device=device)[None, :]
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        r = torch.arange(r0, r1, dtype=torch.int64, device=device)[:, None]
        u = uniform_torch(seed, stream, r * lda + c, dtype)
        if tri_n is not None:
            u = _tri_condition(u.to(torch.float64), r, c, tri_n, torch.where).to(dtype)
        out[r0:r1] = u
    return out
