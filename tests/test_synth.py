"""The seeded generator: numpy and torch back-ends give identical bits, values are uniform on
[-1, 1), and any slice / scattered sample equals the corresponding part of the whole."""
import numpy as np
import pytest
import torch

from paper_2411_07211_b200 import synth


@pytest.mark.parametrize("dtype,tdtype", [(np.float32, torch.float32), (np.float64, torch.float64)])
def test_numpy_and_torch_agree(dtype, tdtype):
    n = 100_003
    a = synth.vector_np(7, 3, n, dtype)
    b = synth.vector_torch(7, 3, n, tdtype, "cpu", chunk=30_000).numpy()
    assert a.dtype == dtype and np.array_equal(a, b)
    assert a.min() >= -1 and a.max() < 1
    assert abs(a.mean()) < 0.02 and abs(a.std() - 1 / np.sqrt(3)) < 0.01
    # counter-based: a slice is the same as generating from `start`
    assert np.array_equal(a[500:700], synth.vector_np(7, 3, 200, dtype, start=500))
    # different streams / seeds differ
    assert not np.array_equal(a, synth.vector_np(7, 4, n, dtype))
    assert not np.array_equal(a, synth.vector_np(8, 3, n, dtype))


@pytest.mark.parametrize("dtype,tdtype", [(np.float32, torch.float32), (np.float64, torch.float64)])
def test_matrix_backends_and_samples(dtype, tdtype):
    rows, cols, lda = 37, 29, 32
    for tri_n in (None, cols):
        a = synth.matrix_np(1, 2, rows, cols, lda, dtype, tri_n=tri_n)
        b = synth.matrix_torch(1, 2, rows, cols, lda, tdtype, "cpu", tri_n=tri_n, chunk_rows=5).numpy()
        assert np.array_equal(a, b)
        r = np.array([0, 5, 36, 12])
        c = np.array([3, 5, 28, 12])
        assert np.array_equal(a[r, c], synth.matrix_entries_np(1, 2, r, c, lda, dtype, tri_n=tri_n))
        # a whole row / a whole column sampled without the matrix
        assert np.array_equal(a[9, :cols], synth.matrix_entries_np(1, 2, 9, np.arange(cols), lda, dtype, tri_n=tri_n))
        assert np.array_equal(a[:, 4], synth.matrix_entries_np(1, 2, np.arange(rows), 4, lda, dtype, tri_n=tri_n))
    t = synth.matrix_np(1, 2, 29, 29, 29, dtype, tri_n=29)
    d = np.diag(t)
    off = t[~np.eye(29, dtype=bool)]
    assert d.min() >= 1 and d.max() < 2 and np.abs(off).max() <= 1 / 29
