"""Pins of the logistic-regression gradient oracle: numerical differentiation of the
loss it is the gradient of, and agreement of the sparse form with the dense one."""
import numpy as np

from oracle import logreg_oracle as L


def _loss(X, y, rows, x):
    s = X[rows].astype(np.float64) @ x
    return float(np.mean(np.logaddexp(0.0, -y[rows].astype(np.float64) * s)))


def test_dense_gradient_is_the_derivative_of_the_minibatch_loss():
    rng = np.random.default_rng(0)
    n, d = 40, 12
    X = rng.standard_normal((n, d)).astype(np.float32)
    y = np.where(rng.random(n) < 0.5, -1.0, 1.0).astype(np.float32)
    x = rng.standard_normal(d) * 0.5
    rows = np.array([3, 7, 8, 20, 39])
    g, margins = L.grad_dense(X, y, rows, x)
    assert np.allclose(margins, X[rows].astype(np.float64) @ x)
    eps = 1e-6
    for i in range(d):
        e = np.zeros(d)
        e[i] = eps
        num = (_loss(X, y, rows, x + e) - _loss(X, y, rows, x - e)) / (2 * eps)
        assert abs(num - g[i]) < 1e-8


def test_extreme_margins_do_not_overflow():
    X = np.array([[1000.0], [-1000.0]], dtype=np.float32)
    y = np.array([1.0, 1.0], dtype=np.float32)
    g, _ = L.grad_dense(X, y, np.array([0, 1]), np.array([1.0]))
    # row 0: sigma(-1000) ~ 0 ; row 1: sigma(1000) = 1 -> coef = -1/2 * a = +500
    assert np.isfinite(g).all() and abs(g[0] - 500.0) < 1e-9


def test_csr_matches_dense_and_default_batches():
    rng = np.random.default_rng(1)
    n, d, M, B = 30, 50, 3, 4
    dense = rng.standard_normal((n, d)).astype(np.float32) * (rng.random((n, d)) < 0.2)
    rowptr = np.zeros(n + 1, dtype=np.int64)
    cols, vals = [], []
    for r in range(n):
        nz = np.nonzero(dense[r])[0]
        rowptr[r + 1] = rowptr[r] + nz.size
        cols.append(nz.astype(np.int32))
        vals.append(dense[r, nz])
    cols, vals = np.concatenate(cols), np.concatenate(vals)
    y = np.where(rng.random(n) < 0.5, -1.0, 1.0).astype(np.float32)
    x = rng.standard_normal(d)
    shard_row0 = (np.arange(M + 1) * n) // M
    for t in (1, 2, 3, 4):
        a = L.grad_workers_dense(dense, y, shard_row0, B, t, x)
        b = L.grad_workers_csr(rowptr, cols, vals, y, shard_row0, B, t, x, d)
        assert np.allclose(a, b, rtol=1e-12, atol=1e-15)
    # default minibatch: consecutive rows of the shard, wrapping inside the shard
    assert L.batch_rows(shard_row0, 1, 4, 1).tolist() == [10, 11, 12, 13]
    assert L.batch_rows(shard_row0, 1, 4, 3).tolist() == [18, 19, 10, 11]


def test_touched_columns_are_the_union_of_the_minibatch_rows_and_bound_the_support():
    """Brute force with Python sets; and the sparse gradient is exactly +0.0 off the touched set
    (for any x), while a touched entry is non-zero unless contributions cancel."""
    rng = np.random.default_rng(4)
    n, d, M, B = 24, 64, 3, 3
    rowptr = np.zeros(n + 1, dtype=np.int64)
    cols, vals = [], []
    for r in range(n):
        nz = np.sort(rng.choice(d, size=rng.integers(0, 6), replace=False))
        rowptr[r + 1] = rowptr[r] + nz.size
        cols.append(nz.astype(np.int32))
        vals.append(rng.standard_normal(nz.size).astype(np.float32) + 3.0)
    cols, vals = np.concatenate(cols), np.concatenate(vals)
    y = np.where(rng.random(n) < 0.5, -1.0, 1.0).astype(np.float32)
    shard_row0 = (np.arange(M + 1) * n) // M
    for t in (1, 2, 5):
        touched = L.touched_columns(rowptr, cols, shard_row0, B, t, d)
        assert touched.shape == (M, d)
        for m in range(M):
            want = set()
            for r in L.batch_rows(shard_row0, m, B, t):
                want |= set(int(c) for c in cols[rowptr[r]:rowptr[r + 1]])
            assert set(np.nonzero(touched[m])[0].tolist()) == want
        g = L.grad_workers_csr(rowptr, cols, vals, y, shard_row0, B, t, rng.standard_normal(d), d)
        assert (g[~touched] == 0).all() and not np.signbit(g[~touched]).any()
        # positive values and a common label sign leave no cancellation: every touched entry is non-zero
        g1 = L.grad_workers_csr(rowptr, cols, vals, np.ones(n, dtype=np.float32), shard_row0, B, t, np.zeros(d), d)
        assert ((g1 != 0) == touched).all()
    ids = np.array([[0, 1], [9, 9], [20, 23]])
    touched = L.touched_columns(rowptr, cols, shard_row0, 2, 1, d, batch_ids=ids)
    assert set(np.nonzero(touched[1])[0].tolist()) == set(int(c) for c in cols[rowptr[9]:rowptr[10]])
