"""Oracle for the per-worker minibatch gradient of L1-regularised logistic regression
(the linear-model workload of the paper's experiments, Section 5.1).

TEST INFRASTRUCTURE ONLY.  fp64 numpy, one worker after another, one row after another
for the sparse form.  The L1 term is handled by the proximal update, so the gradient
is that of the smooth part only:

    f_m(x) = (1/B) sum_{j in Z_t^(m)} log(1 + exp(-y_j <a_j, x>)),   y_j in {-1, +1}
    f_m'(x) = (1/B) sum_j  -y_j * sigma(-y_j <a_j, x>) * a_j

(the minibatch average of Section 3.1 applied to the logistic loss; no bias term).
"""
import numpy as np

F64 = np.float64


def _sigmoid(s):
    # numerically stable logistic function in fp64
    out = np.empty_like(s)
    pos = s >= 0
    out[pos] = 1.0 / (1.0 + np.exp(-s[pos]))
    e = np.exp(s[~pos])
    out[~pos] = e / (1.0 + e)
    return out


def batch_rows(shard_row0, m, batch, t):
    """Default minibatch of worker m at step t (1-based): `batch` consecutive rows of
    the worker's shard [shard_row0[m], shard_row0[m+1]), starting at offset
    ((t-1)*batch) mod shard size and wrapping around inside the shard."""
    lo, hi = int(shard_row0[m]), int(shard_row0[m + 1])
    n = hi - lo
    start = ((int(t) - 1) * int(batch)) % n
    return lo + (start + np.arange(int(batch))) % n


def grad_dense(X, y, rows, x):
    """Gradient of one worker's minibatch; X is n x d (any float dtype), rows the
    global row ids of the minibatch.  Returns (g fp64[d], margins fp64[B])."""
    A = np.asarray(X)[rows].astype(F64)
    yy = np.asarray(y)[rows].astype(F64)
    margins = A @ np.asarray(x, dtype=F64)
    coef = -yy * _sigmoid(-yy * margins) / F64(len(rows))
    return A.T @ coef, margins


def grad_csr(rowptr, colidx, vals, y, rows, x, d):
    """Same for a CSR matrix (rowptr int64[n+1], colidx int32[nnz], vals[nnz])."""
    x = np.asarray(x, dtype=F64)
    g = np.zeros(int(d), dtype=F64)
    margins = np.zeros(len(rows), dtype=F64)
    inv_b = 1.0 / F64(len(rows))
    for k, r in enumerate(rows):
        lo, hi = int(rowptr[r]), int(rowptr[r + 1])
        cols = np.asarray(colidx[lo:hi], dtype=np.int64)
        a = np.asarray(vals[lo:hi], dtype=F64)
        s = float(a @ x[cols])
        margins[k] = s
        yj = float(y[r])
        c = -yj * float(_sigmoid(np.array([-yj * s]))[0]) * inv_b
        np.add.at(g, cols, c * a)
    return g, margins


def grad_workers_dense(X, y, shard_row0, batch, t, x, batch_ids=None):
    """All M workers' gradients, M x d fp64.  batch_ids (M x B global row ids) overrides
    the default cyclic minibatch."""
    m_workers = len(shard_row0) - 1
    out = np.zeros((m_workers, np.asarray(X).shape[1]), dtype=F64)
    for m in range(m_workers):
        rows = batch_rows(shard_row0, m, batch, t) if batch_ids is None else np.asarray(batch_ids[m])
        out[m], _ = grad_dense(X, y, rows, x)
    return out


def grad_workers_csr(rowptr, colidx, vals, y, shard_row0, batch, t, x, d, batch_ids=None):
    m_workers = len(shard_row0) - 1
    out = np.zeros((m_workers, int(d)), dtype=F64)
    for m in range(m_workers):
        rows = batch_rows(shard_row0, m, batch, t) if batch_ids is None else np.asarray(batch_ids[m])
        out[m], _ = grad_csr(rowptr, colidx, vals, y, rows, x, d)
    return out


def touched_columns(rowptr, colidx, shard_row0, batch, t, d, batch_ids=None):
    """Which coordinates each worker's minibatch can make non-zero: column i is touched by
    worker m when some row of its minibatch stores an entry in column i (Section 5.1: the
    text data sets are sparse, so a minibatch gradient has few non-zero coordinates).  A
    coordinate that is not touched has gradient exactly +0.0.  Returns bool [M, d]."""
    m_workers = len(shard_row0) - 1
    out = np.zeros((m_workers, int(d)), dtype=bool)
    for m in range(m_workers):
        rows = batch_rows(shard_row0, m, batch, t) if batch_ids is None else np.asarray(batch_ids[m])
        for r in rows:
            out[m, np.asarray(colidx[int(rowptr[r]):int(rowptr[r + 1])], dtype=np.int64)] = True
    return out


def objective(X, y, x, lam):
    """Full objective f(x) + lambda*||x||_1 over all rows (dense X), fp64."""
    s = np.asarray(X, dtype=F64) @ np.asarray(x, dtype=F64)
    yy = np.asarray(y, dtype=F64)
    return float(np.mean(np.logaddexp(0.0, -yy * s)) + F64(np.float32(lam)) * np.abs(x).sum())
