"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no arithmetic of the method: it only draws gradients, optimizer
states and logistic-regression problems from seeded generators.  The tests hand the
same bits to the CPU oracle and to the CUDA library; the benchmark uses the same
recipes at full size.

None of the paper's datasets (news20, rcv1, MNIST, CIFAR-10; Section 5.1, Table 1) is
used; these generators stand in for their shapes:

* `optimizer_only_gradients`  - per-worker N(0,1) gradients with a per-worker gain,
  the smallest closed workload (optimizer only, no model).
* `student_t_gradients`       - heavy-tailed gradients for the bandwidth-bound step.
* `normal_gradients`          - Gaussian gradients (the paper's Fig. 4 observation).
* `logreg_dense_problem`      - dense Gaussian design with a sparse ground truth.
* `logreg_csr_problem`        - sparse text-like features: Zipf column ids, log-normal
  values, rows normalised to unit L2 norm.
"""
import numpy as np
import torch


# ------------------------------------------------------------------ gradients / state
def optimizer_only_gradients(d, M, t, seed=0):
    """g^(m) ~ N(0,1) * (1 + 0.1 m), m = 0..M-1, fresh for every step t.  numpy fp32 [M, d]."""
    rng = np.random.default_rng([int(seed), int(t)])
    g = rng.standard_normal((M, d), dtype=np.float32)
    gain = (1.0 + 0.1 * np.arange(M, dtype=np.float32))[:, None]
    return np.ascontiguousarray(g * gain)


def _torch_gen(seed, device):
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    return gen


def student_t_gradients(d, M, seed=2, nu=3, scale=1e-2, device="cpu", ld=None, chunk=1 << 24):
    """scale * Student-t(nu) samples, torch fp32 [M, ld] (ld >= d, default d), built as
    Z / sqrt(chi2_nu / nu) from normals, generated in chunks to bound temporaries."""
    ld = int(d if ld is None else ld)
    gen = _torch_gen(seed, device)
    out = torch.zeros((M, ld), dtype=torch.float32, device=device)
    for m in range(M):
        for lo in range(0, d, chunk):
            n = min(chunk, d - lo)
            z = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
            c = torch.randn((nu, n), generator=gen, device=device, dtype=torch.float32)
            c = (c * c).sum(dim=0) / float(nu)
            out[m, lo:lo + n] = scale * z / torch.sqrt(c)
    return out


def normal_gradients(d, M, seed=4, device="cpu", ld=None, chunk=1 << 26):
    """N(0,1) gradients, torch fp32 [M, ld]."""
    ld = int(d if ld is None else ld)
    gen = _torch_gen(seed, device)
    out = torch.zeros((M, ld), dtype=torch.float32, device=device)
    for m in range(M):
        for lo in range(0, d, chunk):
            n = min(chunk, d - lo)
            out[m, lo:lo + n] = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
    return out


def random_state(d, seed=2, device="cpu"):
    """Random optimizer state for one-off steps: x, z ~ 0.1 * N(0,1), h ~ U[0,1).
    Returns torch fp32 tensors (x, h, z)."""
    gen = _torch_gen(int(seed) + 1000003, device)
    x = 0.1 * torch.randn(d, generator=gen, device=device, dtype=torch.float32)
    h = torch.rand(d, generator=gen, device=device, dtype=torch.float32)
    z = 0.1 * torch.randn(d, generator=gen, device=device, dtype=torch.float32)
    return x, h, z


def bernoulli_mask(d, density, seed=2, device="cpu"):
    """fp32 [d] of zeros and ones, one with probability `density` (for a sparse iterate)."""
    gen = _torch_gen(int(seed) + 2000003, device)
    return (torch.rand(d, generator=gen, device=device, dtype=torch.float32) < float(density)).to(torch.float32)


# ------------------------------------------------------------------ logistic regression
def shard_rows(n, M):
    """Row ranges of M equal contiguous shards: int64 [M+1]."""
    return (np.arange(M + 1, dtype=np.int64) * n) // M


def logreg_dense_problem(n=65536, d=4096, M=8, seed=1, density=0.05, noise=0.1):
    """X ~ N(0,1) fp32 [n, d]; w* with `density` non-zeros ~ N(0,1);
    y = sign(X w* + noise * eps) in {-1, +1} fp32.  Returns dict(X, y, w_star, shard_row0)."""
    rng = np.random.default_rng(int(seed))
    X = rng.standard_normal((n, d), dtype=np.float32)
    w = np.zeros(d, dtype=np.float32)
    k = max(1, int(round(density * d)))
    sup = rng.choice(d, size=k, replace=False)
    w[sup] = rng.standard_normal(k, dtype=np.float32)
    s = X.astype(np.float64) @ w.astype(np.float64) + noise * rng.standard_normal(n)
    y = np.where(s >= 0, 1.0, -1.0).astype(np.float32)
    return dict(X=X, y=y, w_star=w, shard_row0=shard_rows(n, M))


def logreg_csr_problem(n=1_000_000, d=1 << 24, M=16, nnz_per_row=80, seed=3, zipf_s=1.1,
                       density=0.01):
    """Sparse design in CSR: about `nnz_per_row` distinct columns per row with ids drawn
    from a Zipf(zipf_s) law truncated to [0, d), values log-normal(0,1), every row scaled
    to unit L2 norm; labels from a `density`-dense w*.  Duplicate column draws inside a
    row are dropped, so rows hold slightly fewer than nnz_per_row entries.
    Returns dict(rowptr int64, colidx int32, vals fp32, y fp32, w_star fp32, shard_row0)."""
    rng = np.random.default_rng(int(seed))
    ranks = np.arange(1, d + 1, dtype=np.float64)
    cdf = np.cumsum(ranks ** (-float(zipf_s)))
    cdf /= cdf[-1]
    del ranks
    w = np.zeros(d, dtype=np.float32)
    k = max(1, int(round(density * d)))
    w[rng.choice(d, size=k, replace=False)] = rng.standard_normal(k, dtype=np.float32)

    rowptr = np.zeros(n + 1, dtype=np.int64)
    cols_out, vals_out = [], []
    y = np.empty(n, dtype=np.float32)
    block = 1 << 16
    for lo in range(0, n, block):
        b = min(block, n - lo)
        cols = np.searchsorted(cdf, rng.random((b, nnz_per_row)), side="left")
        cols = np.minimum(cols, d - 1).astype(np.int64)
        cols.sort(axis=1)
        keep = np.ones_like(cols, dtype=bool)
        keep[:, 1:] = cols[:, 1:] != cols[:, :-1]
        vals = rng.lognormal(0.0, 1.0, size=(b, nnz_per_row))
        vals = np.where(keep, vals, 0.0)
        vals /= np.sqrt((vals * vals).sum(axis=1, keepdims=True))
        s = (vals * w[cols].astype(np.float64)).sum(axis=1)
        y[lo:lo + b] = np.where(s >= 0, 1.0, -1.0)
        rowptr[lo + 1:lo + b + 1] = keep.sum(axis=1)
        cols_out.append(cols[keep].astype(np.int32))
        vals_out.append(vals[keep].astype(np.float32))
    rowptr = np.cumsum(rowptr)
    return dict(rowptr=rowptr, colidx=np.concatenate(cols_out), vals=np.concatenate(vals_out),
                y=y, w_star=w, shard_row0=shard_rows(n, M))
