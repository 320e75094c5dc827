"""GPU parity of the logistic-regression gradient kernels and of the closed training loop
(gradient -> fused step) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import logreg_oracle as L
from oracle import qasg_oracle as O
from paper_2208_05631_b200 import inputs, libqasg
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu

# fp32 dot products against fp64: |err| <= G_RTOL*|want| + G_ATOL*max|want|
G_RTOL, G_ATOL = 2e-4, 2e-6


def _assert_grad_close(got, want):
    got = got.detach().cpu().numpy().astype(np.float64)
    scale = np.abs(want).max()
    assert (np.abs(got - want) <= G_ATOL * scale + G_RTOL * np.abs(want)).all()


@pytest.fixture(scope="module")
def ctx():
    c = libqasg.Context(1 << 16, 16, device=0)
    yield c
    c.close()


# wide rows, a column count that is not a multiple of 128, more minibatch rows than row lanes
@pytest.mark.parametrize("d,B,explicit", [(4096, 512, False), (260, 7, True), (4, 1, False), (8192, 33, True),
                                          (8196, 9, False), (12000, 5, True), (1028, 300, True)])
def test_dense_gradient(ctx, d, B, explicit):
    M, n = 8, 8192 if d == 4096 else (1024 if d == 1028 else 256)
    prob = inputs.logreg_dense_problem(n=n, d=d, M=M, seed=1)
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(d) * 0.05).astype(np.float32)
    Xd, yd, xd = U.to_dev(prob["X"]), U.to_dev(prob["y"]), U.to_dev(x)
    ld = d + 4
    for t in (1, 3, 40):
        ids = None
        ids_dev = None
        if explicit:
            ids = np.stack([rng.integers(prob["shard_row0"][m], prob["shard_row0"][m + 1], size=B) for m in range(M)])
            ids_dev = U.to_dev(ids.astype(np.uint32).view(np.int32))
        g = torch.full((M, ld), float("nan"), dtype=torch.float32, device=U.dev())
        ctx.logreg_grad_dense(Xd, yd, n, d, M, prob["shard_row0"], ids_dev, B, t, xd, g, ld)
        want = L.grad_workers_dense(prob["X"], prob["y"], prob["shard_row0"], B, t, x, batch_ids=ids)
        _assert_grad_close(g[:, :d], want)


def test_dense_gradient_extreme_margins(ctx):
    X = np.zeros((4, 4), dtype=np.float32)
    X[:, 0] = [1000.0, -1000.0, 200.0, -200.0]
    y = np.array([1.0, 1.0, -1.0, -1.0], dtype=np.float32)
    x = np.array([1.0, 0, 0, 0], dtype=np.float32)
    g = torch.zeros((1, 4), dtype=torch.float32, device=U.dev())
    ctx.logreg_grad_dense(U.to_dev(X), U.to_dev(y), 4, 4, 1, [0, 4], None, 4, 1, U.to_dev(x), g, 4)
    want = L.grad_workers_dense(X, y, np.array([0, 4]), 4, 1, x)
    out = g.cpu().numpy()
    assert np.isfinite(out).all()
    _assert_grad_close(g, want)


def test_csr_gradient(ctx):
    d, n, M, B = 1 << 16, 4000, 16, 64
    prob = inputs.logreg_csr_problem(n=n, d=d, M=M, nnz_per_row=80, seed=3)
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(d) * 0.5).astype(np.float32)
    dev_args = [U.to_dev(prob[k]) for k in ("rowptr", "colidx", "vals", "y")]
    xd = U.to_dev(x)
    for t in (1, 2, 70):
        g = torch.full((M, d), float("nan"), dtype=torch.float32, device=U.dev())
        ctx.logreg_grad_csr(*dev_args, n, d, M, prob["shard_row0"], None, B, t, xd, g, d)
        want = L.grad_workers_csr(prob["rowptr"], prob["colidx"], prob["vals"], prob["y"], prob["shard_row0"],
                                  B, t, x, d)
        _assert_grad_close(g, want)
        assert (g.cpu().numpy()[want == 0] == 0).all()


@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
def test_closed_loop_driven_by_the_oracle(ctx, rule):
    """The oracle runs the training loop (its own gradients, its own steps).  At every step
    the GPU gradient kernel is checked at the oracle's iterate, and the GPU fused step is fed
    the oracle's gradient and must track the oracle's iterate."""
    n, d, M, B, T = 4096, 1024, 8, 128, 30
    lam, eta, delta = 1e-4, 0.1, 1e-8
    prob = inputs.logreg_dense_problem(n=n, d=d, M=M, seed=1)
    Xd, yd = U.to_dev(prob["X"]), U.to_dev(prob["y"])
    params = libqasg.make_params(lam, eta, delta)
    xr, hr, zr = np.zeros(d), np.zeros(d), np.zeros(d)
    x, h, z = (torch.zeros(d, dtype=torch.float32, device=U.dev()) for _ in range(3))
    obj0 = L.objective(prob["X"], prob["y"], xr, lam)
    for t in range(1, T + 1):
        g64 = L.grad_workers_dense(prob["X"], prob["y"], prob["shard_row0"], B, t, xr)
        g_gpu = torch.empty((M, d), dtype=torch.float32, device=U.dev())
        ctx.logreg_grad_dense(Xd, yd, n, d, M, prob["shard_row0"], None, B, t, U.to_dev(xr.astype(np.float32)),
                              g_gpu, d)
        _assert_grad_close(g_gpu, g64)
        g32 = g64.astype(np.float32)
        ctx.step(rule, U.to_dev(g32), d, d, M, t, params, x, h, z)
        ref = O.step(rule, g32, xr, hr, zr, t, lam, eta, delta)
        xr, hr, zr = ref["x"], ref["h"], ref["z"] if rule == libqasg.RULE_RDA else zr
        U.assert_close(x, xr, "x step %d" % t)
        U.assert_close(h, hr, "h step %d" % t)
        U.assert_zero_pattern(x, xr, ref["a"], lam)
    assert L.objective(prob["X"], prob["y"], xr, lam) < obj0
