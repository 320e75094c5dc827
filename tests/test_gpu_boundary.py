"""GPU tests of the library boundary: the unquantized step (Q = identity), lambda = 0, refused calls
that must enqueue nothing, indices taken from the caller's sparse data, guard words behind every
output buffer, and the thresholds and scales against a sum that knows nothing of tiles."""
import math

import numpy as np
import pytest
import torch

from oracle import logreg_oracle as L
from oracle import qasg_oracle as O
from paper_2208_05631_b200 import inputs, libqasg
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu

LAM, ETA, DELTA = 1e-3, 0.1, 1e-8


@pytest.fixture(scope="module")
def ctx():
    c = libqasg.Context(1 << 21, 64, device=0)
    yield c
    c.close()


def _status_of(call):
    with pytest.raises(libqasg.QasgError) as e:
        call()
    return e.value.status


# ------------------------------------------------------------------ Q = identity (32-bit CMD / RDA adagrad)
@pytest.mark.parametrize("d,M", [(1, 1), (3, 2), (4098, 8), (70_003, 13), (200_001, 5), (9_999, 64)])
@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
def test_unquantized_step_against_the_oracle(ctx, d, M, rule):
    t = 5
    g = inputs.optimizer_only_gradients(d, M, t, seed=d + M) * np.float32(0.02)
    x0, h0, z0 = (v.numpy() for v in inputs.random_state(d, seed=M))
    h0[::5] = 0.0
    g_dev, ld = U.grad_to_dev(g)
    x, h, z = U.to_dev(x0), U.to_dev(h0), U.to_dev(z0)
    params = libqasg.make_params(LAM, ETA, DELTA, quantizer=libqasg.Q_NONE)
    before = ctx.launch_count()
    ctx.step(rule, g_dev, d, ld, M, t, params, x, h, z)
    assert ctx.launch_count() == before + 1            # one pass over the gradients
    assert ctx.last_async_status() == libqasg.OK
    ref = O.step(rule, g, x0, h0, z0, t, LAM, ETA, DELTA, quantizer=O.QUANT_NONE)
    U.assert_close(x, ref["x"], "x"), U.assert_close(h, ref["h"], "h")
    if rule == libqasg.RULE_RDA:
        U.assert_close(z, ref["z"], "z", atol=U.ATOL + 2.0 ** -23 * (np.abs(z0) + np.abs(ref["q"])))
    else:
        assert np.array_equal(z.cpu().numpy(), z0)
    U.assert_zero_pattern(x, ref["x"], ref["a"], LAM)


def test_unquantized_cmd_step_is_diagonal_adagrad(ctx):
    # lambda = 0, one worker: Eq. CMD adagrad is x <- x - eta * g / (delta + sqrt(sum g^2)), the library
    # routine torch.optim.Adagrad(eps = delta) run on the same device values.
    d, steps = 30_001, 6
    params = libqasg.make_params(0.0, ETA, DELTA, quantizer=libqasg.Q_NONE)
    rng = np.random.default_rng(17)
    x0 = rng.standard_normal(d).astype(np.float32)
    x, h = U.to_dev(x0), torch.zeros(d, dtype=torch.float32, device=U.dev())
    w = torch.nn.Parameter(U.to_dev(x0).double())
    opt = torch.optim.Adagrad([w], lr=float(np.float32(ETA)), eps=float(np.float32(DELTA)))
    for t in range(1, steps + 1):
        g = (rng.standard_normal((1, d)) * 0.3).astype(np.float32)
        g_dev, ld = U.grad_to_dev(g)
        ctx.step(libqasg.RULE_CMD, g_dev, d, ld, 1, t, params, x, h)
        w.grad = g_dev[0, :d].double()
        opt.step()
        U.assert_close(x, w.detach().cpu().numpy(), "x after step %d" % t)
    assert ctx.last_async_status() == libqasg.OK


def test_unquantized_step_reports_a_nonfinite_mean(ctx):
    d, M = 5000, 3
    g = np.ones((M, d), dtype=np.float32)
    g[1, 4321] = np.inf
    g_dev, ld = U.grad_to_dev(g)
    x, h = (torch.zeros(d, dtype=torch.float32, device=U.dev()) for _ in range(2))
    ctx.step(libqasg.RULE_CMD, g_dev, d, ld, M, 1, libqasg.make_params(LAM, ETA, DELTA, quantizer=libqasg.Q_NONE), x, h)
    assert ctx.last_async_status() == libqasg.ERR_NONFINITE
    assert ctx.last_async_status() == libqasg.OK


def test_identity_quantizer_is_refused_where_codes_are_asked_for(ctx):
    d, M = 1000, 2
    g = torch.zeros((M, d), dtype=torch.float32, device=U.dev())
    codes, scales = U.new_codes(M, d), torch.zeros(M, dtype=torch.float32, device=U.dev())
    none = libqasg.make_params(LAM, ETA, DELTA, quantizer=libqasg.Q_NONE)
    before = ctx.launch_count()
    assert _status_of(lambda: ctx.quantize_pack(g, d, d, M, 1, none, codes, scales)) == libqasg.ERR_INVALID_ARG
    x, h = (torch.zeros(d, dtype=torch.float32, device=U.dev()) for _ in range(2))
    assert _status_of(lambda: ctx.step_double(0, g, d, d, M, 1, none, x, h)) == libqasg.ERR_INVALID_ARG
    assert _status_of(lambda: ctx.step_select(0, 0, g, d, d, M, 1, none, x, h)) == libqasg.ERR_INVALID_ARG
    bad = libqasg.make_params(LAM, ETA, DELTA, quantizer=3)
    assert _status_of(lambda: ctx.step(0, g, d, d, M, 1, bad, x, h)) == libqasg.ERR_INVALID_ARG
    assert ctx.launch_count() == before


# ------------------------------------------------------------------ lambda = 0 (Theorems 1 and 2 allow lambda >= 0)
@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
@pytest.mark.parametrize("quantizer", [libqasg.Q_THRESHOLD, libqasg.Q_TERNARY_STOCH])
def test_fused_step_without_regularisation(ctx, rule, quantizer):
    d, M, t = 70_003, 8, 9
    g = inputs.optimizer_only_gradients(d, M, t, seed=3) * np.float32(0.05)
    x0, h0, z0 = (v.numpy() for v in inputs.random_state(d, seed=3))
    x0[::3] = 0.0
    z0[::7] = 0.0
    g_dev, ld = U.grad_to_dev(g)
    x, h, z = U.to_dev(x0), U.to_dev(h0), U.to_dev(z0)
    codes = U.new_codes(M, d)
    ctx.step(rule, g_dev, d, ld, M, t, libqasg.make_params(0.0, ETA, DELTA, quantizer=quantizer, seed=11), x, h, z,
             codes_out=codes)
    assert ctx.last_async_status() == libqasg.OK
    ref = O.step(rule, g, x0, h0, z0, t, 0.0, ETA, DELTA, quantizer=quantizer, seed=11)
    assert np.array_equal(U.codes_np(codes), ref["quant"]["codes"])
    U.assert_close(x, ref["x"], "x"), U.assert_close(h, ref["h"], "h")
    if rule == libqasg.RULE_RDA:
        U.assert_close(z, ref["z"], "z", atol=U.ATOL + 2.0 ** -23 * (np.abs(z0) + np.abs(ref["q"])))
    U.assert_zero_pattern(x, ref["x"], ref["a"], 0.0)
    # without the L1 term an iterate is zero only where the closed form's argument is exactly zero
    assert np.count_nonzero(ref["x"]) > 0.5 * d


@pytest.mark.parametrize("d", [3, 4098, 100_003])
def test_dense_q_steps_without_regularisation(ctx, d):
    rng = np.random.default_rng(d)
    q = (rng.standard_normal(d) * 1e-2).astype(np.float32)
    q[::7] = 0.0
    x0, h0, z0 = (v.numpy() for v in inputs.random_state(d, seed=d))
    x0[::7] = 0.0                      # q = 0 and x = 0 together: stays exactly +0.0
    z0[::7] = 0.0
    params = libqasg.make_params(0.0, ETA, DELTA)
    x, h = U.to_dev(x0), U.to_dev(h0)
    ctx.cmd_step(U.to_dev(q), x, h, d, 3, params)
    xr, hr, a = O.cmd_step(q, x0, h0, 0.0, ETA, DELTA)
    U.assert_close(x, xr, "x cmd"), U.assert_close(h, hr, "h cmd")
    U.assert_zero_pattern(x, xr, a, 0.0)
    x, h, z = torch.full((d,), 9.0, dtype=torch.float32, device=U.dev()), U.to_dev(h0), U.to_dev(z0)
    ctx.rda_step(U.to_dev(q), x, h, z, d, 16, params)
    xr, hr, zr, a = O.rda_step(q, h0, z0, 16, 0.0, ETA, DELTA)
    U.assert_close(x, xr, "x rda"), U.assert_close(h, hr, "h rda"), U.assert_close(z, zr, "z rda")
    U.assert_zero_pattern(x, xr, a, 0.0)
    assert (xr[::7] == 0).all()


# ------------------------------------------------------------------ qasg_step_host refuses before it copies
def test_step_host_refuses_bad_arguments_before_any_copy(ctx):
    d, M = 1000, 2
    ld = d + 8
    gh = torch.ones((M, ld), dtype=torch.float32).pin_memory()
    xh, hh, zh = (torch.ones(d, dtype=torch.float32).pin_memory() for _ in range(3))
    g_dev = torch.full((M, ld), 7.0, dtype=torch.float32, device=U.dev())
    xd, hd, zd = (torch.full((d + 4,), 7.0, dtype=torch.float32, device=U.dev()) for _ in range(3))
    good = libqasg.make_params(LAM, ETA, DELTA)
    before = ctx.launch_count()

    def call(rule=0, d_=d, ld_=ld, M_=M, t=1, params=good, x_host=xh, h_host=hh, z_host=zh, g_d=g_dev, x_d=xd, h_d=hd,
             z_d=zd, g_host=gh):
        return lambda: ctx.step_host(rule, g_host, d_, ld_, M_, t, params, x_host, h_host, z_host, g_d, x_d, h_d, z_d)

    assert _status_of(call(params=libqasg.make_params(LAM, ETA, 0.0))) == libqasg.ERR_INVALID_ARG      # delta = 0
    assert _status_of(call(params=libqasg.make_params(LAM, -1.0, DELTA))) == libqasg.ERR_INVALID_ARG    # eta < 0
    assert _status_of(call(params=libqasg.make_params(LAM, ETA, DELTA, quantizer=5))) == libqasg.ERR_INVALID_ARG
    assert _status_of(call(rule=2)) == libqasg.ERR_INVALID_ARG
    assert _status_of(call(t=0)) == libqasg.ERR_INVALID_ARG
    assert _status_of(call(ld_=d + 6)) == libqasg.ERR_ALIGNMENT                                         # ld % 4
    assert _status_of(call(ld_=d - 4)) == libqasg.ERR_INVALID_ARG                                       # ld < d
    assert _status_of(call(g_d=g_dev.data_ptr() + 4)) == libqasg.ERR_ALIGNMENT
    assert _status_of(call(x_d=xd.data_ptr() + 4)) == libqasg.ERR_ALIGNMENT
    assert _status_of(call(rule=1, z_d=None)) == libqasg.ERR_INVALID_ARG                                # RDA, no z
    assert _status_of(call(rule=1, z_host=None)) == libqasg.ERR_INVALID_ARG
    assert _status_of(call(g_host=None)) == libqasg.ERR_INVALID_ARG
    assert _status_of(call(M_=65)) == libqasg.ERR_INVALID_ARG
    assert _status_of(call(d_=3_000_000, ld_=3_000_000)) == libqasg.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert ctx.launch_count() == before
    for buf in (g_dev, xd, hd, zd):                  # no copy reached the staging buffers
        assert bool((buf == 7.0).all())
    for buf in (xh, hh, zh):
        assert bool((buf == 1.0).all())


# ------------------------------------------------------------------ indices of the caller's sparse data
def test_csr_gradient_skips_and_reports_indices_out_of_range():
    ctx = libqasg.Context(1 << 16, 4, device=0)
    d, n, M, B, t = 5000, 256, 4, 16, 1
    prob = inputs.logreg_csr_problem(n=n, d=d, M=M, nnz_per_row=12, seed=5)
    rng = np.random.default_rng(6)
    x = (rng.standard_normal(d) * 0.1).astype(np.float32)
    rowptr, colidx, vals = prob["rowptr"], prob["colidx"].copy(), prob["vals"].copy()
    rows = [L.batch_rows(prob["shard_row0"], m, B, t) for m in range(M)]
    # entries of minibatch rows whose column is pushed out of [0, d): above d, far above d, negative
    victims = [int(rowptr[rows[0][0]]) + 1, int(rowptr[rows[1][3]]), int(rowptr[rows[3][15] + 1]) - 1]
    bad_cols = [d, 2_000_000_000, -7]
    clean_cols = colidx.copy()
    for k, c in zip(victims, bad_cols):
        colidx[k] = c
    ld = d + 8
    guard = 64

    def run(cols, touched):
        flat = torch.full((M * ld + guard,), float("nan"), dtype=torch.float32, device=U.dev())
        g = flat[: M * ld].view(M, ld)
        args = (U.to_dev(rowptr), U.to_dev(cols), U.to_dev(vals), U.to_dev(prob["y"]), n, d, M, prob["shard_row0"],
                None, B, t, U.to_dev(x), g, ld)
        if touched:
            g.zero_()
            bits = torch.zeros((M, (d + 31) // 32), dtype=torch.int32, device=U.dev())
            ctx.logreg_grad_csr_touched(*args, bits)
        else:
            ctx.logreg_grad_csr(*args)
        status = ctx.last_async_status()
        out = flat.cpu().numpy()
        return status, out[: M * ld].reshape(M, ld), out[M * ld:]

    for touched in (False, True):
        status, got, tail = run(colidx, touched)
        assert status == libqasg.ERR_BAD_INDEX
        assert np.isnan(tail).all()                                  # nothing written behind g
        assert touched or np.isnan(got[:, d:]).all()                 # nor into the padding of its rows
        # the oracle on the data with the three entries removed (value 0) gives what the kernel must give:
        # a skipped entry adds nothing to the margin nor to the gradient
        vals0 = vals.copy()
        vals0[victims] = 0.0
        want = L.grad_workers_csr(rowptr, clean_cols, vals0, prob["y"], prob["shard_row0"], B, t, x.astype(np.float64), d)
        scale = np.abs(want).max()
        assert (np.abs(got[:, :d].astype(np.float64) - want) <= 2e-6 * scale + 2e-4 * np.abs(want)).all()
        status, _, _ = run(clean_cols, touched)
        assert status == libqasg.OK

    # a minibatch row id outside the matrix, and a rowptr pair that runs backwards
    ids = np.stack(rows).astype(np.uint32)
    ids[2, 5] = n + 3
    g = torch.zeros((M, ld), dtype=torch.float32, device=U.dev())
    ctx.logreg_grad_csr(U.to_dev(rowptr), U.to_dev(clean_cols), U.to_dev(vals), U.to_dev(prob["y"]), n, d, M,
                        prob["shard_row0"], U.to_dev(ids.view(np.int32)), B, t, U.to_dev(x), g, ld)
    assert ctx.last_async_status() == libqasg.ERR_BAD_INDEX
    broken = rowptr.copy()
    broken[rows[1][2] + 1] = broken[rows[1][2]] - 5
    ctx.logreg_grad_csr(U.to_dev(broken), U.to_dev(clean_cols), U.to_dev(vals), U.to_dev(prob["y"]), n, d, M,
                        prob["shard_row0"], None, B, t, U.to_dev(x), g, ld)
    assert ctx.last_async_status() == libqasg.ERR_BAD_INDEX
    # dense entry point: a row id outside X
    dense = inputs.logreg_dense_problem(n=64, d=260, M=M, seed=1)
    ids = np.stack([L.batch_rows(dense["shard_row0"], m, 4, 1) for m in range(M)]).astype(np.uint32)
    want = L.grad_workers_dense(dense["X"], dense["y"], dense["shard_row0"], 4, 1, x[:260], batch_ids=ids.astype(np.int64))
    ids[1, 2] = 64
    gd = torch.zeros((M, 260), dtype=torch.float32, device=U.dev())
    ctx.logreg_grad_dense(U.to_dev(dense["X"]), U.to_dev(dense["y"]), 64, 260, M, dense["shard_row0"],
                          U.to_dev(ids.view(np.int32)), 4, 1, U.to_dev(x[:260].copy()), gd, 260)
    assert ctx.last_async_status() == libqasg.ERR_BAD_INDEX
    got = gd.cpu().numpy()
    scale = np.abs(want).max()
    for m in (0, 2, 3):                              # the other workers' gradients are untouched by it
        assert (np.abs(got[m] - want[m]) <= 2e-6 * scale + 2e-4 * np.abs(want[m])).all()
    ctx.close()


# ------------------------------------------------------------------ guard words behind every output
GUARD = 64          # words


class Guarded:
    """A device buffer of `n` elements followed by GUARD elements of a bit pattern no kernel writes."""

    def __init__(self, n, dtype, fill=0):
        self.n = n
        self.flat = torch.empty(n + GUARD, dtype=dtype, device=U.dev())
        self.flat[:n] = fill
        self.pattern = -1.2345e33 if dtype == torch.float32 else 0x5A5A5A5A
        self.flat[n:] = self.pattern
        self.t = self.flat[:n]

    def intact(self):
        return bool((self.flat[self.n:] == self.pattern).all())


@pytest.mark.parametrize("d,M", [(4099, 3), (70_001, 8), (8 * 512 * 3 + 5, 16)])
def test_no_entry_point_writes_behind_its_outputs(ctx, d, M):
    """Every output buffer is exactly as long as the header says and is followed by guard words; after each
    entry point the guards are checked.  (No memory checker runs on the GPU here: this is its stand-in.)"""
    t = 4
    W, IW = libqasg.code_words(d), (d + 31) // 32
    g = inputs.optimizer_only_gradients(d, M, t, seed=d) * np.float32(0.05)
    g_dev, ld = U.grad_to_dev(g)
    x0, h0, z0 = (v.numpy() for v in inputs.random_state(d, seed=2))
    x0[::4] = 0.0

    def state():
        out = [Guarded(d, torch.float32) for _ in range(3)]
        for buf, v in zip(out, (x0, h0, z0)):
            buf.t.copy_(torch.from_numpy(v))
        return out

    def outputs():
        return dict(codes=Guarded(M * W, torch.int32), scales=Guarded(M, torch.float32),
                    thresholds=Guarded(M, torch.float32), counts=Guarded(M, torch.int64),
                    indicators=Guarded(M * IW, torch.int32), selected=Guarded(M, torch.int64),
                    isyn=Guarded(IW, torch.int32), ksyn=Guarded(1, torch.int64),
                    qcodes=Guarded(W, torch.int32), qscale=Guarded(1, torch.float32), gbar=Guarded(d, torch.float32))

    def check(name, *groups):
        torch.cuda.synchronize()
        for group in groups:
            for key, buf in (group.items() if isinstance(group, dict) else enumerate(group)):
                assert buf.intact(), "%s wrote behind %s" % (name, key)

    for quantizer in (libqasg.Q_THRESHOLD, libqasg.Q_TERNARY_STOCH):
        params = libqasg.make_params(LAM, ETA, DELTA, quantizer=quantizer, seed=9)
        for rule in (libqasg.RULE_CMD, libqasg.RULE_RDA):
            o, (x, h, z) = outputs(), state()
            ctx.quantize_pack(g_dev, d, ld, M, t, params, o["codes"].t, o["scales"].t, o["thresholds"].t, o["counts"].t)
            check("quantize_pack", o)
            ctx.decode_average(o["codes"].t, o["scales"].t, d, M, o["gbar"].t)
            check("decode_average", o)
            ctx.requantize(o["codes"].t, o["scales"].t, d, M, t, params, o["qcodes"].t, o["qscale"].t)
            check("requantize", o)
            if rule == libqasg.RULE_CMD:
                ctx.cmd_step(o["gbar"].t, x.t, h.t, d, t, params)
            else:
                ctx.rda_step(o["gbar"].t, x.t, h.t, z.t, d, t, params)
            check("dense step", o, (x, h, z))
            ctx.step(rule, g_dev, d, ld, M, t, params, x.t, h.t, z.t, codes_out=o["codes"].t, scales_out=o["scales"].t)
            check("step", o, (x, h, z))
            ctx.step_double(rule, g_dev, d, ld, M, t, params, x.t, h.t, z.t, o["codes"].t, o["scales"].t, o["qcodes"].t,
                            o["qscale"].t)
            check("step_double", o, (x, h, z))
            ctx.select_quantize_pack(rule, g_dev, d, ld, M, t, params, x.t, h.t, z.t, o["codes"].t, o["scales"].t,
                                     o["thresholds"].t, o["counts"].t, o["indicators"].t, o["selected"].t)
            check("select_quantize_pack", o)
            ctx.indicator_or(o["indicators"].t, d, M, o["isyn"].t, o["ksyn"].t)
            check("indicator_or", o)
            for double_quant in (0, 1):
                ctx.step_select(rule, double_quant, g_dev, d, ld, M, t, params, x.t, h.t, z.t, o["codes"].t,
                                o["scales"].t, o["indicators"].t, o["selected"].t, o["isyn"].t, o["ksyn"].t)
                check("step_select", o, (x, h, z))
            ctx.step(rule, g_dev, d, ld, M, t, libqasg.make_params(LAM, ETA, DELTA, quantizer=libqasg.Q_NONE),
                     x.t, h.t, z.t)
            check("unquantized step", (x, h, z))
    assert ctx.last_async_status() == libqasg.OK
    if M <= libqasg.STATIC_MAX_WORKERS:
        o = outputs()
        libqasg.quantize_pack_static(0, g_dev, d, ld, M, 0.75, o["codes"].t, o["scales"].t, o["thresholds"].t,
                                     o["counts"].t)
        check("quantize_pack_static", o)


# ------------------------------------------------------------------ thresholds and scales without any tile logic
@pytest.mark.parametrize("d", [5, 4097, 70_001, 3 * 4096 * 64 + 1234, 1_500_007])
def test_threshold_and_scale_equal_the_exactly_rounded_definitions(ctx, d):
    """Delta_m = fp32(0.75 * sum|v| / d) and s_m = fp32(sum of kept |v| / n) with the sums taken exactly
    (math.fsum) and rounded once: no tile, column or tree appears on this side.  The fixed-order fp64
    sums of the kernels are accurate to ~1e-15 relative, so the two fp32 results can differ only where
    the exact quotient lies within that distance of a rounding boundary; the seeded cases below do not."""
    M = 3
    rng = np.random.default_rng(d)
    g = rng.standard_normal((M, d)).astype(np.float32) * np.array([[1.0], [3e-4], [700.0]], dtype=np.float32)
    g_dev, ld = U.grad_to_dev(g)
    codes = U.new_codes(M, d)
    scales, thr = (torch.zeros(M, dtype=torch.float32, device=U.dev()) for _ in range(2))
    cnt = torch.zeros(M, dtype=torch.int64, device=U.dev())
    ctx.quantize_pack(g_dev, d, ld, M, 1, libqasg.make_params(), codes, scales, thr, cnt)
    assert ctx.last_async_status() == libqasg.OK
    scales, thr, cnt = scales.cpu().numpy(), thr.cpu().numpy(), cnt.cpu().numpy()
    for m in range(M):
        mags = [abs(float(v)) for v in g[m]]
        delta = np.float32(0.75 * math.fsum(mags) / d)
        assert thr[m] == delta
        kept = [a for a in mags if a > float(delta)]
        assert cnt[m] == len(kept)
        assert scales[m] == np.float32(math.fsum(kept) / len(kept))
