"""GPU parity: every entry point of libqasg, called through the C-ABI, against the CPU
oracle on the same seeded inputs.  Integer results (codes, counts, Philox decisions) and
the fp32 statistics rounded from the fixed-order sums (Delta_m, s_m) are bit-exact; fp32
iterates are within 1e-7 + 1e-5*|oracle| of the fp64 oracle after every step."""
import numpy as np
import pytest
import torch

from oracle import qasg_oracle as O
from paper_2208_05631_b200 import inputs, libqasg
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu

LAM, ETA, DELTA = 1e-3, 0.1, 1e-8


@pytest.fixture(scope="module")
def ctx():
    c = libqasg.Context(6_000_000, 64, device=0)
    yield c
    c.close()


def _quantize_gpu(ctx, g, quantizer=libqasg.Q_THRESHOLD, t=1, seed=0):
    M, d = g.shape
    g_dev, ld = U.grad_to_dev(g)
    codes = U.new_codes(M, d)
    scales = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    thresholds = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    counts = torch.full((M,), -1, dtype=torch.int64, device=U.dev())
    params = libqasg.make_params(LAM, ETA, DELTA, quantizer=quantizer, seed=seed)
    ctx.quantize_pack(g_dev, d, ld, M, t, params, codes, scales, thresholds, counts)
    status = ctx.last_async_status()
    return dict(codes=U.codes_np(codes), scales=scales.cpu().numpy(), thresholds=thresholds.cpu().numpy(),
                counts=counts.cpu().numpy(), status=status)


def _assert_quant_equal(got, ref):
    assert np.array_equal(got["codes"], ref["codes"])
    assert np.array_equal(U.f32_bits(got["scales"]), U.f32_bits(ref["scales"]))
    assert np.array_equal(U.f32_bits(got["thresholds"]), U.f32_bits(ref["thresholds"]))
    assert np.array_equal(got["counts"], ref["counts"])


# ------------------------------------------------------------------ quantize + pack
@pytest.mark.parametrize("d", [1, 5, 16, 17, 1023, 4095, 4096, 4097, 10_000, 3 * 4096 + 17, 200_003])
def test_threshold_codes_bit_exact(ctx, d):
    rng = np.random.default_rng(d)
    g = rng.standard_normal((3, d)).astype(np.float32) * np.array([[1.0], [1e-3], [50.0]], dtype=np.float32)
    got = _quantize_gpu(ctx, g)
    assert got["status"] == libqasg.OK
    _assert_quant_equal(got, O.quantize_workers(g, O.QUANT_THRESHOLD))


def test_threshold_codes_many_tiles_per_chunk(ctx):
    # 1221 tiles -> chunks of 2 tiles, ragged last chunk and ragged last tile
    d = 5_000_001
    g = inputs.normal_gradients(d, 2, seed=4).numpy()
    got = _quantize_gpu(ctx, g)
    _assert_quant_equal(got, O.quantize_workers(g, O.QUANT_THRESHOLD))


@pytest.mark.parametrize("M", [1, 2, 32, 64])
def test_threshold_codes_worker_counts(ctx, M):
    g = inputs.optimizer_only_gradients(9001, M, t=1, seed=M)
    _assert_quant_equal(_quantize_gpu(ctx, g), O.quantize_workers(g, O.QUANT_THRESHOLD))


def test_threshold_edge_cases(ctx):
    d = 4100
    rng = np.random.default_rng(0)
    rows = [np.zeros(d, np.float32),                                  # zero gradient
            np.full(d, 0.37, np.float32) * rng.choice([-1, 1], d).astype(np.float32),  # all |g| equal
            rng.standard_normal(d).astype(np.float32),                # one huge outlier
            (rng.standard_normal(d) * 1e-41).astype(np.float32),      # denormals
            np.where(rng.random(d) < 0.5, 0.0, -0.0).astype(np.float32)]  # signed zeros
    rows[2][77] = 3e30
    g = np.stack(rows)
    got = _quantize_gpu(ctx, g)
    assert got["status"] == libqasg.OK
    ref = O.quantize_workers(g, O.QUANT_THRESHOLD)
    _assert_quant_equal(got, ref)
    assert got["counts"][0] == 0 and got["scales"][0] == 0 and got["counts"][1] == d


def test_threshold_boundary_is_strict(ctx):
    # |v| = (3, 3, 6, 4): Delta = 3 exactly; components equal to Delta code 0
    g = np.array([[3.0, -3.0, 6.0, -4.0]], dtype=np.float32)
    got = _quantize_gpu(ctx, g)
    assert got["thresholds"][0] == 3.0 and got["scales"][0] == 5.0 and got["counts"][0] == 2
    assert O.unpack_codes(got["codes"][0], 4).tolist() == [0, 0, 1, -1]


def test_nonfinite_gradient_is_reported(ctx):
    g = np.ones((2, 5000), dtype=np.float32)
    g[1, 4321] = np.nan
    got = _quantize_gpu(ctx, g)
    assert got["status"] == libqasg.ERR_NONFINITE
    ref = O.quantize_workers(g, O.QUANT_THRESHOLD)
    assert np.array_equal(got["codes"], ref["codes"]) and not got["codes"][1].any()
    g[1, 4321] = np.inf
    assert _quantize_gpu(ctx, g)["status"] == libqasg.ERR_NONFINITE
    assert _quantize_gpu(ctx, np.ones((2, 5000), dtype=np.float32))["status"] == libqasg.OK


@pytest.mark.parametrize("d,t,seed", [(1, 1, 0), (4099, 7, 123456789), (70_001, (1 << 32) + 5, (0xDEADBEEF << 32) | 0x1234)])
def test_stochastic_codes_bit_exact(ctx, d, t, seed):
    rng = np.random.default_rng(d)
    g = rng.standard_normal((5, d)).astype(np.float32)
    g[3] = 0.0
    got = _quantize_gpu(ctx, g, quantizer=libqasg.Q_TERNARY_STOCH, t=t, seed=seed)
    assert got["status"] == libqasg.OK
    _assert_quant_equal(got, O.quantize_workers(g, O.QUANT_TERNARY_STOCH, t=t, seed=seed))


# ------------------------------------------------------------------ decode + average
@pytest.mark.parametrize("d,M", [(1, 1), (18, 3), (4099, 8), (100_001, 33),
                                 (1, 13), (7, 16), (8, 17), (4103, 20), (70_005, 29), (100_001, 32)])
def test_decode_average(ctx, d, M):
    g = inputs.optimizer_only_gradients(d, M, t=2, seed=5)
    ref = O.quantize_workers(g, O.QUANT_THRESHOLD)
    codes = U.to_dev(ref["codes"].view(np.int32))
    scales = U.to_dev(ref["scales"])
    gbar = torch.full((d,), 7.0, dtype=torch.float32, device=U.dev())
    ctx.decode_average(codes, scales, d, M, gbar)
    assert ctx.last_async_status() == libqasg.OK
    U.assert_close(gbar, O.decode_average(ref["terns"], ref["scales"]), "gbar")


def test_invalid_code_is_reported_and_decodes_to_zero(ctx):
    d, M = 64, 2
    words = np.zeros((M, 4), dtype=np.uint32)
    words[0, 0] = 0b11 | (0b01 << 2)          # coordinate 0 invalid, coordinate 1 = +1
    gbar = torch.zeros(d, dtype=torch.float32, device=U.dev())
    ctx.decode_average(U.to_dev(words.view(np.int32)), U.to_dev(np.array([2.0, 4.0], np.float32)), d, M, gbar)
    assert ctx.last_async_status() == libqasg.ERR_BAD_CODE
    out = gbar.cpu().numpy()
    assert out[0] == 0.0 and out[1] == 1.0 and not out[2:].any()


@pytest.mark.parametrize("M", [13, 16, 29, 32])
def test_invalid_codes_among_many_workers(ctx, M):
    """13 to 32 workers are decoded eight coordinates at a time through radix-3 tables, where a code
    value 3 is not a digit: it must still decode to 0, be reported, and leave every other worker's
    and coordinate's contribution as it is."""
    d = 8 * 512 * 3 + 5
    rng = np.random.default_rng(M)
    tern = rng.integers(-1, 2, size=(M, d)).astype(np.int8)
    scales = (1.0 + rng.random(M)).astype(np.float32)
    words = np.stack([O.pack_codes(tern[m]) for m in range(M)])
    hit = [(0, 0), (M - 1, 9), (M // 2, 4100), (3, d - 1), (M - 2, d - 1)]   # (worker, coordinate)
    for m, i in hit:
        words[m, i >> 4] |= np.uint32(3) << np.uint32(2 * (i & 15))
        tern[m, i] = 0
    gbar = torch.full((d,), 7.0, dtype=torch.float32, device=U.dev())
    ctx.decode_average(U.to_dev(words.view(np.int32)), U.to_dev(scales), d, M, gbar)
    assert ctx.last_async_status() == libqasg.ERR_BAD_CODE
    U.assert_close(gbar, O.decode_average(tern, scales), "gbar")


# ------------------------------------------------------------------ dense updates
@pytest.mark.parametrize("d", [1, 3, 4, 4098, 100_003])
def test_cmd_and_rda_step_from_dense_q(ctx, d):
    rng = np.random.default_rng(d)
    q = (rng.standard_normal(d) * 1e-2).astype(np.float32)
    q[::7] = 0.0
    x0, h0, z0 = (v.numpy() for v in inputs.random_state(d, seed=d))
    h0[::5] = 0.0
    params = libqasg.make_params(LAM, ETA, DELTA)
    x, h = U.to_dev(x0), U.to_dev(h0)
    ctx.cmd_step(U.to_dev(q), x, h, d, 3, params)
    xr, hr, a = O.cmd_step(q, x0, h0, LAM, ETA, DELTA)
    U.assert_close(x, xr, "x cmd"), U.assert_close(h, hr, "h cmd")
    U.assert_zero_pattern(x, xr, a, LAM)
    t = 16
    x, h, z = torch.full((d,), 9.0, dtype=torch.float32, device=U.dev()), U.to_dev(h0), U.to_dev(z0 * t * 0.01)
    ctx.rda_step(U.to_dev(q), x, h, z, d, t, params)
    xr, hr, zr, a = O.rda_step(q, h0, z0 * np.float32(t * 0.01), t, LAM, ETA, DELTA)
    U.assert_close(x, xr, "x rda"), U.assert_close(h, hr, "h rda"), U.assert_close(z, zr, "z rda")
    U.assert_zero_pattern(x, xr, a, LAM)
    assert d < 100 or ((xr == 0).any() and (xr != 0).any())


# ------------------------------------------------------------------ the fused step
@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
@pytest.mark.parametrize("quantizer", [libqasg.Q_THRESHOLD, libqasg.Q_TERNARY_STOCH])
def test_optimizer_only_run_100_steps(ctx, rule, quantizer):
    """d = 10,000, M = 4, g ~ N(0,1)(1+0.1m), x = h = z = 0, 100 steps.

    The oracle runs its own fp64 trajectory.  After every step two GPU results are checked:
    (a) one step taken from the oracle's previous state rounded to fp32 - strict tolerance;
    (b) the GPU's own free-running fp32 trajectory - the same tolerance widened by the drift
        fp32 storage allows: a state that has been as large as s carries a rounding error of
        2^-24 * s per step whatever its present size, so after t steps the absolute term
        grows by 2^-23 * sqrt(t) * (largest |state| so far).
    """
    d, M, T, seed = 10_000, 4, 100, 0
    params = libqasg.make_params(LAM, ETA, DELTA, quantizer=quantizer, seed=seed)
    free = [torch.zeros(d, dtype=torch.float32, device=U.dev()) for _ in range(3)]
    xr, hr, zr = np.zeros(d), np.zeros(d), np.zeros(d)
    peak = {"x": 0.0, "h": 0.0, "z": 0.0}
    names = ("x", "h", "z") if rule == libqasg.RULE_RDA else ("x", "h")
    for t in range(1, T + 1):
        g = inputs.optimizer_only_gradients(d, M, t, seed=seed)
        g_dev, ld = U.grad_to_dev(g)
        driven = [U.to_dev(v.astype(np.float32)) for v in (xr, hr, zr)]
        ref = O.step(rule, g, xr, hr, zr, t, LAM, ETA, DELTA, quantizer=quantizer, seed=seed)
        z_prev = zr
        xr, hr = ref["x"], ref["h"]
        zr = ref["z"] if rule == libqasg.RULE_RDA else zr
        want = {"x": xr, "h": hr, "z": zr}
        # (a) driven by the oracle's state
        codes = U.new_codes(M, d)
        scales = torch.zeros(M, dtype=torch.float32, device=U.dev())
        ctx.step(rule, g_dev, d, ld, M, t, params, *driven, codes_out=codes, scales_out=scales)
        assert np.array_equal(U.codes_np(codes), ref["quant"]["codes"]), t
        assert np.array_equal(U.f32_bits(scales), U.f32_bits(ref["quant"]["scales"])), t
        # z_prev and q enter z = z_prev + q rounded to fp32 and may cancel: that sum is as exact as
        # its operands, 2^-24 of each, whatever is left of them
        slack = {"x": U.ATOL, "h": U.ATOL, "z": U.ATOL + 2.0 ** -23 * (np.abs(z_prev) + np.abs(ref["q"]))}
        for name, got in zip(names, driven):
            U.assert_close(got, want[name], "%s step %d (driven)" % (name, t), atol=slack[name])
        U.assert_zero_pattern(driven[0], xr, ref["a"], LAM)
        # (b) free running
        ctx.step(rule, g_dev, d, ld, M, t, params, *free)
        for name, got in zip(names, free):
            peak[name] = max(peak[name], float(np.abs(want[name]).max()))
            U.assert_close(got, want[name], "%s step %d (free)" % (name, t),
                           atol=U.ATOL + 2.0 ** -23 * np.sqrt(t) * peak[name])
    assert ctx.last_async_status() == libqasg.OK
    assert np.count_nonzero(xr) > 0


@pytest.mark.parametrize("d,M", [(1 << 20, 2), (1 << 20, 4), (1 << 20, 8), (1 << 20, 16), (1 << 20, 32),
                                 (1 << 22, 2), (1 << 22, 8), ((1 << 20) + 4099, 3)])
@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
def test_sweep_one_step(ctx, d, M, rule):
    g = inputs.normal_gradients(d, M, seed=4).numpy()
    x0, h0, z0 = (v.numpy() for v in inputs.random_state(d, seed=4))
    g_dev, ld = U.grad_to_dev(g)
    x, h, z = U.to_dev(x0), U.to_dev(h0), U.to_dev(z0)
    params = libqasg.make_params(LAM, ETA, DELTA)
    ctx.step(rule, g_dev, d, ld, M, 16, params, x, h, z)        # codes in the context's scratch
    ref = O.step(rule, g, x0, h0, z0, 16, LAM, ETA, DELTA)
    U.assert_close(x, ref["x"], "x"), U.assert_close(h, ref["h"], "h")
    if rule == libqasg.RULE_RDA:
        U.assert_close(z, ref["z"], "z")
    else:
        assert np.array_equal(z.cpu().numpy(), z0)
    U.assert_zero_pattern(x, ref["x"], ref["a"], LAM)


@pytest.mark.parametrize("M", [1, 5, 9, 12, 13, 16, 28, 31, 52, 53, 64])
@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
def test_fused_step_worker_counts(ctx, M, rule):
    # every dispatch of the decode: per-lane tables (M <= 12), shared tables, short last group
    d = 70_003
    g = inputs.optimizer_only_gradients(d, M, t=3, seed=M) * np.float32(0.01)
    x0, h0, z0 = (v.numpy() for v in inputs.random_state(d, seed=M))
    g_dev, ld = U.grad_to_dev(g)
    x, h, z = U.to_dev(x0), U.to_dev(h0), U.to_dev(z0)
    codes = U.new_codes(M, d)
    ctx.step(rule, g_dev, d, ld, M, 3, libqasg.make_params(LAM, ETA, DELTA), x, h, z, codes_out=codes)
    assert ctx.last_async_status() == libqasg.OK
    ref = O.step(rule, g, x0, h0, z0, 3, LAM, ETA, DELTA)
    assert np.array_equal(U.codes_np(codes), ref["quant"]["codes"])
    U.assert_close(x, ref["x"], "x"), U.assert_close(h, ref["h"], "h")
    if rule == libqasg.RULE_RDA:
        U.assert_close(z, ref["z"], "z")
    U.assert_zero_pattern(x, ref["x"], ref["a"], LAM)


@pytest.mark.parametrize("d,M", [(4097, 3), (70_003, 8), (30_000, 13)])
@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
def test_fused_step_gives_the_bits_of_the_unfused_sequence(ctx, d, M, rule):
    """qasg_step against quantize_pack -> decode_average -> cmd_step / rda_step: same arithmetic, other kernels."""
    t = 7
    g = inputs.optimizer_only_gradients(d, M, t, seed=d + M) * np.float32(0.02)
    x0, h0, z0 = (v.numpy() for v in inputs.random_state(d, seed=M))
    params = libqasg.make_params(LAM, ETA, DELTA)
    g_dev, ld = U.grad_to_dev(g)
    x, h, z = U.to_dev(x0), U.to_dev(h0), U.to_dev(z0)
    codes, scales = U.new_codes(M, d), torch.zeros(M, dtype=torch.float32, device=U.dev())
    ctx.step(rule, g_dev, d, ld, M, t, params, x, h, z, codes_out=codes, scales_out=scales)
    codes2, scales2 = U.new_codes(M, d), torch.zeros(M, dtype=torch.float32, device=U.dev())
    ctx.quantize_pack(g_dev, d, ld, M, t, params, codes2, scales2)
    gbar = torch.zeros((d + 3) // 4 * 4, dtype=torch.float32, device=U.dev())
    ctx.decode_average(codes2, scales2, d, M, gbar)
    x2, h2, z2 = U.to_dev(x0), U.to_dev(h0), U.to_dev(z0)
    if rule == libqasg.RULE_CMD:
        ctx.cmd_step(gbar, x2, h2, d, t, params)
    else:
        ctx.rda_step(gbar, x2, h2, z2, d, t, params)
    assert np.array_equal(U.codes_np(codes), U.codes_np(codes2))
    assert np.array_equal(U.f32_bits(scales), U.f32_bits(scales2))
    for a, b in ((x, x2), (h, h2), (z, z2)):
        assert np.array_equal(U.f32_bits(a), U.f32_bits(b))


def test_step_host_matches_step(ctx):
    d, M, t = 50_003, 4, 5
    g = inputs.optimizer_only_gradients(d, M, t, seed=1)
    ld = (d + 3) // 4 * 4
    gh = torch.zeros((M, ld), dtype=torch.float32).pin_memory()
    gh[:, :d] = torch.from_numpy(g)
    x0, h0, z0 = inputs.random_state(d, seed=1)
    params = libqasg.make_params(LAM, ETA, DELTA)
    for rule in (libqasg.RULE_CMD, libqasg.RULE_RDA):
        xh, hh, zh = (v.clone().pin_memory() for v in (x0, h0, z0))
        g_dev = torch.empty((M, ld), dtype=torch.float32, device=U.dev())
        xd, hd, zd = (torch.empty(d, dtype=torch.float32, device=U.dev()) for _ in range(3))
        ctx.step_host(rule, gh, d, ld, M, t, params, xh, hh, zh, g_dev, xd, hd, zd)
        torch.cuda.synchronize()
        ref = O.step(rule, g, x0.numpy(), h0.numpy(), z0.numpy(), t, LAM, ETA, DELTA)
        U.assert_close(xh, ref["x"], "x"), U.assert_close(hh, ref["h"], "h")
        if rule == libqasg.RULE_RDA:
            U.assert_close(zh, ref["z"], "z")


# ------------------------------------------------------------------ argument errors on a live context
def test_argument_errors(ctx):
    d, M = 1000, 2
    g = torch.zeros((M, d + 8), dtype=torch.float32, device=U.dev())
    x, h = (torch.zeros(d + 4, dtype=torch.float32, device=U.dev()) for _ in range(2))
    params = libqasg.make_params(LAM, ETA, DELTA)
    before = ctx.launch_count()

    def status_of(call):
        with pytest.raises(libqasg.QasgError) as e:
            call()
        return e.value.status

    assert status_of(lambda: ctx.step(0, g, d, d + 6, M, 1, params, x, h)) == libqasg.ERR_ALIGNMENT      # ld % 4
    assert status_of(lambda: ctx.step(0, g.data_ptr() + 4, d, d + 8, M, 1, params, x, h)) == libqasg.ERR_ALIGNMENT
    assert status_of(lambda: ctx.step(0, g, d, d - 4, M, 1, params, x, h)) == libqasg.ERR_INVALID_ARG    # ld < d
    assert status_of(lambda: ctx.step(1, g, d, d + 8, M, 1, params, x, h, None)) == libqasg.ERR_INVALID_ARG  # RDA, no z
    assert status_of(lambda: ctx.step(0, g, d, d + 8, M, 0, params, x, h)) == libqasg.ERR_INVALID_ARG    # t = 0
    assert status_of(lambda: ctx.step(0, g, 7_000_000, 7_000_000, M, 1, params, x, h)) == libqasg.ERR_WORKSPACE
    assert status_of(lambda: ctx.step(0, g, d, d + 8, 65, 1, params, x, h)) == libqasg.ERR_INVALID_ARG
    bad = libqasg.make_params(LAM, ETA, 0.0)
    assert status_of(lambda: ctx.step(0, g, d, d + 8, M, 1, bad, x, h)) == libqasg.ERR_INVALID_ARG       # delta = 0
    bad = libqasg.make_params(-1.0, ETA, DELTA)
    assert status_of(lambda: ctx.step(0, g, d, d + 8, M, 1, bad, x, h)) == libqasg.ERR_INVALID_ARG
    assert ctx.launch_count() == before                                                              # nothing enqueued
    no_scratch = libqasg.Context(1000, 2, flags=libqasg.CREATE_NO_CODE_SCRATCH)
    with pytest.raises(libqasg.QasgError) as e:
        no_scratch.step(0, g, d, d + 8, M, 1, params, x, h)
    assert e.value.status == libqasg.ERR_WORKSPACE
    no_scratch.close()
