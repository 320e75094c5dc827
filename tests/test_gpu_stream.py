"""The one-launch quantizer (an option: a row coded out of L2 right after it was summed) against the oracle
and against the default two-launch path, over row counts, lags and chunk shapes; and its bounded waits."""
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
    c = libqasg.Context(1 << 23, 64, device=0)
    yield c
    c.close()


def _quantize(ctx, g_dev, ld, M, d, quantizer, t, seed):
    codes = U.new_codes(M, d)
    scales = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    thresholds = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    counts = torch.full((M,), -1, dtype=torch.int64, device=U.dev())
    params = libqasg.make_params(LAM, ETA, DELTA, quantizer=quantizer, seed=seed)
    before = ctx.launch_count()
    ctx.quantize_pack(g_dev, d, ld, M, t, params, codes, scales, thresholds, counts)
    launches = ctx.launch_count() - before
    assert ctx.last_async_status() == libqasg.OK
    return dict(codes=U.codes_np(codes), scales=scales.cpu().numpy(), thresholds=thresholds.cpu().numpy(),
                counts=counts.cpu().numpy()), launches


def _same(a, b):
    assert np.array_equal(a["codes"], b["codes"])
    assert np.array_equal(U.f32_bits(a["scales"]), U.f32_bits(b["scales"]))
    assert np.array_equal(U.f32_bits(a["thresholds"]), U.f32_bits(b["thresholds"]))
    assert np.array_equal(a["counts"], b["counts"])


@pytest.mark.parametrize("quantizer", [libqasg.Q_THRESHOLD, libqasg.Q_TERNARY_STOCH])
@pytest.mark.parametrize("d,M", [(1, 1), (17, 3), (4097, 1), (70_001, 8), (300_007, 5), (5_000_001, 2),
                                 (1 << 20, 16), (9001, 64)])
def test_one_launch_equals_two_launches_and_the_oracle(ctx, d, M, quantizer):
    t, seed = 7, 12345
    rng = np.random.default_rng(d + M)
    g = rng.standard_normal((M, d)).astype(np.float32) * (1.0 + 0.1 * np.arange(M, dtype=np.float32))[:, None]
    if M > 2:
        g[2] = 0.0                      # a zero gradient among the workers
    g_dev, ld = U.grad_to_dev(g)
    ref = O.quantize_workers(g, quantizer, t=t, seed=seed)
    ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, 0)
    two, launches = _quantize(ctx, g_dev, ld, M, d, quantizer, t, seed)
    assert launches == 2
    _same(two, ref)
    ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, 64 << 20)
    for lag in (libqasg.LAG_AUTO, 0, 1, 2, 64):
        ctx.set_option(libqasg.OPT_STREAM_LAG, lag)
        one, launches = _quantize(ctx, g_dev, ld, M, d, quantizer, t, seed)
        assert launches == 1
        _same(one, ref)
    ctx.set_option(libqasg.OPT_STREAM_LAG, libqasg.LAG_AUTO)
    ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, 0)


def test_repeated_calls_reuse_the_synchronisation_words(ctx):
    # every slot and word is back in its initial state when a call completes: nothing is reset between calls
    ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, 64 << 20)
    d, M = 200_003, 8
    for rep in range(20):
        g = inputs.optimizer_only_gradients(d, M, rep + 1, seed=3)
        g_dev, ld = U.grad_to_dev(g)
        got, launches = _quantize(ctx, g_dev, ld, M, d, libqasg.Q_THRESHOLD, rep + 1, 0)
        assert launches == 1
        _same(got, O.quantize_workers(g, O.QUANT_THRESHOLD))
    ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, 0)


def test_nonfinite_gradient_in_one_launch(ctx):
    ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, 64 << 20)
    g = np.ones((3, 50_000), dtype=np.float32)
    g[1, 4321] = np.nan
    g_dev, ld = U.grad_to_dev(g)
    codes, scales = U.new_codes(3, 50_000), torch.zeros(3, dtype=torch.float32, device=U.dev())
    ctx.quantize_pack(g_dev, 50_000, ld, 3, 1, libqasg.make_params(), codes, scales)
    assert ctx.last_async_status() == libqasg.ERR_NONFINITE
    ref = O.quantize_workers(g, O.QUANT_THRESHOLD)
    assert np.array_equal(U.codes_np(codes), ref["codes"]) and not U.codes_np(codes)[1].any()
    ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, 0)


@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
def test_fused_step_through_both_quantizer_paths(ctx, rule):
    d, M, t = (1 << 21) + 4099, 4, 16
    g = inputs.normal_gradients(d, M, seed=4).numpy()
    x0, h0, z0 = (v.numpy() for v in inputs.random_state(d, seed=4))
    g_dev, ld = U.grad_to_dev(g)
    params = libqasg.make_params(LAM, ETA, DELTA)
    out = []
    for row_bytes in (0, 64 << 20):
        ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, row_bytes)
        x, h, z = U.to_dev(x0), U.to_dev(h0), U.to_dev(z0)
        before = ctx.launch_count()
        ctx.step(rule, g_dev, d, ld, M, t, params, x, h, z)
        assert ctx.launch_count() - before == (3 if row_bytes == 0 else 2)
        out.append((x, h, z))
    assert ctx.last_async_status() == libqasg.OK
    for a, b in zip(*out):
        assert torch.equal(a, b)
    ref = O.step(rule, g, x0, h0, z0, t, LAM, ETA, DELTA)
    U.assert_close(out[1][0], ref["x"], "x"), U.assert_close(out[1][1], ref["h"], "h")
    U.assert_zero_pattern(out[1][0], ref["x"], ref["a"], LAM)
    ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, 0)


def test_a_wait_that_nothing_ends_gives_up(ctx):
    """The bounded wait on a word no one sets: the kernel returns by itself, the status reports the
    time-out once, and the context keeps working."""
    ctx.wait_selftest(2000)
    torch.cuda.synchronize()
    assert ctx.last_async_status() == libqasg.ERR_TIMEOUT
    assert ctx.last_async_status() == libqasg.OK
    d, M = 70_001, 4
    g = inputs.optimizer_only_gradients(d, M, 1, seed=1)
    g_dev, ld = U.grad_to_dev(g)
    ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, 64 << 20)
    got, launches = _quantize(ctx, g_dev, ld, M, d, libqasg.Q_THRESHOLD, 1, 0)
    assert launches == 1
    _same(got, O.quantize_workers(g, O.QUANT_THRESHOLD))
    ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, 0)
    ctx.wait_selftest(1)
    assert ctx.last_async_status() == libqasg.ERR_TIMEOUT


def test_option_values_are_checked(ctx):
    def status_of(call):
        with pytest.raises(libqasg.QasgError) as e:
            call()
        return e.value.status

    assert status_of(lambda: ctx.set_option(libqasg.OPT_STREAM_LAG, 65)) == libqasg.ERR_INVALID_ARG
    assert status_of(lambda: ctx.set_option(libqasg.OPT_WAIT_POLLS, 0)) == libqasg.ERR_INVALID_ARG
    assert status_of(lambda: ctx.set_option(7, 1)) == libqasg.ERR_INVALID_ARG
    assert status_of(lambda: ctx.wait_selftest(0)) == libqasg.ERR_INVALID_ARG
    ctx.set_option(libqasg.OPT_WAIT_POLLS, 1 << 22)
