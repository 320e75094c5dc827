"""The fused step as ONE launch (an option for small problems: passes A, B, C as phases of a launch whose
CTAs meet twice) against the three-launch path, bit for bit, and against the oracle."""
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
    c = libqasg.Context(1 << 22, 64, device=0)
    yield c
    c.close()


def _step(ctx, rule, g_dev, ld, M, d, t, params, state0, one_launch):
    ctx.set_option(libqasg.OPT_ONE_LAUNCH_STEP_BYTES, (1 << 40) if one_launch else 0)
    x, h, z = (U.to_dev(v) for v in state0)
    codes = U.new_codes(M, d)
    scales = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    before = ctx.launch_count()
    ctx.step(rule, g_dev, d, ld, M, t, params, x, h, z, codes, scales)
    launches = ctx.launch_count() - before
    assert ctx.last_async_status() == libqasg.OK
    return dict(x=x, h=h, z=z, codes=U.codes_np(codes), scales=scales.cpu().numpy()), launches


@pytest.mark.parametrize("quantizer", [libqasg.Q_THRESHOLD, libqasg.Q_TERNARY_STOCH])
@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
@pytest.mark.parametrize("d,M", [(1, 1), (3, 2), (4097, 1), (10_000, 4), (70_001, 8), (300_007, 5), (9001, 64),
                                 (1 << 20, 8), (3_000_001, 3)])
def test_one_launch_equals_three_launches_and_the_oracle(ctx, d, M, rule, quantizer):
    t, seed = 9, 4242
    rng = np.random.default_rng(d * 131 + M)
    g = rng.standard_normal((M, d)).astype(np.float32) * (1.0 + 0.1 * np.arange(M, dtype=np.float32))[:, None]
    if M > 2:
        g[1] = 0.0
    state0 = [v.numpy() for v in inputs.random_state(d, seed=d % 1000)]
    g_dev, ld = U.grad_to_dev(g)
    params = libqasg.make_params(LAM, ETA, DELTA, quantizer=quantizer, seed=seed)
    three, n3 = _step(ctx, rule, g_dev, ld, M, d, t, params, state0, False)
    one, n1 = _step(ctx, rule, g_dev, ld, M, d, t, params, state0, True)
    ctx.set_option(libqasg.OPT_ONE_LAUNCH_STEP_BYTES, 0)
    assert (n3, n1) == (3, 1)
    assert np.array_equal(one["codes"], three["codes"])
    assert np.array_equal(U.f32_bits(one["scales"]), U.f32_bits(three["scales"]))
    for name in ("x", "h") + (("z",) if rule == libqasg.RULE_RDA else ()):
        assert torch.equal(one[name], three[name]), name
    q = O.quantize_workers(g, quantizer, t=t, seed=seed)
    assert np.array_equal(one["codes"], q["codes"])
    assert np.array_equal(U.f32_bits(one["scales"]), U.f32_bits(q["scales"]))
    ref = O.step(rule, g, *state0, t, LAM, ETA, DELTA, quantizer=quantizer, seed=seed)
    U.assert_close(one["x"], ref["x"], "x"), U.assert_close(one["h"], ref["h"], "h")
    U.assert_zero_pattern(one["x"], ref["x"], ref["a"], LAM)


def test_repeated_one_launch_steps_follow_the_three_launch_run(ctx):
    """Forty steps of a run: the meeting counters are back at zero after every launch, so nothing is reset
    in between; the iterates are those of the three-launch run, bit for bit."""
    d, M, T = 10_000, 4, 40
    params = libqasg.make_params(LAM, ETA, DELTA)
    runs = []
    for one_launch in (False, True):
        ctx.set_option(libqasg.OPT_ONE_LAUNCH_STEP_BYTES, (1 << 40) if one_launch else 0)
        x, h = (torch.zeros(d, dtype=torch.float32, device=U.dev()) for _ in range(2))
        for t in range(1, T + 1):
            g_dev, ld = U.grad_to_dev(inputs.optimizer_only_gradients(d, M, t, seed=3))
            ctx.step(libqasg.RULE_CMD, g_dev, d, ld, M, t, params, x, h, None)
        assert ctx.last_async_status() == libqasg.OK
        runs.append((x, h))
    ctx.set_option(libqasg.OPT_ONE_LAUNCH_STEP_BYTES, 0)
    assert torch.equal(runs[0][0], runs[1][0]) and torch.equal(runs[0][1], runs[1][1])


def test_one_launch_step_replays_from_a_graph(ctx):
    d, M, t = 70_001, 8, 5
    g = inputs.normal_gradients(d, M, seed=6).numpy()
    state0 = [v.numpy() for v in inputs.random_state(d, seed=6)]
    g_dev, ld = U.grad_to_dev(g)
    params = libqasg.make_params(LAM, ETA, DELTA)
    ref, _ = _step(ctx, libqasg.RULE_RDA, g_dev, ld, M, d, t, params, state0, False)
    ctx.set_option(libqasg.OPT_ONE_LAUNCH_STEP_BYTES, 1 << 40)
    x, h, z = (U.to_dev(v) for v in state0)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):                      # warm-up outside the capture
        ctx.step(libqasg.RULE_RDA, g_dev, d, ld, M, t, params, x, h, z)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    for v, v0 in zip((x, h, z), state0):
        v.copy_(torch.from_numpy(v0))
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx.step(libqasg.RULE_RDA, g_dev, d, ld, M, t, params, x, h, z)
    graph.replay()
    torch.cuda.synchronize()
    ctx.set_option(libqasg.OPT_ONE_LAUNCH_STEP_BYTES, 0)
    assert ctx.last_async_status() == libqasg.OK
    for name, v in (("x", x), ("h", h), ("z", z)):
        assert torch.equal(v, ref[name]), name


def test_non_finite_gradient_in_one_launch(ctx):
    ctx.set_option(libqasg.OPT_ONE_LAUNCH_STEP_BYTES, 1 << 40)
    d, M = 50_000, 3
    g = np.ones((M, d), dtype=np.float32)
    g[1, 4321] = np.inf
    g_dev, ld = U.grad_to_dev(g)
    x, h = (torch.zeros(d, dtype=torch.float32, device=U.dev()) for _ in range(2))
    ctx.step(libqasg.RULE_CMD, g_dev, d, ld, M, 1, libqasg.make_params(), x, h, None)
    ctx.set_option(libqasg.OPT_ONE_LAUNCH_STEP_BYTES, 0)
    assert ctx.last_async_status() == libqasg.ERR_NONFINITE


def test_default_takes_one_launch_for_small_problems_only():
    c = libqasg.Context(1 << 20, 8, device=0)
    params = libqasg.make_params(LAM, ETA, DELTA)
    for d, M, want in ((10_000, 4, 1), (70_001, 8, 1), (1 << 19, 8, 1), ((1 << 19) + 4, 8, 3), (1 << 20, 8, 3)):
        g_dev, ld = U.grad_to_dev(inputs.normal_gradients(d, M, seed=1).numpy())
        x, h = (torch.zeros(d, dtype=torch.float32, device=U.dev()) for _ in range(2))
        before = c.launch_count()
        c.step(libqasg.RULE_CMD, g_dev, d, ld, M, 1, params, x, h, None)
        assert c.launch_count() - before == want, (d, M)
    assert c.last_async_status() == libqasg.OK
    c.close()
