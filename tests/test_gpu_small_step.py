"""The single-launch fused step used for dimensions of a few tiles: against the oracle, and bit for bit
against the unfused sequence quantize_pack -> decode_average -> cmd_step / rda_step (same arithmetic, other
kernels)."""
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
    c = libqasg.Context(1 << 15, 64, device=0)
    yield c
    c.close()


@pytest.mark.parametrize("d", [1, 5, 4095, 4096, 4097, 3 * 4096 + 1, 4 * 4096])
@pytest.mark.parametrize("M", [1, 3, 8, 17, 64])
@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
def test_single_launch_step(ctx, d, M, rule):
    t = 7
    g = inputs.optimizer_only_gradients(d, M, t, seed=d + M) * np.float32(0.02)
    x0, h0, z0 = (v.numpy() for v in inputs.random_state(d, seed=M))
    params = libqasg.make_params(LAM, ETA, DELTA)
    g_dev, ld = U.grad_to_dev(g)
    x, h, z = U.to_dev(x0), U.to_dev(h0), U.to_dev(z0)
    codes = U.new_codes(M, d)
    scales = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    before = ctx.launch_count()
    ctx.step(rule, g_dev, d, ld, M, t, params, x, h, z, codes_out=codes, scales_out=scales)
    assert ctx.launch_count() == before + 1                      # one kernel
    assert ctx.last_async_status() == libqasg.OK
    ref = O.step(rule, g, x0, h0, z0, t, LAM, ETA, DELTA)
    assert np.array_equal(U.codes_np(codes), ref["quant"]["codes"])
    assert np.array_equal(U.f32_bits(scales), U.f32_bits(ref["quant"]["scales"]))
    U.assert_close(x, ref["x"], "x"), U.assert_close(h, ref["h"], "h")
    if rule == libqasg.RULE_RDA:
        U.assert_close(z, ref["z"], "z", atol=U.ATOL + 2.0 ** -23 * (np.abs(z0) + np.abs(ref["q"])))
    U.assert_zero_pattern(x, ref["x"], ref["a"], LAM)
    # the unfused sequence gives the same bits
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
    assert np.array_equal(U.f32_bits(x), U.f32_bits(x2)) and np.array_equal(U.f32_bits(h), U.f32_bits(h2))
    assert np.array_equal(U.f32_bits(z), U.f32_bits(z2))


def test_larger_dimensions_and_the_stochastic_quantizer_take_three_launches(ctx):
    M, t = 4, 2
    for d, quantizer, launches in ((4 * 4096 + 1, libqasg.Q_THRESHOLD, 3), (4096, libqasg.Q_TERNARY_STOCH, 3)):
        g_dev, ld = U.grad_to_dev(inputs.optimizer_only_gradients(d, M, t, seed=1))
        x, h, z = (torch.zeros(d, dtype=torch.float32, device=U.dev()) for _ in range(3))
        before = ctx.launch_count()
        ctx.step(libqasg.RULE_RDA, g_dev, d, ld, M, t, libqasg.make_params(LAM, ETA, DELTA, quantizer=quantizer), x, h, z)
        assert ctx.launch_count() == before + launches


def test_invalid_values_are_reported(ctx):
    d, M = 5000, 2
    g = np.zeros((M, d), dtype=np.float32)
    g[1, 77] = np.inf
    g_dev, ld = U.grad_to_dev(g)
    x, h, z = (torch.zeros(d, dtype=torch.float32, device=U.dev()) for _ in range(3))
    ctx.step(libqasg.RULE_CMD, g_dev, d, ld, M, 1, libqasg.make_params(LAM, ETA, DELTA), x, h, z)
    assert ctx.last_async_status() == libqasg.ERR_NONFINITE
