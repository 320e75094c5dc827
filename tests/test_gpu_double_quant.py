"""GPU parity of double quantization (q_t = Q(SynQ_t), Algorithm 1 as printed) against the oracle:
the server's codes, scale, threshold and count bit for bit; the iterates within tolerance."""
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


@pytest.fixture(scope="module")
def ctx_no_scratch():
    # without scratch the server row is rebuilt from the code bytes twice instead of being stored once
    c = libqasg.Context(6_000_000, 64, device=0, flags=libqasg.CREATE_NO_CODE_SCRATCH)
    yield c
    c.close()


def _requantize_gpu(ctx, quant, d, M, quantizer, t, seed):
    codes = U.to_dev(quant["codes"].view(np.int32))
    scales = U.to_dev(quant["scales"])
    qcodes = U.new_codes(1, d)
    qscale = torch.full((1,), -1.0, dtype=torch.float32, device=U.dev())
    qthr = torch.full((1,), -1.0, dtype=torch.float32, device=U.dev())
    qcnt = torch.full((1,), -1, dtype=torch.int64, device=U.dev())
    params = libqasg.make_params(LAM, ETA, DELTA, quantizer=quantizer, seed=seed)
    ctx.requantize(codes, scales, d, M, t, params, qcodes, qscale, qthr, qcnt)
    assert ctx.last_async_status() == libqasg.OK
    return U.codes_np(qcodes)[0], qscale.cpu().numpy()[0], qthr.cpu().numpy()[0], int(qcnt.cpu().numpy()[0])


@pytest.mark.parametrize("d,M", [(1, 1), (17, 3), (4097, 8), (70_003, 5), (300_001, 16), (5_000_001, 2)])
@pytest.mark.parametrize("quantizer", [libqasg.Q_THRESHOLD, libqasg.Q_TERNARY_STOCH])
@pytest.mark.parametrize("stored", [True, False])
def test_requantize_bit_exact(ctx, ctx_no_scratch, d, M, quantizer, stored):
    ctx = ctx if stored else ctx_no_scratch
    t, seed = 9, 77
    g = inputs.normal_gradients(d, M, seed=d % 1000).numpy() * np.float32(0.05)
    quant = O.quantize_workers(g, quantizer, t=t, seed=seed)
    ref = O.requantize(O.decode_average(quant["terns"], quant["scales"]), quantizer, t=t, seed=seed)
    codes, scale, thr, cnt = _requantize_gpu(ctx, quant, d, M, quantizer, t, seed)
    assert np.array_equal(codes, ref["codes"])
    assert np.float32(scale).view(np.uint32) == ref["scale"].view(np.uint32)
    assert np.float32(thr).view(np.uint32) == ref["threshold"].view(np.uint32)
    assert cnt == ref["count"]


def test_requantizing_one_worker_returns_its_message(ctx):
    # Q(Q(v)) = Q(v)
    d = 50_001
    g = inputs.normal_gradients(d, 1, seed=3).numpy()
    quant = O.quantize_workers(g, O.QUANT_THRESHOLD)
    codes, scale, _, cnt = _requantize_gpu(ctx, quant, d, 1, libqasg.Q_THRESHOLD, 1, 0)
    assert np.array_equal(codes, quant["codes"][0]) and scale == quant["scales"][0] and cnt == quant["counts"][0]


@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
@pytest.mark.parametrize("quantizer", [libqasg.Q_THRESHOLD, libqasg.Q_TERNARY_STOCH])
def test_double_quantized_run_40_steps(ctx, rule, quantizer):
    """Oracle-driven and free-running, as in the one-way 100-step test."""
    d, M, T, seed = 10_000, 4, 40, 0
    params = libqasg.make_params(LAM, ETA, DELTA, quantizer=quantizer, seed=seed)
    free = [torch.zeros(d, dtype=torch.float32, device=U.dev()) for _ in range(3)]
    xr, hr, zr = np.zeros(d), np.zeros(d), np.zeros(d)
    peak = {"x": 0.0, "h": 0.0, "z": 0.0}
    names = ("x", "h", "z") if rule == libqasg.RULE_RDA else ("x", "h")
    for t in range(1, T + 1):
        g = inputs.optimizer_only_gradients(d, M, t, seed=seed)
        g_dev, ld = U.grad_to_dev(g)
        driven = [U.to_dev(v.astype(np.float32)) for v in (xr, hr, zr)]
        ref = O.step(rule, g, xr, hr, zr, t, LAM, ETA, DELTA, quantizer=quantizer, seed=seed, double_quant=True)
        z_prev = zr
        xr, hr = ref["x"], ref["h"]
        zr = ref["z"] if rule == libqasg.RULE_RDA else zr
        want = {"x": xr, "h": hr, "z": zr}
        codes, qcodes = U.new_codes(M, d), U.new_codes(1, d)
        qscale = torch.zeros(1, dtype=torch.float32, device=U.dev())
        ctx.step_double(rule, g_dev, d, ld, M, t, params, *driven, codes_out=codes, qcodes_out=qcodes,
                        qscale_out=qscale)
        assert np.array_equal(U.codes_np(codes), ref["quant"]["codes"]), t
        assert np.array_equal(U.codes_np(qcodes)[0], ref["requant"]["codes"]), t
        assert qscale.cpu().numpy()[0].view(np.uint32) == ref["requant"]["scale"].view(np.uint32), t
        slack = {"x": U.ATOL, "h": U.ATOL, "z": U.ATOL + 2.0 ** -23 * (np.abs(z_prev) + np.abs(ref["q"]))}
        for name, got in zip(names, driven):
            U.assert_close(got, want[name], "%s step %d (driven)" % (name, t), atol=slack[name])
        U.assert_zero_pattern(driven[0], xr, ref["a"], LAM)
        ctx.step_double(rule, g_dev, d, ld, M, t, params, *free)          # scratch for both code sets
        for name, got in zip(names, free):
            peak[name] = max(peak[name], float(np.abs(want[name]).max()))
            U.assert_close(got, want[name], "%s step %d (free)" % (name, t),
                           atol=U.ATOL + 2.0 ** -23 * np.sqrt(t) * peak[name])
    assert ctx.last_async_status() == libqasg.OK


def test_double_quantized_step_many_chunks(ctx):
    # 1221 tiles: the server row uses more than 1024 chunk partials
    d, M = 5_000_001, 3
    g = inputs.normal_gradients(d, M, seed=8).numpy() * np.float32(0.01)
    x0, h0, z0 = (v.numpy() for v in inputs.random_state(d, seed=8))
    x, h, z = U.to_dev(x0), U.to_dev(h0), U.to_dev(z0)
    g_dev, ld = U.grad_to_dev(g)
    ctx.step_double(libqasg.RULE_RDA, g_dev, d, ld, M, 16, libqasg.make_params(LAM, ETA, DELTA), x, h, z)
    ref = O.step(O.RULE_RDA, g, x0, h0, z0, 16, LAM, ETA, DELTA, double_quant=True)
    U.assert_close(x, ref["x"], "x"), U.assert_close(h, ref["h"], "h")
    U.assert_close(z, ref["z"], "z", atol=U.ATOL + 2.0 ** -23 * (np.abs(z0) + np.abs(ref["q"])))
    U.assert_zero_pattern(x, ref["x"], ref["a"], LAM)
