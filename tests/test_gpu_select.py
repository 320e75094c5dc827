"""GPU parity of the sparse selection (indicator, Q on the selected coordinates, OR of the indicators)
against the oracle: indicator bits, k_m, codes, thresholds, scales bit for bit; iterates within tolerance."""
import numpy as np
import pytest
import torch

from oracle import qasg_oracle as O
from paper_2208_05631_b200 import inputs, libqasg
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = libqasg.Context(6_000_000, 64, device=0)
    yield c
    c.close()


def _state(d, seed, sparse=0.6):
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal(d) * 0.1 * (rng.random(d) > sparse)).astype(np.float32)
    h = (rng.random(d) * (rng.random(d) < 0.9)).astype(np.float32)
    z = (rng.standard_normal(d) * 0.02).astype(np.float32)
    return x, h, z


@pytest.mark.parametrize("d,M", [(1, 1), (37, 3), (4097, 4), (70_003, 8), (5_000_001, 2)])
@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
@pytest.mark.parametrize("quantizer", [libqasg.Q_THRESHOLD, libqasg.Q_TERNARY_STOCH])
def test_select_quantize_pack_bit_exact(ctx, d, M, rule, quantizer):
    t, seed, lam, eta, delta = 6, 5, 1e-2, 0.1, 1e-8
    g = inputs.normal_gradients(d, M, seed=d % 997).numpy() * np.float32(0.02)
    x, h, z = _state(d, d)
    ref = O.select_quantize_workers(rule, g, x, h, z, t, lam, eta, delta, quantizer, seed=seed)
    g_dev, ld = U.grad_to_dev(g)
    words = (d + 31) // 32
    codes = U.new_codes(M, d)
    ind = torch.full((M, words), 0x55555555, dtype=torch.int32, device=U.dev())
    scales = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    thr = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    cnt = torch.full((M,), -1, dtype=torch.int64, device=U.dev())
    sel = torch.full((M,), -1, dtype=torch.int64, device=U.dev())
    params = libqasg.make_params(lam, eta, delta, quantizer=quantizer, seed=seed)
    ctx.select_quantize_pack(rule, g_dev, d, ld, M, t, params, U.to_dev(x), U.to_dev(h), U.to_dev(z), codes, scales,
                             thr, cnt, ind, sel)
    assert ctx.last_async_status() == libqasg.OK
    assert np.array_equal(ind.cpu().numpy().view(np.uint32), ref["ind_words"])
    assert np.array_equal(sel.cpu().numpy(), ref["selected"])
    assert np.array_equal(U.codes_np(codes), ref["codes"])
    assert np.array_equal(U.f32_bits(thr), U.f32_bits(ref["thresholds"]))
    assert np.array_equal(U.f32_bits(scales), U.f32_bits(ref["scales"]))
    assert np.array_equal(cnt.cpu().numpy(), ref["counts"])
    isyn = torch.zeros(words, dtype=torch.int32, device=U.dev())
    ksyn = torch.full((1,), -1, dtype=torch.int64, device=U.dev())
    ctx.indicator_or(ind, d, M, isyn, ksyn)
    assert np.array_equal(isyn.cpu().numpy().view(np.uint32), O.pack_bits(ref["isyn"]))
    assert int(ksyn.cpu().numpy()[0]) == int(ref["isyn"].sum())
    if d > 1000:
        assert 0 < ref["selected"].min() and ref["selected"].max() < d        # a real selection


@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
@pytest.mark.parametrize("double_quant", [False, True])
def test_selected_run_40_steps(ctx, rule, double_quant):
    """lambda large enough that many coordinates stay zero: the regime the selection is made for.
    Every step starts from the oracle's state rounded to fp32 (the indicator is a discrete decision:
    a free-running fp32 trajectory may legitimately select another coordinate at the boundary)."""
    d, M, T, lam, eta, delta = 10_000, 4, 40, 1.5, 0.1, 1e-8
    params = libqasg.make_params(lam, eta, delta)
    xr, hr, zr = np.zeros(d), np.zeros(d), np.zeros(d)
    names = ("x", "h", "z") if rule == libqasg.RULE_RDA else ("x", "h")
    words = (d + 31) // 32
    ksum = 0
    for t in range(1, T + 1):
        g = inputs.optimizer_only_gradients(d, M, t, seed=3)
        g_dev, ld = U.grad_to_dev(g)
        state32 = [v.astype(np.float32) for v in (xr, hr, zr)]
        driven = [U.to_dev(v) for v in state32]
        # the oracle steps from the same fp32 state the GPU is given: the indicator is decided in fp32
        ref = O.step(rule, g, *state32, t, lam, eta, delta, double_quant=double_quant, select=True)
        z_prev = state32[2].astype(np.float64)
        xr, hr = ref["x"], ref["h"]
        zr = ref["z"] if rule == libqasg.RULE_RDA else zr
        want = {"x": xr, "h": hr, "z": zr}
        codes = U.new_codes(M, d)
        ind = torch.zeros((M, words), dtype=torch.int32, device=U.dev())
        sel = torch.zeros(M, dtype=torch.int64, device=U.dev())
        isyn = torch.zeros(words, dtype=torch.int32, device=U.dev())
        ksyn = torch.zeros(1, dtype=torch.int64, device=U.dev())
        ctx.step_select(rule, double_quant, g_dev, d, ld, M, t, params, *driven, codes_out=codes, indicators_out=ind,
                        selected_out=sel, isyn_out=isyn, ksyn_out=ksyn)
        assert np.array_equal(ind.cpu().numpy().view(np.uint32), ref["quant"]["ind_words"]), t
        assert np.array_equal(U.codes_np(codes), ref["quant"]["codes"]), t
        assert np.array_equal(sel.cpu().numpy(), ref["quant"]["selected"]), t
        assert int(ksyn.cpu().numpy()[0]) == int(ref["quant"]["isyn"].sum()), t
        ksum += int(ksyn.cpu().numpy()[0])
        slack = {"x": U.ATOL, "h": U.ATOL, "z": U.ATOL + 2.0 ** -23 * (np.abs(z_prev) + np.abs(ref["q"]))}
        for name, got in zip(names, driven):
            U.assert_close(got, want[name], "%s step %d (driven)" % (name, t), atol=slack[name])
        U.assert_zero_pattern(driven[0], xr, ref["a"], lam)
    assert ctx.last_async_status() == libqasg.OK
    assert 0 < ksum < T * d                                                 # the selection does select


@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
@pytest.mark.parametrize("bad", [np.nan, np.inf])
def test_non_finite_gradient_is_marked_and_reported(ctx, rule, bad):
    """The selection compares "greater or unordered": a NaN or infinite component is marked where x = 0
    too, and the call reports it; the other workers' indicators are those of the oracle."""
    d, M, t, lam = 9001, 3, 4, 1e-2
    g = inputs.normal_gradients(d, M, seed=8).numpy() * np.float32(0.02)
    x, h, z = _state(d, 8)
    x[4321] = 0.0
    ref = O.select_quantize_workers(rule, g, x, h, z, t, lam, 0.1, 1e-8, libqasg.Q_THRESHOLD, seed=0)
    g[1, 4321] = bad
    g_dev, ld = U.grad_to_dev(g)
    words = (d + 31) // 32
    codes = U.new_codes(M, d)
    ind = torch.zeros((M, words), dtype=torch.int32, device=U.dev())
    scales = torch.zeros(M, dtype=torch.float32, device=U.dev())
    ctx.select_quantize_pack(rule, g_dev, d, ld, M, t, libqasg.make_params(lam, 0.1, 1e-8), U.to_dev(x), U.to_dev(h),
                             U.to_dev(z), codes, scales, None, None, ind, None)
    assert ctx.last_async_status() == libqasg.ERR_NONFINITE
    got = ind.cpu().numpy().view(np.uint32)
    assert (got[1, 4321 >> 5] >> (4321 & 31)) & 1 == 1
    assert np.array_equal(got[0], ref["ind_words"][0]) and np.array_equal(got[2], ref["ind_words"][2])
    assert ctx.last_async_status() == libqasg.OK
