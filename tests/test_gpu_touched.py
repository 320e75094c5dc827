"""GPU parity of the path for gradients held in sparse form (only the entries a minibatch touched are
stored): the CSR gradient with its touched bits, the quantizers and the fused step on such rows, each
against the oracle's dense definition (codes, thresholds, scales, counts, bits: exact; iterates and
gradient values: within tolerance)."""
import numpy as np
import pytest
import torch

from oracle import logreg_oracle as L
from oracle import qasg_oracle as O
from paper_2208_05631_b200 import inputs, libqasg
from tests import _gpu_util as U
from tests.test_gpu_logreg import _assert_grad_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = libqasg.Context(1 << 20, 16, device=0)
    yield c
    c.close()


def _touched_words(touched):
    return np.stack([O.pack_bits(row) for row in touched])


def _sparse_case(d, M, density, seed):
    """Values where touched, NaN everywhere else (padding included): an unmarked entry that is read
    poisons a sum or a code."""
    rng = np.random.default_rng(seed)
    touched = rng.random((M, d)) < density
    vals = inputs.normal_gradients(d, M, seed=seed).numpy() * np.float32(0.05)
    g = np.where(touched, vals, np.float32(np.nan)).astype(np.float32)
    return g, touched


@pytest.mark.parametrize("d,M,density", [(1, 1, 1.0), (5, 2, 0.5), (4095, 3, 0.01), (4096 + 17, 4, 0.3),
                                         (3 * 4096 + 100, 2, 0.0), (100_003, 8, 0.005), (1 << 20, 5, 0.002),
                                         (70_001, 16, 1.0)])
@pytest.mark.parametrize("quantizer", [libqasg.Q_THRESHOLD, libqasg.Q_TERNARY_STOCH])
def test_quantize_pack_touched_bit_exact(ctx, d, M, density, quantizer):
    t, seed = 9, 21
    g, touched = _sparse_case(d, M, density, seed=d % 1009 + M)
    ref = O.quantize_workers(O.densify_touched(g, touched), quantizer, t=t, seed=seed)
    g_dev, ld = U.grad_to_dev(g)
    words = _touched_words(touched)
    if d % 32:
        words[:, -1] |= np.uint32(0xFFFFFFFF) << np.uint32(d % 32)      # stray bits past d are ignored
    codes = U.new_codes(M, d)
    scales = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    thr = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    cnt = torch.full((M,), -1, dtype=torch.int64, device=U.dev())
    params = libqasg.make_params(1e-3, 0.1, 1e-8, quantizer=quantizer, seed=seed)
    ctx.quantize_pack_touched(g_dev, d, ld, M, t, params, U.to_dev(words.view(np.int32)), codes, scales, thr, cnt)
    assert ctx.last_async_status() == libqasg.OK
    assert np.array_equal(U.codes_np(codes), ref["codes"])
    assert np.array_equal(U.f32_bits(thr), U.f32_bits(ref["thresholds"]))
    assert np.array_equal(U.f32_bits(scales), U.f32_bits(ref["scales"]))
    assert np.array_equal(cnt.cpu().numpy(), ref["counts"])
    if density == 0.0:
        assert not U.codes_np(codes).any() and not scales.cpu().numpy().any()


@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
@pytest.mark.parametrize("quantizer", [libqasg.Q_THRESHOLD, libqasg.Q_TERNARY_STOCH])
def test_step_touched_matches_the_dense_definition(ctx, rule, quantizer):
    d, M, t, lam, eta, delta, seed = 50_000 + 3, 6, 4, 1e-3, 0.1, 1e-8, 8
    g, touched = _sparse_case(d, M, 0.01, seed=77)
    x, h, z = inputs.random_state(d, seed=5)
    x, h, z = x.numpy(), h.numpy(), z.numpy()
    ref = O.step(rule, g, x, h, z, t, lam, eta, delta, quantizer=quantizer, seed=seed, touched=touched)
    g_dev, ld = U.grad_to_dev(g)
    xd, hd, zd = U.to_dev(x), U.to_dev(h), U.to_dev(z)
    codes = U.new_codes(M, d)
    scales = torch.zeros(M, dtype=torch.float32, device=U.dev())
    params = libqasg.make_params(lam, eta, delta, quantizer=quantizer, seed=seed)
    ctx.step_touched(rule, g_dev, d, ld, M, t, params, U.to_dev(_touched_words(touched).view(np.int32)), xd, hd, zd,
                     codes, scales)
    assert ctx.last_async_status() == libqasg.OK
    assert np.array_equal(U.codes_np(codes), ref["quant"]["codes"])
    assert np.array_equal(U.f32_bits(scales), U.f32_bits(ref["quant"]["scales"]))
    U.assert_close(xd, ref["x"], "x")
    U.assert_close(hd, ref["h"], "h")
    if rule == libqasg.RULE_RDA:
        U.assert_close(zd, ref["z"], "z")
    U.assert_zero_pattern(xd, ref["x"], ref["a"], lam)


def _csr_on_device(prob):
    return [U.to_dev(prob[k]) for k in ("rowptr", "colidx", "vals", "y")]


def test_csr_gradient_in_sparse_form_over_consecutive_calls(ctx):
    """g and the bits carry over from call to call: every call must leave exactly the new minibatch's
    entries marked and everything else +0.0."""
    d, n, M, B = 1 << 16, 4000, 16, 64
    prob = inputs.logreg_csr_problem(n=n, d=d, M=M, nnz_per_row=80, seed=3)
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(d) * 0.5).astype(np.float32)
    dev_args = _csr_on_device(prob)
    xd = U.to_dev(x)
    ld = d + 8
    g = torch.zeros((M, ld), dtype=torch.float32, device=U.dev())
    g[:, d:] = float("nan")                                   # the padding is never touched
    bits = torch.zeros((M, d // 32), dtype=torch.int32, device=U.dev())
    for t in (1, 2, 70, 71):
        ctx.logreg_grad_csr_touched(*dev_args, n, d, M, prob["shard_row0"], None, B, t, xd, g, ld, bits)
        want = L.grad_workers_csr(prob["rowptr"], prob["colidx"], prob["vals"], prob["y"], prob["shard_row0"],
                                  B, t, x, d)
        touched = L.touched_columns(prob["rowptr"], prob["colidx"], prob["shard_row0"], B, t, d)
        assert np.array_equal(bits.cpu().numpy().view(np.uint32), _touched_words(touched))
        got = g.cpu().numpy()
        _assert_grad_close(g[:, :d], want)
        assert (got[:, :d][~touched] == 0).all() and not np.signbit(got[:, :d][~touched]).any()
        assert np.isnan(got[:, d:]).all()
        assert 0.001 < touched.mean() < 0.2                   # a sparse gradient indeed


@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
def test_closed_loop_csr_in_sparse_form_driven_by_the_oracle(ctx, rule):
    """The oracle runs the loop.  Every step: the GPU's sparse-form gradient at the oracle's iterate
    is checked (values, bits), and the GPU step on sparse rows is fed the oracle's gradient with the
    oracle's touched set and must track the oracle's iterate."""
    d, n, M, B, T = 1 << 14, 2000, 8, 32, 25
    lam, eta, delta = 1e-4, 0.1, 1e-8
    prob = inputs.logreg_csr_problem(n=n, d=d, M=M, nnz_per_row=40, seed=9)
    dev_args = _csr_on_device(prob)
    params = libqasg.make_params(lam, eta, delta)
    xr, hr, zr = np.zeros(d), np.zeros(d), np.zeros(d)
    x, h, z = (torch.zeros(d, dtype=torch.float32, device=U.dev()) for _ in range(3))
    g_gpu = torch.zeros((M, d), dtype=torch.float32, device=U.dev())
    bits = torch.zeros((M, d // 32), dtype=torch.int32, device=U.dev())
    for t in range(1, T + 1):
        g64 = L.grad_workers_csr(prob["rowptr"], prob["colidx"], prob["vals"], prob["y"], prob["shard_row0"],
                                 B, t, xr, d)
        touched = L.touched_columns(prob["rowptr"], prob["colidx"], prob["shard_row0"], B, t, d)
        ctx.logreg_grad_csr_touched(*dev_args, n, d, M, prob["shard_row0"], None, B, t,
                                    U.to_dev(xr.astype(np.float32)), g_gpu, d, bits)
        _assert_grad_close(g_gpu, g64)
        assert np.array_equal(bits.cpu().numpy().view(np.uint32), _touched_words(touched))
        g32 = np.where(touched, g64.astype(np.float32), np.float32(np.nan))
        ctx.step_touched(rule, U.to_dev(g32), d, d, M, t, params, U.to_dev(_touched_words(touched).view(np.int32)),
                         x, h, z)
        ref = O.step(rule, g32, xr, hr, zr, t, lam, eta, delta, touched=touched)
        xr, hr, zr = ref["x"], ref["h"], ref["z"] if rule == libqasg.RULE_RDA else zr
        U.assert_close(x, xr, "x step %d" % t)
        U.assert_close(h, hr, "h step %d" % t)
        U.assert_zero_pattern(x, xr, ref["a"], lam)
    assert ctx.last_async_status() == libqasg.OK


def test_touched_argument_errors(ctx):
    d, M = 4096, 2
    g = torch.zeros((M, d), dtype=torch.float32, device=U.dev())
    codes = U.new_codes(M, d)
    scales = torch.zeros(M, dtype=torch.float32, device=U.dev())
    params = libqasg.make_params(1e-3, 0.1, 1e-8)
    with pytest.raises(libqasg.QasgError) as e:
        ctx.quantize_pack_touched(g, d, d, M, 1, params, None, codes, scales)
    assert e.value.status == libqasg.ERR_INVALID_ARG
    bits = torch.zeros((M, d // 32 + 4), dtype=torch.int32, device=U.dev())
    with pytest.raises(libqasg.QasgError) as e:
        ctx.quantize_pack_touched(g, d, d, M, 1, params, bits.view(-1)[1:], codes, scales)
    assert e.value.status == libqasg.ERR_ALIGNMENT
