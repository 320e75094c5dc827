"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these compares the oracle with itself or with the CUDA path: each one checks a
function against a closed form, a brute-force search, an invariant the paper states,
a library routine it must reduce to, or published known-answer values.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import qasg_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ canonical sum
def test_canonical_sum_matches_exact_sum_to_fp64_accuracy():
    rng = np.random.default_rng(11)
    for d in (1, 5, 1023, 1024, 4095, 4096, 4097, 3 * 4096 + 17, 100_003):
        a = np.abs(rng.standard_normal(d)).astype(np.float32) * np.float32(10.0 ** rng.integers(-6, 6))
        exact = math.fsum(float(v) for v in a)
        got = float(O.canonical_sum(a))
        levels = 3 + 10 + max(1, math.ceil(math.log2(max(2, d / 4096))))
        assert abs(got - exact) <= levels * 2.0 ** -53 * exact


def test_canonical_sum_exact_when_every_partial_sum_is_representable():
    rng = np.random.default_rng(12)
    a = rng.integers(0, 1 << 20, size=50_001).astype(np.float32)   # integers < 2^20
    assert float(O.canonical_sum(a)) == float(int(a.astype(np.int64).sum()))


def test_canonical_sum_is_not_an_fp32_sum():
    # 2^24 followed by ones: an fp32 accumulator would drop every 1.
    a = np.ones(5000, dtype=np.float32)
    a[0] = 2.0 ** 24
    assert float(O.canonical_sum(a)) == 2.0 ** 24 + 4999


def test_pairwise_sum_tree_shape():
    # With fp64 values chosen so that rounding depends on the pairing, the adjacent-pair
    # tree (a0+a1)+(a2+a3) differs from the left-to-right sum; check the tree is used.
    big, one = 2.0 ** 53, 1.0
    a = [big, one, one, one]                      # ((big+1)+(1+1)) = big+2 ; sequential = big
    assert float(O.pairwise_sum(a)) == big + 2.0
    assert float(O.pairwise_sum([one, one, one])) == 3.0        # padding with +0.0


def test_threshold_equals_exact_definition_on_seeded_cases():
    # Delta from the canonical sum equals Delta from the exactly rounded sum.
    rng = np.random.default_rng(13)
    for d in (7, 4096, 10_000, 65_537):
        v = rng.standard_normal(d).astype(np.float32)
        _, _, delta, _ = O.threshold_quantize(v)
        exact = math.fsum(abs(float(t)) for t in v)
        assert delta == np.float32(0.75 * exact / d)


# ------------------------------------------------------------------ threshold quantizer
def _q_error(v, tern, s):
    return float(((v.astype(np.float64) - float(s) * tern) ** 2).sum())


def test_scale_minimises_the_quadratic_for_fixed_threshold():
    # Section 3.4: for a given Delta the optimal s is the mean of |v| over I_Delta.
    rng = np.random.default_rng(1)
    for d in (3, 8, 33):
        v = rng.standard_normal(d).astype(np.float32)
        tern, s, delta, n = O.threshold_quantize(v)
        assert n == int((np.abs(v) > delta).sum()) and n > 0
        grid = np.linspace(0.0, 2.0 * float(np.abs(v).max()), 200_001)
        absv = np.abs(v).astype(np.float64)
        sel = absv > float(delta)
        obj = n * grid ** 2 - 2.0 * grid * absv[sel].sum() + (absv ** 2).sum()
        assert abs(grid[obj.argmin()] - float(s)) <= grid[1] - grid[0]


def test_error_identity_and_bound():
    # ||v - Q(v)||^2 = ||v||^2 - |I| s^2 at the optimal s, hence <= ||v||^2.
    rng = np.random.default_rng(2)
    v = rng.standard_normal(5000).astype(np.float32)
    tern, s, delta, n = O.threshold_quantize(v)
    err = _q_error(v, tern, s)
    v2 = float((v.astype(np.float64) ** 2).sum())
    assert err == pytest.approx(v2 - n * float(s) ** 2, rel=1e-6)
    assert err <= v2


def _optimal_threshold_objective(v):
    """Section 3.4: rank |v|, try every component as the threshold, maximise
    (sum_{I}|v|)^2 / |I|."""
    a = np.sort(np.abs(v).astype(np.float64))[::-1]
    pref = np.cumsum(a)
    obj = pref ** 2 / np.arange(1, a.size + 1)
    return obj.max()


def test_approximate_threshold_close_to_optimal_for_gaussian():
    rng = np.random.default_rng(3)
    for d in (16, 64):
        for _ in range(20):
            v = rng.standard_normal(d).astype(np.float32)
            tern, s, delta, n = O.threshold_quantize(v)
            if n == 0:
                continue
            got = (np.abs(v.astype(np.float64))[tern != 0].sum()) ** 2 / n
            assert got <= _optimal_threshold_objective(v) * (1 + 1e-12)
    v = rng.standard_normal(200_000).astype(np.float32) * np.float32(3.0)
    tern, s, delta, n = O.threshold_quantize(v)
    got = (np.abs(v.astype(np.float64))[tern != 0].sum()) ** 2 / n
    assert got >= 0.99 * _optimal_threshold_objective(v)
    # 0.75 * E|v| = 0.75 * sigma * sqrt(2/pi) ~ 0.6 sigma  (Section 3.5)
    assert float(delta) == pytest.approx(0.75 * 3.0 * math.sqrt(2 / math.pi), rel=0.01)
    # fraction of non-zero codes = P(|Z| > 0.598)
    assert n / v.size == pytest.approx(math.erfc(0.75 * math.sqrt(2 / math.pi) / math.sqrt(2)), abs=0.005)


def test_boundary_is_strict_and_worked_example():
    # |v| = (3, 3, 6, 4): Delta = 0.75 * 16 / 4 = 3; components equal to Delta code 0.
    v = np.array([3.0, -3.0, 6.0, -4.0], dtype=np.float32)
    tern, s, delta, n = O.threshold_quantize(v)
    assert delta == np.float32(3.0)
    assert tern.tolist() == [0, 0, 1, -1]
    assert n == 2 and s == np.float32(5.0)


def test_zero_gradient_and_nonfinite():
    tern, s, delta, n = O.threshold_quantize(np.zeros(100, dtype=np.float32))
    assert not tern.any() and s == 0 and delta == 0 and n == 0
    v = np.ones(10, dtype=np.float32)
    v[3] = np.nan
    tern, s, _, n = O.threshold_quantize(v)
    assert not tern.any() and s == 0 and n == 0
    v[3] = np.inf
    tern, s, _, n = O.threshold_quantize(v)
    assert not tern.any() and s == 0 and n == 0


def test_power_of_two_equivariance():
    rng = np.random.default_rng(4)
    v = rng.standard_normal(9001).astype(np.float32)
    t0, s0, d0, n0 = O.threshold_quantize(v)
    for k in (-20, 7):
        t1, s1, d1, n1 = O.threshold_quantize(v * np.float32(2.0 ** k))
        assert np.array_equal(t0, t1) and n0 == n1
        assert s1 == s0 * np.float32(2.0 ** k) and d1 == d0 * np.float32(2.0 ** k)


# ------------------------------------------------------------------ encoding
def test_pack_layout_and_bit_budget():
    assert int(O.pack_codes(np.array([1, -1, 0, 1]))[0]) == (1 | (2 << 2) | (1 << 6))
    tern = np.zeros(17, dtype=np.int8)
    tern[16] = -1
    words = O.pack_codes(tern)
    assert words.tolist() == [0, 2]
    rng = np.random.default_rng(5)
    for d in (1, 15, 16, 17, 1000):
        tern = rng.integers(-1, 2, size=d).astype(np.int8)
        words = O.pack_codes(tern)
        assert words.dtype == np.uint32 and words.size == O.code_words(d)
        assert np.array_equal(O.unpack_codes(words, d), tern)
        # Section 3.5: (32 + 2d) bits per worker, up to padding of the last word
        assert O.wire_bits(d) == 32 + 2 * d <= 32 + 32 * words.size < O.wire_bits(d) + 32
    assert O.unpack_codes(np.array([3], dtype=np.uint32), 1).tolist() == [0]


# ------------------------------------------------------------------ Philox / stochastic mode
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = O.philox4x32_10(v[0], v[1], v[2], v[3], v[4], v[5])
        assert [int(o) for o in out] == v[6:]


def test_philox_draws_keying():
    idx = np.arange(64, dtype=np.uint64)
    w, u = O.philox_draws(seed=0x1234567890ABCDEF, t=5, m=3, idx=idx)
    # coordinate i takes word i&3 of the block with counter (i>>2, m, t_lo, t_hi)
    for i in (0, 1, 6, 63):
        blk = O.philox4x32_10(i >> 2, 3, 5, 0, 0x90ABCDEF, 0x12345678)
        assert int(w[i]) == int(blk[i & 3])
    assert u.dtype == np.float32 and (u >= 0).all() and (u < 1).all()
    assert np.array_equal(u.astype(np.float64) * 2 ** 24, (w >> 8).astype(np.float64))
    # every argument of the key changes the stream
    base = O.philox_draws(1, 1, 0, idx)[0]
    for other in (O.philox_draws(2, 1, 0, idx), O.philox_draws(1, 2, 0, idx),
                  O.philox_draws(1, 1, 1, idx), O.philox_draws(1, 1, 0, idx, domain=1),
                  O.philox_draws(1, 1 + (1 << 32), 0, idx)):
        assert not np.array_equal(base, other[0])
    big = O.philox_draws(7, 3, 2, np.arange(1 << 16, dtype=np.uint64))[1]
    assert abs(float(big.mean()) - 0.5) < 0.01


def test_stochastic_quantizer_unbiased_and_variance_identity():
    # E[Q(g)] = g and E||Q(g) - g||^2 = E||Q(g)||^2 - ||g||^2 <= E||Q(g)||^2  (Section 3.3 remark)
    g = np.array([0.9, -0.05, 0.3, 0.0, -1.2, 0.61, 0.007, -0.33], dtype=np.float32)
    trials = 400_000
    t = np.arange(1, trials + 1, dtype=np.uint64)[:, None]
    idx = np.arange(g.size, dtype=np.uint64)[None, :]
    _, u = O.philox_draws(seed=99, t=t, m=2, idx=idx)
    s = np.float32(np.abs(g).max())
    total = np.zeros(g.size)
    sq = 0.0
    err = 0.0
    for lo in range(0, trials, 50_000):
        for row in u[lo:lo + 50_000]:
            tern, s_row = O.ternary_stochastic_quantize(g, row)
            qv = float(s_row) * tern
            total += qv
            sq += float((qv ** 2).sum())
            err += float(((qv - g) ** 2).sum())
    mean = total / trials
    p = np.abs(g.astype(np.float64)) / float(s)
    sigma = float(s) * np.sqrt(p * (1 - p) / trials)
    assert (np.abs(mean - g) <= 5 * sigma + 1e-12).all()
    g2 = float((g.astype(np.float64) ** 2).sum())
    assert err / trials == pytest.approx(sq / trials - g2, rel=0.02)
    assert err / trials <= sq / trials
    # expected squared norm is s * ||g||_1
    assert sq / trials == pytest.approx(float(s) * float(np.abs(g).sum()), rel=0.01)


def test_stochastic_quantizer_edges():
    tern, s = O.ternary_stochastic_quantize(np.zeros(5, dtype=np.float32), np.zeros(5, dtype=np.float32))
    assert not tern.any() and s == 0
    g = np.array([2.0, -2.0, 1.0], dtype=np.float32)
    u = np.array([0.999, 0.0, 0.5], dtype=np.float32)        # p = 1, 1, 0.5 ; u < p strict
    tern, s = O.ternary_stochastic_quantize(g, u)
    assert s == 2 and tern.tolist() == [1, -1, 0]
    # a slice quantized with the whole vector's scaler gives that slice of the whole vector's codes
    rng = np.random.default_rng(8)
    v, uu = rng.standard_normal(1000).astype(np.float32), rng.random(1000).astype(np.float32)
    whole, s = O.ternary_stochastic_quantize(v, uu)
    assert s == np.abs(v).max()
    parts = [O.ternary_stochastic_quantize(v[lo:lo + 300], uu[lo:lo + 300], scale=s)[0] for lo in range(0, 1000, 300)]
    assert np.array_equal(np.concatenate(parts), whole)
    assert not np.array_equal(np.concatenate([O.ternary_stochastic_quantize(v[lo:lo + 300], uu[lo:lo + 300])[0]
                                              for lo in range(0, 1000, 300)]), whole)


# ------------------------------------------------------------------ averaging
def test_average_of_identical_workers_and_single_worker():
    rng = np.random.default_rng(6)
    v = rng.standard_normal(300).astype(np.float32)
    tern, s, _, _ = O.threshold_quantize(v)
    one = O.decode_average(tern[None], np.array([s]))
    assert np.array_equal(one, float(s) * tern)
    many = O.decode_average(np.stack([tern] * 5), np.array([s] * 5, dtype=np.float32))
    assert np.allclose(many, one, rtol=1e-15, atol=0)
    # two different workers: plain mean of the two decoded vectors
    v2 = rng.standard_normal(300).astype(np.float32) * 3
    tern2, s2, _, _ = O.threshold_quantize(v2)
    both = O.decode_average(np.stack([tern, tern2]), np.array([s, s2]))
    assert np.allclose(both, (float(s) * tern + float(s2) * tern2) / 2, rtol=1e-15, atol=0)


# ------------------------------------------------------------------ closed-form updates
def _argmin_convex(fun, lo, hi, iters=200):
    for _ in range(iters):
        a = lo + (hi - lo) / 3
        b = hi - (hi - lo) / 3
        if fun(a) < fun(b):
            hi = b
        else:
            lo = a
    return 0.5 * (lo + hi)


def test_cmd_closed_form_is_the_argmin():
    # minimise eta*q*x + eta*lambda*|x| + H/2 (x - x_t)^2 coordinate-wise (QCMD objective)
    rng = np.random.default_rng(7)
    lam, eta, delta = np.float32(0.05), np.float32(0.3), np.float32(1e-3)
    for _ in range(60):
        q, xt, h = rng.standard_normal() * 0.3, rng.standard_normal() * 0.2, rng.random()
        x_new, h_new, a = O.cmd_step(np.array([q]), np.array([xt]), np.array([h]), lam, eta, delta)
        H = float(delta) + math.sqrt(h + q * q)
        assert h_new[0] == pytest.approx(h + q * q, rel=1e-15)
        f = lambda x: float(eta) * q * x + float(eta) * float(lam) * abs(x) + 0.5 * H * (x - xt) ** 2
        best = _argmin_convex(f, -5.0, 5.0)
        assert x_new[0] == pytest.approx(best, abs=1e-7)
        assert f(x_new[0]) <= f(best) + 1e-15
        assert (x_new[0] == 0.0) == (a[0] <= float(lam))


def test_rda_closed_form_is_the_argmin():
    # minimise eta*(z/t)*x + eta*lambda*|x| + H x^2 / (2t)  (QRDA objective)
    rng = np.random.default_rng(8)
    lam, eta, delta = np.float32(0.05), np.float32(0.3), np.float32(1e-3)
    for _ in range(60):
        t = int(rng.integers(1, 50))
        q, z0, h = rng.standard_normal() * 0.3, rng.standard_normal() * t * 0.05, rng.random()
        x_new, h_new, z_new, a = O.rda_step(np.array([q]), np.array([h]), np.array([z0]), t, lam, eta, delta)
        z = z0 + q
        H = float(delta) + math.sqrt(h + q * q)
        assert z_new[0] == pytest.approx(z, rel=1e-15)
        f = lambda x: float(eta) * (z / t) * x + float(eta) * float(lam) * abs(x) + H * x * x / (2 * t)
        best = _argmin_convex(f, -50.0, 50.0)
        assert x_new[0] == pytest.approx(best, abs=1e-6)
        assert f(x_new[0]) <= f(best) + 1e-15
        assert (x_new[0] == 0.0) == (abs(z) / t <= float(lam))


def test_exact_sparsity_rules():
    lam, eta, delta = np.float32(0.01), np.float32(0.1), np.float32(1e-8)
    q = np.array([0.0099, -0.0099, 0.0101, -0.0101, 0.0])
    # QCMD from x_t = 0, h = 0: zero iff |q| <= lambda
    x_new, _, _ = O.cmd_step(q, np.zeros(5), np.zeros(5), lam, eta, delta)
    assert (x_new == 0).tolist() == [True, True, False, False, True]
    assert np.sign(x_new[2]) == -1 and np.sign(x_new[3]) == 1
    assert not np.signbit(x_new).any() or (x_new[np.signbit(x_new)] != 0).all()   # zeros are +0.0
    # QRDA: zero iff |z|/t <= lambda
    x_new, _, z_new, _ = O.rda_step(q, np.zeros(5), np.zeros(5), 1, lam, eta, delta)
    assert (x_new == 0).tolist() == [True, True, False, False, True]
    x_new, _, _, _ = O.rda_step(np.zeros(5), np.ones(5), np.array([0.5, -0.5, 0.0499, -0.0499, 0.0501]), 5, lam, eta, delta)
    assert (x_new == 0).tolist() == [False, False, True, True, False]


def test_reduces_to_diagonal_adagrad():
    # Q = identity, lambda = 0, M = 1: QCMD is torch.optim.Adagrad(lr=eta, eps=delta).
    rng = np.random.default_rng(9)
    d, steps, eta, delta = 50, 25, 0.1, 1e-3
    p = torch.zeros(d, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adagrad([p], lr=eta, eps=delta, lr_decay=0.0, initial_accumulator_value=0.0)
    x = np.zeros(d)
    h = np.zeros(d)
    for t in range(1, steps + 1):
        g = rng.standard_normal((1, d)).astype(np.float32)
        out = O.step(O.RULE_CMD, g, x, h, None, t, 0.0, eta, delta, quantizer=O.QUANT_NONE)
        x, h = out["x"], out["h"]
        p.grad = torch.from_numpy(g[0].astype(np.float64))
        opt.step()
        # eta and delta are fp32 at the boundary, so agreement is to fp32 rounding of the scalars
        assert np.allclose(x, p.detach().numpy(), rtol=1e-6, atol=1e-12)


def test_accumulator_satisfies_lemma_1():
    # (1/2) sum_t ||q_t||^2_{psi*_t} <= sum_i ||q_{1:T,i}||_2 with H_t including q_t.
    rng = np.random.default_rng(10)
    d, M, T = 200, 3, 40
    x = np.zeros(d)
    h = np.zeros(d)
    lhs = 0.0
    delta = np.float32(1e-8)
    for t in range(1, T + 1):
        g = rng.standard_normal((M, d)).astype(np.float32)
        out = O.step(O.RULE_CMD, g, x, h, None, t, 1e-3, 0.1, delta)
        x, h, q = out["x"], out["h"], out["q"]
        lhs += float((q * q / (float(delta) + np.sqrt(h))).sum())
    assert 0.5 * lhs <= float(np.sqrt(h).sum()) * (1 + 1e-12)


def test_fused_step_composes_its_parts():
    # a planted dropped 1/M, wrong sign or missing h update would break these relations
    rng = np.random.default_rng(14)
    d, M = 500, 4
    g = rng.standard_normal((M, d)).astype(np.float32)
    x0 = rng.standard_normal(d) * 0.1
    h0 = rng.random(d)
    z0 = rng.standard_normal(d) * 0.1
    out = O.step(O.RULE_RDA, g, x0, h0, z0, 16, 1e-3, 0.1, 1e-8)
    quant = out["quant"]
    manual_q = sum(float(quant["scales"][m]) * O.unpack_codes(quant["codes"][m], d) for m in range(M)) / M
    assert np.allclose(out["q"], manual_q, rtol=1e-14, atol=0)
    assert np.allclose(out["z"], z0 + manual_q, rtol=1e-14)
    assert np.allclose(out["h"], h0 + manual_q ** 2, rtol=1e-14)
    assert np.mean(out["x"] == 0) > 0.0                      # some exact zeros
    nzmask = out["x"] != 0
    assert (np.sign(out["x"][nzmask]) == -np.sign(out["z"][nzmask])).all()


# ------------------------------------------------------------------ double quantization
def test_threshold_quantizer_is_idempotent():
    # Q(Q(v)) = Q(v): the entries of Q(v) are 0 or +-s, the threshold 0.75*s*n/d is below s, so
    # exactly the non-zero entries are kept and their mean magnitude is s again.
    rng = np.random.default_rng(21)
    for d in (9, 1000, 50_001):
        v = rng.standard_normal(d).astype(np.float32) * np.float32(0.3)
        tern, s, _, n = O.threshold_quantize(v)
        again = O.requantize(float(s) * tern.astype(np.float64), O.QUANT_THRESHOLD)
        assert np.array_equal(again["tern"], tern) and again["scale"] == s and again["count"] == n
        assert np.array_equal(again["q"], float(s) * tern)


def test_requantize_is_q_applied_to_the_fp32_average():
    rng = np.random.default_rng(22)
    d, M = 3000, 5
    g = rng.standard_normal((M, d)).astype(np.float32)
    quant = O.quantize_workers(g, O.QUANT_THRESHOLD)
    gbar = O.decode_average(quant["terns"], quant["scales"])
    rq = O.requantize(gbar, O.QUANT_THRESHOLD)
    gbar32 = gbar.astype(np.float32)
    # threshold and scale by their definitions (Section 3.5, Section 3.4), from plain fp64 sums
    delta = 0.75 * np.abs(gbar32.astype(np.float64)).sum() / d
    assert float(rq["threshold"]) == pytest.approx(delta, rel=1e-6)
    kept = np.abs(gbar32) > rq["threshold"]
    assert rq["count"] == int(kept.sum()) and np.array_equal(rq["tern"] != 0, kept)
    assert np.array_equal(np.sign(rq["tern"]), np.sign(gbar32) * kept)
    assert float(rq["scale"]) == pytest.approx(np.abs(gbar32.astype(np.float64))[kept].mean(), rel=1e-6)
    # error identity of the second quantization: ||gbar - q||^2 = ||gbar||^2 - n s^2
    err = float(((gbar32.astype(np.float64) - rq["q"]) ** 2).sum())
    assert err == pytest.approx(float((gbar32.astype(np.float64) ** 2).sum()) - rq["count"] * float(rq["scale"]) ** 2, rel=1e-5)
    assert np.array_equal(O.unpack_codes(rq["codes"], d), rq["tern"])


def test_double_quantized_step_uses_q_of_the_average():
    rng = np.random.default_rng(23)
    d, M = 800, 4
    g = rng.standard_normal((M, d)).astype(np.float32)
    x0, h0, z0 = rng.standard_normal(d) * 0.1, rng.random(d), rng.standard_normal(d) * 0.1
    one = O.step(O.RULE_RDA, g, x0, h0, z0, 7, 1e-3, 0.1, 1e-8)
    two = O.step(O.RULE_RDA, g, x0, h0, z0, 7, 1e-3, 0.1, 1e-8, double_quant=True)
    rq = two["requant"]
    assert one["requant"] is None and np.array_equal(two["quant"]["codes"], one["quant"]["codes"])
    assert np.array_equal(rq["gbar32"], one["q"].astype(np.float32))
    assert set(np.unique(two["q"])) <= {-float(rq["scale"]), 0.0, float(rq["scale"])}
    assert np.allclose(two["z"], z0 + two["q"], rtol=1e-15) and np.allclose(two["h"], h0 + two["q"] ** 2, rtol=1e-15)
    # quantizing twice adds error: the paper's remark that one-way quantization is less noisy
    assert ((two["q"] - one["q"]) ** 2).sum() > 0


def test_stochastic_requantize_uses_its_own_stream_and_is_unbiased():
    gbar = np.array([0.5, -0.25, 0.0, 0.125, -0.5, 0.3], dtype=np.float64)
    trials = 60_000
    total = np.zeros(gbar.size)
    for t in range(1, trials + 1):
        total += O.requantize(gbar, O.QUANT_TERNARY_STOCH, t=t, seed=5)["q"]
    p = np.abs(gbar) / 0.5
    sigma = 0.5 * np.sqrt(p * (1 - p) / trials)
    assert (np.abs(total / trials - gbar) <= 5 * sigma + 1e-12).all()
    a = O.requantize(np.linspace(-1, 1, 64), O.QUANT_TERNARY_STOCH, t=3, seed=9)
    _, u_worker0 = O.philox_draws(9, 3, 0, np.arange(64, dtype=np.uint64), domain=0)
    tern_w, _ = O.ternary_stochastic_quantize(np.linspace(-1, 1, 64).astype(np.float32), u_worker0)
    assert not np.array_equal(a["tern"], tern_w)          # domain 1 is a different stream


# ------------------------------------------------------------------ sparse selection
def _random_sparse_state(rng, d):
    x = rng.standard_normal(d) * 0.1 * (rng.random(d) < 0.3)          # 70 % exact zeros
    h = rng.random(d) * (rng.random(d) < 0.8)
    z = rng.standard_normal(d) * 0.05
    return x.astype(np.float32), h.astype(np.float32), z.astype(np.float32)


def test_indicator_is_the_definition_away_from_the_boundary():
    # I = [x != 0 or x_hat != 0] with x_hat from the closed forms in fp64; the fp32 decision may
    # differ only where the compared quantity is within rounding of lambda.
    rng = np.random.default_rng(31)
    d, t, lam, eta, delta = 20_000, 7, 1e-2, 0.1, 1e-8
    x, h, z = _random_sparse_state(rng, d)
    g = (rng.standard_normal(d) * 0.03).astype(np.float32)
    for rule in (O.RULE_CMD, O.RULE_RDA):
        ind = O.indicator(rule, g, x, h, z, t, lam, eta, delta)
        x_hat = O.trial_update(rule, g, x, h, z, t, lam, eta, delta)
        want = (x != 0) | (x_hat != 0)
        if rule == O.RULE_CMD:
            a = O.cmd_step(g, x, h, lam, eta, delta)[2]
        else:
            a = O.rda_step(g, h, z, t, lam, eta, delta)[3]
        decided = np.abs(a - float(np.float32(lam))) > 1e-6
        assert np.array_equal(ind[decided], want[decided])
        assert decided.mean() > 0.999 and 0.2 < ind.mean() < 0.9


def test_unselected_coordinates_stay_zero_when_nothing_is_sent_for_them():
    # If no worker selects coordinate d (x_d = 0 and every trial update leaves it 0) then q_d = 0
    # and the real update leaves x_d = 0: the selection loses nothing there.
    rng = np.random.default_rng(32)
    d, M, t, lam, eta, delta = 5000, 3, 5, 2e-2, 0.1, 1e-8
    x, h, z = _random_sparse_state(rng, d)
    z = (z * 0.1).astype(np.float32)
    g = (rng.standard_normal((M, d)) * 0.02).astype(np.float32)
    for rule in (O.RULE_CMD, O.RULE_RDA):
        out = O.step(rule, g, x, h, z, t, lam, eta, delta, select=True)
        isyn = out["quant"]["isyn"]
        assert 0 < isyn.sum() < d
        assert not out["q"][~isyn].any() and not out["x"][~isyn].any()
        assert np.array_equal(out["h"][~isyn], h[~isyn].astype(np.float64))


def test_selected_quantizer_is_q_on_the_selected_subvector():
    # Q(S(v, I)) equals Q_Delta applied to the compacted vector of the k selected components
    rng = np.random.default_rng(33)
    d = 9000
    v = rng.standard_normal(d).astype(np.float32)
    sel = rng.random(d) < 0.37
    tern, s, delta, n, k = O.threshold_quantize_selected(v, sel)
    sub = v[sel]
    exact = math.fsum(abs(float(a)) for a in sub)
    assert k == sub.size and delta == np.float32(0.75 * exact / k)
    kept = np.abs(sub) > delta
    assert n == int(kept.sum()) and np.array_equal(tern[sel] != 0, kept) and not tern[~sel].any()
    assert float(s) == pytest.approx(np.abs(sub.astype(np.float64))[kept].mean(), rel=1e-6)
    # nothing selected, everything selected
    assert O.threshold_quantize_selected(v, np.zeros(d, bool))[1:] == (0, 0, 0, 0)
    full = O.threshold_quantize_selected(v, np.ones(d, bool))
    ref = O.threshold_quantize(v)
    assert np.array_equal(full[0], ref[0]) and full[1:4] == ref[1:]


def test_selected_stochastic_quantizer_is_the_unbiased_quantizer_of_the_selected_subvector():
    # Section 3.2 / 3.4: Q(S(v, I)) with the unbiased ternary Q.  The scale is the maximum over the
    # SELECTED components (here the two largest magnitudes are not selected), unselected components
    # code 0, and on the selected ones the codes are those of the quantizer applied to the compacted
    # sub-vector with the same draws.
    rng = np.random.default_rng(35)
    d = 4000
    v = rng.standard_normal(d).astype(np.float32)
    sel = rng.random(d) < 0.4
    big = np.argsort(-np.abs(v))[:2]
    sel[big] = False
    assert np.abs(v[sel]).max() < np.abs(v[big]).min()
    u = rng.random(d).astype(np.float32)
    tern, s = O.ternary_stochastic_quantize_selected(v, u, sel)
    assert s == np.abs(v[sel]).max() and s < np.abs(v).max()
    assert not tern[~sel].any()
    want = (u[sel] < np.abs(v[sel]) / s).astype(np.int8) * np.sign(v[sel]).astype(np.int8)
    assert np.array_equal(tern[sel], want)
    sub_tern, sub_s = O.ternary_stochastic_quantize(v[sel], u[sel])
    assert sub_s == s and np.array_equal(tern[sel], sub_tern)
    # nothing selected: nothing is sent
    none, s0 = O.ternary_stochastic_quantize_selected(v, u, np.zeros(d, bool))
    assert s0 == 0 and not none.any()
    # Monte Carlo over Philox draws: unbiased on the selected components, identically 0 elsewhere
    g = np.array([0.9, -0.05, 3.0, 0.0, -1.2, 0.61, -7.0, -0.33], dtype=np.float32)
    pick = np.array([1, 1, 0, 1, 1, 0, 0, 1], dtype=bool)
    trials = 200_000
    t = np.arange(1, trials + 1, dtype=np.uint64)[:, None]
    _, draws = O.philox_draws(seed=5, t=t, m=1, idx=np.arange(g.size, dtype=np.uint64)[None, :])
    total = np.zeros(g.size)
    for row in draws:
        tr, sr = O.ternary_stochastic_quantize_selected(g, row, pick)
        total += float(sr) * tr
    mean = total / trials
    smax = float(np.abs(g[pick]).max())
    p = np.where(pick, np.abs(g.astype(np.float64)) / smax, 0.0)
    sigma = smax * np.sqrt(p * (1 - p) / trials)
    assert (np.abs(mean - np.where(pick, g, 0.0)) <= 5 * sigma + 1e-12).all()
    assert not mean[~pick].any()


def test_indicator_words_or_and_sparse_bit_budget():
    rng = np.random.default_rng(34)
    d, M = 1000, 4
    x, h, z = _random_sparse_state(rng, d)
    g = (rng.standard_normal((M, d)) * 0.01).astype(np.float32)
    out = O.select_quantize_workers(O.RULE_CMD, g, x, h, z, 3, 1e-2, 0.1, 1e-8)
    assert out["ind_words"].shape == (M, 32) and out["ind_words"].dtype == np.uint32
    for m in range(M):
        bits = ((out["ind_words"][m][:, None] >> np.arange(32, dtype=np.uint32)) & 1).ravel()[:d].astype(bool)
        assert np.array_equal(bits, out["indicators"][m]) and out["selected"][m] == bits.sum()
    assert np.array_equal(O.pack_bits(out["isyn"]), np.bitwise_or.reduce(out["ind_words"], axis=0))
    assert int(O.pack_bits(np.array([1, 0, 1] + [0] * 30 + [1], bool))[0]) == 5 and O.pack_bits(np.ones(33, bool))[1] == 1
    k = int(out["selected"][0])
    assert O.sparse_wire_bits(d, k) == 32 + d + 2 * k
    assert (O.sparse_wire_bits(d, k) < O.wire_bits(d)) == (k < d / 2)         # cheaper iff k < d/2


# ------------------------------------------------------------------ sparse (touched) gradients
def test_touched_step_is_the_dense_step_of_the_stored_entries():
    """Entries a worker does not store are +0.0 by definition: whatever the array holds there is
    ignored, they code 0 under both quantizers, and the threshold is 0.75/d times the sum over the
    stored entries alone (checked against an exactly rounded sum), d still the full dimension."""
    rng = np.random.default_rng(41)
    M, d = 3, 9000
    touched = rng.random((M, d)) < 0.02
    touched[0, :40] = True
    vals = rng.standard_normal((M, d)).astype(np.float32)
    clean = np.where(touched, vals, np.float32(0.0)).astype(np.float32)
    dirty = np.where(touched, vals, np.float32(np.nan)).astype(np.float32)
    assert np.array_equal(O.densify_touched(dirty, touched), clean)
    assert not np.signbit(O.densify_touched(-np.abs(dirty), touched)[~touched]).any()
    x, h, z = rng.standard_normal(d) * 0.1, rng.random(d), rng.standard_normal(d) * 0.1
    for quantizer in (O.QUANT_THRESHOLD, O.QUANT_TERNARY_STOCH):
        for rule in (O.RULE_CMD, O.RULE_RDA):
            a = O.step(rule, dirty, x, h, z, 3, 1e-3, 0.1, 1e-8, quantizer=quantizer, seed=5, touched=touched)
            b = O.step(rule, clean, x, h, z, 3, 1e-3, 0.1, 1e-8, quantizer=quantizer, seed=5)
            assert np.array_equal(a["x"], b["x"]) and np.array_equal(a["h"], b["h"])
            assert np.array_equal(a["quant"]["codes"], b["quant"]["codes"])
            assert (a["quant"]["terns"][~touched] == 0).all()
        if quantizer == O.QUANT_THRESHOLD:
            for m in range(M):
                exact = math.fsum(abs(float(v)) for v in vals[m][touched[m]])
                assert a["quant"]["thresholds"][m] == np.float32(0.75 * exact / d)
    with pytest.raises(ValueError):
        O.densify_touched(vals, touched[:, :-1])


# ------------------------------------------------------------------ exact optimal threshold
def test_canonical_prefix_is_a_prefix_sum():
    rng = np.random.default_rng(51)
    # exact on integers (every partial sum representable), across block, group and group-sequence levels
    for d in (1, 31, 33, 1023, 1025, 5000, (1 << 20) + 4321, (1 << 21) + 77):
        a = rng.integers(0, 1 << 16, size=d).astype(np.float64)
        assert np.array_equal(O.canonical_prefix(a), np.cumsum(a))
    a = np.abs(rng.standard_normal(70_001)) * 10.0 ** rng.integers(-5, 5, size=70_001)
    got = O.canonical_prefix(a)
    want = np.array([math.fsum(a[: i + 1]) for i in range(0, 70_001, 997)])
    assert np.all(np.abs(got[::997] - want) <= 64 * 2.0 ** -53 * want)
    assert np.all(np.diff(got) >= 0)


def _best_ternary_error(v):
    """Eq. of the quantization objective by exhaustive search: min over tern in {-1,0,1}^d and s >= 0
    of ||v - s*tern||^2 (for a given tern the best s is max(0, <v, tern>/|tern|_0))."""
    import itertools
    v = v.astype(np.float64)
    best = float((v * v).sum())
    for tern in itertools.product((-1.0, 0.0, 1.0), repeat=v.size):
        t = np.array(tern)
        nnz = np.count_nonzero(t)
        if nnz == 0:
            continue
        s = max(0.0, float(v @ t) / nnz)
        best = min(best, float(((v - s * t) ** 2).sum()))
    return best


def test_optimal_threshold_attains_the_minimum_over_all_ternary_vectors():
    rng = np.random.default_rng(52)
    for d in (1, 2, 3, 5, 7):
        for _ in range(6):
            v = rng.standard_normal(d).astype(np.float32)
            if d > 2 and rng.random() < 0.3:
                v[1] = v[0]                                   # a tie
            tern, s, delta, n = O.optimal_threshold_quantize(v)
            s_exact = np.abs(v.astype(np.float64))[tern != 0].sum() / n
            err = float(((v.astype(np.float64) - s_exact * tern) ** 2).sum())
            assert err <= _best_ternary_error(v) * (1 + 1e-12) + 1e-300
            assert float(s) == pytest.approx(s_exact, rel=1e-6)
            assert n == int((np.abs(v) > delta).sum())
            assert delta == 0 or delta in np.abs(v)           # a component, as the paper's procedure has it


def test_optimal_threshold_beats_every_component_taken_as_threshold():
    rng = np.random.default_rng(53)
    for d, scale in ((50, 1.0), (1000, 1e-3), (4097, 30.0)):
        v = (rng.standard_normal(d) * scale).astype(np.float32)
        v[rng.integers(0, d, size=d // 10)] = 0.0
        v[5] = v[6] = v[7]
        delta, k = O.optimal_threshold(v)
        a = np.abs(v).astype(np.float64)

        def objective(thr):
            sel = a[a > thr]
            return math.fsum(sel) ** 2 / sel.size if sel.size else 0.0
        best = max(objective(float(c)) for c in np.unique(np.concatenate([a, [0.0]])))
        assert objective(float(delta)) >= best * (1 - 1e-13)
        assert k == int((a > float(delta)).sum()) and k > 0
    assert O.optimal_threshold(np.zeros(9, dtype=np.float32)) == (np.float32(0.0), 0)
    # all equal and non-zero: everything is kept, the threshold falls to 0
    assert O.optimal_threshold(np.full(9, -2.5, dtype=np.float32)) == (np.float32(0.0), 9)


def test_optimal_threshold_for_gaussian_data_is_about_0p6_sigma():
    # Section 3.5 quotes Delta* ~ 0.6 sigma for N(0, sigma^2); the 0.75 * E|v| rule approximates it.
    rng = np.random.default_rng(54)
    v = (rng.standard_normal(300_000) * 2.0).astype(np.float32)
    delta, k = O.optimal_threshold(v)
    assert 0.55 * 2.0 < float(delta) < 0.67 * 2.0
    _, _, approx, _ = O.threshold_quantize(v)
    assert abs(float(approx) - float(delta)) < 0.06 * 2.0
    tern, s, d2, n = O.optimal_threshold_quantize(v)
    got = (np.abs(v.astype(np.float64))[tern != 0].sum()) ** 2 / n
    assert got == pytest.approx(_optimal_threshold_objective(v), rel=1e-12)
