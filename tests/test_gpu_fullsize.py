"""Parity at the benchmark's full size (d = 2^28, M = 8, the launch configuration bench.py times).

The oracle computes every worker's threshold, scale and count from the full 2^28-coordinate
reductions and every worker's complete packed code row; those are compared bit for bit.  The
iterates are compared on a sample of coordinates the oracle updates one by one: 2^20 random
ones plus the first and last coordinates and both sides of tile and chunk boundaries."""
import numpy as np
import pytest
import torch

from oracle import qasg_oracle as O
from paper_2208_05631_b200 import inputs, libqasg
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu

D, M, T_STEP = 1 << 28, 8, 16
LAM, ETA, DELTA = 1e-3, 0.1, 1e-8


def _enough_memory():
    if not torch.cuda.is_available():
        return False
    try:
        import psutil
        host_ok = psutil.virtual_memory().available > 24 * 2 ** 30
    except Exception:
        host_ok = True
    return host_ok and torch.cuda.get_device_properties(0).total_memory > 40 * 2 ** 30


def test_full_size_step_against_the_oracle():
    if not _enough_memory():
        pytest.skip("needs 40 GB of device memory and 24 GB of host memory")
    dev = U.dev()
    g = inputs.student_t_gradients(D, M, seed=2, device=dev)
    x0, h0, z0 = inputs.random_state(D, seed=2, device=dev)
    ctx = libqasg.Context(D, M, device=0)
    params = libqasg.make_params(LAM, ETA, DELTA)
    codes = torch.zeros((M, libqasg.code_words(D)), dtype=torch.int32, device=dev)
    scales = torch.zeros(M, dtype=torch.float32, device=dev)
    xc, hc = x0.clone(), h0.clone()
    ctx.step(libqasg.RULE_CMD, g, D, D, M, T_STEP, params, xc, hc, None, codes_out=codes, scales_out=scales)
    xr, hr, zr = x0.clone(), h0.clone(), z0.clone()
    ctx.step(libqasg.RULE_RDA, g, D, D, M, T_STEP, params, xr, hr, zr)     # codes in the context's scratch
    assert ctx.last_async_status() == libqasg.OK

    rng = np.random.default_rng(5)
    edges = np.concatenate([np.arange(0, 4100), np.arange(D - 4100, D),
                            (np.arange(1, 9)[:, None] * (64 * 4096) + np.arange(-3, 3)[None, :]).ravel(),
                            (1 << 27) + np.arange(-8, 8)])
    idx = np.unique(np.concatenate([rng.integers(0, D, size=1 << 20), edges]))
    terns = np.zeros((M, idx.size), dtype=np.int8)
    ref_scales = np.zeros(M, dtype=np.float32)
    gpu_scales = scales.cpu().numpy()
    for m in range(M):
        row = g[m].cpu().numpy()
        tern, s, delta, n = O.threshold_quantize(row)
        assert n > 0 and delta > 0
        assert np.array_equal(U.codes_np(codes[m]), O.pack_codes(tern)), "codes of worker %d" % m
        assert np.float32(s).view(np.uint32) == gpu_scales[m].view(np.uint32), "scale of worker %d" % m
        terns[m] = tern[idx]
        ref_scales[m] = s
        del row, tern
    q = O.decode_average(terns, ref_scales)
    idx_t = torch.from_numpy(idx).to(dev)
    x0s, h0s, z0s = (v[idx_t].cpu().numpy() for v in (x0, h0, z0))
    x_ref, h_ref, a = O.cmd_step(q, x0s, h0s, LAM, ETA, DELTA)
    U.assert_close(xc[idx_t], x_ref, "x (QCMD)")
    U.assert_close(hc[idx_t], h_ref, "h (QCMD)")
    U.assert_zero_pattern(xc[idx_t], x_ref, a, LAM)
    x_ref, h_ref, z_ref, a = O.rda_step(q, h0s, z0s, T_STEP, LAM, ETA, DELTA)
    U.assert_close(xr[idx_t], x_ref, "x (QRDA)")
    U.assert_close(hr[idx_t], h_ref, "h (QRDA)")
    U.assert_close(zr[idx_t], z_ref, "z (QRDA)", atol=U.ATOL + 2.0 ** -23 * (np.abs(z0s) + np.abs(q)))
    U.assert_zero_pattern(xr[idx_t], x_ref, a, LAM)
    assert (x_ref == 0).any() and (x_ref != 0).any()
    ctx.close()


def test_more_than_2_to_31_coordinates():
    """One worker with d = 2^31 + 4099 coordinates: coordinate, byte and word indices pass 2^31 and the
    row is longer than 2^33 bytes.  Threshold, scale, count and the complete code row are compared."""
    try:
        import psutil
        if psutil.virtual_memory().available < 80 * 2 ** 30:
            pytest.skip("needs 80 GB of host memory for the oracle")
    except ImportError:
        pass
    if not torch.cuda.is_available() or torch.cuda.get_device_properties(0).total_memory < 40 * 2 ** 30:
        pytest.skip("needs 40 GB of device memory")
    d = (1 << 31) + 4099
    ld = (d + 3) // 4 * 4
    dev = U.dev()
    g = inputs.normal_gradients(d, 1, seed=6, device=dev, ld=ld)
    ctx = libqasg.Context(d, 1, device=0, flags=libqasg.CREATE_NO_CODE_SCRATCH)
    codes = torch.zeros((1, libqasg.code_words(d)), dtype=torch.int32, device=dev)
    scales = torch.zeros(1, dtype=torch.float32, device=dev)
    thr = torch.zeros(1, dtype=torch.float32, device=dev)
    cnt = torch.zeros(1, dtype=torch.int64, device=dev)
    ctx.quantize_pack(g, d, ld, 1, 1, libqasg.make_params(), codes, scales, thr, cnt)
    assert ctx.last_async_status() == libqasg.OK
    row = g[0, :d].cpu().numpy()
    tern, s, delta, n = O.threshold_quantize(row)
    del row
    assert thr.cpu().numpy()[0].view(np.uint32) == np.float32(delta).view(np.uint32)
    assert scales.cpu().numpy()[0].view(np.uint32) == np.float32(s).view(np.uint32)
    assert int(cnt.cpu().numpy()[0]) == n
    got = U.codes_np(codes[0])
    half = (tern.size // 32) * 16          # pack in two pieces to bound the oracle's temporaries
    assert np.array_equal(got[: half // 16], O.pack_codes(tern[:half]))
    assert np.array_equal(got[half // 16:], O.pack_codes(tern[half:]))
    del got
    # pass C over the same row: both rules read the oracle's own code words and scale (uploaded, not the
    # kernel's), and the iterates are compared on sampled coordinates on both sides of 2^31 and at the ends
    rng = np.random.default_rng(7)
    idx = np.unique(np.concatenate([rng.integers(0, d, size=1 << 19), np.arange(0, 4100), np.arange(d - 4200, d),
                                    (1 << 31) + np.arange(-4100, 4099), (1 << 30) + np.arange(-16, 16)]))
    q = O.decode_average(tern[idx][None, :], np.array([s], dtype=np.float32))
    codes[0, : half // 16].copy_(torch.from_numpy(O.pack_codes(tern[:half]).view(np.int32)))
    codes[0, half // 16:].copy_(torch.from_numpy(O.pack_codes(tern[half:]).view(np.int32)))
    del tern
    scales.copy_(torch.from_numpy(np.array([s], dtype=np.float32)))
    idx_t = torch.from_numpy(idx).to(dev)
    x, h, z = inputs.random_state(d, seed=6, device=dev)
    x0s, h0s, z0s = (v[idx_t].cpu().numpy() for v in (x, h, z))
    gbar = torch.empty(d, dtype=torch.float32, device=dev)
    ctx.decode_average(codes, scales, d, 1, gbar)
    U.assert_close(gbar[idx_t], q, "decoded average")
    params = libqasg.make_params(LAM, ETA, DELTA)
    ctx.cmd_step(gbar, x, h, d, T_STEP, params)
    x_ref, h_ref, a = O.cmd_step(q, x0s, h0s, LAM, ETA, DELTA)
    U.assert_close(x[idx_t], x_ref, "x (QCMD, dense q)")
    U.assert_close(h[idx_t], h_ref, "h (QCMD, dense q)")
    U.assert_zero_pattern(x[idx_t], x_ref, a, LAM)
    del gbar
    # the fused form: quantize again (same codes, checked above) and update in pass C
    x, h, z = inputs.random_state(d, seed=6, device=dev)
    ctx.step(libqasg.RULE_CMD, g, d, ld, 1, T_STEP, params, x, h, None, codes_out=codes)
    U.assert_close(x[idx_t], x_ref, "x (QCMD)")
    U.assert_close(h[idx_t], h_ref, "h (QCMD)")
    U.assert_zero_pattern(x[idx_t], x_ref, a, LAM)
    x, h, z = inputs.random_state(d, seed=6, device=dev)
    ctx.step(libqasg.RULE_RDA, g, d, ld, 1, T_STEP, params, x, h, z, codes_out=codes)
    x_ref, h_ref, z_ref, a = O.rda_step(q, h0s, z0s, T_STEP, LAM, ETA, DELTA)
    U.assert_close(x[idx_t], x_ref, "x (QRDA)")
    U.assert_close(h[idx_t], h_ref, "h (QRDA)")
    U.assert_close(z[idx_t], z_ref, "z (QRDA)", atol=U.ATOL + 2.0 ** -23 * (np.abs(z0s) + np.abs(q)))
    U.assert_zero_pattern(x[idx_t], x_ref, a, LAM)
    assert ctx.last_async_status() == libqasg.OK
    ctx.close()


def test_sparse_form_at_the_size_of_the_sparse_logistic_workload():
    """d = 2^24, 16 workers, minibatch 1024 rows of ~61 entries (the sparse-feature workload), gradients
    held in sparse form: touched bits exact, gradient values within tolerance, then one QRDA step fed
    with the oracle's gradient: thresholds, scales and all code rows exact, iterates on a sample."""
    from oracle import logreg_oracle as L
    from tests.test_gpu_logreg import G_ATOL, G_RTOL
    if not _enough_memory():
        pytest.skip("needs 40 GB of device memory and 24 GB of host memory")
    dev = U.dev()
    d, n, m_workers, batch, t = 1 << 24, 1 << 16, 16, 1024, 3
    lam, eta, delta = 1e-5, 0.1, 1e-8
    prob = inputs.logreg_csr_problem(n=n, d=d, M=m_workers, nnz_per_row=80, seed=3)
    rng = np.random.default_rng(8)
    x0 = (rng.standard_normal(d) * 0.1 * (rng.random(d) < 0.01)).astype(np.float32)
    h0 = (rng.random(d) * 1e-4).astype(np.float32)
    z0 = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    ctx = libqasg.Context(d, m_workers, device=0)
    dev_args = [U.to_dev(prob[k]) for k in ("rowptr", "colidx", "vals", "y")]
    g = torch.zeros((m_workers, d), dtype=torch.float32, device=dev)
    bits = torch.zeros((m_workers, d // 32), dtype=torch.int32, device=dev)
    ctx.logreg_grad_csr_touched(*dev_args, n, d, m_workers, prob["shard_row0"], None, batch, t, U.to_dev(x0), g, d, bits)

    touched = L.touched_columns(prob["rowptr"], prob["colidx"], prob["shard_row0"], batch, t, d)
    assert np.array_equal(bits.cpu().numpy().view(np.uint32), np.stack([O.pack_bits(r) for r in touched]))
    g64 = L.grad_workers_csr(prob["rowptr"], prob["colidx"], prob["vals"], prob["y"], prob["shard_row0"], batch, t,
                             x0.astype(np.float64), d)
    got = g.cpu().numpy()
    assert not got[~touched].any()
    where = np.nonzero(touched)
    err = np.abs(got[where].astype(np.float64) - g64[where])
    assert (err <= G_ATOL * np.abs(g64).max() + G_RTOL * np.abs(g64[where])).all()
    assert 200_000 < where[0].size < 1_000_000

    g32 = np.where(touched, g64.astype(np.float32), np.float32(np.nan))
    del g64, got
    params = libqasg.make_params(lam, eta, delta)
    codes = torch.zeros((m_workers, libqasg.code_words(d)), dtype=torch.int32, device=dev)
    scales = torch.zeros(m_workers, dtype=torch.float32, device=dev)
    x, h, z = U.to_dev(x0), U.to_dev(h0), U.to_dev(z0)
    g.copy_(torch.from_numpy(g32))
    ctx.step_touched(libqasg.RULE_RDA, g, d, d, m_workers, t, params, bits, x, h, z, codes_out=codes, scales_out=scales)
    assert ctx.last_async_status() == libqasg.OK

    idx = np.unique(np.concatenate([rng.integers(0, d, size=1 << 18), np.arange(0, 8200), np.arange(d - 4100, d)]))
    terns = np.zeros((m_workers, idx.size), dtype=np.int8)
    ref_scales = np.zeros(m_workers, dtype=np.float32)
    dense = O.densify_touched(g32, touched)
    for m in range(m_workers):
        tern, s, thr, cnt = O.threshold_quantize(dense[m])
        assert cnt > 0
        assert np.array_equal(U.codes_np(codes[m]), O.pack_codes(tern)), "codes of worker %d" % m
        assert np.float32(s).view(np.uint32) == scales.cpu().numpy()[m].view(np.uint32), "scale of worker %d" % m
        terns[m], ref_scales[m] = tern[idx], s
    q = O.decode_average(terns, ref_scales)
    x_ref, h_ref, z_ref, a = O.rda_step(q, h0[idx], z0[idx], t, lam, eta, delta)
    idx_t = torch.from_numpy(idx).to(dev)
    U.assert_close(x[idx_t], x_ref, "x")
    U.assert_close(h[idx_t], h_ref, "h")
    U.assert_close(z[idx_t], z_ref, "z", atol=U.ATOL + 2.0 ** -23 * (np.abs(z0[idx]) + np.abs(q)))
    U.assert_zero_pattern(x[idx_t], x_ref, a, lam)
    ctx.close()


def test_stochastic_quantizer_at_2_to_26_coordinates(tmp_path):
    """The unbiased ternary quantizer at d = 2^26, M = 8 (the largest size its timings are quoted at): every
    worker's scale, count and complete code row against the oracle, whose Philox draws and comparisons
    run one worker per host process, in slices; then the fused QCMD step on sampled coordinates."""
    from tests import _oracle_pool as P
    if not _enough_memory():
        pytest.skip("needs 40 GB of device memory and 24 GB of host memory")
    dev = U.dev()
    d, m_workers, t, seed = 1 << 26, 8, T_STEP, (0xC0FFEE << 20) | 77
    g = inputs.student_t_gradients(d, m_workers, seed=9, device=dev)
    jobs = []
    for m in range(m_workers):
        path = str(tmp_path / ("row%d.npy" % m))
        np.save(path, g[m].cpu().numpy())
        jobs.append((path, m, t, seed, 1 << 22))
    ctx = libqasg.Context(d, m_workers, device=0)
    params = libqasg.make_params(LAM, ETA, DELTA, quantizer=libqasg.Q_TERNARY_STOCH, seed=seed)
    codes = torch.zeros((m_workers, libqasg.code_words(d)), dtype=torch.int32, device=dev)
    scales = torch.zeros(m_workers, dtype=torch.float32, device=dev)
    counts = torch.zeros(m_workers, dtype=torch.int64, device=dev)
    x0, h0, _ = inputs.random_state(d, seed=9, device=dev)
    x, h = x0.clone(), h0.clone()
    ctx.quantize_pack(g, d, d, m_workers, t, params, codes, scales, None, counts)
    codes2 = torch.zeros_like(codes)
    ctx.step(libqasg.RULE_CMD, g, d, d, m_workers, t, params, x, h, None, codes_out=codes2)
    assert ctx.last_async_status() == libqasg.OK
    assert torch.equal(codes, codes2)
    del codes2
    got_codes, got_scales, got_counts = U.codes_np(codes), scales.cpu().numpy(), counts.cpu().numpy()
    rng = np.random.default_rng(10)
    idx = np.unique(np.concatenate([rng.integers(0, d, size=1 << 19), np.arange(0, 4100), np.arange(d - 4100, d)]))
    terns = np.zeros((m_workers, idx.size), dtype=np.int8)
    ref_scales = np.zeros(m_workers, dtype=np.float32)
    for m, words, scale, count in P.run(P.stochastic_row, jobs):
        assert np.array_equal(got_codes[m], words), "codes of worker %d" % m
        assert np.float32(scale).view(np.uint32) == got_scales[m].view(np.uint32), "scale of worker %d" % m
        assert count == int(got_counts[m]) and 0 < count < d
        terns[m] = O.unpack_codes(words, d)[idx]
        ref_scales[m] = scale
    q = O.decode_average(terns, ref_scales)
    idx_t = torch.from_numpy(idx).to(dev)
    x_ref, h_ref, a = O.cmd_step(q, x0[idx_t].cpu().numpy(), h0[idx_t].cpu().numpy(), LAM, ETA, DELTA)
    U.assert_close(x[idx_t], x_ref, "x (QCMD)")
    U.assert_close(h[idx_t], h_ref, "h (QCMD)")
    U.assert_zero_pattern(x[idx_t], x_ref, a, LAM)
    ctx.close()


def test_thirty_two_workers_at_2_to_26_coordinates():
    """d = 2^26, M = 32 (the eight-coordinate decode of pass C at the size it is timed at): every worker's
    threshold, scale and complete code row, then both rules' iterates on sampled coordinates."""
    if not _enough_memory():
        pytest.skip("needs 40 GB of device memory and 24 GB of host memory")
    dev = U.dev()
    d, m_workers = 1 << 26, 32
    g = inputs.normal_gradients(d, m_workers, seed=4, device=dev)
    x0, h0, z0 = inputs.random_state(d, seed=4, device=dev)
    ctx = libqasg.Context(d, m_workers, device=0)
    params = libqasg.make_params(LAM, ETA, DELTA)
    codes = torch.zeros((m_workers, libqasg.code_words(d)), dtype=torch.int32, device=dev)
    scales = torch.zeros(m_workers, dtype=torch.float32, device=dev)
    xc, hc = x0.clone(), h0.clone()
    ctx.step(libqasg.RULE_CMD, g, d, d, m_workers, T_STEP, params, xc, hc, None, codes_out=codes, scales_out=scales)
    xr, hr, zr = x0.clone(), h0.clone(), z0.clone()
    ctx.step(libqasg.RULE_RDA, g, d, d, m_workers, T_STEP, params, xr, hr, zr)
    assert ctx.last_async_status() == libqasg.OK
    rng = np.random.default_rng(11)
    # both ends, and both sides of the places where one CTA's share of the coordinates ends and the next begins
    seams = ((8 * 512 * 296 * np.arange(1, 8))[:, None] + np.arange(-9, 9)[None, :]).ravel()
    idx = np.unique(np.concatenate([rng.integers(0, d, size=1 << 19), np.arange(0, 4100), np.arange(d - 4100, d), seams]))
    terns = np.zeros((m_workers, idx.size), dtype=np.int8)
    ref_scales = np.zeros(m_workers, dtype=np.float32)
    gpu_scales = scales.cpu().numpy()
    for m in range(m_workers):
        tern, s, delta, n = O.threshold_quantize(g[m].cpu().numpy())
        assert n > 0 and delta > 0
        assert np.array_equal(U.codes_np(codes[m]), O.pack_codes(tern)), "codes of worker %d" % m
        assert np.float32(s).view(np.uint32) == gpu_scales[m].view(np.uint32), "scale of worker %d" % m
        terns[m], ref_scales[m] = tern[idx], s
    q = O.decode_average(terns, ref_scales)
    idx_t = torch.from_numpy(idx).to(dev)
    x0s, h0s, z0s = (v[idx_t].cpu().numpy() for v in (x0, h0, z0))
    x_ref, h_ref, a = O.cmd_step(q, x0s, h0s, LAM, ETA, DELTA)
    U.assert_close(xc[idx_t], x_ref, "x (QCMD)")
    U.assert_close(hc[idx_t], h_ref, "h (QCMD)")
    U.assert_zero_pattern(xc[idx_t], x_ref, a, LAM)
    x_ref, h_ref, z_ref, a = O.rda_step(q, h0s, z0s, T_STEP, LAM, ETA, DELTA)
    U.assert_close(xr[idx_t], x_ref, "x (QRDA)")
    U.assert_close(hr[idx_t], h_ref, "h (QRDA)")
    U.assert_close(zr[idx_t], z_ref, "z (QRDA)", atol=U.ATOL + 2.0 ** -23 * (np.abs(z0s) + np.abs(q)))
    U.assert_zero_pattern(xr[idx_t], x_ref, a, LAM)
    ctx.close()
