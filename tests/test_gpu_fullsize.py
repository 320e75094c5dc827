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
    del g
    tern, s, delta, n = O.threshold_quantize(row)
    del row
    assert thr.cpu().numpy()[0].view(np.uint32) == np.float32(delta).view(np.uint32)
    assert scales.cpu().numpy()[0].view(np.uint32) == np.float32(s).view(np.uint32)
    assert int(cnt.cpu().numpy()[0]) == n
    got = U.codes_np(codes[0])
    half = (tern.size // 32) * 16          # pack in two pieces to bound the oracle's temporaries
    assert np.array_equal(got[: half // 16], O.pack_codes(tern[:half]))
    assert np.array_equal(got[half // 16:], O.pack_codes(tern[half:]))
    ctx.close()
