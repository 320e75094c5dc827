"""Helpers shared by the GPU parity tests (not a test module)."""
import numpy as np
import torch

from paper_2208_05631_b200 import libqasg

ATOL, RTOL = 1e-7, 1e-5          # iterates: |gpu - oracle| <= ATOL + RTOL * |oracle|
ZERO_BAND = 1e-6                 # zero pattern may differ where |a - lambda| <= ZERO_BAND


def dev():
    return torch.device("cuda:0")


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(dev())


def grad_to_dev(g, pad_value=float("nan")):
    """numpy [M, d] -> device [M, ld] with ld = d rounded up to 4 plus 4; the padding holds
    `pad_value` so that a kernel that reads past d is caught."""
    g = np.asarray(g, dtype=np.float32)
    M, d = g.shape
    ld = (d + 3) // 4 * 4 + 4
    buf = np.full((M, ld), pad_value, dtype=np.float32)
    buf[:, :d] = g
    return to_dev(buf), ld


def assert_close(got, want, what="", atol=ATOL):
    got = got.detach().cpu().numpy().astype(np.float64) if isinstance(got, torch.Tensor) else np.asarray(got, np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = np.abs(got - want)
    bound = atol + RTOL * np.abs(want)
    bad = np.nonzero(err > bound)[0]
    assert bad.size == 0, "%s: %d of %d outside tolerance; worst at %d: got %r want %r" % (
        what, bad.size, want.size, bad[0], got[bad[0]], want[bad[0]])


def assert_zero_pattern(x_gpu, x_ref, a_ref, lam):
    """Zeros agree wherever the compared quantity is not within ZERO_BAND of lambda, and
    every zero is +0.0."""
    xg = x_gpu.detach().cpu().numpy()
    lam = float(np.float32(lam))
    decided = np.abs(np.asarray(a_ref) - lam) > ZERO_BAND
    assert np.array_equal((xg == 0)[decided], (np.asarray(x_ref) == 0)[decided])
    assert not np.signbit(xg[xg == 0]).any()


def new_codes(M, d):
    # poisoned so that unwritten words are noticed
    return torch.full((M, libqasg.code_words(d)), 0x7FFFFFFF, dtype=torch.int32, device=dev())


def codes_np(codes):
    return codes.cpu().numpy().view(np.uint32)


def f32_bits(a):
    a = a.detach().cpu().numpy() if isinstance(a, torch.Tensor) else np.asarray(a, dtype=np.float32)
    return a.view(np.uint32)
