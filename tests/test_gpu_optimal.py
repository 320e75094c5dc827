"""GPU parity of the threshold quantizer at the exact optimal threshold (rank, fixed-order prefix sums,
first maximum of the objective) against the oracle: Delta*, |I_Delta*|, codes and scales bit for bit."""
import numpy as np
import pytest
import torch

from oracle import qasg_oracle as O
from paper_2208_05631_b200 import inputs, libqasg
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = libqasg.Context(4_000_000, 8, device=0)
    yield c
    c.close()


def _rows(kind, d, M, seed):
    rng = np.random.default_rng(seed)
    if kind == "normal":
        g = inputs.normal_gradients(d, M, seed=seed).numpy() * np.float32(0.03)
    elif kind == "heavy":
        g = inputs.student_t_gradients(d, M, seed=seed).numpy()
    elif kind == "ties":      # few distinct magnitudes, many zeros: candidates are the strict drops only
        g = (np.round(rng.standard_normal((M, d)) * 4) / 8).astype(np.float32)
    else:
        raise ValueError(kind)
    return np.ascontiguousarray(g[:, :d], dtype=np.float32)


def _run(ctx, g):
    M, d = g.shape
    g_dev, ld = U.grad_to_dev(g)
    codes = U.new_codes(M, d)
    scales = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    thr = torch.full((M,), -1.0, dtype=torch.float32, device=U.dev())
    cnt = torch.full((M,), -1, dtype=torch.int64, device=U.dev())
    scratch = torch.empty(libqasg.optimal_scratch_bytes(d), dtype=torch.uint8, device=U.dev())
    ctx.quantize_pack_optimal(g_dev, d, ld, M, libqasg.make_params(1e-3, 0.1, 1e-8), codes, scales, scratch, thr, cnt)
    assert ctx.last_async_status() == libqasg.OK
    return U.codes_np(codes), scales, thr, cnt.cpu().numpy()


@pytest.mark.parametrize("kind", ["normal", "heavy", "ties"])
@pytest.mark.parametrize("d,M", [(1, 1), (7, 2), (1023, 3), (4096, 1), (3 * 4096 + 5, 2), (70_001, 4),
                                 ((1 << 20) + 4321, 2), (3_000_001, 1)])
def test_optimal_threshold_quantizer_bit_exact(ctx, kind, d, M):
    g = _rows(kind, d, M, seed=d % 1013 + M)
    codes, scales, thr, cnt = _run(ctx, g)
    for m in range(M):
        tern, s, delta, n = O.optimal_threshold_quantize(g[m])
        assert U.f32_bits(thr)[m] == U.f32_bits(np.float32(delta)), (m, float(thr[m]), float(delta))
        assert int(cnt[m]) == n
        assert np.array_equal(codes[m], O.pack_codes(tern))
        assert U.f32_bits(scales)[m] == U.f32_bits(np.float32(s))
    if kind == "normal" and d > 50_000:
        # the rule of Section 3.5 lands close to it on Gaussian data
        assert abs(float(thr[0]) / (0.75 * np.abs(g[0]).mean()) - 1) < 0.1


def test_degenerate_rows(ctx):
    d = 5000
    g = np.zeros((3, d), dtype=np.float32)
    g[1] = -2.5                                    # all equal: everything kept, threshold 0
    g[2, 17] = 3.0                                 # a single non-zero entry
    codes, scales, thr, cnt = _run(ctx, g)
    assert cnt.tolist() == [0, d, 1]
    assert thr.cpu().numpy().tolist() == [0.0, 0.0, 0.0]
    assert scales.cpu().numpy().tolist() == [0.0, 2.5, 3.0]
    assert not codes[0].any() and (codes[1] == 0xAAAAAAAA).sum() == d // 16


def test_optimal_argument_errors(ctx):
    d, M = 4096, 1
    g = torch.zeros((M, d), dtype=torch.float32, device=U.dev())
    codes, scales = U.new_codes(M, d), torch.zeros(M, dtype=torch.float32, device=U.dev())
    small = torch.empty(1024, dtype=torch.uint8, device=U.dev())
    with pytest.raises(libqasg.QasgError) as e:
        ctx.quantize_pack_optimal(g, d, d, M, libqasg.make_params(1e-3, 0.1, 1e-8), codes, scales, small)
    assert e.value.status == libqasg.ERR_WORKSPACE
    stoch = libqasg.make_params(1e-3, 0.1, 1e-8, quantizer=libqasg.Q_TERNARY_STOCH)
    big = torch.empty(libqasg.optimal_scratch_bytes(d), dtype=torch.uint8, device=U.dev())
    with pytest.raises(libqasg.QasgError) as e:
        ctx.quantize_pack_optimal(g, d, d, M, stoch, codes, scales, big)
    assert e.value.status == libqasg.ERR_INVALID_ARG
    assert libqasg.optimal_scratch_bytes(1 << 31) == 0
