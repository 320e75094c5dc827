"""qasg_quantize_pack_static, the entry point for callers that cannot allocate device memory
(a framework that owns all of it through its own pool, or a loop that cannot take the
synchronisation an allocation implies).  It keeps its scratch in a fixed array inside the
library instead of a context's workspace, so its results must be exactly those of
qasg_quantize_pack.  Checked through the C-ABI on two calls in a row: the second, smaller
call runs over whatever the first left in the shared array.

This file is collected last on purpose, so a run that stops at the first failure has
already run every other test."""
import numpy as np
import pytest
import torch

from paper_2208_05631_b200 import inputs, libqasg

pytestmark = pytest.mark.gpu


def _both_ways(ctx, g_np, coef=0.75):
    dev = torch.device("cuda:0")
    M, d = g_np.shape
    ld = (d + 3) // 4 * 4
    g = torch.zeros((M, ld), dtype=torch.float32, device=dev)
    g[:, :d] = torch.from_numpy(g_np).to(dev)
    out = []
    for static in (False, True):
        codes = torch.full((M, libqasg.code_words(d)), 0x7FFFFFFF, dtype=torch.int32, device=dev)
        scales = torch.full((M,), -1.0, dtype=torch.float32, device=dev)
        thresholds = torch.full((M,), -1.0, dtype=torch.float32, device=dev)
        counts = torch.full((M,), -1, dtype=torch.int64, device=dev)
        if static:
            libqasg.quantize_pack_static(0, g, d, ld, M, coef, codes, scales, thresholds, counts)
        else:
            ctx.quantize_pack(g, d, ld, M, 1, libqasg.make_params(thr_coef=coef), codes, scales, thresholds, counts)
        torch.cuda.synchronize()
        out.append([t.cpu().numpy() for t in (codes, scales, thresholds, counts)])
    return out


def test_static_scratch_entry_point_matches_quantize_pack_twice_in_a_row():
    ctx = libqasg.Context(6_000_000, 16, device=0)
    first = inputs.normal_gradients(5_000_001, 3, seed=11).numpy()       # several tiles per chunk, ragged tail
    second = inputs.optimizer_only_gradients(10_000, 16, t=2, seed=12)  # fewer chunks, more workers
    for g in (first, second):
        want, got = _both_ways(ctx, g)
        for a, b in zip(want, got):
            assert np.array_equal(a.view(np.uint32) if a.dtype == np.float32 else a,
                                  b.view(np.uint32) if b.dtype == np.float32 else b)
        assert got[3].min() > 0
    ctx.close()


def test_static_scratch_entry_point_rejects_what_it_cannot_hold():
    dev = torch.device("cuda:0")
    M = libqasg.STATIC_MAX_WORKERS + 1
    g = torch.zeros((M, 64), dtype=torch.float32, device=dev)
    codes = torch.zeros((M, 4), dtype=torch.int32, device=dev)
    scales = torch.zeros(M, dtype=torch.float32, device=dev)
    with pytest.raises(libqasg.QasgError) as e:
        libqasg.quantize_pack_static(0, g, 64, 64, M, 0.75, codes, scales)
    assert e.value.status == libqasg.ERR_WORKSPACE
    with pytest.raises(libqasg.QasgError) as e:
        libqasg.quantize_pack_static(0, g, 64, 62, 2, 0.75, codes, scales)
    assert e.value.status == libqasg.ERR_INVALID_ARG
