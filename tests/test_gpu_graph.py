"""qasg_step only enqueues kernels on the caller's stream (no allocation, no synchronisation), so a
launch-bound loop can be captured once in a CUDA graph and replayed.  The replayed steps must give
exactly the bits of eagerly launched ones."""
import numpy as np
import pytest
import torch

from paper_2208_05631_b200 import inputs, libqasg

pytestmark = pytest.mark.gpu


# the step as three chained launches (option 0) and as the default picks it (one launch at this size)
@pytest.mark.parametrize("one_launch_bytes", [0, None])
@pytest.mark.parametrize("rule", [libqasg.RULE_CMD, libqasg.RULE_RDA])
def test_fused_step_replayed_from_a_cuda_graph(rule, one_launch_bytes):
    dev = torch.device("cuda:0")
    d, M, t = 40_003, 8, 5
    ld = (d + 3) // 4 * 4
    g = torch.zeros((M, ld), dtype=torch.float32, device=dev)
    g[:, :d] = torch.from_numpy(inputs.optimizer_only_gradients(d, M, t, seed=2) * np.float32(0.01)).to(dev)
    x0, h0, z0 = inputs.random_state(d, seed=2, device=dev)
    ctx = libqasg.Context(d, M, device=0)
    if one_launch_bytes is not None:
        ctx.set_option(libqasg.OPT_ONE_LAUNCH_STEP_BYTES, one_launch_bytes)
    params = libqasg.make_params(1e-3, 0.1, 1e-8)

    eager = [v.clone() for v in (x0, h0, z0)]
    for _ in range(3):
        ctx.step(rule, g, d, ld, M, t, params, *eager)
    torch.cuda.synchronize()

    state = [v.clone() for v in (x0, h0, z0)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):                      # warm-up outside the capture
        warm = [v.clone() for v in (x0, h0, z0)]
        ctx.step(rule, g, d, ld, M, t, params, *warm)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx.step(rule, g, d, ld, M, t, params, *state)
    for v, v0 in zip(state, (x0, h0, z0)):
        v.copy_(v0)                                    # the capture itself ran nothing
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    for got, want in zip(state, eager):
        assert torch.equal(got, want)
    assert ctx.last_async_status() == libqasg.OK
    ctx.close()


@pytest.mark.parametrize("one_launch_bytes", [0, None])
def test_chained_launches_give_the_bits_of_serial_launches(one_launch_bytes):
    """By default a step's kernels are launched as programmatic dependents of one another (a kernel is placed,
    and pass B requests its first tile, while its predecessor drains).  The same iterations on a context
    created with QASG_CREATE_SERIAL_LAUNCHES must give the same bits: gradient kernel + fused step, both
    quantizers, state carried over ten iterations."""
    dev = torch.device("cuda:0")
    n, d, M, B = 4096, 1024, 8, 64
    prob = inputs.logreg_dense_problem(n=n, d=d, M=M, seed=1)
    X, y = torch.from_numpy(prob["X"]).to(dev), torch.from_numpy(prob["y"]).to(dev)
    results = []
    for flags in (0, libqasg.CREATE_SERIAL_LAUNCHES):
        ctx = libqasg.Context(d, M, device=0, flags=flags)
        if one_launch_bytes is not None:
            ctx.set_option(libqasg.OPT_ONE_LAUNCH_STEP_BYTES, one_launch_bytes)
        out = []
        for quantizer in (libqasg.Q_THRESHOLD, libqasg.Q_TERNARY_STOCH):
            params = libqasg.make_params(1e-4, 0.1, 1e-8, quantizer=quantizer, seed=5)
            for rule in (libqasg.RULE_CMD, libqasg.RULE_RDA):
                x, h, z = (torch.zeros(d, dtype=torch.float32, device=dev) for _ in range(3))
                g = torch.empty((M, d), dtype=torch.float32, device=dev)
                codes = torch.zeros((M, libqasg.code_words(d)), dtype=torch.int32, device=dev)
                for t in range(1, 11):
                    ctx.logreg_grad_dense(X, y, n, d, M, prob["shard_row0"], None, B, t, x, g, d)
                    ctx.step(rule, g, d, d, M, t, params, x, h, z, codes_out=codes)
                torch.cuda.synchronize()
                out += [x.clone(), h.clone(), z.clone(), codes.clone()]
        assert ctx.last_async_status() == libqasg.OK
        ctx.close()
        results.append(out)
    for a, b in zip(*results):
        assert torch.equal(a, b)
    assert any(bool(t.any()) for t in results[0])
