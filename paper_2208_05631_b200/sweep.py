"""Timing sweeps of libqasg on one GPU, beyond the single workload bench.py reports.

  python -m paper_2208_05631_b200.sweep step   [--quantizer threshold|stochastic] [--double-quant] [--select]
                                               [--min-log2-d 20] [--max-log2-d 28] [--workers 2,4,8,16,32]
  python -m paper_2208_05631_b200.sweep logreg [--steps 50] [--graph] [--csr-only]
  python -m paper_2208_05631_b200.sweep optimal [--min-log2-d 20] [--max-log2-d 28] [--workers 8]
  python -m paper_2208_05631_b200.sweep touched [--steps 50]

`step`   - the fused step over d in {2^20 .. 2^28} x M in {2, 4, 8, 16, 32} simulated workers,
           N(0,1) gradients, both update rules (the paper uses 2-4 workers; this is the scaling
           of the step in d and in the number of workers).  L2 is flushed before every timed
           step, so small sizes are not flattered by gradients that stay in the 126 MB L2.
`logreg` - the two L1-logistic-regression workloads: gradient kernel + fused step per iteration.
           dense: X 65536 x 4096, 8 workers, minibatch 512; sparse: 10^6 x 2^24 CSR, ~80 non-zeros
           per row, 16 workers, minibatch 1024.

`optimal` - the threshold quantizer with the 0.75 * mean|g| rule against the exact optimal threshold
           (sort + prefix sums): time of each and the relative quantization error each reaches, on
           N(0,1) and on Student-t(3) gradients.

`touched` - passes A and B on rows held in sparse form for synthetic patterns of stored entries (d = 2^24,
           16 workers): none, uniform, Zipf-like, full head tiles; replayed from a CUDA graph (both kernels).

`--graph` captures one iteration (fixed step index) in a CUDA graph and replays it: every call of the
library only enqueues kernels on the given stream, so a launch-bound loop can be replayed without
the host in the way.

Prints one JSON line per measured point.  Every number is device time from CUDA events.
"""
import argparse
import json

import numpy as np
import torch

from . import inputs, libqasg

LAM, ETA, DELTA, T_STEP = 1e-3, 0.1, 1e-8, 16


def _flush_l2(buf):
    buf.add_(1.0)


def _time_calls(fn, reps, flush_buf):
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    for _ in range(reps):
        if flush_buf is not None:
            _flush_l2(flush_buf)
        start.record()
        fn()
        stop.record()
        torch.cuda.synchronize()
        times.append(start.elapsed_time(stop))
    return float(np.median(times)), float(min(times))


def sweep_step(args):
    dev = torch.device("cuda", 0)
    flush = torch.zeros(64 << 20, dtype=torch.float32, device=dev)      # 256 MB > L2
    quantizer = libqasg.Q_THRESHOLD if args.quantizer == "threshold" else libqasg.Q_TERNARY_STOCH
    params = libqasg.make_params(LAM, ETA, DELTA, quantizer=quantizer, seed=4)
    for log2d in range(args.min_log2_d, args.max_log2_d + 1, 2):
        d = 1 << log2d
        for M in [int(v) for v in args.workers.split(",")]:
            g = inputs.normal_gradients(d, M, seed=4, device=dev)
            x, h, z = inputs.random_state(d, seed=4, device=dev)
            ctx = libqasg.Context(d, M, device=0)
            for rule, name, state_bytes in ((libqasg.RULE_CMD, "qcmd", 16), (libqasg.RULE_RDA, "qrda", 20)):
                def one():
                    if args.select:
                        ctx.step_select(rule, args.double_quant, g, d, d, M, T_STEP, params, x, h, z)
                    elif args.double_quant:
                        ctx.step_double(rule, g, d, d, M, T_STEP, params, x, h, z)
                    else:
                        ctx.step(rule, g, d, d, M, T_STEP, params, x, h, z)
                for _ in range(3):
                    one()
                torch.cuda.synchronize()
                med, best = _time_calls(one, args.reps, flush)
                ctx.profile_begin()
                one()
                kernel_ms = {k: v[0] / v[1] for k, v in ctx.profile_end().items()}
                # bytes the method must move: g twice, worker codes written and read once, state once;
                # double quantization reads the worker codes three times and writes/reads the server's codes
                moved = d * (8.0 * M + M / 2.0 + state_bytes)
                if args.double_quant:
                    moved = d * (8.0 * M + M / 4.0 + 2.0 * M / 4.0 + 2 * 0.25 + state_bytes)
                what = "step" + ("_select" if args.select else "") + ("_double" if args.double_quant else "")
                print(json.dumps({"what": what, "quantizer": args.quantizer,
                                  "rule": name, "d": d, "M": M, "ms_median": med, "ms_best": best,
                                  "coord_workers_per_s": d * M / (med * 1e-3),
                                  "gbs_moved": moved / 1e9 / (med * 1e-3), "kernel_ms": kernel_ms}), flush=True)
            assert ctx.last_async_status() == libqasg.OK
            ctx.close()
            del g, x, h, z
            torch.cuda.empty_cache()


def _timed_graph(it, warm, steps):
    """Captures one call of `it` in a CUDA graph and times `steps` replays (device time per replay, us)."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(warm):
            it()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        it()
    for _ in range(warm):
        graph.replay()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        graph.replay()
    stop.record()
    torch.cuda.synchronize()
    return start.elapsed_time(stop) * 1e3 / steps


def _timed_iterations(ctx, it, warm, steps):
    for _ in range(warm):
        it()
    torch.cuda.synchronize()
    ctx.profile_begin()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        it()
    stop.record()
    torch.cuda.synchronize()
    kernels = ctx.profile_end()
    return start.elapsed_time(stop) * 1e3 / steps, {k: v[0] * 1e3 / v[1] for k, v in kernels.items()}


def sweep_logreg(args):
    dev = torch.device("cuda", 0)
    # dense: "L1-regularised logistic regression, dense synthetic"
    n, d, M, B = 65536, 4096, 8, 512
    prob = inputs.logreg_dense_problem(n=n, d=d, M=M, seed=1)
    X, y = torch.from_numpy(prob["X"]).to(dev), torch.from_numpy(prob["y"]).to(dev)
    ctx = libqasg.Context(1 << 24, 16, device=0)
    for rule, name in (() if args.csr_only else ((libqasg.RULE_CMD, "qcmd"), (libqasg.RULE_RDA, "qrda"))):
        params = libqasg.make_params(1e-4, ETA, DELTA)
        x, h, z = (torch.zeros(d, dtype=torch.float32, device=dev) for _ in range(3))
        g = torch.empty((M, d), dtype=torch.float32, device=dev)
        t = [0]

        def it():
            t[0] += 1
            ctx.logreg_grad_dense(X, y, n, d, M, prob["shard_row0"], None, B, t[0], x, g, d)
            ctx.step(rule, g, d, d, M, t[0], params, x, h, z)
        us, kernel_us = _timed_iterations(ctx, it, 5, args.steps)
        graph_us = _timed_graph(it, 3, args.steps) if args.graph else None
        print(json.dumps({"what": "logreg_dense", "rule": name, "n": n, "d": d, "M": M, "B": B,
                          "us_per_iteration": us, "us_per_graph_replay": graph_us, "kernel_us": kernel_us,
                          "nnz_x": int((x != 0).sum().item())}), flush=True)
    del X, y
    # sparse: "sparse-feature logistic regression"
    n, d, M, B = args.csr_rows, 1 << 24, 16, 1024
    prob = inputs.logreg_csr_problem(n=n, d=d, M=M, nnz_per_row=80, seed=3)
    dev_args = [torch.from_numpy(prob[k]).to(dev) for k in ("rowptr", "colidx", "vals", "y")]
    params = libqasg.make_params(1e-5, ETA, DELTA)
    x, h, z = (torch.zeros(d, dtype=torch.float32, device=dev) for _ in range(3))
    g = torch.empty((M, d), dtype=torch.float32, device=dev)
    t = [0]

    def it_csr():
        t[0] += 1
        ctx.logreg_grad_csr(*dev_args, n, d, M, prob["shard_row0"], None, B, t[0], x, g, d)
        ctx.step(libqasg.RULE_RDA, g, d, d, M, t[0], params, x, h, z)
    us, kernel_us = _timed_iterations(ctx, it_csr, 3, args.steps)
    graph_us = _timed_graph(it_csr, 3, args.steps) if args.graph else None
    print(json.dumps({"what": "logreg_csr", "rule": "qrda", "n": n, "d": d, "M": M, "B": B,
                      "nnz": int(prob["rowptr"][-1]), "us_per_iteration": us, "us_per_graph_replay": graph_us,
                      "kernel_us": kernel_us,
                      "nnz_x": int((x != 0).sum().item())}), flush=True)
    # the same iteration with the gradients held in sparse form (touched bits; g stays zero elsewhere)
    x.zero_(), h.zero_(), z.zero_(), g.zero_()
    bits = torch.zeros((M, d // 32), dtype=torch.int32, device=dev)
    t[0] = 0

    def it_touched():
        t[0] += 1
        ctx.logreg_grad_csr_touched(*dev_args, n, d, M, prob["shard_row0"], None, B, t[0], x, g, d, bits)
        ctx.step_touched(libqasg.RULE_RDA, g, d, d, M, t[0], params, bits, x, h, z)
    us, kernel_us = _timed_iterations(ctx, it_touched, 3, args.steps)
    graph_us = _timed_graph(it_touched, 3, args.steps) if args.graph else None
    words = bits.cpu().numpy().view("uint32").ravel()
    touched = int(sum(bin(int(w)).count("1") for w in words[words != 0]))
    print(json.dumps({"what": "logreg_csr_touched", "rule": "qrda", "n": n, "d": d, "M": M, "B": B,
                      "nnz": int(prob["rowptr"][-1]), "touched_last_step": touched,
                      "us_per_iteration": us, "us_per_graph_replay": graph_us, "kernel_us": kernel_us,
                      "nnz_x": int((x != 0).sum().item())}), flush=True)
    assert ctx.last_async_status() == libqasg.OK
    ctx.close()


def sweep_optimal(args):
    """The 0.75 * mean|g| rule against the exact optimal threshold: time of each quantizer and the
    quantization error ||g - s*tern||^2 / ||g||^2 = 1 - n s^2 / ||g||^2 each one reaches."""
    dev = torch.device("cuda", 0)
    M = int(args.workers.split(",")[0])
    for log2_d in range(args.min_log2_d, args.max_log2_d + 1, 2):
        d = 1 << log2_d
        ctx = libqasg.Context(d, M, device=0)
        scratch = torch.empty(libqasg.optimal_scratch_bytes(d), dtype=torch.uint8, device=dev)
        params = libqasg.make_params(LAM, ETA, DELTA)
        flush = torch.zeros(64 << 20, dtype=torch.float32, device=dev)      # 256 MB > L2
        for name, gen in (("normal", inputs.normal_gradients), ("student_t3", inputs.student_t_gradients)):
            g = gen(d, M, seed=4, device=dev)
            sq = (g.double() ** 2).sum(dim=1)
            codes = torch.empty((M, libqasg.code_words(d)), dtype=torch.int32, device=dev)
            out = {}
            for which in ("rule", "optimal"):
                scales = torch.zeros(M, dtype=torch.float32, device=dev)
                thr = torch.zeros(M, dtype=torch.float32, device=dev)
                cnt = torch.zeros(M, dtype=torch.int64, device=dev)

                def run():
                    if which == "rule":
                        ctx.quantize_pack(g, d, d, M, 1, params, codes, scales, thr, cnt)
                    else:
                        ctx.quantize_pack_optimal(g, d, d, M, params, codes, scales, scratch, thr, cnt)
                run()
                ms_median, _ = _time_calls(run, args.reps, flush)
                err = 1.0 - cnt.double() * scales.double() ** 2 / sq
                out[which] = {"ms_median": ms_median,
                              "threshold_over_mean_abs": (thr.double() / g.abs().double().mean(dim=1)).tolist(),
                              "kept_fraction": (cnt.double() / d).tolist(),
                              "relative_sq_error": err.tolist()}
            print(json.dumps({"what": "optimal_vs_rule", "input": name, "d": d, "M": M, **out}), flush=True)
            del g
        assert ctx.last_async_status() == libqasg.OK
        ctx.close()
        del scratch


def _bits_from_columns(columns, d, dev):
    """columns: one int64 tensor of column ids per worker -> touched words int32 [M, d/32]."""
    rows = []
    for cols in columns:
        cols = torch.unique(cols)
        acc = torch.zeros(d // 32, dtype=torch.int64, device=dev)
        acc.index_put_(((cols >> 5),), torch.ones_like(cols) << (cols & 31), accumulate=True)   # distinct bits: sum == or
        rows.append(torch.where(acc >= 2 ** 31, acc - 2 ** 32, acc).to(torch.int32))
    return torch.stack(rows)


def sweep_touched(args):
    """Passes A and B on rows held in sparse form, for synthetic patterns of stored entries (d = 2^24, M = 16):
    how the time depends on the number of entries and on where they sit."""
    dev = torch.device("cuda", 0)
    d, M = 1 << 24, 16
    ctx = libqasg.Context(d, M, device=0)
    params = libqasg.make_params(1e-5, ETA, DELTA)
    g = torch.randn((M, d), device=dev) * 0.01
    codes = torch.empty((M, libqasg.code_words(d)), dtype=torch.int32, device=dev)
    scales = torch.zeros(M, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1)
    cdf = torch.cumsum(torch.arange(1, d + 1, device=dev, dtype=torch.float64) ** -1.1, 0)
    cdf = cdf / cdf[-1].clone()

    def uniform(n):
        return [torch.randint(0, d, (n,), device=dev, generator=gen) for _ in range(M)]

    def zipf(n):
        return [torch.searchsorted(cdf, torch.rand(n, device=dev, dtype=torch.float64, generator=gen)).clamp(max=d - 1)
                for _ in range(M)]
    cases = [("no entry", [torch.zeros(0, dtype=torch.int64, device=dev)] * M),
             ("25 000 uniform draws per worker", uniform(25_000)),
             ("250 000 uniform draws per worker", uniform(250_000)),
             ("62 000 Zipf(1.1) draws per worker", zipf(62_000)),
             ("the first tile full", [torch.arange(0, 4096, device=dev)] * M),
             ("the first 16 tiles full", [torch.arange(0, 16 * 4096, device=dev)] * M)]
    for name, columns in cases:
        bits = _bits_from_columns(columns, d, dev)

        def run():
            ctx.quantize_pack_touched(g, d, d, M, 1, params, bits, codes, scales)
        graph_us = _timed_graph(run, 3, args.steps)
        entries = int(sum(torch.unique(c).numel() for c in columns))
        print(json.dumps({"what": "touched_passes_A_B", "pattern": name, "d": d, "M": M, "stored_entries": entries,
                          "us_per_graph_replay": graph_us}), flush=True)
    assert ctx.last_async_status() == libqasg.OK
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["step", "logreg", "optimal", "touched"])
    ap.add_argument("--quantizer", default="threshold", choices=["threshold", "stochastic"])
    ap.add_argument("--double-quant", action="store_true")
    ap.add_argument("--select", action="store_true")
    ap.add_argument("--min-log2-d", type=int, default=20)
    ap.add_argument("--max-log2-d", type=int, default=28)
    ap.add_argument("--workers", default="2,4,8,16,32")
    ap.add_argument("--reps", type=int, default=7)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--csr-rows", type=int, default=1_000_000)
    ap.add_argument("--graph", action="store_true")
    ap.add_argument("--csr-only", action="store_true")
    args = ap.parse_args()
    assert torch.cuda.is_available(), "needs a CUDA device"
    if args.what == "optimal":
        sweep_optimal(args)
    elif args.what == "touched":
        sweep_touched(args)
    elif args.what == "step":
        sweep_step(args)
    else:
        sweep_logreg(args)


if __name__ == "__main__":
    main()
