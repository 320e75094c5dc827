#!/usr/bin/env python
"""Benchmark of the quantized adaptive-subgradient step (libqasg) on synthetic workloads.

  python bench.py [--config 1|2|3|4|5|optimal|touched] [--gpus N] [--steps K] [--warmup W]
                  [--impl ours|reference] [--quantizer threshold|stochastic|none] [--variant step|double|select] [--state-density P]

Workloads (--config; default 3, the headline):
  1  optimizer-only QCMD run: d = 10,000, M = 4, g ~ N(0,1)(1+0.1m), 100 iterations from x = h = 0;
     one bench step = the whole 100-iteration run.
  2  dense L1 logistic regression: X 65536 x 4096, M = 8 shards, minibatch 512; one bench step = one
     iteration (gradient kernel + fused step) of QCMD and one of QRDA.
  3  bandwidth-bound single step: d = 2^28, M = 8, gradients 1e-2 * Student-t(3), random state, t = 16;
     one bench step = one fused QCMD step + one fused QRDA step, each from the stated state.
  4  sparse-feature logistic regression: CSR 10^6 x 2^24, ~80 non-zeros per row, M = 16, minibatch 1024,
     QRDA; one bench step = one iteration with the gradients held in sparse form.
  5  the fused step over d in {2^20 .. 2^28} x M in {2, 4, 8, 16, 32}, N(0,1) gradients, both rules;
     one bench step = one pass over the whole grid (median of --steps repetitions per point).
  optimal, touched: side measurements (exact optimal threshold against the 0.75 rule; passes A and B on
     rows held in sparse form for synthetic patterns); one line per point.

Prints ONE JSON line per run (the side measurements: one per point).  Times are device times from CUDA
events; with N > 1 (torchrun) every rank runs an independent replica and the slowest rank's time counts.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2208_05631_b200 import inputs  # noqa: E402

METRIC = "fused quantized step coords*workers/s and HBM GB/s vs 8 TB/s peak (d=2^28, M=8)"
UNIT = "coords*workers/s"
LAM, ETA, DELTA, T_STEP, SEED = 1e-3, 0.1, 1e-8, 16, 2
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 << 20


# ------------------------------------------------------------------ byte accounting
def bytes_per_coord(M):
    """Algorithmic bytes per coordinate of each kernel of the fused step (fp32 state, 2-bit codes):
    what the method itself must move through device memory."""
    return {
        "abs_sum": 4.0 * M,                       # read g
        "abs_max": 4.0 * M,
        "threshold_codes": 4.0 * M + M / 4.0,     # read g again, write codes
        "stochastic_codes": 4.0 * M + M / 4.0,
        # one launch, each row coded out of L2 right after it was summed: g crosses device memory once
        "quantize_stream_threshold": 4.0 * M + M / 4.0,
        "quantize_stream_stochastic": 4.0 * M + M / 4.0,
        "decode_update_cmd": M / 4.0 + 16.0,      # read codes; h, x read + write
        "decode_update_rda": M / 4.0 + 20.0,      # read codes; h, z read + write; x write
        "mean_update_cmd": 4.0 * M + 16.0,        # no quantization: read g once; h, x read + write
        "mean_update_rda": 4.0 * M + 20.0,
    }


def step_bytes(M, rule, once_through=False):
    """Bytes per coordinate of one fused step: g read twice (threshold, then codes) unless the row is
    coded out of L2 (`once_through`), codes written and read once, state once."""
    state = 16.0 if rule == "qcmd" else 20.0
    return (4.0 * M if once_through else 8.0 * M) + M / 2.0 + state


def minimal_bytes(M, rule):
    """The least a step can move: every gradient once, the state once (codes never leave the chip)."""
    return 4.0 * M + (16.0 if rule == "qcmd" else 20.0)


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per coordinate at M = 8 of the two-launch
# quantizer's kernels, from one ncu capture at d = 2^24 (both kernels stream, so their traffic grows in
# proportion to d).  Valid only for the kernel source it was taken from (checked by hash).
NCU_TRAFFIC = {
    "kernels_sha256": "afcae0653967ed52d457675782f346e923cf18e16314d94894f1e1a64c4b6d06",
    "M": 8,
    "bytes_per_coord": {"abs_sum": 540856320 / 2 ** 24, "threshold_codes": 567921664 / 2 ** 24},
}


def ncu_traffic(kernel, d, M):
    """Bytes per launch from the stored ncu counters, or None once the kernels have changed."""
    import hashlib
    digest = hashlib.sha256()
    try:
        for name in ("qasg_device.cuh", "qasg_kernels.cu"):   # the step kernels and what they inline
            with open(os.path.join(ROOT, "paper_2208_05631_b200", "csrc", name), "rb") as f:
                digest.update(f.read())
        same = digest.hexdigest() == NCU_TRAFFIC["kernels_sha256"]
    except OSError:
        same = False
    if not same or M != NCU_TRAFFIC["M"] or kernel not in NCU_TRAFFIC["bytes_per_coord"]:
        return None
    return NCU_TRAFFIC["bytes_per_coord"][kernel] * d


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU from a thread while the timed region runs
    (NVML in-process, every few ms; the main thread waits inside CUDA calls that release the GIL)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index):
        self.index, self.sm, self.bits, self.max_mhz = index, [], 0, None
        self.stop_flag = threading.Event()
        self.thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nvml = pynvml
            # CUDA_VISIBLE_DEVICES may renumber devices: address the GPU by the UUID torch reports
            uuid = torch.cuda.get_device_properties(index).uuid
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            # first calls are slow: make them before the timed region
            pynvml.nvmlDeviceGetClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
            pynvml.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
        except Exception:
            self.nvml = None

    def _loop(self):
        n = self.nvml
        while not self.stop_flag.is_set():
            try:
                self.sm.append(float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)))
                self.bits |= int(n.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nvml is None:
            return
        self.thread = threading.Thread(target=self._loop, daemon=True)
        self.thread.start()
        time.sleep(0.01)

    def stop(self):
        if self.nvml is None or self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvml unavailable"]}
        self.stop_flag.set()
        self.thread.join(timeout=2)
        reasons = sorted(name for bit, name in self.REASONS.items() if self.bits & bit)
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.max_mhz,
                "samples": len(self.sm), "reasons": reasons}


# ------------------------------------------------------------------ multi-rank aggregation
def max_over_ranks(ms, dist, device):
    """Slowest rank's time: every rank runs an independent replica, the job is as slow as the slowest."""
    if dist is None:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world, d, M, ms_per_step):
    """Coordinate-workers per second over all replicas: one bench step is 2 fused steps of d*M."""
    return world * 2.0 * d * M / (ms_per_step * 1e-3)


class Rig:
    """Device, process group and timing helpers of one rank."""

    def __init__(self, args):
        assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        torch.cuda.set_device(self.local)
        self.dev = torch.device("cuda", self.local)
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=self.dev)
            self.dist = dist
        self.args = args
        self._flush = None

    def fence(self):
        torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
            torch.cuda.synchronize()

    def flush_l2(self):
        """Writes a buffer twice the size of L2, so that nothing of the workload is left in it."""
        if self._flush is None:
            self._flush = torch.zeros(2 * L2_BYTES // 4, dtype=torch.float32, device=self.dev)
        self._flush.add_(1.0)

    def timed(self, fn, steps, warmup, before_each=None):
        """Device time of `steps` calls of fn, each bracketed by its own pair of CUDA events on the current
        stream (so that `before_each`, e.g. restoring the state or flushing L2, stays outside).
        Returns the list of per-call milliseconds."""
        for _ in range(warmup):
            if before_each:
                before_each()
            fn()
        self.fence()
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for start, stop in pairs:
            if before_each:
                before_each()
            start.record()
            fn()
            stop.record()
        self.fence()
        return [s.elapsed_time(e) for s, e in pairs]

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def graph_of(fn, warm=3):
    """Captures one call of fn (which only enqueues library kernels on the current stream) in a CUDA graph."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(warm):
            fn()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        fn()
    return graph


def kernel_table(kernels, units):
    """Per-kernel averages from qasg_profile_end; units[name] = algorithmic bytes per launch (or absent)."""
    total = sum(v[0] for v in kernels.values()) or 1.0
    out = {}
    for name, (ms, n) in kernels.items():
        avg = ms / n
        algo = units.get(name)
        out[name] = {"launches": n, "avg_ms": avg, "share": ms / total,
                     "algorithmic_gb": None if algo is None else algo / 1e9,
                     "gbs": None if algo is None else algo / 1e9 / (avg * 1e-3)}
    return out


def roofline_of(per_kernel, units, traffic=None):
    peak, kind = measured_peak()
    top = max(per_kernel, key=lambda k: per_kernel[k]["share"])
    gbs = per_kernel[top]["gbs"]
    return {"bound": "hbm", "kernel": top, "achieved": gbs, "peak": peak, "peak_kind": kind, "unit": "GB/s",
            "frac": None if gbs is None else gbs / peak,
            "frac_of_nominal_8tbs": None if gbs is None else gbs / NOMINAL_HBM_GBS,
            "algorithmic_bytes": units.get(top), "traffic": traffic(top) if traffic else None,
            "per_kernel": per_kernel}


def emit(rig, args, **fields):
    line = {"metric": METRIC, "unit": UNIT, "n_gpus": rig.world, "steps": args.steps, "warmup": args.warmup,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic"}
    line.update(fields)
    print(json.dumps(line), flush=True)


def quantizer_of(args, libqasg):
    return {"threshold": libqasg.Q_THRESHOLD, "stochastic": libqasg.Q_TERNARY_STOCH, "none": libqasg.Q_NONE}[args.quantizer]


def fused_call(ctx, libqasg, args, rule, g, d, ld, M, t, params, x, h, z):
    """The call a bench step makes for --variant."""
    if args.variant == "double":
        ctx.step_double(rule, g, d, ld, M, t, params, x, h, z)
    elif args.variant == "select":
        ctx.step_select(rule, 0, g, d, ld, M, t, params, x, h, z)
    else:
        ctx.step(rule, g, d, ld, M, t, params, x, h, z)


# ------------------------------------------------------------------ the CPU oracle legs
def oracle_single_step(d_sample, M, steps, warmup, processes=1):
    """Times the CPU oracle (as it stands) on the first d_sample coordinates of workload 3: one QCMD step +
    one QRDA step per bench step.  processes > 1: the same oracle functions driven over that many host
    processes (workers in parallel for the quantizer, coordinate ranges for the update).
    Returns (units/s, seconds per step)."""
    from oracle import qasg_oracle as O
    g = inputs.student_t_gradients(d_sample, M, seed=SEED).numpy()
    x0, h0, z0 = (v.numpy().astype(np.float64) for v in inputs.random_state(d_sample, seed=SEED))
    times = []
    if processes <= 1:
        for i in range(warmup + steps):
            t0 = time.perf_counter()
            O.step(O.RULE_CMD, g, x0, h0, None, T_STEP, LAM, ETA, DELTA)
            O.step(O.RULE_RDA, g, x0, h0, z0, T_STEP, LAM, ETA, DELTA)
            if i >= warmup:
                times.append(time.perf_counter() - t0)
    else:
        from oracle import harness
        with harness.Harness(processes) as hs:
            path_g = hs.put("g", g)
            px, ph, pz = (hs.put(n, v) for n, v in (("x", x0), ("h", h0), ("z", z0)))
            for i in range(warmup + steps):
                t0 = time.perf_counter()
                hs.step(O.RULE_CMD, path_g, M, d_sample, [px, ph, None], T_STEP, LAM, ETA, DELTA)
                hs.step(O.RULE_RDA, path_g, M, d_sample, [px, ph, pz], T_STEP, LAM, ETA, DELTA)
                if i >= warmup:
                    times.append(time.perf_counter() - t0)
    per_step = float(np.mean(times))
    return 2.0 * d_sample * M / per_step, per_step


def cpu_baseline_single_step(d, M):
    """Both oracle legs beside the GPU number of workload 3: 1 process, then all host cores."""
    d_sample = min(d, 1 << 25)
    sample = "first %d coordinates of every worker's gradient, one QCMD + one QRDA oracle step" % d_sample
    v1, s1 = oracle_single_step(d_sample, M, steps=1, warmup=0)
    cores = os.cpu_count() or 1
    out = {"value": v1, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": s1, "sample": sample}
    if cores > 1:
        va, sa = oracle_single_step(d_sample, M, steps=1, warmup=0, processes=cores)
        out["all_cores"] = {"value": va, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": sa,
                            "sample": sample + "; the same oracle functions over %d processes" % cores}
    return out


def run_reference(args):
    """The reference arm: the oracle, as it stands, on the host cores, on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import qasg_oracle as O
    cfg = str(args.config)
    if cfg == "3":
        d_sample, M = min(args.d, 1 << 21), args.M
        value, per_step = oracle_single_step(d_sample, M, args.steps, args.warmup)
        sample = "first %d coordinates of every worker's gradient, both rules, per step" % d_sample
        workload = workload_3(args, "cpu oracle on a bounded sample: " + sample)
    elif cfg == "1":
        d, M, T = 10_000, 4, 100
        times = []
        for i in range(args.warmup + args.steps):
            x, h = np.zeros(d), np.zeros(d)
            t0 = time.perf_counter()
            for t in range(1, T + 1):
                out = O.step(O.RULE_CMD, inputs.optimizer_only_gradients(d, M, t, seed=0), x, h, None, t, 1e-3, 0.1, 1e-8)
                x, h = out["x"], out["h"]
            if i >= args.warmup:
                times.append(time.perf_counter() - t0)
        per_step = float(np.mean(times))
        value = T * d * M / per_step
        sample = "the whole run (100 iterations, gradient generation included)"
        workload = {"workload": WORKLOAD_1, "note": "cpu oracle: " + sample}
    elif cfg == "5":
        d, M = 1 << 20, 8
        g = inputs.normal_gradients(d, M, seed=4).numpy()
        x0, h0, z0 = (v.numpy().astype(np.float64) for v in inputs.random_state(d, seed=4))
        times = []
        for i in range(args.warmup + args.steps):
            t0 = time.perf_counter()
            O.step(O.RULE_CMD, g, x0, h0, None, T_STEP, LAM, ETA, DELTA)
            O.step(O.RULE_RDA, g, x0, h0, z0, T_STEP, LAM, ETA, DELTA)
            if i >= args.warmup:
                times.append(time.perf_counter() - t0)
        per_step = float(np.mean(times))
        value = 2.0 * d * M / per_step
        sample = "the grid point d = 2^20, M = 8 only, both rules"
        workload = {"workload": WORKLOAD_5, "note": "cpu oracle: " + sample}
    else:
        from oracle import logreg_oracle as L
        if cfg == "2":
            prob = inputs.logreg_dense_problem(n=8192, d=4096, M=8, seed=1)
            d, M, B, lam = 4096, 8, 512, 1e-4
            grad = lambda t, x: L.grad_workers_dense(prob["X"], prob["y"], prob["shard_row0"], B, t, x)   # noqa: E731
            rules = (O.RULE_CMD, O.RULE_RDA)
            sample = "8192 of the 65536 rows (the minibatches are the same size), both rules"
            workload = {"workload": WORKLOAD_2, "note": "cpu oracle: " + sample}
        else:
            prob = inputs.logreg_csr_problem(n=1 << 15, d=1 << 20, M=16, nnz_per_row=80, seed=3)
            d, M, B, lam = 1 << 20, 16, 1024, 1e-5
            grad = lambda t, x: L.grad_workers_csr(prob["rowptr"], prob["colidx"], prob["vals"], prob["y"],   # noqa: E731
                                                   prob["shard_row0"], B, t, x, d)
            rules = (O.RULE_RDA,)
            sample = "d = 2^20 features and 2^15 rows instead of 2^24 and 10^6 (minibatches the same size)"
            workload = {"workload": WORKLOAD_4, "note": "cpu oracle: " + sample}
        times = []
        state = {rule: dict(x=np.zeros(d), h=np.zeros(d), z=np.zeros(d)) for rule in rules}
        for i in range(args.warmup + args.steps):
            t0 = time.perf_counter()
            for rule in rules:
                s = state[rule]
                out = O.step(rule, grad(i + 1, s["x"]).astype(np.float32), s["x"], s["h"], s["z"], i + 1, lam, 0.1, 1e-8)
                s["x"], s["h"] = out["x"], out["h"]
                if rule == O.RULE_RDA:
                    s["z"] = out["z"]
            if i >= args.warmup:
                times.append(time.perf_counter() - t0)
        per_step = float(np.mean(times))
        value = len(rules) * d * M / per_step
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------ workload 3: the headline
def workload_3(args, note):
    return {"workload": "bandwidth-bound single step: d=%d fp32, M=%d, gradients 1e-2*Student-t(3), "
                        "x,z~0.1*N(0,1), h~U[0,1), t=%d, lambda=%g, eta=%g, delta=%g, seed %d; one fused QCMD "
                        "step + one fused QRDA step per bench step, each from the stated state (restored, "
                        "untimed, before every step)" % (args.d, args.M, T_STEP, LAM, ETA, DELTA, SEED),
            "d": args.d, "M": args.M, "quantizer": args.quantizer, "variant": args.variant, "rules": ["qcmd", "qrda"],
            "state_density": args.state_density,
            "l2": "inputs (%.1f GiB of gradients) are larger than L2 and the state restore (%.1f GiB copied) "
                  "passes through it between steps" % (args.d * args.M * 4 / 2 ** 30, 5 * args.d * 4 / 2 ** 30),
            "parallelism": "replicas" if args.gpus > 1 else "single", "note": note}


def run_config3(rig, args):
    from paper_2208_05631_b200 import libqasg
    dev, d, M = rig.dev, args.d, args.M
    g = inputs.student_t_gradients(d, M, seed=SEED + rig.rank, device=dev)
    x0, h0, z0 = inputs.random_state(d, seed=SEED + rig.rank, device=dev)
    if args.state_density < 1.0:   # a sparse iterate: the selection masks are then mixed in every tile
        x0 *= inputs.bernoulli_mask(d, args.state_density, seed=SEED + rig.rank, device=dev)
    xc, hc = x0.clone(), h0.clone()                 # QCMD state
    xr, hr, zr = x0.clone(), h0.clone(), z0.clone()  # QRDA state
    ctx = new_context(libqasg, rig, args, d, M)
    params = libqasg.make_params(LAM, ETA, DELTA, quantizer=quantizer_of(args, libqasg), seed=SEED)

    def restore():
        xc.copy_(x0), hc.copy_(h0), xr.copy_(x0), hr.copy_(h0), zr.copy_(z0)

    def bench_step():
        fused_call(ctx, libqasg, args, libqasg.RULE_CMD, g, d, d, M, T_STEP, params, xc, hc, None)
        fused_call(ctx, libqasg, args, libqasg.RULE_RDA, g, d, d, M, T_STEP, params, xr, hr, zr)

    for _ in range(max(3, args.warmup)):
        restore()
        bench_step()
    rig.fence()
    sampler = ClockSampler(rig.local)
    if rig.rank == 0:
        sampler.start()
    launches0 = ctx.launch_count()
    ctx.profile_begin()
    times = rig.timed(bench_step, args.steps, 0, before_each=restore)
    kernels = ctx.profile_end()
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop() if rig.rank == 0 else None
    assert ctx.last_async_status() == libqasg.OK
    ms_per_step = max_over_ranks(sum(times), rig.dist, dev) / args.steps
    value = whole_job_value(rig.world, d, M, ms_per_step)

    e2e = None
    if args.e2e_steps > 0 and args.variant == "step":
        e2e = e2e_single_step(rig, args, ctx, params, g, x0, h0, z0)
    if rig.rank != 0:
        return

    bpc = bytes_per_coord(M)
    units = {k: v * d for k, v in bpc.items()}
    per_kernel = kernel_table(kernels, units)
    roofline = roofline_of(per_kernel, units, traffic=lambda k: ncu_traffic(k, d, M))
    once = 4.0 * d <= args.stream_row_bytes
    moved = (step_bytes(M, "qcmd", once) + step_bytes(M, "qrda", once)) * d
    minimal = (minimal_bytes(M, "qcmd") + minimal_bytes(M, "qrda")) * d
    peak, _ = measured_peak()
    sec = ms_per_step * 1e-3
    cpu = None
    if rig.world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline_single_step(d, M)
    emit(rig, args, value=value, ms_per_step=ms_per_step, config=workload_3(args, "inputs resident in HBM before the timed region"),
         clocks=clocks, e2e=e2e, gpu_launches=launches, roofline=roofline, cpu_baseline=cpu,
         hbm={"minimal_bytes_per_step_gb": minimal / 1e9,
              "minimal_bytes_frac_of_nominal_8tbs": minimal / 1e9 / sec / NOMINAL_HBM_GBS,
              "minimal_bytes_note": "each gradient once + the state once (the stated roofline); at this size a row "
                                    "(%.0f MiB) does not fit on chip and is read twice, see bytes_moved" % (4.0 * d / 2 ** 20),
              "bytes_moved_per_step_gb": moved / 1e9, "gbs_moved": moved / 1e9 / sec,
              "bytes_moved_frac_of_nominal_8tbs": moved / 1e9 / sec / NOMINAL_HBM_GBS,
              "bytes_moved_frac_of_peak": moved / 1e9 / sec / peak})


def new_context(libqasg, rig, args, d, M):
    ctx = libqasg.Context(d, M, device=rig.local)
    if args.stream_row_bytes:
        ctx.set_option(libqasg.OPT_STREAM_ROW_BYTES, args.stream_row_bytes)
    if args.one_launch_step_bytes is not None:
        ctx.set_option(libqasg.OPT_ONE_LAUNCH_STEP_BYTES, args.one_launch_step_bytes)
    return ctx


def e2e_single_step(rig, args, ctx, params, g, x0, h0, z0):
    """The same bench step through qasg_step_host: gradients and state start in pinned host memory,
    the new state ends there; host<->device copies are inside the timed region."""
    from paper_2208_05631_b200 import libqasg
    d, M, dev = args.d, args.M, rig.dev
    try:
        gh = torch.empty((M, d), dtype=torch.float32, pin_memory=True)
        gh.copy_(g)
        host = [torch.empty(d, dtype=torch.float32, pin_memory=True) for _ in range(5)]
    except RuntimeError as e:  # not enough pinned host memory on this machine
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": None, "d2h_bytes_per_step": None,
                "error": "pinned host allocation failed: %s" % str(e).splitlines()[0]}
    xch, hch, xrh, hrh, zrh = host
    xd, hd, zd = (torch.empty(d, dtype=torch.float32, device=dev) for _ in range(3))
    steps = max(1, min(args.steps, args.e2e_steps))

    def restore():
        for dst, src in ((xch, x0), (hch, h0), (xrh, x0), (hrh, h0), (zrh, z0)):
            dst.copy_(src)

    def host_step():
        ctx.step_host(libqasg.RULE_CMD, gh, d, d, M, T_STEP, params, xch, hch, None, g, xd, hd, None)
        ctx.step_host(libqasg.RULE_RDA, gh, d, d, M, T_STEP, params, xrh, hrh, zrh, g, xd, hd, zd)

    times = rig.timed(host_step, steps, 1, before_each=restore)
    ms = max_over_ranks(sum(times), rig.dist, dev) / steps
    vec = 4 * d
    h2d = 2 * 4 * d * M + (2 * vec) + (2 * vec)      # g twice; QCMD: x, h; QRDA: h, z
    d2h = (2 * vec) + (3 * vec)                      # QCMD: x, h; QRDA: x, h, z
    return {"value": whole_job_value(rig.world, d, M, ms), "unit": UNIT, "ms_per_step": ms,
            "steps": steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}


# ------------------------------------------------------------------ workload 1: optimizer-only run
WORKLOAD_1 = ("QCMD adagrad optimizer-only run: d=10000 fp32 parameters from 0, M=4, g^(m)~N(0,1)*(1+0.1m) fresh per "
              "iteration (seed 0), threshold quantizer, lambda=1e-3, eta=0.1, delta=1e-8, T=100 iterations; one bench "
              "step = the whole run")


def run_config1(rig, args):
    from paper_2208_05631_b200 import libqasg
    dev, d, M, T = rig.dev, 10_000, 4, 100
    ld = d
    gs = torch.stack([torch.from_numpy(inputs.optimizer_only_gradients(d, M, t, seed=0)) for t in range(1, T + 1)]).to(dev)
    x, h = (torch.zeros(d, dtype=torch.float32, device=dev) for _ in range(2))
    ctx = new_context(libqasg, rig, args, d, M)
    params = libqasg.make_params(1e-3, 0.1, 1e-8, quantizer=quantizer_of(args, libqasg), seed=0)

    def run():
        x.zero_(), h.zero_()
        for t in range(1, T + 1):
            ctx.step(libqasg.RULE_CMD, gs[t - 1], d, ld, M, t, params, x, h)

    sampler = ClockSampler(rig.local)
    eager = rig.timed(run, args.steps, max(3, args.warmup))
    graph = graph_of(run)
    if rig.rank == 0:
        sampler.start()
    launches0 = ctx.launch_count()
    replay = rig.timed(graph.replay, args.steps, max(3, args.warmup))
    clocks = sampler.stop() if rig.rank == 0 else None
    ctx.profile_begin()
    run()
    torch.cuda.synchronize()
    kernels = ctx.profile_end()
    assert ctx.last_async_status() == libqasg.OK
    nnz = int((x != 0).sum().item())
    ms = max_over_ranks(float(np.mean(replay)), rig.dist, dev)
    ms_eager = max_over_ranks(float(np.mean(eager)), rig.dist, dev)
    # end to end: every iteration's gradients come from pinned host memory, the iterate goes back
    gh = gs.cpu().pin_memory()
    xh, hh = (torch.zeros(d, dtype=torch.float32).pin_memory() for _ in range(2))
    gd = torch.empty((M, ld), dtype=torch.float32, device=dev)

    def host_run():
        xh.zero_(), hh.zero_()
        for t in range(1, T + 1):
            ctx.step_host(libqasg.RULE_CMD, gh[t - 1], d, ld, M, t, params, xh, hh, None, gd, x, h, None)
    e2e_ms = max_over_ranks(float(np.mean(rig.timed(host_run, max(1, min(args.steps, 5)), 1))), rig.dist, dev)
    if rig.rank != 0:
        return
    bpc = bytes_per_coord(M)
    units = {k: v * d for k, v in bpc.items()}
    per_kernel = kernel_table(kernels, units)
    emit(rig, args, value=rig.world * T * d * M / (ms * 1e-3), ms_per_step=ms,
         config={"workload": WORKLOAD_1, "d": d, "M": M, "iterations": T, "quantizer": args.quantizer,
                 "l2": "the whole workload (16 MB of gradients) fits in L2: not flushed, this run is bound by launches",
                 "note": "value: the run replayed from one CUDA graph (%d launches); eager from Python: see `eager`" % (2 * T)},
         us_per_iteration=ms * 1e3 / T, eager={"ms_per_step": ms_eager, "us_per_iteration": ms_eager * 1e3 / T},
         clocks=clocks, gpu_launches=(ctx.launch_count() - launches0) or 2 * T * args.steps,
         e2e={"value": rig.world * T * d * M / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
              "h2d_bytes_per_step": T * (M * d + 2 * d) * 4, "d2h_bytes_per_step": T * 2 * d * 4},
         roofline=roofline_of(per_kernel, units), cpu_baseline=None, nonzeros_in_x=nnz)


# ------------------------------------------------------------------ workloads 2 and 4: logistic regression
WORKLOAD_2 = ("L1-regularised logistic regression, dense synthetic: X 65536x4096 fp32 N(0,1), w* 5% non-zeros, "
              "y=sign(Xw*+0.1eps), M=8 shards, minibatch 512 per worker, lambda=1e-4, eta=0.1, delta=1e-8, seed 1; one "
              "bench step = one iteration (gradient + fused step) of QCMD and one of QRDA")
WORKLOAD_4 = ("sparse-feature logistic regression: CSR 10^6 x 2^24, ~80 non-zeros per row, columns Zipf(1.1), values "
              "log-normal(0,1) row-normalised, labels from a 1%-dense w*, M=16, minibatch 1024, QRDA, lambda=1e-5, "
              "eta=0.1, delta=1e-8, seed 3; one bench step = one iteration")


def _logreg_timing(rig, args, ctx, libqasg, iteration, reset, units_of, iters_per_graph=20):
    """Eager and graph-replayed device time per iteration, and the per-kernel profile of one pass."""
    steps, warm = max(args.steps, 20), max(3, args.warmup)
    reset()
    eager = rig.timed(iteration, steps, warm)
    reset()

    def block():
        for _ in range(iters_per_graph):
            iteration()
    graph = graph_of(block, warm=1)
    replay = rig.timed(graph.replay, max(3, steps // iters_per_graph), 2)
    reset()
    for _ in range(warm):
        iteration()
    torch.cuda.synchronize()
    ctx.profile_begin()
    for _ in range(10):
        iteration()
    torch.cuda.synchronize()
    kernels = ctx.profile_end()
    return (max_over_ranks(float(np.median(eager)), rig.dist, rig.dev),
            max_over_ranks(float(np.median(replay)), rig.dist, rig.dev) / iters_per_graph, kernels)


def run_config2(rig, args):
    from paper_2208_05631_b200 import libqasg
    dev = rig.dev
    n, d, M, B = 65536, 4096, 8, 512
    prob = inputs.logreg_dense_problem(n=n, d=d, M=M, seed=1)
    X, y = torch.from_numpy(prob["X"]).to(dev), torch.from_numpy(prob["y"]).to(dev)
    ctx = new_context(libqasg, rig, args, d, M)
    params = libqasg.make_params(1e-4, ETA, DELTA, quantizer=quantizer_of(args, libqasg), seed=1)
    state = {r: [torch.zeros(d, dtype=torch.float32, device=dev) for _ in range(3)] for r in (0, 1)}
    g = torch.empty((M, d), dtype=torch.float32, device=dev)
    t = [0]

    def reset():
        t[0] = 0
        for vs in state.values():
            for v in vs:
                v.zero_()

    def iteration():
        t[0] += 1
        for rule in (libqasg.RULE_CMD, libqasg.RULE_RDA):
            x, h, z = state[rule]
            ctx.logreg_grad_dense(X, y, n, d, M, prob["shard_row0"], None, B, t[0], x, g, d)
            ctx.step(rule, g, d, d, M, t[0], params, x, h, z)

    sampler = ClockSampler(rig.local)
    if rig.rank == 0:
        sampler.start()
    launches0 = ctx.launch_count()
    eager_ms, replay_ms, kernels = _logreg_timing(rig, args, ctx, libqasg, iteration, reset, None)
    clocks = sampler.stop() if rig.rank == 0 else None
    launches = ctx.launch_count() - launches0
    # end to end: the minibatch row ids come from the host every iteration, the status word goes back
    ids_host = torch.empty((M, B), dtype=torch.int32).pin_memory()
    ids_dev = torch.empty((M, B), dtype=torch.int32, device=dev)
    shard = np.asarray(prob["shard_row0"])

    def host_iteration():
        t[0] += 1
        for m in range(M):
            lo, size = int(shard[m]), int(shard[m + 1] - shard[m])
            ids_host[m] = torch.from_numpy((lo + ((t[0] - 1) * B + np.arange(B)) % size).astype(np.int32))
        ids_dev.copy_(ids_host, non_blocking=True)
        for rule in (libqasg.RULE_CMD, libqasg.RULE_RDA):
            x, h, z = state[rule]
            ctx.logreg_grad_dense(X, y, n, d, M, prob["shard_row0"], ids_dev, B, t[0], x, g, d)
            ctx.step(rule, g, d, d, M, t[0], params, x, h, z)
        assert ctx.last_async_status() == libqasg.OK
    reset()
    e2e_ms = max_over_ranks(float(np.median(rig.timed(host_iteration, 50, 3))), rig.dist, dev)
    assert ctx.last_async_status() == libqasg.OK
    if rig.rank != 0:
        return
    bpc = bytes_per_coord(M)
    units = {k: v * d for k, v in bpc.items()}
    units["logreg_dense"] = float(M * B * d * 4)          # the minibatch rows once (the second pass reads them from L2)
    per_kernel = kernel_table(kernels, units)
    emit(rig, args, value=rig.world * 2 * d * M / (replay_ms * 1e-3), ms_per_step=replay_ms,
         config={"workload": WORKLOAD_2, "d": d, "M": M, "quantizer": args.quantizer,
                 "l2": "per iteration 8 MiB of minibatch rows per rule out of a 1 GiB matrix: not flushed, "
                       "consecutive iterations read other rows",
                 "note": "value: iterations replayed from a CUDA graph (20 per graph); eager from Python: see `eager`"},
         us_per_iteration_pair=replay_ms * 1e3, eager={"ms_per_step": eager_ms},
         clocks=clocks, gpu_launches=launches,
         e2e={"value": rig.world * 2 * d * M / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
              "h2d_bytes_per_step": M * B * 4, "d2h_bytes_per_step": 4},
         roofline=roofline_of(per_kernel, units), cpu_baseline=None,
         nonzeros_in_x={"qcmd": int((state[0][0] != 0).sum().item()), "qrda": int((state[1][0] != 0).sum().item())})


def run_config4(rig, args):
    from paper_2208_05631_b200 import libqasg
    dev = rig.dev
    n, d, M, B = args.csr_rows, 1 << 24, 16, 1024
    prob = inputs.logreg_csr_problem(n=n, d=d, M=M, nnz_per_row=80, seed=3)
    dev_args = [torch.from_numpy(prob[k]).to(dev) for k in ("rowptr", "colidx", "vals", "y")]
    ctx = new_context(libqasg, rig, args, d, M)
    params = libqasg.make_params(1e-5, ETA, DELTA, quantizer=quantizer_of(args, libqasg), seed=3)
    x, h, z = (torch.zeros(d, dtype=torch.float32, device=dev) for _ in range(3))
    g = torch.zeros((M, d), dtype=torch.float32, device=dev)
    bits = torch.zeros((M, d // 32), dtype=torch.int32, device=dev)
    t = [0]

    def reset():
        t[0] = 0
        x.zero_(), h.zero_(), z.zero_(), g.zero_(), bits.zero_()

    def sparse_form():
        t[0] += 1
        ctx.logreg_grad_csr_touched(*dev_args, n, d, M, prob["shard_row0"], None, B, t[0], x, g, d, bits)
        ctx.step_touched(libqasg.RULE_RDA, g, d, d, M, t[0], params, bits, x, h, z)

    def dense_rows():
        t[0] += 1
        ctx.logreg_grad_csr(*dev_args, n, d, M, prob["shard_row0"], None, B, t[0], x, g, d)
        ctx.step(libqasg.RULE_RDA, g, d, d, M, t[0], params, x, h, z)

    sampler = ClockSampler(rig.local)
    if rig.rank == 0:
        sampler.start()
    launches0 = ctx.launch_count()
    eager_ms, replay_ms, kernels = _logreg_timing(rig, args, ctx, libqasg, sparse_form, reset, None, iters_per_graph=10)
    clocks = sampler.stop() if rig.rank == 0 else None
    launches = ctx.launch_count() - launches0
    nnz_x = int((x != 0).sum().item())
    dense_eager, dense_replay, dense_kernels = _logreg_timing(rig, args, ctx, libqasg, dense_rows, reset, None,
                                                              iters_per_graph=10)
    reset()

    def host_iteration():
        sparse_form()
        assert ctx.last_async_status() == libqasg.OK
    e2e_ms = max_over_ranks(float(np.median(rig.timed(host_iteration, 30, 3))), rig.dist, dev)
    if rig.rank != 0:
        return
    per_kernel = kernel_table(kernels, {})
    emit(rig, args, value=rig.world * d * M / (replay_ms * 1e-3), ms_per_step=replay_ms,
         config={"workload": WORKLOAD_4, "d": d, "M": M, "rows": n, "non_zeros": int(prob["rowptr"][-1]),
                 "quantizer": args.quantizer,
                 "l2": "not flushed: the touched sectors and 32 MiB of bits per pass; the state (3 x 64 MiB) does not stay in L2",
                 "note": "value: gradients held in sparse form, iterations replayed from a CUDA graph (10 per graph); "
                         "`dense_rows`: the same iteration with dense gradient rows"},
         us_per_iteration=replay_ms * 1e3, eager={"ms_per_step": eager_ms},
         dense_rows={"ms_per_step": dense_replay, "eager_ms_per_step": dense_eager,
                     "per_kernel": kernel_table(dense_kernels, {})},
         clocks=clocks, gpu_launches=launches,
         e2e={"value": rig.world * d * M / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
              "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 4,
              "note": "the minibatch is the default cyclic one (row ids computed on the device): nothing to copy in"},
         roofline=roofline_of(per_kernel, {}), cpu_baseline=None, nonzeros_in_x=nnz_x)


# ------------------------------------------------------------------ workload 5: the d x M grid
WORKLOAD_5 = ("scaling sweep of the fused step: d in {2^20, 2^22, 2^24, 2^26, 2^28} x M in {2, 4, 8, 16, 32}, N(0,1) "
              "gradients, random state, t=16, both update rules, seed 4; L2 flushed before every timed step; one bench "
              "step = one pass over the grid (per point the median of the timed repetitions)")


def run_config5(rig, args):
    from paper_2208_05631_b200 import libqasg
    dev = rig.dev
    params = libqasg.make_params(LAM, ETA, DELTA, quantizer=quantizer_of(args, libqasg), seed=4)
    grid, total_units, total_ms, launches = [], 0.0, 0.0, 0
    sampler = ClockSampler(rig.local)
    if rig.rank == 0:
        sampler.start()
    for log2d in range(args.min_log2_d, args.max_log2_d + 1, 2):
        d = 1 << log2d
        for M in [int(v) for v in args.workers.split(",")]:
            g = inputs.normal_gradients(d, M, seed=4, device=dev)
            x0, h0, z0 = inputs.random_state(d, seed=4, device=dev)
            x, h, z = x0.clone(), h0.clone(), z0.clone()
            ctx = new_context(libqasg, rig, args, d, M)
            for rule, name in ((libqasg.RULE_CMD, "qcmd"), (libqasg.RULE_RDA, "qrda")):
                def before():
                    x.copy_(x0), h.copy_(h0), z.copy_(z0)
                    rig.flush_l2()

                def one():
                    fused_call(ctx, libqasg, args, rule, g, d, d, M, T_STEP, params, x, h, z)
                times = rig.timed(one, args.steps, max(3, args.warmup), before_each=before)
                med = max_over_ranks(float(np.median(times)), rig.dist, dev)
                ctx.profile_begin()
                before()
                one()
                torch.cuda.synchronize()
                kernel_ms = {k: v[0] / v[1] for k, v in ctx.profile_end().items()}
                once = 4.0 * d <= args.stream_row_bytes and args.variant == "step" and args.quantizer != "none"
                moved = step_bytes(M, name, once) * d if args.quantizer != "none" else minimal_bytes(M, name) * d
                grid.append({"d": d, "M": M, "rule": name, "ms_median": med, "ms_best": min(times),
                             "coord_workers_per_s": d * M / (med * 1e-3),
                             "gbs_moved": moved / 1e9 / (med * 1e-3),
                             "gbs_minimal": minimal_bytes(M, name) * d / 1e9 / (med * 1e-3),
                             "kernel_ms": kernel_ms})
                total_units += d * M
                total_ms += med
            launches += ctx.launch_count()
            assert ctx.last_async_status() == libqasg.OK
            ctx.close()
            del g, x0, h0, z0, x, h, z
            torch.cuda.empty_cache()
    clocks = sampler.stop() if rig.rank == 0 else None
    if rig.rank != 0:
        return
    emit(rig, args, value=rig.world * total_units / (total_ms * 1e-3), ms_per_step=total_ms,
         config={"workload": WORKLOAD_5, "quantizer": args.quantizer, "variant": args.variant,
                 "l2": "flushed (a 252 MiB buffer written) and the state restored before every timed step",
                 "one_launch_quantizer_row_bytes": args.stream_row_bytes,
                 "one_launch_step_bytes": args.one_launch_step_bytes,
                 "note": "gbs_moved: bytes the step must move through device memory (g twice; once where the one-launch "
                         "quantizer codes a row out of L2); gbs_minimal: each gradient once + state once"},
         clocks=clocks, gpu_launches=launches, e2e=None, roofline=None, cpu_baseline=None, grid=grid)


# ------------------------------------------------------------------ side measurements
def run_optimal(rig, args):
    """The 0.75 * mean|g| rule against the exact optimal threshold: time of each quantizer and the
    quantization error ||g - s*tern||^2 / ||g||^2 = 1 - n s^2 / ||g||^2 each one reaches."""
    from paper_2208_05631_b200 import libqasg
    dev = rig.dev
    M = int(args.workers.split(",")[0])
    for log2_d in range(args.min_log2_d, args.max_log2_d + 1, 2):
        d = 1 << log2_d
        ctx = new_context(libqasg, rig, args, d, M)
        scratch = torch.empty(libqasg.optimal_scratch_bytes(d), dtype=torch.uint8, device=dev)
        params = libqasg.make_params(LAM, ETA, DELTA)
        for name, gen in (("normal", inputs.normal_gradients), ("student_t3", inputs.student_t_gradients)):
            g = gen(d, M, seed=4, device=dev)
            sq = (g.double() ** 2).sum(dim=1)
            codes = torch.empty((M, libqasg.code_words(d)), dtype=torch.int32, device=dev)
            out = {}
            for which in ("rule", "optimal"):
                scales, thr = (torch.zeros(M, dtype=torch.float32, device=dev) for _ in range(2))
                cnt = torch.zeros(M, dtype=torch.int64, device=dev)

                def run():
                    if which == "rule":
                        ctx.quantize_pack(g, d, d, M, 1, params, codes, scales, thr, cnt)
                    else:
                        ctx.quantize_pack_optimal(g, d, d, M, params, codes, scales, scratch, thr, cnt)
                times = rig.timed(run, args.steps, 1, before_each=rig.flush_l2)
                err = 1.0 - cnt.double() * scales.double() ** 2 / sq
                out[which] = {"ms_median": float(np.median(times)),
                              "threshold_over_mean_abs": (thr.double() / g.abs().double().mean(dim=1)).tolist(),
                              "kept_fraction": (cnt.double() / d).tolist(), "relative_sq_error": err.tolist()}
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


def run_touched(rig, args):
    """Passes A and B on rows held in sparse form, for synthetic patterns of stored entries (d = 2^24, M = 16):
    how the time depends on the number of entries and on where they sit."""
    from paper_2208_05631_b200 import libqasg
    dev = rig.dev
    d, M = 1 << 24, 16
    ctx = new_context(libqasg, rig, args, d, M)
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
        graph = graph_of(run)
        us = float(np.median(rig.timed(graph.replay, max(args.steps, 20), 3))) * 1e3
        entries = int(sum(torch.unique(c).numel() for c in columns))
        print(json.dumps({"what": "touched_passes_A_B", "pattern": name, "d": d, "M": M, "stored_entries": entries,
                          "us_per_graph_replay": us}), flush=True)
    assert ctx.last_async_status() == libqasg.OK
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="3", choices=["1", "2", "3", "4", "5", "optimal", "touched"])
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quantizer", default="threshold", choices=["threshold", "stochastic", "none"])
    ap.add_argument("--variant", default="step", choices=["step", "double", "select"])
    ap.add_argument("--state-density", type=float, default=1.0,
                    help="config 3: fraction of the iterate x that is non-zero (seeded Bernoulli mask)")
    ap.add_argument("--d", type=int, default=1 << 28, help="workload 3: coordinates")
    ap.add_argument("--M", type=int, default=8, help="workload 3: workers")
    ap.add_argument("--min-log2-d", type=int, default=20, help="workload 5 and optimal")
    ap.add_argument("--max-log2-d", type=int, default=28)
    ap.add_argument("--workers", default="2,4,8,16,32", help="workload 5 and optimal")
    ap.add_argument("--csr-rows", type=int, default=1_000_000, help="workload 4: rows of the CSR matrix")
    ap.add_argument("--one-launch-step-bytes", type=int, default=None,
                    help="qasg_step as one launch up to this many bytes of gradients (default: the library's)")
    ap.add_argument("--stream-row-bytes", type=int, default=0,
                    help="workloads 3 and 5: quantize rows up to this size with the one-launch kernel (library option; 0 = default path)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    rig = Rig(args)
    {"1": run_config1, "2": run_config2, "3": run_config3, "4": run_config4, "5": run_config5,
     "optimal": run_optimal, "touched": run_touched}[args.config](rig, args)
    rig.close()


if __name__ == "__main__":
    main()
