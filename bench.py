#!/usr/bin/env python
"""Benchmark of the fused quantized adaptive-subgradient step.

Workload (the bandwidth-bound single step): d = 2^28 fp32 coordinates, M = 8 workers,
gradients 1e-2 * Student-t(3), random state, t = 16, lambda = 1e-3, eta = 0.1, delta = 1e-8.
One bench step = one fused QCMD step followed by one fused QRDA step on the same gradients
(2 * d * M coordinate-workers).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (torchrun) every rank runs an independent replica of the workload (the path has
no exchange step); the time is the maximum over ranks.  `--impl reference` times the CPU
oracle on a bounded sample of the same workload.
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


# ------------------------------------------------------------------ byte accounting
def bytes_per_coord(M):
    """Algorithmic bytes per coordinate of each kernel of the fused step (fp32 state, 2-bit codes)."""
    return {
        "abs_sum": 4.0 * M,                       # read g
        "threshold_codes": 4.0 * M + M / 4.0,     # read g again, write codes
        "decode_update_cmd": M / 4.0 + 16.0,      # read codes; h, x read + write
        "decode_update_rda": M / 4.0 + 20.0,      # read codes; h, z read + write; x write
    }


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per coordinate at M = 8, from the ncu
# capture summarised in profiles/step_kernels_d2p24_M8_ncu_full.md (d = 2^24; passes A and B stream,
# so their traffic grows in proportion to d).  Valid only for the kernel source it was taken from.
NCU_TRAFFIC = {
    "kernels_sha256": "15c39fbd299dd161025ec37617c0e0ae9bcdeef5e5b886510ff02a86c5f49841",
    "M": 8,
    "bytes_per_coord": {"abs_sum": 541067520 / 2 ** 24, "threshold_codes": 568647424 / 2 ** 24},
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
    (NVML in-process, every 5 ms; the main thread waits inside CUDA calls that release the GIL)."""

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

    def stop(self):
        if self.nvml is None or self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvml unavailable"]}
        self.stop_flag.set()
        self.thread.join(timeout=2)
        reasons = sorted(name for bit, name in self.REASONS.items() if self.bits & bit)
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.max_mhz,
                "samples": len(self.sm), "reasons": reasons}


# ------------------------------------------------------------------ the CPU oracle legs
def oracle_throughput(d_sample, M, steps, warmup):
    """Times the CPU oracle (as it stands) on the first d_sample coordinates of the workload:
    one QCMD step + one QRDA step per bench step.  Returns (units/s, seconds per step)."""
    from oracle import qasg_oracle as O
    g = inputs.student_t_gradients(d_sample, M, seed=SEED).numpy()
    x0, h0, z0 = (v.numpy().astype(np.float64) for v in inputs.random_state(d_sample, seed=SEED))
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        O.step(O.RULE_CMD, g, x0, h0, None, T_STEP, LAM, ETA, DELTA)
        O.step(O.RULE_RDA, g, x0, h0, z0, T_STEP, LAM, ETA, DELTA)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    per_step = float(np.mean(times))
    return 2.0 * d_sample * M / per_step, per_step


def run_reference(args, rank):
    if rank != 0:
        return
    d_sample = min(args.d, 1 << 21)
    value, per_step = oracle_throughput(d_sample, args.M, args.steps, args.warmup)
    sample = "first %d coordinates of every worker's gradient, both rules, per step" % d_sample
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(args, "cpu oracle on a bounded sample: " + sample),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def workload_config(args, note):
    return {"workload": "bandwidth-bound single step: d=%d fp32, M=%d, gradients 1e-2*Student-t(3), "
                        "x,z~0.1*N(0,1), h~U[0,1), t=%d, lambda=%g, eta=%g, delta=%g, seed %d; one fused QCMD "
                        "step + one fused QRDA step per bench step" % (args.d, args.M, T_STEP, LAM, ETA, DELTA, SEED),
            "d": args.d, "M": args.M, "quantizer": "threshold", "rules": ["qcmd", "qrda"],
            "l2": "inputs (%.1f GiB of gradients) are larger than L2; no flush" % (args.d * args.M * 4 / 2 ** 30),
            "parallelism": "replicas" if args.gpus > 1 else "single", "note": note}


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


# ------------------------------------------------------------------ our arm
def run_ours(args, rank, world):
    from paper_2208_05631_b200 import libqasg
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    d, M = args.d, args.M
    g = inputs.student_t_gradients(d, M, seed=SEED + rank, device=dev)
    x0, h0, z0 = inputs.random_state(d, seed=SEED + rank, device=dev)
    xc, hc = x0.clone(), h0.clone()                 # QCMD state
    xr, hr, zr = x0.clone(), h0.clone(), z0.clone()  # QRDA state
    ctx = libqasg.Context(d, M, device=local)
    params = libqasg.make_params(LAM, ETA, DELTA)

    def bench_step():
        ctx.step(libqasg.RULE_CMD, g, d, d, M, T_STEP, params, xc, hc)
        ctx.step(libqasg.RULE_RDA, g, d, d, M, T_STEP, params, xr, hr, zr)

    def fence():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        bench_step()
    fence()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.01)
    launches0 = ctx.launch_count()
    ctx.profile_begin()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(args.steps):
        bench_step()
    stop.record()
    fence()
    elapsed_ms = start.elapsed_time(stop)
    kernels = ctx.profile_end()
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    assert ctx.last_async_status() == libqasg.OK
    elapsed_ms = max_over_ranks(elapsed_ms, dist, dev)
    ms_per_step = elapsed_ms / args.steps
    value = whole_job_value(world, d, M, ms_per_step)

    # ---------------------------------------------------------------- end to end, host buffers
    e2e = None
    if args.e2e_steps > 0 and (rank == 0 or world > 1):
        e2e = run_e2e(args, ctx, params, g, x0, h0, z0, dev, dist, world)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---------------------------------------------------------------- roofline of the dominant kernel
    peak, peak_kind = measured_peak()
    bpc = bytes_per_coord(M)
    per_kernel = {}
    for name, (ms, n) in kernels.items():
        avg = ms / n
        algo = bpc.get(name, 0.0) * d
        per_kernel[name] = {"launches": n, "avg_ms": avg, "algorithmic_gb": algo / 1e9,
                            "gbs": algo / 1e9 / (avg * 1e-3), "share": ms / sum(v[0] for v in kernels.values())}
    top = max(per_kernel, key=lambda k: per_kernel[k]["share"])
    roofline = {"bound": "hbm", "kernel": top, "achieved": per_kernel[top]["gbs"], "peak": peak,
                "peak_kind": peak_kind, "unit": "GB/s", "frac": per_kernel[top]["gbs"] / peak,
                "frac_of_nominal_8tbs": per_kernel[top]["gbs"] / NOMINAL_HBM_GBS,
                "algorithmic_bytes": bpc.get(top, 0.0) * d, "traffic": ncu_traffic(top, d, M),
                "per_kernel": per_kernel}
    step_bytes = sum(bpc.values()) * d + bpc["abs_sum"] * d + bpc["threshold_codes"] * d  # A and B run twice
    moved_gbs = step_bytes / 1e9 / (ms_per_step * 1e-3)
    once_through = ((4 * M + 16) + (4 * M + 20)) * d / 1e9 / (ms_per_step * 1e-3)

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        d_sample = min(d, 1 << 25)
        v, per = oracle_throughput(d_sample, M, steps=1, warmup=0)
        cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": per,
               "sample": "first %d coordinates of every worker's gradient, one QCMD + one QRDA oracle step" % d_sample}

    print(json.dumps({
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(args, "inputs resident in HBM before the timed region"),
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu,
        "hbm": {"bytes_moved_per_step_gb": step_bytes / 1e9, "gbs_moved": moved_gbs,
                "frac_of_nominal_8tbs": moved_gbs / NOMINAL_HBM_GBS, "frac_of_peak": moved_gbs / peak,
                "once_through_frac_of_nominal_8tbs": once_through / NOMINAL_HBM_GBS},
    }))
    if dist is not None:
        dist.destroy_process_group()


def run_e2e(args, ctx, params, g, x0, h0, z0, dev, dist, world):
    """The same bench step through qasg_step_host: gradients and state start in pinned host memory,
    the new state ends there; host<->device copies are inside the timed region."""
    from paper_2208_05631_b200 import libqasg
    d, M = args.d, args.M
    try:
        gh = torch.empty((M, d), dtype=torch.float32, pin_memory=True)
        gh.copy_(g)
        host = [torch.empty(d, dtype=torch.float32, pin_memory=True) for _ in range(5)]
    except RuntimeError as e:  # not enough pinned host memory on this machine
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": None, "d2h_bytes_per_step": None,
                "error": "pinned host allocation failed: %s" % str(e).splitlines()[0]}
    xch, hch, xrh, hrh, zrh = host
    for dst, src in ((xch, x0), (hch, h0), (xrh, x0), (hrh, h0), (zrh, z0)):
        dst.copy_(src)
    xd, hd, zd = (torch.empty(d, dtype=torch.float32, device=dev) for _ in range(3))
    steps = max(1, min(args.steps, args.e2e_steps))

    def host_step():
        ctx.step_host(libqasg.RULE_CMD, gh, d, d, M, T_STEP, params, xch, hch, None, g, xd, hd, None)
        ctx.step_host(libqasg.RULE_RDA, gh, d, d, M, T_STEP, params, xrh, hrh, zrh, g, xd, hd, zd)

    host_step()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        host_step()
    stop.record()
    torch.cuda.synchronize()
    ms = max_over_ranks(start.elapsed_time(stop), dist, dev)
    vec = 4 * d
    h2d = 2 * 4 * d * M + (2 * vec) + (2 * vec)      # g twice; QCMD: x, h; QRDA: h, z
    d2h = (2 * vec) + (3 * vec)                      # QCMD: x, h; QRDA: x, h, z
    return {"value": whole_job_value(world, d, M, ms / steps), "unit": UNIT, "ms_per_step": ms / steps,
            "steps": steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--d", type=int, default=1 << 28)
    ap.add_argument("--M", type=int, default=8)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, world)


if __name__ == "__main__":
    main()
