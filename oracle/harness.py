"""The oracle's own functions driven over several host processes.

TEST INFRASTRUCTURE ONLY (see the package docstring): used by the benchmark's CPU-baseline leg and
by the tests, never by the library.  Nothing here computes anything of the method: every number
comes from a function of `qasg_oracle`, called on one worker's row (the quantizer: its sums run
over the whole row) or on one range of coordinates (decode, average, accumulator, update: these
act coordinate by coordinate, so a slice of the result is the result of the slice).  The results
are therefore those of the single-process oracle bit for bit, which `tests/test_bench_host.py`
checks.

Processes are started with `spawn`, so a harness may be opened after the parent has initialised
CUDA.  Arrays travel as .npy files in a scratch directory (memory-mapped by the children).
"""
import multiprocessing as mp
import os
import shutil
import tempfile

import numpy as np

from . import qasg_oracle as O


def _quantize_row(args):
    path_g, m, quantizer, t, seed, coef, out_path = args
    row = np.load(path_g, mmap_mode="r")[m]
    if quantizer == O.QUANT_THRESHOLD:
        tern, scale, thr, count = O.threshold_quantize(np.asarray(row), coef)
    else:
        _, u = O.philox_draws(seed, t, m, np.arange(row.size, dtype=np.uint64))
        tern, scale = O.ternary_stochastic_quantize(np.asarray(row), u)
        thr, count = np.float32(0.0), int(np.count_nonzero(tern))
    np.save(out_path, tern)
    return float(scale), float(thr), int(count)


def _update_range(args):
    rule, tern_paths, scales, state_paths, lo, hi, t, lam, eta, delta = args
    terns = np.stack([np.load(p, mmap_mode="r")[lo:hi] for p in tern_paths])
    q = O.decode_average(terns, np.asarray(scales, dtype=np.float32))
    x, h, z = (None if p is None else np.load(p, mmap_mode="r")[lo:hi] for p in state_paths)
    if rule == O.RULE_CMD:
        x_new, h_new, a = O.cmd_step(q, x, h, lam, eta, delta)
        return x_new, h_new, None, a, q
    x_new, h_new, z_new, a = O.rda_step(q, h, z, t, lam, eta, delta)
    return x_new, h_new, z_new, a, q


class Harness:
    """A pool of `processes` oracle processes and a scratch directory."""

    def __init__(self, processes=None):
        self.processes = int(processes or os.cpu_count() or 1)
        self.pool = mp.get_context("spawn").Pool(self.processes)
        base = "/dev/shm" if os.path.isdir("/dev/shm") and os.access("/dev/shm", os.W_OK) else None
        self.dir = tempfile.mkdtemp(prefix="qasg_oracle_", dir=base)

    def close(self):
        self.pool.close()
        self.pool.join()
        shutil.rmtree(self.dir, ignore_errors=True)

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def put(self, name, array):
        """Stores an array in the scratch directory; returns its path."""
        path = os.path.join(self.dir, name + ".npy")
        np.save(path, np.ascontiguousarray(array))
        return path

    def step(self, rule, path_g, m_workers, d, state_paths, t, lam, eta, delta, quantizer=O.QUANT_THRESHOLD,
             seed=0, coef=0.75, range_len=1 << 20):
        """`qasg_oracle.step` (one-way quantization) with the workers quantized in parallel and the
        update taken over ranges of `range_len` coordinates (a multiple of the 4096-coordinate tile).
        path_g: file of the fp32 [M, d] gradients; state_paths: files of x, h, z (z None for QCMD).
        Returns dict(x, h, z, a, q, scales, thresholds, counts)."""
        assert range_len % O.TILE == 0
        tern_paths = [os.path.join(self.dir, "tern%d.npy" % m) for m in range(m_workers)]
        stats = self.pool.map(_quantize_row, [(path_g, m, quantizer, t, seed, coef, tern_paths[m])
                                              for m in range(m_workers)])
        scales = [s[0] for s in stats]
        jobs = [(rule, tern_paths, scales, state_paths, lo, min(d, lo + range_len), t, lam, eta, delta)
                for lo in range(0, d, range_len)]
        parts = self.pool.map(_update_range, jobs)
        cat = lambda k: None if parts[0][k] is None else np.concatenate([p[k] for p in parts])   # noqa: E731
        return dict(x=cat(0), h=cat(1), z=cat(2), a=cat(3), q=cat(4), scales=np.array(scales, dtype=np.float32),
                    thresholds=np.array([s[1] for s in stats], dtype=np.float32),
                    counts=np.array([s[2] for s in stats], dtype=np.int64), tern_paths=tern_paths)
