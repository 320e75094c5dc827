"""Runs oracle functions over several host processes (not a test module).

The oracle stays as it is: each process calls its functions on one worker's row, in slices that
bound the temporaries.  Processes are started with `spawn`, so a pool may be opened after CUDA has
been initialised in the parent.  Rows travel as .npy files (memory-mapped by the child)."""
import multiprocessing as mp
import os

import numpy as np


def stochastic_row(args):
    """Codes and count of one worker's row under the unbiased ternary quantizer: Philox draws for
    (seed, t, m, i), kept iff u < |v|/s with s the row's maximum (Section 3.4, first paragraph)."""
    from oracle import qasg_oracle as O
    path, m, t, seed, chunk = args
    row = np.load(path, mmap_mode="r")
    d = row.size
    scale = np.float32(np.abs(row).max())
    words, count = [], 0
    for lo in range(0, d, chunk):                     # chunk is a multiple of 16: whole code words
        hi = min(d, lo + chunk)
        _, u = O.philox_draws(seed, t, m, np.arange(lo, hi, dtype=np.uint64))
        tern, _ = O.ternary_stochastic_quantize(np.asarray(row[lo:hi]), u, scale=scale)
        words.append(O.pack_codes(tern))
        count += int(np.count_nonzero(tern))
    return m, np.concatenate(words), float(scale), count


def run(fn, jobs, processes=None):
    processes = processes or min(len(jobs), os.cpu_count() or 1)
    with mp.get_context("spawn").Pool(processes) as pool:
        return pool.map(fn, jobs)
