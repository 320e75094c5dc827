"""Host-side logic of bench.py that needs no GPU: the multi-rank aggregation (two gloo ranks on
CPU), the byte accounting, and the reference arm's JSON line."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    out[rank] = ms
    dist.destroy_process_group()


def test_max_over_two_gloo_ranks():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
        assert dict(out) == {0: 15.0, 1: 15.0}
    # replicas: the whole job processes world * 2 * d * M coordinate-workers per bench step
    assert bench.whole_job_value(2, 1 << 20, 8, 1.0) == 2 * 2 * (1 << 20) * 8 / 1e-3
    assert bench.max_over_ranks(3.5, None, None) == 3.5


def test_byte_accounting_matches_the_method():
    b = bench.bytes_per_coord(8)
    # per coordinate: g read twice (4M each), codes written and read once (M/4 each), state once
    assert b["abs_sum"] == 32 and b["threshold_codes"] == 34
    assert b["decode_update_cmd"] == 2 + 16 and b["decode_update_rda"] == 2 + 20
    assert b["abs_sum"] + b["threshold_codes"] + b["decode_update_cmd"] == 8 * 8 + 8 / 2 + 16   # 84 B
    assert b["abs_sum"] + b["threshold_codes"] + b["decode_update_rda"] == 8 * 8 + 8 / 2 + 20   # 88 B


def test_reference_arm_prints_one_json_line():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--d", "65536",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0, res.stderr
    lines = [l for l in res.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["value"] > 0 and rec["unit"] == bench.UNIT
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["e2e"]["h2d_bytes_per_step"] == 0
    # other ranks print nothing
    env["RANK"] = "1"
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--d", "65536",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_all_cores_harness_gives_the_single_process_oracle_bit_for_bit():
    """The benchmark's second CPU leg drives the oracle over several processes (workers in parallel for
    the quantizer, coordinate ranges for the update).  It must be the same oracle: every output equals
    `qasg_oracle.step` bit for bit."""
    import numpy as np
    from oracle import harness
    from oracle import qasg_oracle as O
    from paper_2208_05631_b200 import inputs
    d, M, t = 20_001, 3, 5
    lam, eta, delta = 1e-3, 0.1, 1e-8
    g = inputs.optimizer_only_gradients(d, M, t, seed=4) * np.float32(0.05)
    x0, h0, z0 = (v.numpy().astype(np.float64) for v in inputs.random_state(d, seed=4))
    with harness.Harness(processes=3) as hs:
        path_g = hs.put("g", g)
        paths = [hs.put(n, v) for n, v in (("x", x0), ("h", h0), ("z", z0))]
        for quantizer in (O.QUANT_THRESHOLD, O.QUANT_TERNARY_STOCH):
            for rule in (O.RULE_CMD, O.RULE_RDA):
                state = paths if rule == O.RULE_RDA else [paths[0], paths[1], None]
                got = hs.step(rule, path_g, M, d, state, t, lam, eta, delta, quantizer=quantizer, seed=9,
                              range_len=4096)
                ref = O.step(rule, g, x0, h0, z0, t, lam, eta, delta, quantizer=quantizer, seed=9)
                for key in ("x", "h", "a", "q") + (("z",) if rule == O.RULE_RDA else ()):
                    assert np.array_equal(got[key].view(np.uint64), np.asarray(ref[key]).view(np.uint64)), key
                assert np.array_equal(got["scales"].view(np.uint32), ref["quant"]["scales"].view(np.uint32))
                assert np.array_equal(got["counts"], ref["quant"]["counts"])
