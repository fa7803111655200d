"""Host logic of bench.py that needs no GPU: the over-ranks aggregation (two gloo ranks on CPU),
the reference arm's rank handling and JSON shape, and the CPU-baseline sample."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, units = bench.aggregate_over_ranks(10.0 * (rank + 1), 5.0 + rank, dist)
    out.put((rank, ms, units))
    dist.barrier()
    dist.destroy_process_group()


def test_aggregate_is_max_time_and_sum_of_units_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get() for _ in range(2))
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert got == [(0, 20.0, 11.0), (1, 20.0, 11.0)]


def test_aggregate_single_process_is_identity():
    assert bench.aggregate_over_ranks(3.5, 7.0, None) == (3.5, 7.0)


def test_reference_arm_prints_one_line_on_rank0_and_nothing_elsewhere():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["metric"] == bench.METRIC and j["unit"] == bench.UNIT
    assert j["value"] > 0 and j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["value"] == j["value"]
    assert j["e2e"]["h2d_bytes_per_step"] == 0 and j["e2e"]["d2h_bytes_per_step"] == 0


def test_oracle_sample_is_seeded_and_row_sliced():
    a, sp = bench.oracle_sample("c2_1p6b", 1, rows_fraction=0.125)
    b, _ = bench.oracle_sample("c2_1p6b", 1, rows_fraction=0.125)
    assert len(a) == 8 and sp["d"] == 2048
    for i, j in zip(a, b):
        assert i["oc"] % 256 == 0 and np.array_equal(i["codes"]["q"], j["codes"]["q"])
        assert np.array_equal(i["x"], j["x"])
    ys = bench.oracle_step(a)
    assert [y.shape for y in ys] == [(1, it["oc"]) for it in a]
