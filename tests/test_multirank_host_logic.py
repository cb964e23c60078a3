"""Host-side logic of the multi-GPU bench path, run as two gloo ranks on CPU: rows are
sharded as independent replicas (no data-path collective); only the timing is combined
(max over ranks) and the value summed over ranks."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2512_23424_b200 import workloads as wl  # noqa: E402


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local = 0.010 * (rank + 1)                       # rank 1 is the slow one
        slow = bench.slowest_rank(local, world, "cpu")
        w = wl.make_config(2, rows=4, seed_offset=rank)  # each rank generates its own rows
        value = bench.whole_job_value(w.algorithmic_bytes(), world, slow)
        with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as fh:
            json.dump({"slow": slow, "value": value, "x00": float(w.x[0, 0]), "bytes": w.algorithmic_bytes()}, fh)
    finally:
        dist.destroy_process_group()


def test_two_ranks_combine_time_and_value(tmp_path):
    world, port = 2, 29000 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r0 = json.load(open(tmp_path / "rank0.json"))
    r1 = json.load(open(tmp_path / "rank1.json"))
    assert r0["slow"] == r1["slow"] == pytest.approx(0.020)          # max over ranks, on every rank
    assert r0["value"] == r1["value"] == pytest.approx(2 * r0["bytes"] / 0.020 / 1e9)
    assert r0["x00"] != r1["x00"]                                    # different seeds per rank
    assert r0["bytes"] == r1["bytes"]                                # same per-rank work (weak scaling)


def test_single_rank_helpers():
    assert bench.slowest_rank(0.5, 1, "cpu") == 0.5
    assert bench.whole_job_value(10**9, 4, 0.5) == pytest.approx(8.0)
    w = wl.make_config(5, rows=8192)
    # rows 0..4095 have 1..4096 live entries, twice
    assert w.algorithmic_bytes() == (2 * sum(range(1, 4097)) + 8192 * 4096) * 2
    assert bench.pairs_for(wl.make_config(2, rows=8)) >= 2


def test_reference_arm_prints_one_line_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["config"]["workload"] == wl.CONFIG_NAMES[bench.HEADLINE]
