"""Host-side logic of bench.py: the replica bookkeeping over two gloo ranks on
the CPU, and the reference (oracle) arm's JSON line."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from helpers import ROOT

sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = 10.0 + 5.0 * rank                     # the slower rank must set the time
        worst = bench.reduce_max(mine, world, torch.device("cpu"))
        rows = list(bench.global_rows(rank, 4))
        gathered = [None] * world
        dist.all_gather_object(gathered, rows)
        out[rank] = (worst, gathered)
    finally:
        dist.destroy_process_group()


def test_two_replicas_over_gloo():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29533, out), nprocs=world, join=True)
    for rank in range(world):
        worst, gathered = out[rank]
        assert worst == 15.0
        assert gathered == [[0, 1, 2, 3], [4, 5, 6, 7]]      # disjoint, rank-ordered rows
    # whole-job value: all ranks' units over the slowest rank's time
    assert bench.whole_job_throughput(1000, 2, 10, 15.0) == pytest.approx(2 * 1000 * 10 / 0.015)
    assert bench.reduce_max(3.0, 1, torch.device("cpu")) == 3.0


def test_reference_arm_prints_one_json_line():
    env = dict(os.environ, OMP_NUM_THREADS="4")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "1", "--warmup", "1"], capture_output=True, text=True,
                         env=env, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == bench.METRIC and d["unit"] == bench.UNIT
    assert d["config"]["workload"] == bench.WORKLOAD and d["higher_is_better"] is True
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0}
    assert d["value"] > 0 and d["steps"] == 1


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--gpus", "2", "--steps", "1", "--warmup", "1"], capture_output=True,
                         text=True, env=env, timeout=120, cwd=ROOT)
    assert res.returncode == 0 and res.stdout.strip() == ""
