"""Host-side logic of the multi-GPU bench on CPU: two gloo ranks aggregate their
timings (max over ranks, points summed), every rank draws its own shape table,
and the reference arm stays silent on ranks other than 0."""
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    v = bench.aggregate_over_ranks(dist, torch.device("cpu"), 10.0 * (rank + 1), 100.0 * (world - rank),
                                   world, 1000, 5, 3)
    out[rank] = v
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_aggregate_by_max_time_and_summed_points():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29531 + os.getpid() % 1000, out), nprocs=world, join=True)
    for rank in range(world):
        value, e2e_value, total_ms, e2e_ms = out[rank]
        assert total_ms == 20.0 and e2e_ms == 200.0           # the slowest rank
        assert value == 1000 * 5 * world / 0.020              # points of all ranks
        assert e2e_value == 1000 * 3 * world / 0.200


def test_each_rank_gets_its_own_table_of_the_same_distribution():
    import bench
    a = bench.workload("C4", 32, rank=0)["models"]
    b = bench.workload("C4", 32, rank=1)["models"]
    assert a.tobytes() != b.tobytes()
    for t in (a, b):
        assert t["layers"].max() <= 160 and t["seq"].max() <= 32768 and t["micro_batch"].max() <= 64
    assert bench.workload("C4", 32, rank=0)["models"].tobytes() == a.tobytes()


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1", "--models", "2"], env=env, capture_output=True, text=True)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_window_is_inside_the_space_and_not_group_aligned():
    import bench
    first, count = bench.window_of(6_963_200_000, 25)
    assert count == 1 << 25 and first % 625 != 0 and first + count <= 6_963_200_000
    assert bench.window_of(4375, 25) == (0, 4375)


def test_reference_arm_prints_the_contract_line():
    """Rank 0 of the reference arm prints one JSON line with the keys the bench
    contract names; its value is the oracle's own throughput."""
    import json
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "1",
                        "--steps", "1", "--warmup", "1", "--workload", "C3", "--models", "2"],
                       env=env, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    line = json.loads(lines[0])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
                "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["value"] > 0 and line["vs_baseline"] is None
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0,
                           "d2h_bytes_per_step": 0}
    assert "workload" in line["config"]
