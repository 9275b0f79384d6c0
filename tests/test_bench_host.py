"""Host-side logic of bench.py without a GPU: the N > 1 aggregation over gloo ranks, the reference
arm's rank handling, and the JSON contract of the reference line."""
import json
import os
import subprocess
import sys

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

    times, counts = bench.reduce_over_ranks([1.0 + rank, 10.0 - rank], [100.0 * (rank + 1)], world, "cpu")
    if rank == 0:
        with open(out, "w") as f:
            json.dump({"times": times, "counts": counts}, f)
    dist.destroy_process_group()


def test_two_rank_aggregation_takes_max_time_and_sum_of_work(tmp_path):
    out = str(tmp_path / "agg.json")
    mp.spawn(_worker, args=(2, 29517, out), nprocs=2, join=True)
    got = json.load(open(out))
    assert got["times"] == [2.0, 10.0]          # max over ranks, per entry
    assert got["counts"] == [300.0]             # units summed over ranks


def test_reference_arm_prints_one_line_on_rank_zero_only():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1", "--steps", "1",
           "--warmup", "0", "--gpus", "2"]
    r1 = subprocess.run(cmd, env=dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1"), capture_output=True, text=True)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0"), capture_output=True, text=True)
    assert r0.returncode == 0, r0.stderr
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "lookups/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]
