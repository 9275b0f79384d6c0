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


def test_profiler_traffic_record_is_dropped_when_the_kernel_source_changes(tmp_path, monkeypatch):
    import bench

    files = ["tbe_backward.cu", "common.cuh"]
    rec = {"reduce_chunks": {"cfg2": {"dram_bytes_per_lookup": 168.5, "source_files": files,
                                      "source_sha256": bench.kernel_source_hash(files), "capture": "test"}}}
    path = tmp_path / "traffic.json"
    path.write_text(json.dumps(rec))
    monkeypatch.setattr(bench, "TRAFFIC_FILE", str(path))
    assert bench.ncu_traffic_per_lookup("reduce_chunks", "cfg2")[0] == 168.5
    assert bench.ncu_traffic_per_lookup("reduce_chunks", "cfg3")[0] is None          # another workload
    assert bench.ncu_traffic_per_lookup("tbe_forward_kernel", "cfg2")[0] is None     # no record
    rec["reduce_chunks"]["cfg2"]["source_sha256"] = "0" * 64                                 # the kernel changed since
    path.write_text(json.dumps(rec))
    assert bench.ncu_traffic_per_lookup("reduce_chunks", "cfg2")[0] is None


def test_every_workload_has_a_spec_for_both_arms():
    import argparse

    import bench

    a = argparse.Namespace(tables=0, budget_gb=0.01, warmup=1, steps=1, rows=1000, batch=8, pooling=3, alpha=1.0,
                           cache_fraction=0.1)
    for name, cached in (("cfg1", False), ("cfg2", False), ("cfg3", False), ("cfg4", True), ("cfg5", True)):
        spec = bench.make_spec(name, 0, a)
        assert spec.name == name and spec.cached == cached
    f = bench.fractions(4000.0, 6547.2)
    assert abs(f["frac_of_measured"] - 4000.0 / 6547.2) < 1e-12 and abs(f["frac_of_nominal"] - 0.5) < 1e-12
