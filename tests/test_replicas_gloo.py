"""The N > 1 path of the benchmark on CPU: two gloo ranks.

The hot path has no exchange step, so multi-GPU runs are independent replicas; the only multi-rank logic
is the timing aggregation (max over ranks, whole-job throughput) and the rule that the reference arm runs
on rank 0 only.
"""
import json
import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist
    sys.path.insert(0, str(ROOT))
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    worst = bench.reduce_max(local_ms)
    value = bench.job_throughput(2_000_000_000, world, worst * 1e-3)
    dist.barrier()
    Path(out_dir, f"rank{rank}.json").write_text(json.dumps({"worst": worst, "value": value}))
    dist.destroy_process_group()


def test_two_ranks_agree_on_max_time_and_whole_job_throughput(tmp_path):
    import torch.multiprocessing as mp
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = json.loads((tmp_path / "rank0.json").read_text())
    r1 = json.loads((tmp_path / "rank1.json").read_text())
    assert r0 == r1
    assert r0["worst"] == 15.0                          # max over ranks, not the mean
    assert r0["value"] == pytest.approx(2 * 2.0 / 15e-3)  # two replicas of 2 GFLOP each per 15 ms step


def test_single_process_reduce_is_identity():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.reduce_max(3.5) == 3.5
    assert bench.job_throughput(10**9, 4, 0.5) == pytest.approx(8.0)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_reference_arm_prints_one_json_line():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--workload", "cfg1",
                          "--steps", "2", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr
    lines = [l for l in res.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["cpu_baseline"]["kind"] == "oracle"
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["value"] > 0
