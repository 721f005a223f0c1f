"""The N > 1 arm of the benchmark is "replicas only": each rank runs the same workload and the
job time is the maximum over ranks.  These tests run that reduction on two gloo ranks on CPU,
and check that the reference arm leaves all work to rank 0."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    torch.distributed.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [10.0 + rank, 5.0 - rank, float("nan")]
        got = bench.reduce_max_over_ranks(mine, world, "cpu")
        with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
            json.dump(got, f)
    finally:
        torch.distributed.destroy_process_group()


def test_time_is_the_maximum_over_two_gloo_ranks(tmp_path):
    port = 29000 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for rank in (0, 1):
        got = json.load(open(tmp_path / f"r{rank}.json"))
        assert got[0] == 11.0 and got[1] == 5.0 and got[2] != got[2]      # NaN stays NaN


def test_value_counts_all_ranks_and_workers():
    sys.path.insert(0, ROOT)
    import bench
    one = bench.whole_job_value(1000, 2, 1, 10, 1.0)
    assert bench.whole_job_value(1000, 2, 4, 10, 1.0) == pytest.approx(4 * one)
    assert one == pytest.approx(4.0 * 1000 * 2 * 10 / 1e-3 / 1e9)
    assert bench.reduce_max_over_ranks([1.0, 2.0], 1, "cpu") == [1.0, 2.0]


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--config", "0"], env=env, capture_output=True,
                         text=True, timeout=300)
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
