"""The multi-rank bookkeeping of bench.py on CPU: two gloo ranks, maximum over ranks of the timings, whole-job
throughput of independent replicas, and the reference arm running on rank 0 only."""
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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 100.0 - 30.0 * rank])
    out[rank] = (ms, e2e, bench.whole_job_gbs(world, 1e9, 4, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time_and_add_the_work():
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(2, 29571, out), nprocs=2, join=True)
        assert out[0] == out[1]
        ms, e2e, gbs = out[0]
        assert ms == 15.0 and e2e == 100.0                 # slowest rank each
        assert abs(gbs - 2 * 1e9 * 4 / 0.015 / 1e9) < 1e-9  # both ranks' bytes over the slowest rank's time


def test_without_a_process_group_the_values_pass_through():
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.whole_job_gbs(1, 2e9, 10, 1000.0) == 20.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=600)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2
