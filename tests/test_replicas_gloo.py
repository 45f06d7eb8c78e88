"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The hot path has no exchange
step, so ranks are independent replicas; what they share is the job-level aggregation
(slowest rank's time, sum of tokens), distinct query seeds, and the rule that only
rank 0 of the reference arm prints."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, tokens = bench.job_aggregate(10.0 + 5.0 * rank, 1000.0 * (rank + 1), dist, torch.device("cpu"))
    out[rank] = (ms, tokens, bench.rank_seed(7, rank))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_aggregate_max_time_and_sum_tokens():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][:2] == (15.0, 3000.0) and res[1][:2] == (15.0, 3000.0)
    assert res[0][2] == 7 and res[1][2] == 107            # same pool, different queries


def test_single_process_aggregate_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.job_aggregate(3.5, 42.0, None, torch.device("cpu")) == (3.5, 42.0)


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "cfg1", "--steps", "1", "--warmup", "0"], env=env, capture_output=True,
                       text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "cfg1", "--steps", "1", "--warmup", "0"], env=env, capture_output=True,
                       text=True, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
