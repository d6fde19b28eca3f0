"""Host-side logic of the multi-rank benchmark, on CPU with two gloo ranks (no GPU, no kernels).

The path shards over independent layer inputs, so the only cross-rank step is the timing reduction:
every rank reports its own device time, the job's time is the maximum, and the value is the whole-job
token rate.  The reference arm runs on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2509_24899_b200 import workloads as W
    wl = W.CONFIGS["tiny"]
    mine = bench.rank_workload(wl, rank)
    ms, e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 100.0 - 7.0 * rank], "cpu")
    value = bench.whole_job_value(wl, world, 4, ms)
    with open(os.path.join(out_dir, "rank%d.json" % rank), "w") as f:
        json.dump({"seed": mine.seed, "ms": ms, "e2e": e2e, "value": value}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_maximum_time_and_count_all_tokens(tmp_path):
    world, port = 2, 29541
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(world)]
    from paper_2509_24899_b200 import workloads as W
    wl = W.CONFIGS["tiny"]
    assert [r["seed"] for r in res] == [wl.seed, wl.seed + 1]            # independent inputs per rank
    for r in res:
        assert r["ms"] == 15.0 and r["e2e"] == 100.0                      # slowest rank decides, per quantity
        assert abs(r["value"] - wl.B * wl.N * 2 * 4 / 15e-3) < 1e-6       # whole-job tokens / max time


def test_max_over_ranks_without_a_process_group_is_the_identity():
    import bench
    assert bench.max_over_ranks([1.5, 2.5], "cpu") == [1.5, 2.5]


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True)
    assert r.returncode == 0 and r.stdout.strip() == ""                   # other ranks exit 0 without work
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
