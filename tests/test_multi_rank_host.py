"""The multi-GPU path of bench.py shards by replication (every rank holds its own batch shard and
cache, no data-path collective); what ranks exchange is the timing: a barrier and one all-reduce
(max).  Checked here with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local = [10.0 + rank, 5.0 - rank, 1.0, 0.25 * (rank + 1)]           # each rank's own timings (ms)
    dist.barrier()
    agg = bench.max_over_ranks(local, torch.device("cpu"), world)
    value = bench.whole_job_throughput(1.0e6, agg[0], world)
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"agg": agg, "value": value}, f)
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_rank(tmp_path):
    world, port = 2, 29611 + os.getpid() % 200
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    assert res[0]["agg"] == res[1]["agg"] == [11.0, 5.0, 1.0, 0.5]
    # weak scaling: both ranks processed 1e6 units within the slower rank's 11 ms
    assert abs(res[0]["value"] - 2 * 1.0e6 / 11.0e-3) < 1e-6 * res[0]["value"]


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 1.0], torch.device("cpu"), 1) == [3.0, 1.0]
    assert bench.whole_job_throughput(2.0, 1000.0, 1) == 2.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
