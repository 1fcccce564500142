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


def _shard_rank_main(rank, world, port, out_dir):
    """Sequence-sharded decode as two ranks would run it: each rank holds a token shard (quantized on its
    own, as Algorithm 3 over the tokens it holds), computes its (max, sum, out) triples, the triples are
    all-gathered into every rank's own memory and merged.  Oracle arithmetic on CPU, gloo exchange."""
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import vidkv_oracle as O
    from workloads import CONFIGS, make_layer_kv, make_step_inputs
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = CONFIGS["tiny"]
    T, cut = 640, 384
    K, V = make_layer_kv(wl, 0, "cpu", T=T, B=1)
    q, k_new, v_new = make_step_inputs(wl, 0, 0, "cpu", T=T, B=1)
    lo, hi = (0, cut) if rank == 0 else (cut, T)
    sc = O.SlabCache()
    sc.prefill(K[0, 1, lo:hi].float().numpy(), V[0, 1, lo:hi].float().numpy(), None)
    Kd, Vd = sc.dequant_k(), sc.dequant_v()
    if rank == world - 1:                                   # the last shard owns the newest token
        Kd = np.concatenate([Kd, k_new[0, 1].float().numpy()[None].astype(np.float64)])
        Vd = np.concatenate([Vd, v_new[0, 1].float().numpy()[None].astype(np.float64)])
    m, l, o = O.attention_partial(q[0, 7:14].float().numpy(), Kd, Vd, 1.0 / np.sqrt(128.0))
    mine = torch.from_numpy(np.concatenate([m[:, None], l[:, None], o], axis=1))      # [7, 130]
    got = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(got, mine)
    parts = [(g[:, 0].numpy(), g[:, 1].numpy(), g[:, 2:].numpy()) for g in got]
    np.save(os.path.join(out_dir, f"merged{rank}.npy"), O.merge_partials(parts))
    np.save(os.path.join(out_dir, f"kd{rank}.npy"), Kd)
    np.save(os.path.join(out_dir, f"vd{rank}.npy"), Vd)
    dist.destroy_process_group()


def test_two_gloo_ranks_merge_token_shards(tmp_path):
    import numpy as np
    from oracle import vidkv_oracle as O
    from workloads import CONFIGS, make_step_inputs
    world, port = 2, 29411 + os.getpid() % 200
    mp.spawn(_shard_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    merged = [np.load(tmp_path / f"merged{r}.npy") for r in range(world)]
    assert np.array_equal(merged[0], merged[1])              # every rank ends with the same output
    Kd = np.concatenate([np.load(tmp_path / f"kd{r}.npy") for r in range(world)])
    Vd = np.concatenate([np.load(tmp_path / f"vd{r}.npy") for r in range(world)])
    q, _, _ = make_step_inputs(CONFIGS["tiny"], 0, 0, "cpu", T=640, B=1)
    whole = O.attention(q[0, 7:14].float().numpy(), Kd, Vd, 1.0 / np.sqrt(128.0))
    assert np.allclose(merged[0], whole, rtol=1e-12, atol=1e-13)
