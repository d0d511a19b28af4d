"""The multi-GPU path is "replicas only": each rank runs its own stream with no data-path collective, and
the only exchange is the maximum of the ranks' timings.  Covered here on CPU with two gloo ranks."""
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
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r "measured" (r + 1) ms per step and its own kernel times
    mine = [1.0 + rank, 0.5 - 0.1 * rank, 7.0 * (rank + 1)]
    got = bench.max_over_ranks(mine, world, "cpu")
    per_replica = 100.0 / got[0]
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"got": got, "value": bench.whole_job(per_replica, world)}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_two_gloo_ranks(tmp_path):
    world, port = 2, 29541 + os.getpid() % 200
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    for r in res:
        assert r["got"] == [2.0, 0.5, 14.0]                 # slowest replica per entry, same on every rank
        assert r["value"] == 2 * (100.0 / 2.0)              # whole-job value: replicas x per-replica rate at the max time


def test_reference_arm_prints_on_rank_zero_only():
    """Under a multi-rank launch of `bench.py --impl reference` the ranks other than 0 do no work and print nothing."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    env["LOCAL_RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
