"""The multi-process side of the benchmark, on CPU with the gloo backend (world size 2).

The path does not shard across devices: with N GPUs the benchmark runs N independent replicas.
What the ranks share is the timing rule (the job is as slow as its slowest rank) and the rule that
only rank 0 reports; both are exercised here without a GPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 100.0 * (rank + 1)                   # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, dist, torch.device("cpu"))
    value = bench.job_steps_per_s(ms, world, steps=50)
    dist.barrier()
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"ms": ms, "value": value}, f)
    dist.destroy_process_group()


def test_max_over_ranks_and_job_throughput(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, 29631, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        r = json.load(open(tmp_path / f"rank{rank}.json"))
        assert r["ms"] == 200.0                      # the slowest rank's time, on every rank
        assert abs(r["value"] - 2 * 50 / 0.2) < 1e-9  # two replicas x 50 steps in 0.2 s


def test_reference_arm_runs_on_rank_zero_only():
    """`--impl reference` times the CPU oracle on rank 0; other ranks exit 0 without output."""
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
           "--steps", "2", "--warmup", "1", "--gpus", "2"]
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29632")
    r1 = subprocess.run(cmd, env=dict(env, RANK="1", LOCAL_RANK="1"), capture_output=True, text=True, timeout=600)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=dict(env, RANK="0", LOCAL_RANK="0"), capture_output=True, text=True, timeout=600)
    assert r0.returncode == 0, r0.stderr
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "steps/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["n_gpus"] == 2 and line["config"]["N"] == 4
