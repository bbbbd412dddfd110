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


# ---------------------------------------------------------------------------------------------
# worker-sharded step: the orchestration (which calls, which collectives, which N) under gloo,
# world size 2, with a CPU stand-in for the CUDA context that computes each call from the oracle
# ---------------------------------------------------------------------------------------------
class _OracleContext:
    """The four calls ShardedStep makes, computed on CPU tensors by the oracle (a test double: the
    product's context runs the same calls on the GPU)."""

    def mv_vote(self, grads, err, votes=None, K=None, **_):
        from oracle import mv_oracle as O
        v = O.mv_vote(grads.numpy(), err.numpy(), K)
        err.copy_(torch.from_numpy(v["acc"]))
        votes.copy_(torch.from_numpy(v["votes"]))

    def mv_select(self, votes, N, out_idx, K=None, **_):
        from oracle import mv_oracle as O
        assert int(votes.max()) <= N
        out_idx.copy_(torch.from_numpy(O.select_mask(votes.numpy(), K)[0]))

    def mv_aggregate_partial(self, acc, idx, out_sum):
        cols = idx.long()
        total = torch.zeros(idx.numel(), dtype=torch.float64)
        for n in range(acc.shape[0]):
            total += acc[n, cols].double()
        out_sum.copy_(total)
        acc[:, cols] = 0.0

    def mv_finish_mean(self, total, N_total, out_val):
        out_val.copy_((total / float(N_total)).float())


def _sharded_rank(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import numpy as np
    from paper_2011_06495_b200.sharded import ShardedStep
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N, d, K, steps = 6, 5003, 60, 3
    rows = slice(rank * N // world, (rank + 1) * N // world)
    g = torch.Generator().manual_seed(77)
    err = torch.zeros(N, d)[rows].clone()
    step = ShardedStep(_OracleContext(), N, d, K, "cpu")
    out_idx = torch.empty(K, dtype=torch.int32)
    out_val = torch.empty(K, dtype=torch.float32)
    outs = []
    for _ in range(steps):
        grads = torch.randn(N, d, generator=g)          # the same stream on both ranks; each takes its rows
        step.step(grads[rows].clone(), err, out_idx, out_val)
        outs.append((out_idx.clone(), out_val.clone()))
    torch.save({"outs": outs, "err": err}, os.path.join(out_dir, f"sharded{rank}.pt"))
    dist.destroy_process_group()


def test_worker_sharded_step_equals_the_unsharded_step(tmp_path):
    import numpy as np
    from oracle import mv_oracle as O
    world = 2
    mp.spawn(_sharded_rank, args=(world, 29633, str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(tmp_path / f"sharded{r}.pt") for r in range(world)]
    N, d, K, steps = 6, 5003, 60, 3
    g = torch.Generator().manual_seed(77)
    err = np.zeros((N, d), dtype=np.float32)
    for s in range(steps):
        ref = O.mv_sparse_step(torch.randn(N, d, generator=g).numpy(), err, K)
        err = ref["err"]
        for r in range(world):
            idx, val = res[r]["outs"][s]
            assert np.array_equal(idx.numpy(), ref["out_idx"])                       # every rank holds the same mask
            np.testing.assert_allclose(val.numpy(), ref["out_val"], rtol=1e-6, atol=1e-12)
    got_err = np.concatenate([res[r]["err"].numpy() for r in range(world)], axis=0)
    assert np.array_equal(got_err.view(np.uint32), err.view(np.uint32))              # residuals, rank by rank


def _rows_rank(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seen = {}
    for N in (2, 5, 10, 25):
        lo, hi = bench.shard_rows(N, world, rank)
        mine = torch.zeros(N, dtype=torch.int32)
        mine[lo:hi] = 1
        dist.all_reduce(mine)                        # every worker row is held by exactly one rank
        seen[N] = (lo, hi, mine.tolist())
    with open(os.path.join(out_dir, f"rows{rank}.json"), "w") as f:
        json.dump(seen, f)
    dist.destroy_process_group()


def test_sharded_bench_splits_the_workers_over_the_ranks(tmp_path):
    world = 2
    mp.spawn(_rows_rank, args=(world, 29634, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        seen = json.load(open(tmp_path / f"rows{rank}.json"))
        for N, (lo, hi, cover) in seen.items():
            assert cover == [1] * int(N) and hi > lo
