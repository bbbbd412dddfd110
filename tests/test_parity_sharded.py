"""GPU parity of the worker-sharded step (workers spread over ranks).  One GPU is available, so
(a) R ranks are emulated one after the other on the same device, each with its own context and
its own rows, the two sums over ranks being plain tensor additions, and (b) the real
orchestration (`ShardedStep`) runs in a one-rank NCCL group.  Both are compared with the oracle's
unsharded step: mask and residual bit for bit, values within 1e-6."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist

from oracle import mv_oracle as O
from paper_2011_06495_b200 import binding as B
from paper_2011_06495_b200 import workloads as WL
from paper_2011_06495_b200.sharded import ShardedStep
from tests import parity as PT

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("N,d,K,R", [(6, 100_003, 1000, 2), (8, 300_007, 300, 4), (5, 50_001, 500, 5), (10, 1_000_003, 10_000, 2)])
def test_emulated_ranks_match_the_unsharded_oracle(N, d, K, R):
    w = WL.scaled(WL.resnet_like("c3"), d=d, N=N, K=K, steps=3)
    bounds = [r * N // R for r in range(R + 1)]
    ctxs = [B.MvContext(N, d, K, device=DEV, mode=B.MV_MODE_TRACK) for _ in range(R)]
    errs = [torch.zeros((bounds[r + 1] - bounds[r], d), dtype=torch.float32, device=DEV) for r in range(R)]
    err_ref = np.zeros((N, d), dtype=np.float32)
    votes = [torch.empty(d, dtype=torch.uint8, device=DEV) for _ in range(R)]
    part = [torch.empty(K, dtype=torch.float64, device=DEV) for _ in range(R)]
    out_idx = [torch.empty(K, dtype=torch.int32, device=DEV) for _ in range(R)]
    out_val = torch.empty(K, dtype=torch.float32, device=DEV)
    for step in range(w.steps):
        grads = WL.gradients(w, step, device=DEV)
        ref = O.mv_sparse_step(grads.cpu().numpy(), err_ref, K)
        for r in range(R):
            ctxs[r].mv_vote(grads[bounds[r]:bounds[r + 1]].clone(), errs[r], votes=votes[r], K=K)
        total_votes = torch.stack(votes).sum(dim=0, dtype=torch.uint8)          # stands in for the all-reduce
        PT.first_diff(PT.npy(total_votes), ref["votes"], f"step {step} summed votes")
        for r in range(R):
            ctxs[r].mv_select(total_votes, N, out_idx[r], K=K)
            PT.first_diff(PT.npy(out_idx[r]), ref["out_idx"], f"step {step} rank {r} out_idx")
            ctxs[r].mv_aggregate_partial(errs[r], out_idx[r], part[r])
        total = torch.stack(part).sum(dim=0)                                    # stands in for the all-reduce
        ctxs[0].mv_finish_mean(total, N, out_val)
        torch.cuda.synchronize()
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), f"step {step} out_val")
        got_err = torch.cat(errs, dim=0)
        PT.first_diff(PT.bits(PT.npy(got_err)), PT.bits(ref["err"]), f"step {step} err")
        err_ref = ref["err"]


def test_sharded_step_in_a_one_rank_nccl_group():
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29641")
    torch.cuda.set_device(0)
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device(DEV))
    try:
        N, d, K = 6, 200_003, 2000
        w = WL.scaled(WL.resnet_like("c2"), d=d, N=N, K=K, steps=3)
        ctx = B.MvContext(N, d, K, device=DEV)
        step = ShardedStep(ctx, N, d, K, DEV)
        err = torch.zeros((N, d), dtype=torch.float32, device=DEV)
        err_ref = np.zeros((N, d), dtype=np.float32)
        out_idx = torch.empty(K, dtype=torch.int32, device=DEV)
        out_val = torch.empty(K, dtype=torch.float32, device=DEV)
        for s in range(w.steps):
            grads = WL.gradients(w, s, device=DEV)
            ref = O.mv_sparse_step(grads.cpu().numpy(), err_ref, K)
            step.step(grads, err, out_idx, out_val)
            torch.cuda.synchronize()
            PT.first_diff(PT.npy(out_idx), ref["out_idx"], f"step {s} out_idx")
            PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), f"step {s} out_val")
            PT.first_diff(PT.bits(PT.npy(err)), PT.bits(ref["err"]), f"step {s} err")
            err_ref = ref["err"]
    finally:
        if created:
            dist.destroy_process_group()


def test_sharded_bench_with_one_rank_gives_the_unsharded_mask():
    """`bench.py --sharded` in a one-rank NCCL group ends on the same mask as the plain step of the same run
    length would (checked through the line it prints and through a short plain run of the library)."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1", MASTER_PORT="29642")
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--sharded", "--workload", "c1", "--steps", "4",
                        "--warmup", "3"], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["scaling"] == "strong" and line["n_gpus"] == 1 and line["same_mask_on_every_rank"] is True
    assert line["setup"]["workers_per_rank"] == [4] and line["launches_per_step"] >= 4 and line["value"] > 0
