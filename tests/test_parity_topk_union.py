"""GPU parity of mv_topk_union_step (SSGD-top-K, the paper's comparison scheme: Section 2, Eq. 6-7) against the
CPU oracle: the union of the workers' masks index for index, the residual bit for bit, the values within the
tolerance of the aggregate (1e-6 relative; both sides add in binary64 in worker order and round once)."""
import numpy as np
import pytest
import torch

from oracle import mv_oracle as O
from paper_2011_06495_b200 import binding as B
from paper_2011_06495_b200 import workloads as WL
from tests import parity as PT
from tests.test_parity_small import make

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run(ctx, grads, err, K, extra=0):
    N, d = grads.shape
    cap = min(d, N * K) + extra
    out_idx = torch.full((cap,), -7, dtype=torch.int32, device=DEV)
    out_val = torch.full((cap,), float("nan"), dtype=torch.float32, device=DEV)
    count = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    e = err.to(DEV).clone()
    ctx.mv_topk_union_step(grads.to(DEV), e, out_idx, out_val, count, K=K)
    torch.cuda.synchronize()
    return PT.npy(out_idx), PT.npy(out_val), int(count.item()), PT.npy(e)


def check(ctx, grads, err, K, label, extra=0):
    ref = O.topk_union_step(grads.numpy(), err.numpy(), K)
    idx, val, cnt, e = run(ctx, grads, err, K, extra)
    U = ref["union_idx"].size
    assert cnt == U, f"{label}: union size {cnt} vs {U}"
    PT.first_diff(idx[:U], ref["union_idx"], label + " union_idx")
    assert np.all(idx[U:] == -1) and np.all(val[U:] == 0)
    cols = ref["union_idx"].astype(np.int64)
    scale = np.maximum(np.abs(ref["union_val"].astype(np.float64)), np.abs(ref["acc"][:, cols].astype(np.float64)).mean(axis=0))
    assert np.all(np.abs(val[:U].astype(np.float64) - ref["union_val"].astype(np.float64)) <= PT.REL_TOL * scale), label + " union_val"
    PT.first_diff(PT.bits(e), PT.bits(ref["err"]), label + " err")
    return ref


@pytest.mark.parametrize("mode", [B.MV_MODE_AUTO, B.MV_MODE_GENERAL, B.MV_MODE_TRACK], ids=["auto", "general", "track"])
@pytest.mark.parametrize("kind", ["gauss", "ties", "sparse"])
@pytest.mark.parametrize("N,d,K", [(1, 1, 1), (1, 5000, 50), (3, 33, 33), (4, 4097, 7), (5, 10001, 1000), (9, 65538, 655),
                                   (33, 5000, 50), (6, 300_007, 3000)])
def test_shapes(N, d, K, kind, mode):
    grads, err = make(N, d, kind, seed=N * 1000 + K)
    ctx = B.MvContext(N, d, K, device=DEV, mode=mode)
    check(ctx, grads, err, K, f"[{N}x{d} K={K} {kind}]", extra=(5 if d > 100 else 0))


def test_identical_workers_and_single_worker_reduce_to_majority_voting():
    N, d, K = 4, 50_021, 500
    g1, e1 = make(1, d, "gauss", seed=3)
    grads, err = g1.repeat(N, 1).contiguous(), e1.repeat(N, 1).contiguous()
    ctx = B.MvContext(N, d, K, device=DEV)
    ref = check(ctx, grads, err, K, "[identical]")
    mv = O.mv_sparse_step(grads.numpy(), err.numpy(), K)
    assert np.array_equal(ref["union_idx"], mv["out_idx"]) and np.array_equal(ref["err"], mv["err"])
    ctx1 = B.MvContext(1, d, K, device=DEV)
    check(ctx1, g1, e1, K, "[single]")


def test_error_feedback_over_steps_and_mixed_with_majority_voting():
    """Residuals carried over steps of SSGD-top-K stay bit-identical to the oracle's; a majority-vote step on the
    same context in between does not disturb it."""
    w = WL.scaled(WL.resnet_like("c2"), d=200_003, N=6, steps=4)
    ctx = B.MvContext(w.N, w.d, w.K, device=DEV, mode=B.MV_MODE_TRACK)
    err_t = WL.initial_err(w)
    oi = torch.empty(w.K, dtype=torch.int32, device=DEV)
    ov = torch.empty(w.K, dtype=torch.float32, device=DEV)
    for step in range(w.steps):
        grads = WL.gradients(w, step)
        ref = check(ctx, grads, err_t, w.K, f"[step {step}]")
        err_t = torch.from_numpy(ref["err"])
        g2 = WL.gradients(w, 100 + step)
        e2 = torch.zeros(w.N, w.d, device=DEV)
        ctx.mv_sparse_step(g2.to(DEV), e2, oi, ov)
        torch.cuda.synchronize()
        PT.first_diff(PT.npy(oi), O.mv_sparse_step(g2.numpy(), np.zeros((w.N, w.d), np.float32), w.K)["out_idx"], f"[step {step}] mv")


def test_full_size_c2():
    w = WL.resnet_like("c2")
    ctx = B.MvContext(w.N, w.d, w.K, device=DEV)
    grads = WL.gradients(w, 0, device=DEV).cpu()
    err = torch.zeros(w.N, w.d)
    check(ctx, grads, err, w.K, "[c2]")


def test_capacity_is_checked_before_anything_runs():
    N, d, K = 3, 1000, 100
    ctx = B.MvContext(N, d, K, device=DEV)
    g = torch.zeros(N, d, device=DEV)
    e = torch.zeros(N, d, device=DEV)
    idx = torch.zeros(N * K - 1, dtype=torch.int32, device=DEV)
    val = torch.zeros(N * K - 1, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int32, device=DEV)
    with pytest.raises(B.MvError) as ei:
        ctx.mv_topk_union_step(g, e, idx, val, cnt)
    assert ei.value.status == B.MV_ERR_INVALID_ARG
