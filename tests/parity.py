"""Shared machinery of the GPU parity tests: runs every C-ABI entry point on one input and
compares each result with the CPU oracle, element by element."""
from __future__ import annotations

import numpy as np
import torch

from oracle import mv_oracle as O
from paper_2011_06495_b200 import binding as B

REL_TOL = 1e-6   # out_val: |gpu - oracle| <= REL_TOL * max(|oracle|, mean_n |acc[n, j]|); everything else is bit-exact


def bits(a):
    return np.ascontiguousarray(a).view(np.uint32) if a.dtype == np.float32 else a


def first_diff(a, b, what):
    a, b = np.asarray(a), np.asarray(b)
    assert a.shape == b.shape, f"{what}: shape {a.shape} vs {b.shape}"
    ne = np.flatnonzero(a.ravel() != b.ravel())
    if ne.size:
        i = int(ne[0])
        raise AssertionError(f"{what}: {ne.size} of {a.size} differ; first at flat {i}: gpu={a.ravel()[i]!r} oracle={b.ravel()[i]!r}; "
                             f"next {ne[:8].tolist()}")


def check_out_val(gpu_val, ref, acc, idx, what="out_val"):
    gv = gpu_val.astype(np.float64)
    rv = ref["out_val"].astype(np.float64) if isinstance(ref, dict) else ref.astype(np.float64)
    scale = np.maximum(np.abs(rv), np.abs(acc[:, idx].astype(np.float64)).mean(axis=0))
    with np.errstate(invalid="ignore"):
        bad = ~(np.abs(gv - rv) <= REL_TOL * scale)
    bad &= ~((gv == rv) | (np.isnan(gv) & np.isnan(rv)))
    if bad.any():
        i = int(np.flatnonzero(bad)[0])
        raise AssertionError(f"{what}: {int(bad.sum())} of {gv.size} outside {REL_TOL} rel; first k={i}: gpu={gv[i]!r} oracle={rv[i]!r}")


def run_phases(ctx, grads_t, err_t, K):
    """mv_vote -> mv_select -> mv_aggregate with every optional output requested."""
    N, d = grads_t.shape
    dev = grads_t.device
    W = (d + 31) // 32
    out = dict(
        acc=err_t.clone(),
        worker_idx=torch.full((N, K), -7, dtype=torch.int32, device=dev),
        worker_bits=torch.full((N, W), 0x5A5A5A5A, dtype=torch.int32, device=dev),
        votes=torch.full((d,), 77, dtype=torch.uint8, device=dev),
        thresh=torch.zeros((N, 3), dtype=torch.int32, device=dev),
        out_idx=torch.full((K,), -7, dtype=torch.int32, device=dev),
        mask_bits=torch.full((W,), 0x5A5A5A5A, dtype=torch.int32, device=dev),
        out_val=torch.full((K,), float("nan"), dtype=torch.float32, device=dev),
    )
    ctx.mv_vote(grads_t, out["acc"], out["worker_idx"], out["worker_bits"], out["votes"], out["thresh"], K=K)
    out["launches_vote"] = ctx.last_launches()
    out["diag"] = ctx.read_diag(N)
    ctx.mv_select(out["votes"], N, out["out_idx"], out["mask_bits"], K=K)
    out["err"] = out["acc"].clone()
    ctx.mv_aggregate(out["err"], out["out_idx"], out["out_val"])
    torch.cuda.synchronize()
    return out


def run_step(ctx, grads_t, err_t, K):
    dev = grads_t.device
    err = err_t.clone()
    out_idx = torch.full((K,), -7, dtype=torch.int32, device=dev)
    out_val = torch.full((K,), float("nan"), dtype=torch.float32, device=dev)
    ctx.mv_sparse_step(grads_t, err, out_idx, out_val, K=K)
    torch.cuda.synchronize()
    return dict(err=err, out_idx=out_idx, out_val=out_val, launches=ctx.last_launches())


def npy(t, dtype=None):
    a = t.detach().cpu().numpy()
    return a.view(dtype) if dtype is not None else a


def compare_all(ctx, grads_t, err_t, K, ref=None, by_sort=False, label=""):
    """Runs the phased calls and the fused step and compares everything with the oracle.
    Returns (oracle result, phased result, fused result)."""
    g_np, e_np = npy(grads_t), npy(err_t)
    if ref is None:
        ref = O.mv_sparse_step(g_np, e_np, K, by_sort=by_sort)
    ph = run_phases(ctx, grads_t, err_t, K)
    L = label
    first_diff(bits(npy(ph["acc"])), bits(ref["acc"]), L + "acc (err after mv_vote)")
    first_diff(npy(ph["thresh"], np.uint32), ref["thresh"], L + "thresh (T_n, cnt_gt, cnt_eq)")
    first_diff(npy(ph["worker_bits"], np.uint32), ref["worker_bits"], L + "worker_bits")
    first_diff(npy(ph["worker_idx"]), ref["worker_idx"], L + "worker_idx")
    first_diff(npy(ph["votes"]), ref["votes"], L + "votes")
    first_diff(npy(ph["out_idx"]), ref["out_idx"], L + "out_idx (mv_select)")
    first_diff(npy(ph["mask_bits"], np.uint32), ref["mask_bits"], L + "mask_bits")
    check_out_val(npy(ph["out_val"]), ref, ref["acc"], ref["out_idx"].astype(np.int64), L + "out_val (mv_aggregate)")
    first_diff(bits(npy(ph["err"])), bits(ref["err"]), L + "err (residual after mv_aggregate)")
    fu = run_step(ctx, grads_t, err_t, K)
    first_diff(npy(fu["out_idx"]), ref["out_idx"], L + "out_idx (mv_sparse_step)")
    first_diff(bits(npy(fu["out_val"])), bits(npy(ph["out_val"])), L + "out_val fused vs phased bytes")
    first_diff(bits(npy(fu["err"])), bits(ref["err"]), L + "err (mv_sparse_step)")
    fu2 = run_step(ctx, grads_t, err_t, K)   # same input again: identical bytes
    for k in ("out_idx", "out_val", "err"):
        assert torch.equal(fu[k].view(torch.int32), fu2[k].view(torch.int32)), L + f"{k} differs between two runs"
    # the whole step has two implementations of what follows the streaming pass (a sequence of kernels, and one
    # persistent kernel with grid barriers): both, forced, against the oracle and against each other
    for setting, name in ((2, "single-kernel tail"), (0, "kernel sequence")):
        ctx.set_tail_kernel(setting)
        try:
            fv = run_step(ctx, grads_t, err_t, K)
        finally:
            ctx.set_tail_kernel(1)
        first_diff(npy(fv["out_idx"]), ref["out_idx"], L + f"out_idx ({name})")
        first_diff(bits(npy(fv["err"])), bits(ref["err"]), L + f"err ({name})")
        first_diff(bits(npy(fv["out_val"])), bits(npy(fu["out_val"])), L + f"out_val bytes ({name})")
    return ref, ph, fu
