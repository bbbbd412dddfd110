"""GPU parity of majority voting with add-drop (mv_ad_step, Algorithm 2) against the CPU oracle:
the workers' vote masks, what they added and dropped, the running vote sum, the shared mask, the
aggregated values and the residual, over several steps with masks and residual carried."""
import numpy as np
import pytest
import torch

from oracle import mv_oracle as O
from paper_2011_06495_b200 import binding as B
from paper_2011_06495_b200 import workloads as WL
from tests import parity as PT

pytestmark = pytest.mark.gpu
DEV = "cuda"


def pack(mask_bool):
    """bool[N, d] -> uint32[N, ceil(d/32)] with bit b of word w = coordinate 32*w + b."""
    N, d = mask_bool.shape
    return np.stack([O.support_to_bits(np.flatnonzero(mask_bool[n]), d) for n in range(N)])


def lists_to_mask(lists, d):
    m = np.zeros((len(lists), d), dtype=bool)
    for n, l in enumerate(lists):
        m[n, l] = True
    return m


def run_steps(N, d, K, K_ad, steps, kind, seed, prev0=None, mode=B.MV_MODE_AUTO, want_lists=True):
    g = torch.Generator().manual_seed(seed)
    base = torch.randn(1, d, generator=g)
    W = (d + 31) // 32
    ctx = B.MvContext(N, d, K, device=DEV, mode=mode)
    err_ref = np.zeros((N, d), dtype=np.float32)
    prev_ref = np.zeros((N, d), dtype=bool) if prev0 is None else prev0.copy()
    err = torch.from_numpy(err_ref.copy()).to(DEV)
    prev_bits = torch.from_numpy(pack(prev_ref).view(np.int32)).to(DEV)
    out_idx = torch.empty(K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(K, dtype=torch.float32, device=DEV)
    add_bits = torch.empty((N, W), dtype=torch.int32, device=DEV)
    drop_bits = torch.empty((N, W), dtype=torch.int32, device=DEV)
    msum = torch.empty(d, dtype=torch.uint8, device=DEV)
    for step in range(steps):
        grads = 0.8 * base + 0.6 * torch.randn(N, d, generator=g)       # votes correlate over workers and steps
        if kind == "ties":
            grads = (grads * 4).round() / 4
        grads = grads.float().contiguous()
        ref = O.mv_ad_step(grads.numpy(), err_ref, prev_ref, K, K_ad)
        if want_lists:
            ctx.mv_ad_step(grads.to(DEV), err, prev_bits, K_ad, out_idx, out_val, add_bits, drop_bits, msum)
        else:       # without the add/drop outputs the vote masks are updated in place
            ctx.mv_ad_step(grads.to(DEV), err, prev_bits, K_ad, out_idx, out_val, None, None, msum)
        torch.cuda.synchronize()
        tag = f"[ad {N}x{d} K={K} K_ad={K_ad} {kind} step {step}] "
        if want_lists:
            PT.first_diff(PT.npy(add_bits, np.uint32), pack(lists_to_mask(ref["add"], d)), tag + "add_bits")
            PT.first_diff(PT.npy(drop_bits, np.uint32), pack(lists_to_mask(ref["drop"], d)), tag + "drop_bits")
        PT.first_diff(PT.npy(prev_bits, np.uint32), pack(ref["prev"]), tag + "vote masks")
        PT.first_diff(PT.npy(msum), ref["msum"], tag + "msum")
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], tag + "out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), tag + "out_val")
        PT.first_diff(PT.bits(PT.npy(err)), PT.bits(ref["err"]), tag + "err")
        err_ref, prev_ref = ref["err"], ref["prev"]


@pytest.mark.parametrize("kind", ["gauss", "ties"])
@pytest.mark.parametrize("N,d,K,K_ad", [(2, 8, 3, 1), (3, 1000, 50, 5), (4, 10001, 300, 30), (5, 65538, 655, 65),
                                        (3, 4097, 40, 40), (33, 5000, 50, 7), (2, 300007, 3000, 300)])
def test_add_drop_from_empty_votes(N, d, K, K_ad, kind):
    run_steps(N, d, K, K_ad, steps=5, kind=kind, seed=N * 100 + d)


@pytest.mark.parametrize("kind", ["gauss", "ties"])
@pytest.mark.parametrize("N,d,K,K_ad", [(3, 1000, 50, 5), (4, 10001, 300, 30), (33, 5000, 50, 7), (2, 300007, 3000, 300)])
def test_add_drop_in_place_update(N, d, K, K_ad, kind):
    run_steps(N, d, K, K_ad, steps=5, kind=kind, seed=N * 7 + d, want_lists=False)


def test_add_drop_from_given_votes():
    """Starting masks that share little with the workers' top-K: drops and adds both saturate."""
    N, d, K, K_ad = 4, 20011, 400, 40
    rng = np.random.default_rng(1)
    prev0 = np.zeros((N, d), dtype=bool)
    for n in range(N):
        prev0[n, rng.choice(d, size=K - 3 * n, replace=False)] = True
    run_steps(N, d, K, K_ad, steps=4, kind="gauss", seed=5, prev0=prev0)


@pytest.mark.parametrize("mode", [B.MV_MODE_AUTO, B.MV_MODE_TRACK], ids=["auto", "track"])
def test_add_drop_from_full_votes_across_boundaries(mode):
    """Starting masks with exactly K members (the most the contract allows), among them runs of coordinates that
    straddle a chunk boundary, word boundaries and the end of the row: the streaming pass lists every member with
    its key (the drop selection reads |acc| there), and that list is full to the last slot."""
    N, d, K, K_ad = 4, 20011, 400, 40
    rng = np.random.default_rng(2)
    prev0 = np.zeros((N, d), dtype=bool)
    prev0[:, 4090:4102] = True
    prev0[:, 8191:8193] = True
    prev0[:, 63:66] = True
    prev0[:, d - 5:] = True
    for n in range(N):
        free = np.flatnonzero(~prev0[n])
        prev0[n, rng.choice(free, size=K - int(prev0[n].sum()) - (3 * n if n else 0), replace=False)] = True
    assert prev0[0].sum() == K
    run_steps(N, d, K, K_ad, steps=4, kind="gauss", seed=6, prev0=prev0, mode=mode)
    run_steps(N, d, K, K_ad, steps=3, kind="ties", seed=7, prev0=prev0, mode=mode, want_lists=False)


def test_add_drop_without_sampling():
    run_steps(3, 50021, 500, 50, steps=3, kind="gauss", seed=9, mode=B.MV_MODE_GENERAL)


@pytest.mark.parametrize("N,d,K,K_ad", [(4, 300007, 3000, 300), (6, 100003, 500, 50)])
def test_add_drop_with_a_tracked_threshold(N, d, K, K_ad):
    """The bench's configuration: candidate threshold carried from step to step."""
    run_steps(N, d, K, K_ad, steps=6, kind="gauss", seed=13, mode=B.MV_MODE_TRACK, want_lists=False)


def test_large_K_ad_equals_plain_majority_voting():
    """K_ad = K: the step gives the same bytes as mv_sparse_step."""
    N, d, K = 5, 70001, 700
    g = torch.Generator().manual_seed(3)
    grads = torch.randn(N, d, generator=g).to(DEV)
    err0 = (0.3 * torch.randn(N, d, generator=g)).to(DEV)
    ctx = B.MvContext(N, d, K, device=DEV)
    W = (d + 31) // 32
    prev_bits = torch.zeros((N, W), dtype=torch.int32, device=DEV)
    a_idx = torch.empty(K, dtype=torch.int32, device=DEV)
    a_val = torch.empty(K, dtype=torch.float32, device=DEV)
    a_err = err0.clone()
    ctx.mv_ad_step(grads, a_err, prev_bits, K, a_idx, a_val)
    b_idx, b_val, b_err = torch.empty_like(a_idx), torch.empty_like(a_val), err0.clone()
    ctx.mv_sparse_step(grads, b_err, b_idx, b_val)
    torch.cuda.synchronize()
    assert torch.equal(a_idx, b_idx) and torch.equal(a_val.view(torch.int32), b_val.view(torch.int32))
    assert torch.equal(a_err.view(torch.int32), b_err.view(torch.int32))


def test_add_drop_at_resnet_size():
    """c2-sized (N=10, d=11,173,962, K=d/100) with K_ad = K/10, the paper's setting; three steps."""
    w = WL.resnet_like("c2")
    K_ad = w.K // 10
    std = WL.std_vector(w, DEV)
    ctx = B.MvContext(w.N, w.d, w.K, device=DEV, mode=B.MV_MODE_TRACK)
    W = (w.d + 31) // 32
    err = WL.initial_err(w, device=DEV)
    err_ref = err.cpu().numpy()
    prev_ref = np.zeros((w.N, w.d), dtype=bool)
    prev_bits = torch.zeros((w.N, W), dtype=torch.int32, device=DEV)
    out_idx = torch.empty(w.K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(w.K, dtype=torch.float32, device=DEV)
    msum = torch.empty(w.d, dtype=torch.uint8, device=DEV)
    grads = torch.empty((w.N, w.d), dtype=torch.float32, device=DEV)
    for step in range(3):
        WL.gradients(w, step, out=grads, std=std)
        ref = O.mv_ad_step(grads.cpu().numpy(), err_ref, prev_ref, w.K, K_ad)
        ctx.mv_ad_step(grads, err, prev_bits, K_ad, out_idx, out_val, None, None, msum)
        torch.cuda.synchronize()
        tag = f"[ad c2 step {step}] "
        PT.first_diff(PT.npy(prev_bits, np.uint32), pack(ref["prev"]), tag + "vote masks")
        PT.first_diff(PT.npy(msum), ref["msum"], tag + "msum")
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], tag + "out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), tag + "out_val")
        PT.first_diff(PT.bits(PT.npy(err)), PT.bits(ref["err"]), tag + "err")
        err_ref, prev_ref = ref["err"], ref["prev"]
