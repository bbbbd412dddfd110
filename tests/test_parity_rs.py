"""GPU parity of majority voting with random selection (SSGD-MV-RS) against the CPU oracle: the same
seed and draw counter must give the same mask index for index (the generator, the logarithm and the
ring-time rounding are fixed operation by operation), the values within 1e-6, the residual bit for bit."""
import numpy as np
import pytest
import torch

from tests import parity as PT
from oracle import mv_oracle as O
from oracle import rs_oracle as R
from paper_2011_06495_b200 import binding as B
from paper_2011_06495_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def gpu_select(ctx, votes_np, N, K, seed, draw, want_bits=True):
    d = votes_np.shape[0]
    votes = torch.from_numpy(votes_np).to(DEV)
    out_idx = torch.full((K,), -7, dtype=torch.int32, device=DEV)
    bits = torch.full(((d + 31) // 32,), -1, dtype=torch.int32, device=DEV) if want_bits else None
    ctx.mv_select_rs(votes, N, seed, draw, out_idx, bits, K=K)
    torch.cuda.synchronize()
    return out_idx.cpu().numpy(), (bits.cpu().numpy().view(np.uint32) if want_bits else None)


def votes_of(rng, N, d, K, pool):
    """Vote count of N workers that each vote for K coordinates out of a common pool of `pool` coordinates."""
    cand = rng.choice(d, size=min(d, max(K, pool)), replace=False)
    votes = np.zeros(d, dtype=np.uint8)
    for _ in range(N):
        votes[rng.choice(cand, size=K, replace=False)] += 1
    return votes


@pytest.mark.parametrize("N,d,K,pool", [
    (4, 1, 1, 1), (3, 37, 5, 12), (4, 4096, 100, 150), (4, 4097, 7, 4097), (6, 100_003, 1000, 3000),
    (10, 1_000_003, 10_000, 80_000), (25, 300_007, 300, 2000), (64, 50_000, 500, 50_000), (2, 12_289, 12_000, 12_289)])
def test_select_rs_matches_the_oracle(N, d, K, pool):
    rng = np.random.default_rng(d + K)
    votes = votes_of(rng, N, d, K, pool)
    ctx = B.MvContext(N, d, K, device=DEV)
    for seed, draw in ((1, 0), (0xDEADBEEFCAFE, 3), (7, (1 << 40) + 5)):
        want = R.select_mask_rs(votes, K, seed, draw)
        got, bits = gpu_select(ctx, votes, N, K, seed, draw)
        PT.first_diff(got, want, f"[rs {N}x{d} K={K} seed={seed} draw={draw}] out_idx")
        PT.first_diff(bits, O.support_to_bits(want, d), "mask_bits")
    a, _ = gpu_select(ctx, votes, N, K, 5, 1, False)
    b, _ = gpu_select(ctx, votes, N, K, 5, 2, False)
    if K < (votes > 0).sum():
        assert not np.array_equal(a, b)                        # another draw, another mask


def test_select_rs_with_fewer_voted_coordinates_than_K():
    N, d, K = 4, 10_000, 200
    votes = np.zeros(d, dtype=np.uint8)
    voted = np.sort(np.random.default_rng(1).choice(d, size=120, replace=False))
    votes[voted] = 2
    ctx = B.MvContext(N, d, K, device=DEV)
    got, bits = gpu_select(ctx, votes, N, K, 3, 4)
    assert np.array_equal(got[:120], voted) and np.all(got[120:] == -1)
    assert np.array_equal(got[:120], R.select_mask_rs(votes, K, 3, 4))
    PT.first_diff(bits, O.support_to_bits(voted.astype(np.int32), d), "mask_bits")
    # more voted coordinates than N workers with K votes each can produce: refused on the device, nothing selected
    votes[:] = 1
    got, bits = gpu_select(ctx, votes, N, K, 3, 4)
    assert np.all(got == -1) and not bits.any()


def test_select_rs_ties_in_ring_time():
    """Enough coordinates that binary32 ring times collide; K cut inside a tie group."""
    d, N = 400_000, 255
    votes = np.ones(d, dtype=np.uint8)
    t = R.ring_times(votes, 1, 1)
    srt = np.sort(t)
    dup = np.flatnonzero(srt[1:] == srt[:-1])
    dup = dup[dup >= 2000]                                   # K must be at least d / N for the votes to be admissible
    assert dup.size > 0
    K = int(dup[0]) + 1                                      # keeps the first of the two equal times only
    ctx = B.MvContext(N, d, K, device=DEV)
    got, _ = gpu_select(ctx, votes, N, K, 1, 1, False)
    want = R.select_mask_rs(votes, K, 1, 1)
    tied = np.flatnonzero(t == srt[dup[0]])
    assert tied[0] in want and tied[1] not in want
    PT.first_diff(got, want, "tie cut")


def test_selection_frequencies_on_the_gpu():
    """The GPU's own draws follow the votes: frequencies against the exact successive-sampling law."""
    from tests.test_oracle_rs import successive_sampling_probabilities
    votes = np.array([3, 1, 0, 2, 1, 0, 4], dtype=np.uint8)
    K, draws = 2, 3000
    exact = successive_sampling_probabilities(votes, K)
    ctx = B.MvContext(4, 7, K, device=DEV)
    v = torch.from_numpy(votes).to(DEV)
    out = torch.empty((draws, 4), dtype=torch.int32, device=DEV)       # rows 16-byte aligned
    for t in range(draws):
        ctx.mv_select_rs(v, 4, 99, t, out[t], None, K=K)
    torch.cuda.synchronize()
    sel = out.cpu().numpy()[:, :2]
    for k, p in exact.items():
        p = float(p)
        n = int(((sel[:, 0] == k[0]) & (sel[:, 1] == k[1])).sum())
        assert abs(n - draws * p) < 4.5 * np.sqrt(draws * p * (1 - p)), (k, n, draws * p)


@pytest.mark.parametrize("name,d,N,K", [("c2", 300_011, 4, 3000), ("c3", 1_000_003, 8, 1000), ("c2", 11_173_962, 10, 111_739)])
def test_rs_step_matches_the_oracle(name, d, N, K):
    w = WL.scaled(WL.resnet_like(name), d=d, N=N, K=K, steps=3)
    ctx = B.MvContext(w.N, w.d, w.K, device=DEV, mode=B.MV_MODE_TRACK)
    err = WL.initial_err(w, device=DEV)
    err_ref = err.cpu().numpy()
    out_idx = torch.empty(w.K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(w.K, dtype=torch.float32, device=DEV)
    masks = []
    for step in range(w.steps):
        grads = WL.gradients(w, step, device=DEV)
        ref = R.mv_rs_step(grads.cpu().numpy(), err_ref, w.K, seed=2011, draw=step, threads=8)
        ctx.mv_rs_step(grads, err, 2011, step, out_idx, out_val)
        torch.cuda.synchronize()
        tag = f"[rs step {step} {w.name}] "
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], tag + "out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), tag + "out_val")
        PT.first_diff(PT.bits(PT.npy(err)), PT.bits(ref["err"]), tag + "err")
        err_ref = ref["err"]
        masks.append(ref["out_idx"])
        # not the K most voted: the random mask differs from the deterministic one
        assert not np.array_equal(ref["out_idx"], O.select_mask(ref["votes"], w.K)[0])


@pytest.mark.parametrize("mode", [B.MV_MODE_AUTO, B.MV_MODE_GENERAL], ids=["auto", "general"])
def test_rs_step_in_the_other_threshold_modes(mode):
    """The whole random-selection step with the threshold sampled every call and with no sampling at all (the picks
    kernel of either route clears the list state of the selection that follows), a stand-alone selection of another
    size in between (which clears that state by itself), against the oracle."""
    w = WL.scaled(WL.resnet_like("c2"), d=200_003, N=5, K=2000, steps=3)
    ctx = B.MvContext(w.N, w.d, w.K, device=DEV, mode=mode)
    err = WL.initial_err(w, device=DEV)
    err_ref = err.cpu().numpy()
    out_idx = torch.empty(w.K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(w.K, dtype=torch.float32, device=DEV)
    g = torch.Generator().manual_seed(8)
    for step in range(w.steps):
        grads = WL.gradients(w, step, device=DEV)
        ref = R.mv_rs_step(grads.cpu().numpy(), err_ref, w.K, seed=77, draw=step, threads=8)
        ctx.mv_rs_step(grads, err, 77, step, out_idx, out_val)
        torch.cuda.synchronize()
        tag = f"[rs step {step}] "
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], tag + "out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), tag + "out_val")
        PT.first_diff(PT.bits(PT.npy(err)), PT.bits(ref["err"]), tag + "err")
        err_ref = ref["err"]
        if step == 0:
            d2, K2 = 50_021, 300
            votes2 = (torch.randint(1, w.N + 1, (d2,), generator=g) * (torch.rand(d2, generator=g) < 0.02)).to(torch.uint8).to(DEV)
            assert K2 <= int((votes2 > 0).sum()) <= w.N * K2
            oi2 = torch.empty(K2, dtype=torch.int32, device=DEV)
            ctx.mv_select_rs(votes2, w.N, 5, 9, oi2, K=K2)
            torch.cuda.synchronize()
            assert np.array_equal(oi2.cpu().numpy(), R.select_mask_rs(votes2.cpu().numpy(), K2, seed=5, draw=9))
