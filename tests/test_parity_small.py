"""GPU parity, small and mid sizes: every entry point against the CPU oracle, element by element,
in both threshold modes, over shapes that cover several chunks, ragged tails, misaligned rows,
ties, degenerate inputs and the fallback from the sampled pass to the exact select."""
import numpy as np
import pytest
import torch

from oracle import mv_oracle as O
from paper_2011_06495_b200 import binding as B
from paper_2011_06495_b200 import workloads as WL
from tests import parity as PT

pytestmark = pytest.mark.gpu
DEV = "cuda"
MODES = [B.MV_MODE_AUTO, B.MV_MODE_GENERAL, B.MV_MODE_TRACK]
MODE_IDS = ["auto", "general", "track"]


def make(N, d, kind, seed):
    g = torch.Generator().manual_seed(seed)
    grads = torch.randn(N, d, generator=g)
    err = 0.3 * torch.randn(N, d, generator=g)
    if kind == "gauss":
        pass
    elif kind == "ties":
        grads = (grads * 4).round() / 4
        err = (err * 4).round() / 4
    elif kind == "ties_fine":       # a fine grid: a handful of equal magnitudes at every level
        grads = (grads * 2048).round() / 2048
        err = torch.zeros(N, d)
    elif kind == "equal":
        grads = torch.full((N, d), 0.5)
        grads[::2] *= -1
        err = torch.full((N, d), 0.25)
        err[::2] *= -1
    elif kind == "zeros":
        grads = torch.zeros(N, d)
        err = torch.zeros(N, d)
    elif kind == "sparse":          # mostly zero, a few large values: threshold lands on the zero ties
        keep = torch.rand(N, d, generator=g) < 0.01
        grads = grads * keep
        err = torch.zeros(N, d)
    elif kind == "layers":          # scale changes by decades along the row
        scale = 10.0 ** (-3 * torch.arange(d) / max(d - 1, 1))
        grads = grads * scale
        err = err * scale
    else:
        raise ValueError(kind)
    return grads.float().contiguous(), err.float().contiguous()


SHAPES = [
    # N, d, K
    (1, 1, 1), (1, 5, 5), (3, 31, 4), (2, 33, 33), (4, 4096, 10), (4, 4097, 7), (3, 8191, 100),
    (5, 10001, 1000), (7, 12289, 1), (9, 65538, 655), (10, 100003, 1000), (33, 5000, 50), (64, 20000, 200),
    (2, 12288, 12288), (3, 9001, 9000),
]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("kind", ["gauss", "ties", "layers"])
@pytest.mark.parametrize("N,d,K", SHAPES)
def test_shapes(N, d, K, kind, mode):
    grads, err = make(N, d, kind, seed=N * 1000 + d + K)
    ctx = B.MvContext(N, d, K, device=DEV, mode=mode)
    PT.compare_all(ctx, grads.to(DEV), err.to(DEV), K, by_sort=(d <= 20000), label=f"[{N}x{d} K={K} {kind}] ")


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
@pytest.mark.parametrize("kind", ["equal", "zeros", "sparse"])
@pytest.mark.parametrize("N,d,K", [(3, 5000, 17), (4, 20011, 300), (2, 300007, 10)])
def test_degenerate(N, d, K, kind, mode):
    grads, err = make(N, d, kind, seed=d + K)
    ctx = B.MvContext(N, d, K, device=DEV, mode=mode)
    PT.compare_all(ctx, grads.to(DEV), err.to(DEV), K, label=f"[{N}x{d} K={K} {kind}] ")


def test_max_workers():
    N, d, K = 255, 3001, 30
    grads, err = make(N, d, "ties", seed=255)
    ctx = B.MvContext(N, d, K, device=DEV)
    PT.compare_all(ctx, grads.to(DEV), err.to(DEV), K, label="[N=255] ")


def test_longest_row():
    """d at the documented limit (2^31 - 8193) with two workers, so that coordinates, flat offsets
    n*d + j and chunk numbers reach their largest values.  The expected result follows from the
    definition alone: a background of small values, a few hundred planted distinct large magnitudes
    (always selected) and a few thousand planted equal magnitudes of which only the lowest indices
    fit - placed at the very start, the very end and around 2^30 and 2^31 - 2^13 as well."""
    N, K = 2, 2000
    d = (1 << 31) - 8193
    rng = np.random.default_rng(31)
    ctx = B.MvContext(N, d, K, device=DEV)
    grads = torch.empty((N, d), dtype=torch.float32, device=DEV)
    err = torch.empty((N, d), dtype=torch.float32, device=DEV)
    g = torch.Generator(device=DEV).manual_seed(31)
    for n in range(N):
        grads[n].normal_(0.0, 0.01, generator=g)
        err[n].normal_(0.0, 0.001, generator=g)
    special = np.array([0, 1, 31, 4095, 4096, (1 << 30) - 1, 1 << 30, (1 << 31) - 16384, d - 4097, d - 4096, d - 33, d - 2, d - 1])
    planted = []
    for n in range(N):
        pos = np.unique(np.concatenate([special, rng.integers(0, d, size=3200)]))
        rng.shuffle(pos)
        big, tied = np.sort(pos[:500]), np.sort(pos[500:3000])
        if n == 1:                                                  # half of worker 1's distinct picks coincide with worker 0's
            big = np.unique(np.concatenate([planted[0][0][::2], big[:250]]))
            tied = np.setdiff1d(tied, big)
        planted.append((big, tied))
        tpos = torch.from_numpy(np.concatenate([big, tied])).to(DEV)
        vals = torch.cat([torch.arange(big.size, device=DEV, dtype=torch.float32) * (1 if n == 0 else -1) + (200.0 if n == 0 else -200.0),
                          torch.full((tied.size,), -100.0 if n == 0 else 100.0, device=DEV)])
        grads[n, tpos] = vals
        err[n, tpos] = 0.0
    # the definition, on the planted positions only: each worker keeps its distinct values and the lowest-index ties
    worker_sets = [np.sort(np.concatenate([b, t[:K - b.size]])) for b, t in planted]
    pos, votes = np.unique(np.concatenate(worker_sets), return_counts=True)
    order = np.lexsort((pos, -votes))                               # votes descending, index ascending
    want_idx = np.sort(pos[order[:K]]).astype(np.int64)
    out_idx = torch.empty(K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(K, dtype=torch.float32, device=DEV)
    widx = torch.empty((N, K), dtype=torch.int32, device=DEV)
    acc_at = (grads[:, torch.from_numpy(want_idx).to(DEV)] + err[:, torch.from_numpy(want_idx).to(DEV)]).double().cpu().numpy()
    probe = torch.from_numpy(np.concatenate([special, rng.integers(0, d, size=100_000)])).to(DEV)
    acc_probe = grads[:, probe] + err[:, probe]
    e = err.clone()
    ctx.mv_vote(grads, e, worker_idx=widx)                          # sampled threshold
    torch.cuda.synchronize()
    for n in range(N):
        PT.first_diff(PT.npy(widx[n]).astype(np.int64), worker_sets[n].astype(np.int64), f"worker {n} top-K")
    ctx.set_mode(B.MV_MODE_TRACK)
    launches = []
    for call in range(2):                                           # the second call runs with a carried threshold
        e.copy_(err)
        ctx.mv_sparse_step(grads, e, out_idx, out_val)
        torch.cuda.synchronize()
        launches.append(ctx.last_launches())
        # K/d is 1e-6 here: a sample of 2^20 elements cannot bracket the K-th key (both workers take the
        # full-row select on the first call); the carried threshold of the second call can
        assert ctx.read_diag(N)[:, 2].tolist() == ([1, 1] if call == 0 else [0, 0])
        PT.first_diff(PT.npy(out_idx).astype(np.int64), want_idx, f"call {call} out_idx")
        np.testing.assert_allclose(PT.npy(out_val).astype(np.float64), acc_at.sum(axis=0) / N, rtol=1e-6, atol=0)
        got = e[:, probe]
        in_mask = torch.from_numpy(np.isin(PT.npy(probe), want_idx)).to(DEV)
        assert bool((got[:, in_mask] == 0).all()) and torch.equal(got[:, ~in_mask], acc_probe[:, ~in_mask])
        assert int((e[:, torch.from_numpy(want_idx).to(DEV)] != 0).sum()) == 0
    assert launches[1] == launches[0] - 1


@pytest.mark.parametrize("name", ["c1", "c1_ties"])
@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
def test_config_c1(name, mode):
    w = WL.resnet_like(name)
    grads = WL.gradients(w, 0)
    err = WL.initial_err(w)
    if name == "c1":
        key = O.magnitude_key(grads.numpy())
        assert all(np.unique(key[n]).size == w.d for n in range(w.N)), "c1 is meant to be tie-free"
    ctx = B.MvContext(w.N, w.d, w.K, device=DEV, mode=mode)
    ref, ph, fu = PT.compare_all(ctx, grads.to(DEV), err.to(DEV), w.K, by_sort=True, label=f"[{name}] ")
    if name == "c1_ties":
        assert (ref["thresh"][:, 2] > 1).all(), "forced ties should straddle every worker's threshold"


def test_special_values():
    """Signed zeros, denormals and infinities follow the bit-pattern order; residual bytes are exact."""
    N, d, K = 3, 4500, 40
    grads, err = make(N, d, "gauss", seed=4500)
    grads[0, 7] = float("inf")
    grads[1, 4099] = float("-inf")
    grads[2, 10:60] = 1e-41          # denormals
    err[2, 10:60] = 0.0
    grads[0, 100:200] = -0.0
    err[0, 100:200] = -0.0
    for mode in MODES:
        ctx = B.MvContext(N, d, K, device=DEV, mode=mode)
        PT.compare_all(ctx, grads.to(DEV), err.to(DEV), K, by_sort=True, label="[special] ")


@pytest.mark.parametrize("N,d,K", [(4, 300007, 3000), (3, 1000003, 250), (16, 1 << 20, 1048)])
def test_sampled_threshold_path(N, d, K):
    """d large enough that the threshold bound comes from a strided sample; the streaming pass must
    succeed for every worker (no fallback) on smooth data, and all results stay exact."""
    grads, err = make(N, d, "gauss", seed=d)
    ctx = B.MvContext(N, d, K, device=DEV)
    ref, ph, fu = PT.compare_all(ctx, grads.to(DEV), err.to(DEV), K, label=f"[sampled {N}x{d}] ")
    diag = ph["diag"]
    assert (diag[:, 2] == 0).all(), f"fallback used: {diag.tolist()}"
    assert (diag[:, 0] >= K).all() and (diag[:, 0] <= 4 * K + 4096).all()


@pytest.mark.parametrize("kind", ["ties", "ties_fine"])
@pytest.mark.parametrize("N,d,K", [(3, 300007, 2500), (2, 1000003, 300)])
def test_sampled_threshold_path_with_ties(N, d, K, kind):
    """Threshold ties that are only partly kept, in the sampled regime: a few of them (ranked in a small
    list) and thousands of them (walked chunk by chunk)."""
    grads, err = make(N, d, kind, seed=d + 17)
    ctx = B.MvContext(N, d, K, device=DEV)
    ref, ph, fu = PT.compare_all(ctx, grads.to(DEV), err.to(DEV), K, label=f"[sampled {kind} {N}x{d}] ")
    assert (ref["thresh"][:, 2] > ref["thresh"][:, 1] * 0 + 1).all(), "the threshold should be tied"


def test_threshold_beyond_the_sampled_range():
    """The sample misses a group of huge values (they sit only in lines it does not visit), so the
    K-th largest key lies far above the sampled bound: the candidate select must still be exact."""
    N, d, K = 2, 400_000, 1000
    g = torch.Generator().manual_seed(77)
    grads = torch.randn(N, d, generator=g)
    err = torch.zeros(N, d)
    lines = torch.arange(d) // 32
    hidden = torch.nonzero(lines % 2 == 1).flatten()          # the sample visits lines 0, 10, 20, ... only
    pick = hidden[torch.randperm(hidden.numel(), generator=g)[:2000]]
    grads[:, pick] = grads[:, pick] * 1e6 + 1e6
    ctx = B.MvContext(N, d, K, device=DEV)
    ref, ph, fu = PT.compare_all(ctx, grads.contiguous().to(DEV), err.to(DEV), K, label="[beyond range] ")
    assert (ph["diag"][:, 2] == 0).all(), "the candidate path should have been kept"
    assert (ref["thresh"][:, 0] > 0x49000000).all()            # T_n is one of the huge values


@pytest.mark.parametrize("N,d,K", [(2, 500_000, 1), (2, 500_000, 499_999), (3, 400_001, 200_000), (2, 1_000_003, 7)])
def test_sampled_regime_extreme_K(N, d, K):
    """K = 1, K close to d and K = d/2 at sizes where the threshold bound comes from a sample: whatever
    path each worker ends up on, the results are exact."""
    grads, err = make(N, d, "gauss", seed=K + d)
    ctx = B.MvContext(N, d, K, device=DEV)
    PT.compare_all(ctx, grads.to(DEV), err.to(DEV), K, label=f"[extreme K {N}x{d} K={K}] ")


def test_fallback_per_worker():
    """One smooth worker next to one whose values are all equal (its candidate count overflows):
    the second takes the exact multi-pass select, the first does not, results are exact."""
    N, d, K = 3, 300007, 100
    grads, err = make(N, d, "gauss", seed=99)
    grads[1] = 0.125
    err[1] = 0.0
    ctx = B.MvContext(N, d, K, device=DEV)
    ref, ph, fu = PT.compare_all(ctx, grads.to(DEV), err.to(DEV), K, label="[fallback] ")
    assert ph["diag"][:, 2].tolist() == [0, 1, 0]
    assert ref["worker_idx"][1].tolist() == list(range(K))


def test_error_feedback_over_steps():
    """Residuals carried over several steps stay bit-identical to the oracle's."""
    w = WL.scaled(WL.resnet_like("c2"), d=200003, N=6, steps=5)
    ctx = B.MvContext(w.N, w.d, w.K, device=DEV)
    err_gpu = WL.initial_err(w).to(DEV)
    err_ref = WL.initial_err(w).numpy()
    out_idx = torch.empty(w.K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(w.K, dtype=torch.float32, device=DEV)
    for step in range(w.steps):
        grads = WL.gradients(w, step)
        ref = O.mv_sparse_step(grads.numpy(), err_ref, w.K)
        ctx.mv_sparse_step(grads.to(DEV), err_gpu, out_idx, out_val)
        torch.cuda.synchronize()
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], f"step {step} out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), f"step {step} out_val")
        PT.first_diff(PT.bits(PT.npy(err_gpu)), PT.bits(ref["err"]), f"step {step} err")
        err_ref = ref["err"]


@pytest.mark.parametrize("N,d,K", [(6, 200003, 2000), (3, 1000003, 250), (4, 50000, 5000), (2, 4097, 7),
                                   (2, (1 << 21) + 3, 300_000)])   # the last: candidate buffers beyond 2^20 entries
def test_threshold_tracking_over_steps(N, d, K):
    """MV_MODE_TRACK: after the first call the candidate threshold comes from the previous call's key
    histogram (one kernel fewer); every step stays bit-identical to the oracle, and on slowly
    changing data no worker needs the fallback."""
    w = WL.scaled(WL.resnet_like("c2"), d=d, N=N, K=K, steps=7)
    ctx = B.MvContext(w.N, w.d, w.K, device=DEV, mode=B.MV_MODE_TRACK)
    err_gpu = WL.initial_err(w).to(DEV)
    err_ref = WL.initial_err(w).numpy()
    out_idx = torch.empty(w.K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(w.K, dtype=torch.float32, device=DEV)
    launches = []
    for step in range(w.steps):
        grads = WL.gradients(w, step)
        ref = O.mv_sparse_step(grads.numpy(), err_ref, w.K)
        ctx.mv_sparse_step(grads.to(DEV), err_gpu, out_idx, out_val)
        torch.cuda.synchronize()
        launches.append(ctx.last_launches())
        diag = ctx.read_diag(w.N)
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], f"step {step} out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), f"step {step} out_val")
        PT.first_diff(PT.bits(PT.npy(err_gpu)), PT.bits(ref["err"]), f"step {step} err")
        if step >= 2:
            assert (diag[:, 2] == 0).all(), f"step {step}: fallback with a tracked threshold: {diag.tolist()}"
        err_ref = ref["err"]
    if d <= 32768:
        assert set(launches) == {1}            # a row that fits a CTA's shared memory: the whole step is one kernel
    else:
        assert launches[0] == launches[1] + 1 and len(set(launches[1:])) == 1      # the sampling kernel runs once


@pytest.mark.parametrize("mode", [B.MV_MODE_AUTO, B.MV_MODE_TRACK], ids=["auto", "track"])
def test_magnitudes_spread_over_many_binades(mode):
    """Magnitudes log-uniform over sixty binades: the candidates above the threshold bound span many
    powers of two, so the K-th key lies far outside the narrow window of keys that the select looks
    at first and the three-digit radix select over the candidates has to find it; with ties (every
    magnitude is a power of 2^(1/8), so there are only a few hundred distinct keys) on top."""
    N, d, K = 3, 300_007, 2000
    g = torch.Generator().manual_seed(4242)
    ctx = B.MvContext(N, d, K, device=DEV, mode=mode)
    err_gpu = torch.zeros(N, d, device=DEV)
    err_ref = np.zeros((N, d), dtype=np.float32)
    out_idx = torch.empty(K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(K, dtype=torch.float32, device=DEV)
    for step in range(3):
        expo = torch.randint(-240, 240, (N, d), generator=g).float() / 8.0
        sign = torch.randint(0, 2, (N, d), generator=g).float() * 2 - 1
        grads = (sign * torch.exp2(expo)).float().contiguous()
        ref = O.mv_sparse_step(grads.numpy(), err_ref, K)
        ctx.mv_sparse_step(grads.to(DEV), err_gpu, out_idx, out_val)
        torch.cuda.synchronize()
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], f"step {step} out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), f"step {step} out_val")
        PT.first_diff(PT.bits(PT.npy(err_gpu)), PT.bits(ref["err"]), f"step {step} err")
        err_ref = ref["err"]


@pytest.mark.parametrize("name,N,d,K", [("c3", 8, 400_009, 400), ("c2", 6, 300_007, 3000), ("c4", 4, 500_003, 125)])
def test_threshold_tracking_long_run(name, N, d, K):
    """Hundreds of consecutive steps: the tracked threshold neither drifts out of the usable range
    (no fallback once the residuals have built up) nor oscillates; the last step is compared with
    the oracle from the device's own residual state."""
    w = WL.scaled(WL.resnet_like(name), d=d, N=N, K=K, steps=1)
    ctx = B.MvContext(w.N, w.d, w.K, device=DEV, mode=B.MV_MODE_TRACK)
    pool = [WL.gradients(w, s, device=DEV) for s in range(5)]
    err = WL.initial_err(w, device=DEV)
    out_idx = torch.empty(w.K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(w.K, dtype=torch.float32, device=DEV)
    fallbacks, ratio = [], []
    steps = 600
    for step in range(steps):
        if step == steps - 1:
            err_before = err.cpu().numpy()
        ctx.mv_sparse_step(pool[step % 5], err, out_idx, out_val)
        if step % 7 == 0 or step == steps - 1:
            diag = ctx.read_diag(w.N)
            fallbacks.append(int(diag[:, 2].sum()))
            ratio.append(float(diag[:, 0].max()) / w.K)
    torch.cuda.synchronize()
    assert sum(fallbacks[2:]) == 0, f"fallbacks at sampled steps: {fallbacks}"
    assert max(ratio[2:]) < 3.5 and min(ratio[2:]) >= 1.0, f"candidates per K out of range: {ratio}"
    ref = O.mv_sparse_step(PT.npy(pool[(steps - 1) % 5]), err_before, w.K)
    PT.first_diff(PT.npy(out_idx), ref["out_idx"], "last step out_idx")
    PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), "last step out_val")
    PT.first_diff(PT.bits(PT.npy(err)), PT.bits(ref["err"]), "last step err")


def test_threshold_tracking_survives_a_change_of_scale():
    """The tracked threshold is only a guess: when the data jumps by orders of magnitude between two
    calls the affected workers take the exact multi-pass select for that call and results stay exact;
    the call after that is back on the fast path.  Another (d, K) on the same context samples again."""
    N, d, K = 4, 300007, 3000
    ctx = B.MvContext(N, d, K, device=DEV, mode=B.MV_MODE_TRACK)
    grads, err = make(N, d, "gauss", seed=31)
    scales = [1.0, 1.0, 1e3, 1e3, 1e-4, 1e-4, 1.0]
    fell_back = []
    for step, sc in enumerate(scales):
        g = (grads * sc).roll(step, dims=1).contiguous()
        e = (err * sc).contiguous()
        g[1] = grads[1].roll(step)                      # worker 1 keeps its scale throughout
        e[1] = err[1]
        ref = O.mv_sparse_step(g.numpy(), e.numpy(), K)
        fu = PT.run_step(ctx, g.to(DEV), e.to(DEV), K)
        fell_back.append(ctx.read_diag(N)[:, 2].tolist())
        PT.first_diff(PT.npy(fu["out_idx"]), ref["out_idx"], f"step {step} out_idx")
        PT.check_out_val(PT.npy(fu["out_val"]), ref, ref["acc"], ref["out_idx"].astype(np.int64), f"step {step} out_val")
        PT.first_diff(PT.bits(PT.npy(fu["err"])), PT.bits(ref["err"]), f"step {step} err")
    assert fell_back[0] == [0, 0, 0, 0] and fell_back[1] == [0, 0, 0, 0]
    assert fell_back[2] == [1, 0, 1, 1] and fell_back[4] == [1, 0, 1, 1] and fell_back[6] == [1, 0, 1, 1]
    assert fell_back[3] == [0, 0, 0, 0] and fell_back[5] == [0, 0, 0, 0]
    # a smaller problem on the same context: nothing is carried over
    d2, K2 = 100003, 500
    g2, e2 = make(N, d2, "gauss", seed=32)
    ref = O.mv_sparse_step(g2.numpy(), e2.numpy(), K2)
    out_idx = torch.empty(K2, dtype=torch.int32, device=DEV)
    out_val = torch.empty(K2, dtype=torch.float32, device=DEV)
    e2g = e2.to(DEV)
    before = None
    for rep in range(2):
        e2g.copy_(e2)
        ctx.mv_sparse_step(g2.to(DEV), e2g, out_idx, out_val, K=K2)
        torch.cuda.synchronize()
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], f"second problem, call {rep}")
        PT.first_diff(PT.bits(PT.npy(e2g)), PT.bits(ref["err"]), f"second problem, call {rep} err")
        assert (ctx.read_diag(N)[:, 2] == 0).all()
        if rep == 0:
            before = ctx.last_launches()
    assert ctx.last_launches() == before - 1


@pytest.mark.parametrize("mode", [B.MV_MODE_AUTO, B.MV_MODE_TRACK], ids=["auto", "track"])
def test_one_context_changing_K_and_entry_points(mode):
    """One context serves steps whose K changes from call to call, with other entry points (the
    three phases, with buffers of their own) called in between: every call starts from clean
    scratch counters, masks and votes whatever the call before it left, and a tracked threshold
    of another K is not reused."""
    N, d = 5, 200_003
    Ks = [2000, 150, 2000, 2000, 7000, 150, 2000]
    g = torch.Generator().manual_seed(9001)
    ctx = B.MvContext(N, d, max(Ks), device=DEV, mode=mode)
    err_gpu = torch.zeros(N, d, device=DEV)
    err_ref = np.zeros((N, d), dtype=np.float32)
    W = (d + 31) // 32
    for step, K in enumerate(Ks):
        grads = torch.randn(N, d, generator=g) * (1.0 + 0.1 * step)
        ref = O.mv_sparse_step(grads.numpy(), err_ref, K)
        out_idx = torch.full((K,), -7, dtype=torch.int32, device=DEV)
        out_val = torch.full((K,), float("nan"), dtype=torch.float32, device=DEV)
        ctx.mv_sparse_step(grads.to(DEV), err_gpu, out_idx, out_val, K=K)
        torch.cuda.synchronize()
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], f"step {step} K={K} out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), f"step {step} out_val")
        PT.first_diff(PT.bits(PT.npy(err_gpu)), PT.bits(ref["err"]), f"step {step} err")
        err_ref = ref["err"]
        if step % 2 == 0:
            # the phases on other data, another K, outputs in caller buffers: must not disturb the next step
            K2 = 333
            g2 = torch.randn(N, d, generator=g)
            acc2 = torch.zeros(N, d, device=DEV)
            votes = torch.full((d,), 9, dtype=torch.uint8, device=DEV)
            bits_ = torch.full((N, W), -1, dtype=torch.int32, device=DEV)
            idx2 = torch.empty(K2, dtype=torch.int32, device=DEV)
            val2 = torch.empty(K2, dtype=torch.float32, device=DEV)
            ref2 = O.mv_sparse_step(g2.numpy(), np.zeros((N, d), dtype=np.float32), K2)
            ctx.mv_vote(g2.to(DEV), acc2, None, bits_, votes, None, K=K2)
            ctx.mv_select(votes, N, idx2, None, K=K2)
            ctx.mv_aggregate(acc2, idx2, val2)
            torch.cuda.synchronize()
            PT.first_diff(PT.npy(votes), ref2["votes"], f"step {step} phases votes")
            PT.first_diff(PT.npy(idx2), ref2["out_idx"], f"step {step} phases out_idx")
            PT.first_diff(PT.bits(PT.npy(acc2)), PT.bits(ref2["err"]), f"step {step} phases err")


def test_checkpoint_resume():
    """The residual is the only state: saving and restoring it mid-run changes nothing."""
    w = WL.scaled(WL.resnet_like("c3"), d=50021, N=5, steps=6)
    outs = []
    for split in (None, 3):
        ctx = B.MvContext(w.N, w.d, w.K, device=DEV)
        err = WL.initial_err(w).to(DEV)
        out_idx = torch.empty(w.K, dtype=torch.int32, device=DEV)
        out_val = torch.empty(w.K, dtype=torch.float32, device=DEV)
        for step in range(w.steps):
            if split is not None and step == split:
                saved = err.cpu().clone()
                ctx = B.MvContext(w.N, w.d, w.K, device=DEV)
                err = saved.to(DEV)
            ctx.mv_sparse_step(WL.gradients(w, step).to(DEV), err, out_idx, out_val)
        torch.cuda.synchronize()
        outs.append((err.cpu(), out_idx.cpu(), out_val.cpu()))
    for a, b in zip(*outs):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))


def test_host_entry_point():
    """mv_sparse_step_host: gradients in pinned host memory, results back in host memory."""
    N, d, K = 4, 70001, 700
    grads, err = make(N, d, "gauss", seed=5)
    ref = O.mv_sparse_step(grads.numpy(), err.numpy(), K)
    ctx = B.MvContext(N, d, K, device=DEV)
    h_grads = grads.pin_memory()
    h_idx = torch.empty(K, dtype=torch.int32).pin_memory()
    h_val = torch.empty(K, dtype=torch.float32).pin_memory()
    d_grads = torch.empty(N, d, device=DEV)
    d_err = err.to(DEV)
    d_idx = torch.empty(K, dtype=torch.int32, device=DEV)
    d_val = torch.empty(K, dtype=torch.float32, device=DEV)
    ctx.mv_sparse_step_host(h_grads, h_idx, h_val, d_grads, d_err, d_idx, d_val)
    PT.first_diff(h_idx.numpy(), ref["out_idx"], "host out_idx")
    PT.check_out_val(h_val.numpy(), ref, ref["acc"], ref["out_idx"].astype(np.int64), "host out_val")
    PT.first_diff(PT.bits(PT.npy(d_err)), PT.bits(ref["err"]), "host err")


def test_argument_errors_on_device_pointers():
    N, d, K = 2, 1000, 10
    ctx = B.MvContext(N, d, K, device=DEV)
    g = torch.zeros(N, d, device=DEV)
    e = torch.zeros(N, d, device=DEV)
    oi = torch.zeros(K, dtype=torch.int32, device=DEV)
    ov = torch.zeros(K, device=DEV)
    with pytest.raises(B.MvError) as ei:
        ctx.mv_sparse_step(g, g, oi, ov)                    # grads aliases err
    assert ei.value.status == B.MV_ERR_INVALID_ARG
    with pytest.raises(B.MvError) as ei:
        ctx.mv_sparse_step(g, e, oi, ov, K=d + 1)           # K > d
    assert ei.value.status == B.MV_ERR_INVALID_ARG
    big = torch.zeros(N, 100 * d, device=DEV)
    with pytest.raises(B.MvError) as ei:
        ctx.mv_sparse_step(big, big.clone(), oi, ov)        # workspace sized for a smaller problem
    assert ei.value.status == B.MV_ERR_WORKSPACE
    ctx.mv_sparse_step(g, e, oi, ov)                        # the context is still usable
    torch.cuda.synchronize()


def test_random_selection_of_another_size_between_steps():
    """A stand-alone mv_select_rs of a much smaller problem writes its list state at the offsets of its
    own (N, d, K), inside what a whole step of the larger problem left cleared: the step that follows
    must start from clean counters all the same (compared with the oracle, residual carried)."""
    from oracle import rs_oracle as R
    N, d, K = 16, 120_011, 1200
    ctx = B.MvContext(N, d, K, device=DEV, mode=B.MV_MODE_TRACK)
    g = torch.Generator().manual_seed(4242)
    err_gpu = torch.zeros(N, d, device=DEV)
    err_ref = np.zeros((N, d), dtype=np.float32)
    out_idx = torch.empty(K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(K, dtype=torch.float32, device=DEV)
    N2, d2, K2 = 2, 9001, 40
    for step in range(4):
        grads = torch.randn(N, d, generator=g)
        ref = O.mv_sparse_step(grads.numpy(), err_ref, K)
        ctx.mv_sparse_step(grads.to(DEV), err_gpu, out_idx, out_val)
        torch.cuda.synchronize()
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], f"step {step} out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), f"step {step} out_val")
        PT.first_diff(PT.bits(PT.npy(err_gpu)), PT.bits(ref["err"]), f"step {step} err")
        err_ref = ref["err"]
        # the small random selection in between (votes of N2 workers with K2 votes each)
        votes2 = np.zeros(d2, dtype=np.uint8)
        rng = np.random.default_rng(step)
        for _ in range(N2):
            votes2[rng.choice(d2, K2, replace=False)] += 1
        idx2 = torch.empty(K2, dtype=torch.int32, device=DEV)
        ctx.mv_select_rs(torch.from_numpy(votes2).to(DEV), N2, 77, step, idx2, None, K=K2)
        torch.cuda.synchronize()
        PT.first_diff(PT.npy(idx2), R.select_mask_rs(votes2, K2, 77, step), f"step {step} small random selection")


def _debug_context(N, d, K, mode=B.MV_MODE_AUTO):
    from paper_2011_06495_b200 import build as BLD
    BLD.build(debug=True)                      # no-op when the checked library is up to date
    ctx = B.MvContext(N, d, K, device=DEV, mode=mode, debug=True)
    assert ctx.lib.mv_debug_build() == 1 and B.load().mv_debug_build() == 0
    return ctx


@pytest.mark.parametrize("name", ["c1", "c1_ties"])
def test_checked_build_reports_nothing_on_valid_input(name):
    """The checked build (device-side bounds checks that set status bits) runs the tiny configuration,
    with and without ties, to the oracle's results and with an empty status word."""
    w = WL.resnet_like(name)
    ctx = _debug_context(w.N, w.d, w.K)
    grads, err = WL.gradients(w, 0).to(DEV), WL.initial_err(w).to(DEV)
    PT.compare_all(ctx, grads, err, w.K, label=f"[checked {name}] ")
    assert ctx.debug_status() == 0
    assert ctx.debug_status() == 0             # reading clears; still nothing
    # the normal build answers 0 whatever happened
    plain = B.MvContext(w.N, w.d, w.K, device=DEV)
    PT.run_step(plain, grads, err, w.K)
    assert plain.debug_status() == 0


def test_checked_build_reports_the_fallback_and_the_overflow():
    """Valid inputs that take the slow but exact routes: a jump of scale under threshold tracking (the
    carried threshold admits every element: candidate overflow, then the full-row select) and a row of
    equal magnitudes.  The results are the oracle's; the status word names the detours and nothing else."""
    N, d, K = 3, 300_007, 3000
    ctx = _debug_context(N, d, K, mode=B.MV_MODE_TRACK)
    grads, err = make(N, d, "gauss", seed=77)
    seen = []
    for step, sc in enumerate([1.0, 1.0, 1e3, 1e3]):
        g, e = (grads * sc).roll(step, dims=1).contiguous(), (err * sc).contiguous()
        ref = O.mv_sparse_step(g.numpy(), e.numpy(), K)
        fu = PT.run_step(ctx, g.to(DEV), e.to(DEV), K)
        PT.first_diff(PT.npy(fu["out_idx"]), ref["out_idx"], f"step {step} out_idx")
        PT.first_diff(PT.bits(PT.npy(fu["err"])), PT.bits(ref["err"]), f"step {step} err")
        seen.append(ctx.debug_status())
    assert seen[0] == 0 and seen[1] == 0 and seen[3] == 0
    assert seen[2] == B.MV_DBG_CAND_OVERFLOW | B.MV_DBG_FALLBACK
    # equal magnitudes: every element is a candidate of the sampled threshold
    g2, e2 = make(N, d, "equal", seed=1)
    ctx.set_mode(B.MV_MODE_AUTO)
    PT.compare_all(ctx, g2.to(DEV), e2.to(DEV), K, label="[checked equal] ")
    assert ctx.debug_status() == B.MV_DBG_CAND_OVERFLOW | B.MV_DBG_FALLBACK
    # an index list that is not one: mv_aggregate refuses the entries outside [0, d) and says so
    idx = torch.tensor([5, -1, d, 7], dtype=torch.int32, device=DEV)
    val = torch.full((4,), float("nan"), device=DEV)
    acc = g2.to(DEV).clone()
    ctx.mv_aggregate(acc, idx, val)
    torch.cuda.synchronize()
    assert ctx.debug_status() == B.MV_DBG_GATHER_RANGE
    assert val.cpu().tolist()[1:3] == [0.0, 0.0]


@pytest.mark.parametrize("tail", [2, 0], ids=["single-kernel", "sequence"])
def test_both_tails_through_fallbacks_and_tracking(tail):
    """Whole steps with either implementation of the part after the streaming pass, over a run that visits the
    rare routes: a tracked threshold that misses after a jump of scale (full-row select), rows with heavy ties
    (threshold ties kept in part), equal rows, and ordinary steps in between; residual carried, every step
    compared with the oracle."""
    N, d, K = 5, 260_003, 2600
    ctx = B.MvContext(N, d, K, device=DEV, mode=B.MV_MODE_TRACK)
    ctx.set_tail_kernel(tail)
    g = torch.Generator().manual_seed(777)
    err_gpu = torch.zeros(N, d, device=DEV)
    err_ref = np.zeros((N, d), dtype=np.float32)
    out_idx = torch.empty(K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(K, dtype=torch.float32, device=DEV)
    fell = []
    for step, kind in enumerate(["gauss", "gauss", "big", "big", "ties", "ties", "gauss", "equal", "gauss", "gauss"]):
        grads = torch.randn(N, d, generator=g)
        if kind == "big":
            grads[1:] *= 1e3
        elif kind == "ties":
            grads = (grads * 8).round() / 8
        elif kind == "equal":
            grads[2] = 0.5
        ref = O.mv_sparse_step(grads.numpy(), err_ref, K)
        ctx.mv_sparse_step(grads.to(DEV), err_gpu, out_idx, out_val)
        torch.cuda.synchronize()
        fell.append(int(ctx.read_diag(N)[:, 2].sum()))
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], f"step {step} ({kind}) out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), f"step {step} out_val")
        PT.first_diff(PT.bits(PT.npy(err_gpu)), PT.bits(ref["err"]), f"step {step} ({kind}) err")
        err_ref = ref["err"]
    assert fell[0] == 0 and fell[2] >= 1, fell          # the jump of scale sends workers over their full rows
    assert ctx.last_launches() == (2 if tail == 2 else 6)


@pytest.mark.parametrize("mode", [B.MV_MODE_AUTO, B.MV_MODE_TRACK], ids=["auto", "track"])
def test_single_kernel_step_for_rows_that_fit_a_cta(mode):
    """d <= 32768: the whole step is one kernel (a CTA per worker, exact select in shared memory, two vote arrays
    that alternate).  Several steps with the residual carried, ties, K changing on the same context, another entry
    point in between (which uses the vote array), and the sequence of kernels forced for comparison."""
    N, d = 7, 20_011
    g = torch.Generator().manual_seed(2024)
    ctx = B.MvContext(N, d, 2000, device=DEV, mode=mode)
    err_gpu = torch.zeros(N, d, device=DEV)
    err_ref = np.zeros((N, d), dtype=np.float32)
    for step, (K, kind) in enumerate([(200, "g"), (200, "g"), (200, "ties"), (2000, "g"), (200, "g"), (1, "g"), (200, "votes"),
                                      (200, "g"), (200, "seq"), (200, "g")]):
        grads = torch.randn(N, d, generator=g)
        if kind == "ties":
            grads = (grads * 2).round() / 2
        if kind == "votes":      # the phases in between: mv_vote counts into the workspace's vote array
            acc2 = torch.zeros(N, d, device=DEV)
            ctx.mv_vote(torch.randn(N, d, generator=g).to(DEV), acc2, K=300)
        ctx.set_tail_kernel(0 if kind == "seq" else 1)
        ref = O.mv_sparse_step(grads.numpy(), err_ref, K)
        out_idx = torch.full((K,), -7, dtype=torch.int32, device=DEV)
        out_val = torch.full((K,), float("nan"), dtype=torch.float32, device=DEV)
        ctx.mv_sparse_step(grads.to(DEV), err_gpu, out_idx, out_val, K=K)
        torch.cuda.synchronize()
        assert ctx.last_launches() == (1 if kind != "seq" else ctx.last_launches())
        if kind != "seq":
            assert ctx.last_launches() == 1
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], f"step {step} ({kind}, K={K}) out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), f"step {step} out_val")
        PT.first_diff(PT.bits(PT.npy(err_gpu)), PT.bits(ref["err"]), f"step {step} ({kind}) err")
        err_ref = ref["err"]


@pytest.mark.parametrize("mode", [B.MV_MODE_AUTO, B.MV_MODE_TRACK], ids=["auto", "track"])
def test_single_kernel_step_routes_to_the_kth_key(mode):
    """The one-kernel step finds T_n from a lower bound (carried or sampled) and falls back to three radix digits.
    Steps that take each route, on one context, against the oracle: a carried bound that suddenly lies far above every
    key (residual reset, gradients 1e-4 times smaller), one far below (1e3 times larger), a row of a few distinct
    magnitudes (the bin of rank K is too crowded to rank: radix digits), all-equal magnitudes, and a selection of
    another size in between, whose scratch lands where the kernel keeps its alternating state."""
    N, d, K = 5, 30_001, 300
    g = torch.Generator().manual_seed(77)
    ctx = B.MvContext(N, d, K, device=DEV, mode=mode)
    err_gpu = torch.zeros(N, d, device=DEV)
    err_ref = np.zeros((N, d), dtype=np.float32)
    plan = [("gauss", 1.0, False), ("gauss", 1.0, False), ("gauss", 1e-4, True), ("gauss", 1.0, False), ("gauss", 1e3, False),
            ("coarse", 1.0, True), ("gauss", 1.0, False), ("equal", 1.0, True), ("other", 1.0, False), ("gauss", 1.0, False),
            ("gauss", 1.0, False)]
    for step, (kind, scale, reset) in enumerate(plan):
        grads = torch.randn(N, d, generator=g) * scale
        if kind == "coarse":
            grads = (grads * 2).round() / 2
        if kind == "equal":
            grads = torch.full((N, d), 0.75)
            grads[:, ::3] *= -1
        if reset:
            err_gpu.zero_()
            err_ref[:] = 0
        if kind == "other":      # mv_select for another problem size on the same context
            d2, K2 = 25_000, 100
            votes2 = torch.randint(0, N + 1, (d2,), generator=g).to(torch.uint8).to(DEV)
            oi2 = torch.empty(K2, dtype=torch.int32, device=DEV)
            ctx.mv_select(votes2, N, oi2, K=K2)
            torch.cuda.synchronize()
            assert np.array_equal(oi2.cpu().numpy(), O.select_mask(votes2.cpu().numpy(), K2)[0])
        ref = O.mv_sparse_step(grads.numpy(), err_ref, K)
        out_idx = torch.full((K,), -7, dtype=torch.int32, device=DEV)
        out_val = torch.full((K,), float("nan"), dtype=torch.float32, device=DEV)
        ctx.mv_sparse_step(grads.to(DEV), err_gpu, out_idx, out_val, K=K)
        torch.cuda.synchronize()
        assert ctx.last_launches() == 1
        PT.first_diff(PT.npy(out_idx), ref["out_idx"], f"step {step} ({kind} x{scale}) out_idx")
        PT.check_out_val(PT.npy(out_val), ref, ref["acc"], ref["out_idx"].astype(np.int64), f"step {step} out_val")
        PT.first_diff(PT.bits(PT.npy(err_gpu)), PT.bits(ref["err"]), f"step {step} ({kind}) err")
        err_ref = ref["err"]


@pytest.mark.parametrize("N,d,K", [(4, 10_000, 100), (5, 300_007, 3000)], ids=["one-kernel step", "single-kernel tail"])
def test_a_wait_that_was_given_up_is_reported(N, d, K):
    """The two persistent kernels bound their grid-barrier waits; a CTA that gives up sets a sticky word in the
    workspace header, every CTA that sees it leaves at its next barrier, and the calls that wait for the stream
    return MV_ERR_TIMEOUT.  Here the word is set by the host before the launch (no wait actually runs out): the
    kernel leaves at its first barrier, the status comes back through the ABI, and the CUDA context stays usable
    (a fresh context on the same stream gives the oracle's result afterwards)."""
    grads, err = make(N, d, "gauss", seed=5)
    ctx = B.MvContext(N, d, K, device=DEV)
    ctx.set_tail_kernel(2)
    out_idx = torch.empty(K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(K, dtype=torch.float32, device=DEV)
    e = err.to(DEV)
    ctx.mv_sparse_step(grads.to(DEV), e, out_idx, out_val)       # (the first call clears the header)
    torch.cuda.synchronize()
    assert ctx.fallback_count() >= 0
    ctx.workspace[8:12] = torch.tensor([1, 0, 0, 0], dtype=torch.uint8, device=DEV)   # header word 2: "a wait gave up"
    ctx.mv_sparse_step(grads.to(DEV), e, out_idx, out_val)
    with pytest.raises(B.MvError) as ei:
        ctx.read_diag(N)
    assert ei.value.status == B.MV_ERR_TIMEOUT
    assert "wait" in B.status_string(B.MV_ERR_TIMEOUT).lower()
    torch.cuda.synchronize()
    ctx.close()
    ctx2 = B.MvContext(N, d, K, device=DEV)
    PT.compare_all(ctx2, grads.to(DEV), err.to(DEV), K, label="[after a reported timeout] ")


@pytest.mark.parametrize("d,K", [(3001, 30), (50_021, 500)], ids=["one-kernel step", "single-kernel tail"])
def test_one_cta_per_worker_at_the_device_limit(d, K):
    """As many workers as the device has multiprocessors: the largest cooperative grid of the one-kernel step (a
    CTA per worker) and, for the longer row, the single-kernel tail with a single CTA serving each worker; one
    worker more and the step takes the kernel sequence.  All against the oracle."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for N in (sms, min(sms + 1, 255)):
        grads, err = make(N, d, "gauss", seed=N + d)
        ctx = B.MvContext(N, d, K, device=DEV, mode=B.MV_MODE_TRACK)
        ref = O.mv_sparse_step(grads.numpy(), err.numpy(), K, threads=8)
        PT.compare_all(ctx, grads.to(DEV), err.to(DEV), K, ref=ref, label=f"[N={N} d={d}] ")
        ctx.set_tail_kernel(2)
        fu = PT.run_step(ctx, grads.to(DEV), err.to(DEV), K)
        few = 1 if d <= 32768 else 2
        assert (fu["launches"] <= few + 1) == (N <= sms), (N, fu["launches"])
