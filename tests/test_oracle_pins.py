"""Pins for the CPU oracle: things fixed by the paper's definitions and by plain
mathematics, none of which is computed by the oracle itself.

  * hand-worked fixtures under tests/golden/ (forced ties, error feedback, signed zero);
  * a pure-Python brute force (full sort with the (key desc, index asc) order);
  * special cases that reduce to library routines (torch.topk, a dense mean);
  * invariants (|mask| = K, vote ordering, residual + transmitted = acc, Eq. 8 linearity).
"""
import glob
import json
import os
import struct

import numpy as np
import pytest
import torch

from oracle import mv_oracle as O

GOLDEN = sorted(p for p in glob.glob(os.path.join(os.path.dirname(__file__), "golden", "*.json"))
                if not os.path.basename(p).startswith(("add_drop", "topk_union")))   # (those have tests of their own)


def f32_bits(x):
    return np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)


# ---------------------------------------------------------------- hand-worked fixtures
@pytest.mark.parametrize("path", GOLDEN, ids=[os.path.basename(p) for p in GOLDEN])
@pytest.mark.parametrize("by_sort", [False, True])
def test_golden(path, by_sort):
    g = json.load(open(path))
    grads = np.array(g["grads"], dtype=np.float32)
    err = np.array(g["err"], dtype=np.float32)
    r = O.mv_sparse_step(grads, err, g["K"], by_sort=by_sort)
    assert np.array_equal(f32_bits(r["acc"]), f32_bits(np.array(g["acc"], dtype=np.float32)))
    assert r["worker_idx"].tolist() == g["worker_idx"]
    tkey = [struct.unpack("<I", struct.pack("<f", abs(v)))[0] for v in g["thresh_value"]]
    assert r["thresh"][:, 0].tolist() == tkey
    assert r["thresh"][:, 1].tolist() == g["thresh_cnt_gt"]
    assert r["thresh"][:, 2].tolist() == g["thresh_cnt_eq"]
    assert r["votes"].tolist() == g["votes"]
    assert r["out_idx"].tolist() == g["out_idx"]
    assert list(r["vote_thresh"]) == g["vote_thresh"]
    want = np.array([np.float32(np.float64(a) / np.float64(g["out_val_den"])) for a in g["out_val_num"]],
                    dtype=np.float32)
    assert np.array_equal(f32_bits(r["out_val"]), f32_bits(want))
    assert np.array_equal(f32_bits(r["err"]), f32_bits(np.array(g["err_new"], dtype=np.float32)))
    # bit masks agree with the lists
    for n in range(g["N"]):
        bits = r["worker_bits"][n]
        got = [j for j in range(g["d"]) if (int(bits[j // 32]) >> (j % 32)) & 1]
        assert got == g["worker_idx"][n]


# ---------------------------------------------------------------- brute force
def brute_stop(score, K):
    """First K of the strict total order (score descending, index ascending)."""
    order = sorted(range(len(score)), key=lambda j: (-int(score[j]), j))
    return sorted(order[:K])


def brute_key(x):
    return [struct.unpack("<I", struct.pack("<f", float(v)))[0] & 0x7FFFFFFF for v in x]


@pytest.mark.parametrize("seed", range(6))
def test_topk_brute_force_all_K(seed):
    rng = np.random.default_rng(seed)
    d = int(rng.integers(1, 40))
    # few distinct magnitudes => many ties, both signs
    vals = rng.choice(np.array([-2.5, -1.0, -0.0, 0.0, 0.5, 1.0, 2.5, 1e-40, -1e-40], dtype=np.float32), size=d)
    keys = brute_key(vals)
    for K in range(1, d + 1):
        want = brute_stop(keys, K)
        for fn in (O.worker_topk, O.worker_topk_by_sort):
            idx, T, cnt_gt, cnt_eq = fn(vals, K)
            assert idx.tolist() == want
            kth = sorted(keys, reverse=True)[K - 1]
            assert T == kth
            assert cnt_gt == sum(k > kth for k in keys)
            assert cnt_eq == sum(k == kth for k in keys)


@pytest.mark.parametrize("seed", range(6))
def test_vote_select_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    d = int(rng.integers(1, 50))
    N = int(rng.integers(1, 7))
    votes = rng.integers(0, N + 1, size=d).astype(np.uint8)
    for K in range(1, d + 1):
        want = brute_stop(votes, K)
        assert O.select_mask(votes, K)[0].tolist() == want
        assert O.select_mask_by_sort(votes, K)[0].tolist() == want


def test_count_votes_by_definition():
    rng = np.random.default_rng(7)
    d, N, K = 37, 5, 9
    lists = [np.sort(rng.choice(d, size=K, replace=False)).astype(np.int32) for _ in range(N)]
    votes = O.count_votes(lists, d)
    for j in range(d):
        assert votes[j] == sum(int(j in set(l.tolist())) for l in lists)
    assert int(votes.sum()) == N * K


def test_full_step_brute_force_python():
    """Whole step recomputed with Python scalars on a small tied input."""
    rng = np.random.default_rng(11)
    N, d, K = 4, 29, 6
    grads = (np.round(rng.standard_normal((N, d)) * 2) / 2).astype(np.float32)
    err = (np.round(rng.standard_normal((N, d))) / 4).astype(np.float32)
    r = O.mv_sparse_step(grads, err, K)
    acc = [[float(np.float32(np.float32(err[n, j]) + np.float32(grads[n, j]))) for j in range(d)] for n in range(N)]
    lists = [brute_stop(brute_key(acc[n]), K) for n in range(N)]
    votes = [sum(j in l for l in lists) for j in range(d)]
    mask = brute_stop(votes, K)
    assert r["worker_idx"].tolist() == lists
    assert r["votes"].tolist() == votes
    assert r["out_idx"].tolist() == mask
    for k, j in enumerate(mask):
        s = 0.0
        for n in range(N):
            s += acc[n][j]                       # Python floats are binary64
        assert float(r["out_val"][k]) == float(np.float32(s / N))
    for n in range(N):
        for j in range(d):
            want = 0.0 if j in mask else acc[n][j]
            assert f32_bits(r["err"][n, j]) == f32_bits(np.float32(want))


# ---------------------------------------------------------------- mid-size: selection routine == definition
@pytest.mark.parametrize("ties", [False, True])
def test_partition_variant_equals_sort_variant(ties):
    rng = np.random.default_rng(3)
    N, d, K = 5, 20011, 517
    grads = rng.standard_normal((N, d)).astype(np.float32)
    err = (0.1 * rng.standard_normal((N, d))).astype(np.float32)
    if ties:
        grads = (np.round(grads * 10) / 10).astype(np.float32)
        err = np.zeros_like(err)
    a = O.mv_sparse_step(grads, err, K, by_sort=False)
    b = O.mv_sparse_step(grads, err, K, by_sort=True)
    for k in ("worker_idx", "worker_bits", "votes", "thresh", "out_idx", "mask_bits"):
        assert np.array_equal(a[k], b[k]), k
    assert a["vote_thresh"] == b["vote_thresh"]
    assert np.array_equal(f32_bits(a["out_val"]), f32_bits(b["out_val"]))
    assert np.array_equal(f32_bits(a["err"]), f32_bits(b["err"]))


# ---------------------------------------------------------------- special cases -> library routines
def test_single_worker_is_classic_topk_with_error_feedback():
    """N = 1: the mask is the worker's own top-K (torch.topk on |acc| gives the
    same set when there are no ties), out_val = acc on it, residual zeroed there."""
    d, K = 5003, 250
    for seed in range(5, 50):                      # reseed until no two magnitudes coincide
        g = torch.Generator().manual_seed(seed)
        grads = torch.randn(1, d, generator=g)
        err = 0.3 * torch.randn(1, d, generator=g)
        acc = err + grads
        if torch.unique(acc.abs()).numel() == d:
            break
    assert torch.unique(acc.abs()).numel() == d
    want = torch.topk(acc[0].abs(), K).indices.sort().values.numpy()
    r = O.mv_sparse_step(grads.numpy(), err.numpy(), K)
    assert np.array_equal(r["worker_idx"][0], want)
    assert np.array_equal(r["out_idx"], want)
    assert np.array_equal(f32_bits(r["out_val"]), f32_bits(acc[0, want].numpy()))
    keep = np.ones(d, bool)
    keep[want] = False
    assert np.all(r["err"][0, want] == 0) and np.array_equal(r["err"][0, keep], acc[0].numpy()[keep])


def test_K_equals_d_is_the_dense_mean():
    """K = d: every coordinate is selected; out_val is the plain average of Eq. 4."""
    rng = np.random.default_rng(9)
    N, d = 6, 257
    grads = rng.standard_normal((N, d)).astype(np.float32)
    err = rng.standard_normal((N, d)).astype(np.float32)
    r = O.mv_sparse_step(grads, err, d)
    assert r["out_idx"].tolist() == list(range(d))
    assert np.all(r["votes"] == N)
    acc = (err + grads).astype(np.float32)
    dense = acc.astype(np.float64).mean(axis=0)
    np.testing.assert_allclose(r["out_val"].astype(np.float64), dense, rtol=1e-6, atol=1e-7)
    assert not r["err"].any()


def test_identical_workers_vote_unanimously():
    rng = np.random.default_rng(13)
    N, d, K = 7, 1000, 40
    row = rng.standard_normal(d).astype(np.float32)
    grads = np.tile(row, (N, 1))
    r = O.mv_sparse_step(grads, np.zeros_like(grads), K)
    assert set(np.unique(r["votes"]).tolist()) == {0, N}
    assert np.array_equal(r["out_idx"], r["worker_idx"][0])
    assert np.array_equal(f32_bits(r["out_val"]), f32_bits(row[r["out_idx"]]))


def test_all_equal_magnitudes_pick_lowest_indices():
    N, d, K = 3, 100, 17
    grads = np.full((N, d), -0.75, dtype=np.float32)
    grads[1] *= -1
    r = O.mv_sparse_step(grads, np.zeros_like(grads), K)
    for n in range(N):
        assert r["worker_idx"][n].tolist() == list(range(K))
        assert r["thresh"][n].tolist() == [int(f32_bits(np.float32(0.75)).ravel()[0]), 0, d]
    assert r["out_idx"].tolist() == list(range(K))


# ---------------------------------------------------------------- invariants
@pytest.mark.parametrize("seed", range(8))
def test_invariants(seed):
    rng = np.random.default_rng(1000 + seed)
    N = int(rng.integers(1, 12))
    d = int(rng.integers(8, 3000))
    K = int(rng.integers(1, d + 1))
    scale = 10.0 ** rng.uniform(-3, 0, size=(1, d))
    grads = (rng.standard_normal((N, d)) * scale).astype(np.float32)
    if seed % 2:
        grads = (np.round(grads * 8) / 8).astype(np.float32)
    err = (0.5 * rng.standard_normal((N, d)) * scale).astype(np.float32)
    r = O.mv_sparse_step(grads, err, K)
    acc, votes, mask = r["acc"], r["votes"].astype(int), r["out_idx"]
    key = O.magnitude_key(acc)
    for n in range(N):
        idx = r["worker_idx"][n]
        assert len(idx) == K and np.all(np.diff(idx) > 0)
        inside = np.zeros(d, bool)
        inside[idx] = True
        T, cnt_gt, cnt_eq = (int(v) for v in r["thresh"][n])
        if K < d:
            assert key[n][inside].min() >= key[n][~inside].max()
        assert cnt_gt < K <= cnt_gt + cnt_eq
        assert key[n][inside].min() == T
        ties = np.flatnonzero(key[n] == T)
        assert np.array_equal(np.flatnonzero(inside & (key[n] == T)), ties[: K - cnt_gt])
    assert votes.sum() == N * K and votes.max() <= N
    assert len(mask) == K and np.all(np.diff(mask) > 0)
    inm = np.zeros(d, bool)
    inm[mask] = True
    if K < d:
        assert votes[inm].min() >= votes[~inm].max()
    assert votes[inm].min() >= 1                       # a union of K-sets has at least K members
    # residual + transmitted == acc, exactly, per coordinate
    transmitted = np.where(inm[None, :], acc, np.float32(0))
    assert np.array_equal(f32_bits(r["err"] + transmitted), f32_bits(acc + np.float32(0)))
    assert not f32_bits(r["err"][:, inm]).any()
    assert np.array_equal(f32_bits(r["err"][:, ~inm]), f32_bits(acc[:, ~inm]))
    # linearity (Eq. 8): mean of the masked vectors == masked mean
    col_mean = acc.astype(np.float64).mean(axis=0)[mask]
    scale_k = np.abs(acc.astype(np.float64)).mean(axis=0)[mask]
    assert np.all(np.abs(r["out_val"].astype(np.float64) - col_mean) <= 1e-6 * scale_k + 1e-45)


def test_nonfinite_and_denormal_ordering():
    """Order is by the sign-cleared bit pattern: NaN > inf > finite > denormal > zero."""
    nan = np.float32(np.nan)
    x = np.array([1e-45, np.inf, -0.0, 3.0, nan, -np.inf, 1e-39, -3.0], dtype=np.float32)
    idx, T, cnt_gt, cnt_eq = O.worker_topk(x, 4)
    assert idx.tolist() == [1, 3, 4, 5]           # NaN, both infs, then the first |3.0|
    assert (T, cnt_gt, cnt_eq) == (int(f32_bits(np.float32(3.0)).ravel()[0]), 3, 2)
    idx, *_ = O.worker_topk(x, 7)
    assert idx.tolist() == [0, 1, 3, 4, 5, 6, 7]  # only the zero is left out
