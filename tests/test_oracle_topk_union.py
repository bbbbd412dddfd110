"""Pins of the oracle's SSGD-top-K step (the paper's comparison scheme: every worker sparsifies with its own
top-K mask, the server averages what it receives; Section 2, Eq. 6-7; Table 1, row SSGD-top-K): a hand-worked
fixture, a dense recomputation from the definition, the special cases N = 1 (classic top-K with error
feedback), identical workers (equal to majority voting) and K = d (the dense mean, Eq. 4), the paper's
downlink figure for disjoint masks, and invariants."""
import json
import os

import numpy as np
import pytest

from oracle import mv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_hand_worked_fixture():
    fx = json.load(open(os.path.join(GOLDEN, "topk_union_n3_d8_k2.json")))
    g, e = np.array(fx["grads"], np.float32), np.array(fx["err"], np.float32)
    for by_sort in (False, True):
        r = O.topk_union_step(g, e, fx["K"], by_sort=by_sort)
        assert r["worker_idx"].tolist() == fx["worker_idx"]
        assert r["votes"].tolist() == fx["votes"]
        assert r["union_idx"].tolist() == fx["union_idx"]
        want = (np.array(fx["union_val_num"], np.float64) / fx["union_val_den"]).astype(np.float32)
        assert np.array_equal(r["union_val"].view(np.uint32), want.view(np.uint32))
        assert np.array_equal(r["err"].view(np.uint32), np.array(fx["err_new"], np.float32).view(np.uint32))


def _dense_definition(grads, err, K):
    """Eq. 6-7 executed densely with Python scalars: full vectors M_n (x) acc_n, summed and divided by N."""
    acc = (grads.astype(np.float32) + err.astype(np.float32)).astype(np.float32)
    N, d = acc.shape
    masks = np.zeros((N, d), bool)
    for n in range(N):
        order = sorted(range(d), key=lambda j: (-(int(acc[n, j].view(np.uint32)) & 0x7fffffff), j))
        masks[n, order[:K]] = True
    dense = [sum(float(acc[n, j]) for n in range(N) if masks[n, j]) / N for j in range(d)]
    return acc, masks, np.array(dense, np.float64)


@pytest.mark.parametrize("N,d,K,seed", [(1, 9, 3, 0), (3, 17, 4, 1), (5, 40, 7, 2), (4, 33, 33, 3), (6, 64, 1, 4)])
def test_against_the_dense_definition(N, d, K, seed):
    rng = np.random.default_rng(seed)
    grads = (rng.standard_normal((N, d)) * 4).round() / 4            # many ties
    err = (rng.standard_normal((N, d))).round() / 2
    grads, err = grads.astype(np.float32), err.astype(np.float32)
    acc, masks, dense = _dense_definition(grads, err, K)
    r = O.topk_union_step(grads, err, K)
    assert np.array_equal(r["union_idx"], np.flatnonzero(masks.any(axis=0)))
    assert np.array_equal(r["union_val"], dense[r["union_idx"]].astype(np.float32))
    assert K <= r["union_idx"].size <= min(d, N * K)
    # the residual: zero on the worker's own mask, acc elsewhere; residual + what was sent = acc exactly
    sent = np.where(masks, acc, np.float32(0))
    assert np.array_equal((r["err"] + sent).view(np.uint32), (acc + np.float32(0)).view(np.uint32))
    assert not r["err"][masks].any()


def test_single_worker_is_classic_topk_with_error_feedback():
    rng = np.random.default_rng(7)
    g = rng.standard_normal((1, 200)).astype(np.float32)
    e = rng.standard_normal((1, 200)).astype(np.float32)
    K = 20
    r = O.topk_union_step(g, e, K)
    acc = g + e
    top = np.sort(np.argsort(-np.abs(acc[0]), kind="stable")[:K])
    assert np.array_equal(r["union_idx"], top)
    assert np.array_equal(r["union_val"], acc[0, top])
    mv = O.mv_sparse_step(g, e, K)                                    # and it is majority voting with one voter
    assert np.array_equal(mv["out_idx"], r["union_idx"]) and np.array_equal(mv["err"], r["err"])


def test_identical_workers_equal_majority_voting():
    rng = np.random.default_rng(8)
    row = rng.standard_normal(300).astype(np.float32)
    g = np.tile(row, (4, 1))
    e = np.zeros_like(g)
    K = 25
    r, mv = O.topk_union_step(g, e, K), O.mv_sparse_step(g, e, K)
    assert np.array_equal(r["union_idx"], mv["out_idx"])
    assert np.array_equal(r["union_val"].view(np.uint32), mv["out_val"].view(np.uint32))
    assert np.array_equal(r["err"].view(np.uint32), mv["err"].view(np.uint32))


def test_K_equal_d_is_the_dense_mean():
    rng = np.random.default_rng(9)
    g = rng.standard_normal((5, 50)).astype(np.float32)
    e = rng.standard_normal((5, 50)).astype(np.float32)
    r = O.topk_union_step(g, e, 50)
    acc = g + e
    assert np.array_equal(r["union_idx"], np.arange(50))
    assert np.array_equal(r["union_val"], (acc.astype(np.float64).sum(axis=0) / 5).astype(np.float32))
    assert not r["err"].any()


def test_disjoint_masks_give_the_downlink_load_of_table_1():
    """Table 1, row SSGD-top-K at phi = 1e-2 with N = 10 workers: 0.32 value bits per parameter on the uplink
    and 3.2 on the downlink, i.e. N times as many non-zeros when the workers' masks do not overlap."""
    N, d, K = 10, 2000, 20                                            # phi = 1e-2
    g = np.zeros((N, d), np.float32)
    for n in range(N):
        g[n, n * K:(n + 1) * K] = 1.0 + n                             # every worker's large entries in a block of its own
    r = O.topk_union_step(g, np.zeros_like(g), K)
    assert r["union_idx"].size == N * K
    assert 32.0 * K / d == pytest.approx(0.32) and 32.0 * r["union_idx"].size / d == pytest.approx(3.2)
    assert np.array_equal(r["union_val"], np.repeat((1.0 + np.arange(N)) / N, K).astype(np.float32))
