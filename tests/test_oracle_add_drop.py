"""Pins for the add-drop part of the CPU oracle (Algorithm 2): a hand-worked fixture, a pure-Python
brute force, the update rule of Eq. 16, set invariants, and the special case K_ad >= K in which the
scheme reduces to plain majority voting whatever the previous votes were."""
import json
import os

import numpy as np
import pytest

from oracle import mv_oracle as O
from tests.test_oracle_pins import brute_key, brute_stop, f32_bits

HERE = os.path.dirname(__file__)


def masks_from_lists(lists, d):
    m = np.zeros((len(lists), d), dtype=bool)
    for n, l in enumerate(lists):
        m[n, l] = True
    return m


def test_golden_add_drop():
    g = json.load(open(os.path.join(HERE, "golden", "add_drop_n2_d8_k3.json")))
    grads = np.array(g["grads"], dtype=np.float32)
    err = np.array(g["err"], dtype=np.float32)
    prev = masks_from_lists(g["prev"], g["d"])
    r = O.mv_ad_step(grads, err, prev, g["K"], g["K_ad"])
    assert r["worker_idx"].tolist() == g["worker_idx"]
    assert [a.tolist() for a in r["add"]] == g["add"]
    assert [a.tolist() for a in r["drop"]] == g["drop"]
    assert np.array_equal(r["prev"], masks_from_lists(g["prev_new"], g["d"]))
    assert r["msum"].tolist() == g["msum"]
    assert r["out_idx"].tolist() == g["out_idx"]
    assert list(r["vote_thresh"]) == g["vote_thresh"]
    assert np.array_equal(f32_bits(r["out_val"]), f32_bits(np.array(g["out_val"], dtype=np.float32)))
    assert np.array_equal(f32_bits(r["err"]), f32_bits(np.array(g["err_new"], dtype=np.float32)))


@pytest.mark.parametrize("seed", range(8))
def test_add_drop_brute_force(seed):
    rng = np.random.default_rng(300 + seed)
    d = int(rng.integers(6, 60))
    K = int(rng.integers(1, d))
    K_ad = int(rng.integers(1, K + 2))
    acc = rng.choice(np.array([-2, -1, -0.5, 0, 0.5, 1, 2, 3], dtype=np.float32), size=d)   # many ties
    prev = np.zeros(d, dtype=bool)
    prev[rng.choice(d, size=int(rng.integers(0, K + 1)), replace=False)] = True
    top, add, drop, new = O.ad_vote_row(acc, prev, K, K_ad)
    keys = brute_key(acc)
    cur = set(brute_stop(keys, K))
    assert top.tolist() == sorted(cur)
    a_set = sorted(j for j in cur if not prev[j])
    d_set = sorted(j for j in range(d) if prev[j] and j not in cur)
    want_add = sorted(sorted(a_set, key=lambda j: (-keys[j], j))[:K_ad])
    want_drop = sorted(sorted(d_set, key=lambda j: (keys[j], j))[:K_ad])
    assert add.tolist() == want_add and drop.tolist() == want_drop
    want_new = (set(np.flatnonzero(prev).tolist()) | set(want_add)) - set(want_drop)
    assert sorted(np.flatnonzero(new).tolist()) == sorted(want_new)


@pytest.mark.parametrize("seed", range(5))
def test_invariants_over_steps(seed):
    rng = np.random.default_rng(400 + seed)
    N, d = int(rng.integers(2, 7)), int(rng.integers(50, 600))
    K = int(rng.integers(2, d // 3))
    K_ad = max(1, K // int(rng.integers(2, 9)))
    prev = np.zeros((N, d), dtype=bool)
    err = np.zeros((N, d), dtype=np.float32)
    base = rng.standard_normal((1, d))
    msum = prev.sum(axis=0).astype(np.int64)
    for step in range(6):
        grads = (0.7 * base + 0.7 * rng.standard_normal((N, d))).astype(np.float32)
        r = O.mv_ad_step(grads, err, prev, K, K_ad)
        key = O.magnitude_key(r["acc"])
        for n in range(N):
            cur = np.zeros(d, bool)
            cur[r["worker_idx"][n]] = True
            A, D = cur & ~prev[n], prev[n] & ~cur
            add, drop = r["add"][n], r["drop"][n]
            assert A[add].all() and D[drop].all()
            assert len(add) == min(K_ad, A.sum()) and len(drop) == min(K_ad, D.sum())
            rest_a = A.copy()
            rest_a[add] = False
            if len(add) and rest_a.any():
                assert key[n][add].min() >= key[n][rest_a].max()
            rest_d = D.copy()
            rest_d[drop] = False
            if len(drop) and rest_d.any():
                assert key[n][drop].max() <= key[n][rest_d].min()
            assert r["prev"][n].sum() == prev[n].sum() + len(add) - len(drop) <= K
            # Eq. 16: the server's running sum moves by the adds and the drops
            msum[add] += 1
            msum[drop] -= 1
        assert np.array_equal(msum, r["msum"].astype(np.int64))
        inm = np.zeros(d, bool)
        inm[r["out_idx"]] = True
        assert inm.sum() == K and r["msum"][inm].min() >= r["msum"][~inm].max()
        prev, err = r["prev"], r["err"]


def test_large_K_ad_is_plain_majority_voting():
    """K_ad >= K: every worker's vote becomes its current top-K, whatever it voted before."""
    rng = np.random.default_rng(9)
    N, d, K = 5, 400, 30
    grads = rng.standard_normal((N, d)).astype(np.float32)
    err = (0.2 * rng.standard_normal((N, d))).astype(np.float32)
    prev = rng.random((N, d)) < 0.05
    for n in range(N):                       # at most K previous votes per worker
        on = np.flatnonzero(prev[n])
        prev[n, on[K:]] = False
    a = O.mv_ad_step(grads, err, prev, K, K_ad=K)
    b = O.mv_sparse_step(grads, err, K)
    assert np.array_equal(a["msum"], b["votes"])
    assert np.array_equal(a["out_idx"], b["out_idx"])
    assert np.array_equal(f32_bits(a["out_val"]), f32_bits(b["out_val"]))
    assert np.array_equal(f32_bits(a["err"]), f32_bits(b["err"]))
    for n in range(N):
        assert np.array_equal(np.flatnonzero(a["prev"][n]), b["worker_idx"][n])
