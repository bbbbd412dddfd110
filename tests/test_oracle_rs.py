"""Pins for the random-selection oracle: the generator against its published known-answer vectors,
the hand-rolled logarithm against the library one, and the one-number-per-coordinate selection
against the distribution that the paper's sequential procedure defines (exact by enumeration on a
tiny case, and against that procedure run as written)."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import rs_oracle as R


def test_philox_known_answers():
    """Known-answer vectors of Philox4x32-10 from the Random123 distribution (Salmon et al., SC'11)."""
    kat = [
        ((0, 0, 0, 0), (0, 0), (0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8)),
        ((0xFFFFFFFF,) * 4, (0xFFFFFFFF,) * 2, (0x408F276D, 0x41C83B0E, 0xA20BC7C6, 0x6D5451FD)),
        ((0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344), (0xA4093822, 0x299F31D0),
         (0xD16CFE09, 0x94FDCCEB, 0x5001E420, 0x24126EA1)),
    ]
    for ctr, key, want in kat:
        got = R.philox4x32_10(*[np.array([c]) for c in ctr], *key)
        assert tuple(int(g[0]) for g in got) == want


def test_philox_is_a_bijection_on_a_small_slice_and_vectorises():
    j = np.arange(5000)
    x = R.philox4x32_10(j, 0, 7, 0, 123, 456)
    one = R.philox4x32_10(np.array([4321]), 0, 7, 0, 123, 456)
    assert all(int(a[4321]) == int(b[0]) for a, b in zip(x, one))
    assert len({tuple(int(w[i]) for w in x) for i in range(5000)}) == 5000


def test_neg_log_against_the_library_logarithm():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.integers(0, 1 << 32, size=200_000, dtype=np.uint64).astype(np.uint32),
                        np.array([0, 1, 2, 3, (1 << 31) - 1, 1 << 31, (1 << 32) - 2, (1 << 32) - 1], dtype=np.uint32),
                        (np.uint64(1) << np.arange(32, dtype=np.uint64)).astype(np.uint32)])
    got = R.neg_log_u(x)
    want = np.array([-math.log((int(v) + 0.5) / 4294967296.0) for v in x[-300:]])
    np.testing.assert_allclose(got[-300:], want, rtol=0, atol=2e-14)
    u = (x.astype(np.float64) + 0.5) / 4294967296.0
    np.testing.assert_allclose(got, -np.log(u), rtol=0, atol=2e-14)
    assert got.min() > 0 and got.max() < 33 * R.LN2 + 1e-9           # u in (0, 1): E in (0, 33 ln 2)


def successive_sampling_probabilities(votes, K):
    """Exact probability of every K-subset under 'draw proportionally to votes, discard repeats'."""
    w = [Fraction(int(v)) for v in votes]
    items = [i for i, v in enumerate(votes) if v > 0]
    prob = {}
    for perm in itertools.permutations(items, K):
        p, rest = Fraction(1), sum(w)
        for i in perm:
            p *= w[i] / rest
            rest -= w[i]
        key = tuple(sorted(perm))
        prob[key] = prob.get(key, Fraction(0)) + p
    return prob


def test_selection_follows_the_papers_distribution():
    votes = np.array([3, 1, 0, 2, 1, 0, 4], dtype=np.uint8)
    K, draws = 2, 40_000
    exact = successive_sampling_probabilities(votes, K)
    assert sum(exact.values()) == 1
    count = {k: 0 for k in exact}
    for t in range(draws):
        sel = tuple(int(i) for i in R.select_mask_rs(votes, K, seed=2011, draw=t))
        count[sel] += 1                                   # a subset with an unvoted coordinate would raise KeyError
    for k, p in exact.items():
        p = float(p)
        sigma = math.sqrt(draws * p * (1 - p))
        assert abs(count[k] - draws * p) < 4.5 * sigma, (k, count[k], draws * p)
    # the procedure as the paper words it, run as written, lands on the same frequencies
    rng = np.random.default_rng(5)
    seq = {k: 0 for k in exact}
    for _ in range(10_000):
        seq[tuple(int(i) for i in R.select_sequential(votes, K, rng))] += 1
    for k, p in exact.items():
        p = float(p)
        assert abs(seq[k] - 10_000 * p) < 4.5 * math.sqrt(10_000 * p * (1 - p))


def test_selection_invariants():
    rng = np.random.default_rng(3)
    d, K = 5000, 300
    votes = rng.binomial(6, 0.05, size=d).astype(np.uint8)
    a = R.select_mask_rs(votes, K, seed=9, draw=0)
    assert a.shape == (K,) and np.all(np.diff(a) > 0) and np.all(votes[a] > 0)
    assert np.array_equal(a, R.select_mask_rs(votes, K, seed=9, draw=0))
    assert not np.array_equal(a, R.select_mask_rs(votes, K, seed=9, draw=1))
    assert not np.array_equal(a, R.select_mask_rs(votes, K, seed=10, draw=0))
    # as many voted coordinates as K, or fewer: all of them, whatever the draw
    voted = np.flatnonzero(votes > 0)
    assert np.array_equal(R.select_mask_rs(votes, voted.size, 1, 2), voted)
    assert np.array_equal(R.select_mask_rs(votes, voted.size + 50, 1, 2), voted)
    # more votes, more often selected
    freq = np.zeros(7)
    tot = np.zeros(7)
    for t in range(200):
        m = np.zeros(d, bool)
        m[R.select_mask_rs(votes, K, 77, t)] = True
        for v in range(1, 7):
            freq[v] += m[votes == v].sum()
            tot[v] += (votes == v).sum()
    rate = freq[1:4] / tot[1:4]
    assert rate[0] < rate[1] < rate[2]


def test_ties_in_ring_time_go_to_the_lowest_index():
    """binary32 ring times collide now and then; the stable order then decides."""
    votes = np.ones(200_000, dtype=np.uint8)
    t = R.ring_times(votes, 1, 1)
    srt = np.sort(t)
    dup = srt[1:][srt[1:] == srt[:-1]]
    assert dup.size > 0                                   # collisions do occur at this size
    v = dup[0]
    tied = np.flatnonzero(t == v)
    K = int((t < v).sum()) + 1                            # room for exactly one of the tied coordinates
    sel = R.select_mask_rs(votes, K, 1, 1)
    assert tied[0] in sel and tied[1] not in sel


def test_rs_step_keeps_the_error_feedback_identity():
    rng = np.random.default_rng(8)
    N, d, K = 4, 3000, 60
    grads = rng.standard_normal((N, d)).astype(np.float32)
    err = (0.3 * rng.standard_normal((N, d))).astype(np.float32)
    r = R.mv_rs_step(grads, err, K, seed=5, draw=3)
    assert np.all(r["votes"][r["out_idx"]] > 0) and r["out_idx"].shape == (K,)
    sent = np.zeros_like(r["acc"])
    sent[:, r["out_idx"]] = r["acc"][:, r["out_idx"]]
    assert np.array_equal((r["err"] + sent).view(np.uint32) & 0x7FFFFFFF, r["acc"].view(np.uint32) & 0x7FFFFFFF)
    np.testing.assert_allclose(r["out_val"], r["acc"][:, r["out_idx"]].astype(np.float64).mean(axis=0), rtol=1e-6)
