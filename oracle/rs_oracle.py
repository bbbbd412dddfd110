"""CPU oracle for majority voting with random selection (SSGD-MV-RS; Algorithm 1, the red line,
and the description in Section 4.1: indices are drawn at random with probabilities proportional to
their votes until K distinct ones have been drawn).

TEST INFRASTRUCTURE ONLY (see mv_oracle.py); numpy, no code shared with the CUDA library.

Two statements of S_rand-weighted live here:

* `select_sequential` is the paper's procedure taken literally: draw an index with probability
  votes_j / sum(votes), keep it if it is new, repeat until K distinct indices are held.  It consumes
  a data-dependent number of random numbers one after the other, so it is the *definition of the
  distribution*, used by the pins, not something a parallel implementation can reproduce draw by draw.

* `select_mask_rs` draws from the same distribution with one random number per coordinate
  (Efraimidis and Spirakis 2006, weighted sampling without replacement by exponential clocks:
  coordinate j rings at time E_j / votes_j with E_j ~ Exp(1); the K earliest ring times are a draw of
  "successive sampling proportional to votes until K distinct").  This is what the CUDA library is
  compared with bit for bit, so everything that decides an index is fixed here:
    - x_j = first output word of Philox4x32-10 (Salmon et al. 2011) with key (seed_lo, seed_hi) and
      counter (j, 0, draw_lo, draw_hi); u_j = (x_j + 1/2) / 2^32;
    - E_j = -ln(u_j) by `neg_log_u`: a fixed sequence of binary64 additions, multiplications and
      divisions (no library logarithm), so that any IEEE-754 machine gets the same bits;
    - t_j = E_j / votes_j in binary64, rounded once to binary32; the K smallest t_j win, equal t_j go
      to the lowest index; coordinates without a vote never ring.
  If fewer than K coordinates hold a vote, all of them are selected and nothing else.
"""
from __future__ import annotations

import numpy as np

M0, M1 = 0xD2511F53, 0xCD9E8D57          # Philox4x32 multipliers
W0, W1 = 0x9E3779B9, 0xBB67AE85          # Weyl key increments
LN2 = 0.6931471805599453
SQRT2 = 1.4142135623730951


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten rounds of Philox4x32 on uint32 arrays (counters) and scalar keys; returns the four output words."""
    c0, c1, c2, c3 = (np.asarray(c, dtype=np.uint64) & 0xFFFFFFFF for c in (c0, c1, c2, c3))
    k0, k1 = int(k0) & 0xFFFFFFFF, int(k1) & 0xFFFFFFFF
    for _ in range(10):
        p0 = np.uint64(M0) * c0                     # 64-bit products of 32-bit operands
        p1 = np.uint64(M1) * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & np.uint64(0xFFFFFFFF)
        hi1, lo1 = p1 >> np.uint64(32), p1 & np.uint64(0xFFFFFFFF)
        c0, c1, c2, c3 = hi1 ^ c1 ^ np.uint64(k0), lo1, hi0 ^ c3 ^ np.uint64(k1), lo0
        k0, k1 = (k0 + W0) & 0xFFFFFFFF, (k1 + W1) & 0xFFFFFFFF
    return tuple(c.astype(np.uint32) for c in (c0, c1, c2, c3))


def neg_log_u(x):
    """-ln((x + 1/2) / 2^32) for uint32 x, from binary64 +, *, / only (see the module text)."""
    v = 2 * np.asarray(x, dtype=np.int64) + 1                          # odd integer below 2^33, exact in binary64
    e = np.floor(np.log2(v.astype(np.float64))).astype(np.int64)       # bit length - 1 ...
    e = np.where((np.int64(1) << e) > v, e - 1, e)                      # ... made exact whatever log2 rounds to
    e = np.where((np.int64(1) << (e + 1)) <= v, e + 1, e)
    m = v.astype(np.float64) / (np.int64(1) << e).astype(np.float64)   # [1, 2), exact
    big = m > SQRT2
    m = np.where(big, m * 0.5, m)
    e = np.where(big, e + 1, e)
    s = (m - 1.0) / (m + 1.0)
    z = s * s
    poly = np.full_like(z, 1.0 / 23.0)
    for k in range(21, 0, -2):                                          # 1/21, 1/19, ..., 1/3, 1
        poly = poly * z + (1.0 / k)
    logm = (2.0 * s) * poly
    return (33 - e).astype(np.float64) * LN2 - logm


def ring_times(votes: np.ndarray, seed: int, draw: int) -> np.ndarray:
    """binary32 ring time of every coordinate (inf where votes == 0)."""
    d = votes.shape[0]
    j = np.arange(d, dtype=np.uint64)
    x, _, _, _ = philox4x32_10(j, 0, draw & 0xFFFFFFFF, (draw >> 32) & 0xFFFFFFFF, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    E = neg_log_u(x)
    with np.errstate(divide="ignore"):
        t = E / votes.astype(np.float64)
    return t.astype(np.float32)


def select_mask_rs(votes: np.ndarray, K: int, seed: int, draw: int) -> np.ndarray:
    """Ascending int32 indices of the K earliest ring times among voted coordinates (ties: lowest index)."""
    t = ring_times(votes, seed, draw)
    voted = np.flatnonzero(votes > 0)
    order = voted[np.argsort(t[voted], kind="stable")]                  # stable: equal times keep index order
    return np.sort(order[:K]).astype(np.int32)


def select_sequential(votes: np.ndarray, K: int, rng: np.random.Generator) -> np.ndarray:
    """The paper's procedure: draw proportionally to the votes, with replacement, until K distinct indices."""
    p = votes.astype(np.float64) / votes.sum()
    K = min(K, int((votes > 0).sum()))
    chosen = set()
    while len(chosen) < K:
        chosen.add(int(rng.choice(votes.shape[0], p=p)))
    return np.array(sorted(chosen), dtype=np.int32)


def mv_rs_step(grads: np.ndarray, err: np.ndarray, K: int, seed: int, draw: int, threads: int = 1):
    """One SSGD-MV-RS step: Algorithm 1 with the red line in place of the blue one."""
    from oracle import mv_oracle as O
    v = O.mv_vote(grads, err, K, threads=threads)
    out_idx = select_mask_rs(v["votes"], K, seed, draw)
    out_val = O.aggregate(v["acc"], out_idx)
    new_err = O.residual(v["acc"], out_idx)
    return dict(acc=v["acc"], votes=v["votes"], worker_idx=v["worker_idx"], out_idx=out_idx, out_val=out_val, err=new_err)
