"""CPU oracle for the majority-vote sparse DSGD step (SSGD-MV, Algorithm 1).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what one
step computes, written from the paper's definitions with numpy.  It is imported
by the tests, by the smoke check and by the benchmark's CPU-baseline leg, and by
nothing else; it shares no code with the CUDA library and never imports it.

One step, for N workers holding d parameters each (Algorithm 1, worker side and
parameter-server side collapsed onto one machine):

  1. acc_n   = grads_n + err_n                      error feedback (Alg. 1, accumulate step)
  2. M_n     = S_top(|acc_n|, K)                    per-worker top-K mask (Eq. 6 / S_top)
  3. votes   = sum_n M_n                            vote count per coordinate (Eq. 9)
  4. M       = S_top(votes, K)                      the K most voted coordinates (Eq. 9)
  5. out_val = (1/N) sum_n (M (x) acc_n) on supp(M) shared-mask aggregate (Eq. 8; mean as in the text)
  6. err_n   = acc_n - M (x) acc_n                  residual (Alg. 1, error update)

Readings where the paper is silent (each is also listed in the design notes):
  * "largest absolute value" is ordered by key(x) = bits(x) & 0x7fffffff, the
    IEEE-754 binary32 pattern with the sign cleared, which is monotone in |x|.
  * ties in either S_top go to the lowest coordinate index, so the selected set
    is the first K elements of the strict total order (key descending, index
    ascending) and is therefore unique.
  * supports are reported as ascending index lists.
  * the aggregate is the mean (the text's 1/N), accumulated in binary64 in
    worker order, divided by N and rounded once to binary32.
  * the residual is "+0.0 on the mask, a bit copy elsewhere" (equal to the
    subtraction for all finite values).
  * acc is one binary32 round-to-nearest add, denormals kept.

Every selection is written twice: `*_by_sort` is the definition executed with a
full stable sort; the plain name reaches the same unique set with a library
selection routine (numpy.partition) so that full-size inputs finish in seconds.
The tests pin the two against each other, against a pure-Python brute force and
against hand-worked examples.
"""
from __future__ import annotations

import numpy as np

_SIGN_CLEAR = np.uint32(0x7FFFFFFF)


# ----------------------------------------------------------------------------
# step 1: error feedback (Algorithm 1, "Delta-bar = Delta + e")
# ----------------------------------------------------------------------------
def accumulate(grads: np.ndarray, err: np.ndarray) -> np.ndarray:
    """acc[n, j] = fl32(err[n, j] + grads[n, j])."""
    grads = np.asarray(grads, dtype=np.float32)
    err = np.asarray(err, dtype=np.float32)
    assert grads.shape == err.shape
    with np.errstate(all="ignore"):
        return np.add(err, grads, dtype=np.float32)


def magnitude_key(x: np.ndarray) -> np.ndarray:
    """key(x): the binary32 pattern with the sign bit cleared (monotone in |x|)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return x.view(np.uint32) & _SIGN_CLEAR


# ----------------------------------------------------------------------------
# S_top on an integer score vector: the K largest scores, ties to the lowest index
# ----------------------------------------------------------------------------
def _stop_by_sort(score: np.ndarray, K: int):
    """Definition executed: stable sort by descending score, take the first K."""
    score = np.asarray(score)
    d = score.shape[0]
    assert 1 <= K <= d
    # ascending stable sort of (max - score) == descending score, index ascending
    inv = score.max().astype(np.int64) - score.astype(np.int64)
    order = np.argsort(inv, kind="stable")
    chosen = order[:K]
    thr = score[chosen[-1]]
    cnt_gt = int(np.count_nonzero(score > thr))
    cnt_eq = int(np.count_nonzero(score == thr))
    return np.sort(chosen).astype(np.int32), thr, cnt_gt, cnt_eq


def _stop(score: np.ndarray, K: int):
    """Same set via a selection routine: threshold = K-th largest score, then
    everything above it plus the lowest-index (K - cnt_gt) elements equal to it."""
    score = np.asarray(score)
    d = score.shape[0]
    assert 1 <= K <= d
    thr = np.partition(score, d - K)[d - K]          # K-th largest value
    gt = score > thr
    eq = score == thr
    cnt_gt = int(np.count_nonzero(gt))
    cnt_eq = int(np.count_nonzero(eq))
    need = K - cnt_gt
    assert 1 <= need <= cnt_eq
    take = gt
    take[np.flatnonzero(eq)[:need]] = True             # the `need` lowest-index ties
    return np.flatnonzero(take).astype(np.int32), thr, cnt_gt, cnt_eq


# ----------------------------------------------------------------------------
# step 2: per-worker top-K of |acc_n| (S_top, Eq. 6; Algorithm 1 worker side)
# ----------------------------------------------------------------------------
def worker_topk_by_sort(acc_row: np.ndarray, K: int):
    """Returns (ascending int32 indices, threshold key T, cnt_gt, cnt_eq)."""
    idx, thr, cnt_gt, cnt_eq = _stop_by_sort(magnitude_key(acc_row), K)
    return idx, int(thr), cnt_gt, cnt_eq


def worker_topk(acc_row: np.ndarray, K: int):
    idx, thr, cnt_gt, cnt_eq = _stop(magnitude_key(acc_row), K)
    return idx, int(thr), cnt_gt, cnt_eq


def support_to_bits(idx: np.ndarray, d: int) -> np.ndarray:
    """d-bit mask as ceil(d/32) uint32 words; bit b of word w is coordinate 32*w+b."""
    flags = np.zeros(((d + 31) // 32) * 32, dtype=np.uint8)
    flags[np.asarray(idx, dtype=np.int64)] = 1
    return np.packbits(flags, bitorder="little").view(np.uint32).copy()


# ----------------------------------------------------------------------------
# step 3: vote count (Eq. 9, inner sum)
# ----------------------------------------------------------------------------
def count_votes(worker_idx, d: int) -> np.ndarray:
    """votes[j] = number of workers whose top-K support contains j."""
    votes = np.zeros(d, dtype=np.int64)
    for idx in worker_idx:
        votes[np.asarray(idx, dtype=np.int64)] += 1   # indices within one list are distinct
    assert votes.max(initial=0) <= 255
    return votes.astype(np.uint8)


# ----------------------------------------------------------------------------
# step 4: global mask = the K most voted coordinates (Eq. 9, outer S_top)
# ----------------------------------------------------------------------------
def select_mask_by_sort(votes: np.ndarray, K: int):
    idx, thr, cnt_gt, cnt_eq = _stop_by_sort(np.asarray(votes), K)
    return idx, int(thr), cnt_gt, cnt_eq


def select_mask(votes: np.ndarray, K: int):
    idx, thr, cnt_gt, cnt_eq = _stop(np.asarray(votes), K)
    return idx, int(thr), cnt_gt, cnt_eq


# ----------------------------------------------------------------------------
# step 5: aggregate on the shared mask (Eq. 8 with the 1/N of the text)
# ----------------------------------------------------------------------------
def aggregate(acc: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """out_val[k] = fl32( (sum over workers, in worker order, in binary64) / N )."""
    acc = np.asarray(acc, dtype=np.float32)
    N = acc.shape[0]
    cols = np.asarray(idx, dtype=np.int64)
    total = np.zeros(cols.shape[0], dtype=np.float64)
    with np.errstate(all="ignore"):
        for n in range(N):
            total = total + acc[n, cols].astype(np.float64)
        return (total / np.float64(N)).astype(np.float32)


# ----------------------------------------------------------------------------
# step 6: residual (Algorithm 1, "e = Delta-bar - Delta-tilde")
# ----------------------------------------------------------------------------
def residual(acc: np.ndarray, idx: np.ndarray) -> np.ndarray:
    out = np.array(acc, dtype=np.float32, copy=True)
    out[:, np.asarray(idx, dtype=np.int64)] = np.float32(0.0)
    return out


# ----------------------------------------------------------------------------
# the whole step
# ----------------------------------------------------------------------------
def mv_vote(grads, err, K: int, by_sort: bool = False, threads: int = 1):
    """Steps 1-3.  Returns a dict with acc, worker_idx [N,K], worker_bits
    [N,ceil(d/32)], votes [d] and thresh [N,3] = (T_n, cnt_gt, cnt_eq).
    The workers' rows are independent; `threads` > 1 only lets several rows be
    selected at the same time (same functions, same results)."""
    acc = accumulate(grads, err)
    N, d = acc.shape
    topk = worker_topk_by_sort if by_sort else worker_topk
    worker_idx = np.empty((N, K), dtype=np.int32)
    worker_bits = np.empty((N, (d + 31) // 32), dtype=np.uint32)
    thresh = np.empty((N, 3), dtype=np.uint32)

    def one_row(n):
        idx, T, cnt_gt, cnt_eq = topk(acc[n], K)
        worker_idx[n] = idx
        worker_bits[n] = support_to_bits(idx, d)
        thresh[n] = (T, cnt_gt, cnt_eq)

    if threads > 1:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(one_row, range(N)))
    else:
        for n in range(N):
            one_row(n)
    votes = count_votes(worker_idx, d)
    return dict(acc=acc, worker_idx=worker_idx, worker_bits=worker_bits,
                votes=votes, thresh=thresh)


def mv_sparse_step(grads, err, K: int, by_sort: bool = False, threads: int = 1):
    """One full step.  Returns a dict with everything the step defines:
    acc, worker_idx, worker_bits, votes, thresh, out_idx [K], mask_bits,
    vote_thresh = (v*, cnt_gt, cnt_eq), out_val [K] and the new err [N,d]."""
    r = mv_vote(grads, err, K, by_sort=by_sort, threads=threads)
    sel = select_mask_by_sort if by_sort else select_mask
    out_idx, vstar, vgt, veq = sel(r["votes"], K)
    r["out_idx"] = out_idx
    r["mask_bits"] = support_to_bits(out_idx, r["acc"].shape[1])
    r["vote_thresh"] = (vstar, vgt, veq)
    r["out_val"] = aggregate(r["acc"], out_idx)
    r["err"] = residual(r["acc"], out_idx)
    return r


# ============================================================================
# Majority voting with add-drop (Algorithm 2, MV-AD)
#
# Each worker keeps a vote mask Mt_n (the paper's M-tilde) from the previous
# iteration and changes at most K_ad entries in each direction:
#   M_n     = S_top(|acc_n|, K)                                   as before
#   add_n   = the K_ad largest  |acc_n| among  M_n and not Mt_n   (Alg. 2, add line)
#   drop_n  = the K_ad smallest |acc_n| among  Mt_n and not M_n   (Alg. 2, drop line)
#   Mt_n   <- Mt_n + add_n - drop_n
#   M_sum  <- M_sum + sum_n (add_n - drop_n)                      (Eq. 16)
#   M       = S_top(M_sum, K)
# followed by the same aggregation and residual as Algorithm 1.
#
# Readings (the paper is silent): if fewer than K_ad coordinates are eligible,
# all of them are taken and nothing else (the selections are restricted to the
# eligible set); ties go to the lowest index in both selections; M_sum equals
# the per-coordinate count of the workers' current masks (true by induction when
# it starts that way), so the server state is recomputed as that count; with
# fewer than K voted coordinates the mask is filled up with unvoted coordinates
# in index order, as S_top on the count vector dictates.
# ============================================================================
def masked_select(key: np.ndarray, eligible: np.ndarray, k: int, largest: bool) -> np.ndarray:
    """Ascending indices of the min(k, #eligible) eligible coordinates with the largest (or
    smallest) key, ties to the lowest index: a full stable sort of the eligible set."""
    cand = np.flatnonzero(eligible)
    if cand.size == 0 or k <= 0:
        return np.zeros(0, dtype=np.int32)
    kk = key[cand].astype(np.int64)
    order = np.argsort(-kk if largest else kk, kind="stable")   # stable: equal keys stay in index order
    return np.sort(cand[order[:k]]).astype(np.int32)


def ad_vote_row(acc_row: np.ndarray, prev_row: np.ndarray, K: int, K_ad: int):
    """One worker's add-drop vote.  prev_row: bool[d].  Returns (top-K indices, add indices,
    drop indices, new mask bool[d])."""
    d = acc_row.shape[0]
    key = magnitude_key(acc_row)
    top, _, _, _ = worker_topk(acc_row, K)
    cur = np.zeros(d, dtype=bool)
    cur[top] = True
    add = masked_select(key, cur & ~prev_row, K_ad, largest=True)
    drop = masked_select(key, prev_row & ~cur, K_ad, largest=False)
    new = prev_row.copy()
    new[add] = True
    new[drop] = False
    return top, add, drop, new


def mv_ad_step(grads, err, prev, K: int, K_ad: int):
    """One MV-AD step.  prev: bool[N, d] (the workers' previous vote masks).  Returns a dict with
    acc, worker_idx [N,K], add / drop (lists of index arrays), prev (new masks, bool[N,d]),
    msum (uint8[d]), out_idx [K], vote_thresh, out_val [K], err [N,d]."""
    acc = accumulate(grads, err)
    N, d = acc.shape
    prev = np.asarray(prev, dtype=bool)
    worker_idx = np.empty((N, K), dtype=np.int32)
    adds, drops = [], []
    new_prev = np.empty_like(prev)
    for n in range(N):
        top, add, drop, new = ad_vote_row(acc[n], prev[n], K, K_ad)
        worker_idx[n] = top
        adds.append(add)
        drops.append(drop)
        new_prev[n] = new
    msum = new_prev.sum(axis=0).astype(np.uint8)        # Eq. 16, by induction from M_sum = count of the masks
    out_idx, vstar, vgt, veq = select_mask(msum, K)
    return dict(acc=acc, worker_idx=worker_idx, add=adds, drop=drops, prev=new_prev, msum=msum,
                out_idx=out_idx, vote_thresh=(vstar, vgt, veq), out_val=aggregate(acc, out_idx),
                err=residual(acc, out_idx))


# ============================================================================
# SSGD-top-K (the paper's comparison scheme: Section 2, first paragraph, the
# masked gradient of Eq. 6 and the update of Eq. 7; Table 1, row "SSGD-top-K")
#
# Every worker keeps the K largest |acc_n| under its OWN mask and the server
# averages what it receives:
#   M_n   = S_top(|acc_n|, K)
#   G     = (1/N) sum_n M_n (x) acc_n        non-zero only on the union of the masks
#   err_n = acc_n - M_n (x) acc_n            each worker's residual on its own mask
# The union holds between K and N K coordinates (the masks need not match: this
# is why the scheme's downlink is up to N times heavier than its uplink).
#
# Readings: error accumulation as in Algorithm 1 (the paper runs all schemes
# with it); the union is reported as an ascending index list, defined by the
# masks and not by the values (a coordinate whose kept values cancel stays in
# it); a value is the binary64 sum, in worker order, over the workers that kept
# the coordinate, divided by N (all N workers, as in Eq. 7's 1/N), rounded once
# to binary32; ties in S_top to the lowest index; the residual is +0.0 where the
# worker's own mask is set and a bit copy elsewhere.
# ============================================================================
def topk_union_step(grads, err, K: int, by_sort: bool = False, threads: int = 1):
    """One SSGD-top-K step.  Returns a dict with acc, worker_idx [N,K], worker_bits, votes [d],
    union_idx (ascending int32), union_val (float32, same length) and the new err [N,d]."""
    r = mv_vote(grads, err, K, by_sort=by_sort, threads=threads)
    acc = r["acc"]
    N, d = acc.shape
    union = np.flatnonzero(r["votes"] > 0).astype(np.int32)          # coordinates at least one worker kept
    cols = union.astype(np.int64)
    total = np.zeros(cols.shape[0], dtype=np.float64)
    new_err = np.array(acc, dtype=np.float32, copy=True)
    with np.errstate(all="ignore"):
        for n in range(N):                                             # worker order
            kept = np.zeros(d, dtype=bool)
            kept[r["worker_idx"][n].astype(np.int64)] = True
            k = kept[cols]
            total[k] = total[k] + acc[n, cols[k]].astype(np.float64)
            new_err[n, kept] = np.float32(0.0)
        r["union_val"] = (total / np.float64(N)).astype(np.float32)
    r["union_idx"] = union
    r["err"] = new_err
    return r
