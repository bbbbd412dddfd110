"""mv_select_static: the shared-mask selection for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is off limits (a real-time loop, a plug-in whose
host forbids allocation after start-up, a process whose memory pool is fully handed out), so they
cannot provide the workspace that mv_create wants.  mv_select_static keeps its scratch in an array
compiled into the library instead.  These tests call it through the C ABI and require the same bytes
as mv_select gives -- and as the CPU oracle's S_top over the votes gives -- on two calls in a row (the
array keeps the first call's leftovers, which the second call must not see), at the largest size the
array is built for, and check that a size beyond that limit is refused.

This file is named so that pytest collects it last.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import mv_oracle as O
from paper_2011_06495_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _votes(d, N, seed, dense):
    g = torch.Generator().manual_seed(seed)
    if dense:
        v = torch.randint(0, N + 1, (d,), generator=g)
    else:                                   # mostly zero, as after a sparse vote
        v = torch.randint(0, N + 1, (d,), generator=g) * (torch.rand(d, generator=g) < 0.02)
    return v.to(torch.uint8).to(DEV)


def _both(votes, N, K):
    d = votes.numel()
    W = (d + 31) // 32
    ctx = B.MvContext(N, d, K, device=DEV)
    ref_idx = torch.full((K,), -1, dtype=torch.int32, device=DEV)
    ref_bits = torch.full((W,), 0x5A5A5A5A, dtype=torch.int32, device=DEV)
    ctx.mv_select(votes, N, ref_idx, ref_bits, K=K)
    got_idx = torch.full((K,), -2, dtype=torch.int32, device=DEV)
    got_bits = torch.full((W,), 0x3C3C3C3C, dtype=torch.int32, device=DEV)
    B.mv_select_static(votes, N, K, got_idx, got_bits)
    torch.cuda.synchronize()
    return ref_idx, ref_bits, got_idx, got_bits


def test_two_calls_in_a_row_match_mv_select():
    # first call: a larger problem, dense votes; second call: smaller and sparse, so anything the
    # first call left in the array (ticket, histogram, per-chunk counts) would show
    cases = [(9, 1_000_003, 20_000, True, 1), (5, 300_007, 700, False, 2), (9, 1_000_003, 20_000, True, 1)]
    for N, d, K, dense, seed in cases:
        votes = _votes(d, N, seed, dense)
        ref_idx, ref_bits, got_idx, got_bits = _both(votes, N, K)
        assert torch.equal(got_idx, ref_idx), f"out_idx differs for N={N} d={d} K={K}"
        assert torch.equal(got_bits, ref_bits), f"mask_bits differs for N={N} d={d} K={K}"
        # the oracle's selection over the same votes (Eq. 9, outer S_top; ties to the lowest index)
        want_idx = O.select_mask(votes.cpu().numpy(), K)[0]
        assert np.array_equal(got_idx.cpu().numpy(), want_idx), f"out_idx differs from the oracle for N={N} d={d} K={K}"
        assert np.array_equal(got_bits.cpu().numpy().view(np.uint32), O.support_to_bits(want_idx, d))
        # and both are right: K strictly ascending indices, every chosen vote >= every other vote
        idx = got_idx.cpu().numpy().astype(np.int64)
        v = votes.cpu().numpy()
        assert np.all(np.diff(idx) > 0) and idx[0] >= 0 and idx[-1] < d
        inside = np.zeros(d, bool)
        inside[idx] = True
        assert v[inside].min() >= v[~inside].max()


def test_largest_size_the_array_is_built_for():
    """d = MV_SELECT_STATIC_MAX_D exactly (every per-chunk slot of the array in use), twice in a row with
    different votes, against mv_select and against the oracle."""
    d = B.MV_SELECT_STATIC_MAX_D
    for N, K, dense, seed in [(64, d // 100, False, 11), (3, 4194, True, 12)]:
        votes = _votes(d, N, seed, dense)
        ref_idx, ref_bits, got_idx, got_bits = _both(votes, N, K)
        assert torch.equal(got_idx, ref_idx) and torch.equal(got_bits, ref_bits)
        want_idx = O.select_mask(votes.cpu().numpy(), K)[0]
        assert np.array_equal(got_idx.cpu().numpy(), want_idx), f"out_idx differs from the oracle for N={N} K={K}"


def test_mask_may_be_omitted_and_small_inputs_work():
    for N, d, K in [(1, 1, 1), (3, 33, 33), (7, 4097, 5)]:
        votes = _votes(d, N, d, True)
        ctx = B.MvContext(N, d, K, device=DEV)
        ref = torch.empty(K, dtype=torch.int32, device=DEV)
        got = torch.empty(K, dtype=torch.int32, device=DEV)
        ctx.mv_select(votes, N, ref, None, K=K)
        B.mv_select_static(votes, N, K, got, None)
        torch.cuda.synchronize()
        assert torch.equal(got, ref)


def test_sizes_beyond_the_array_are_refused():
    lib = B.load()
    d = B.MV_SELECT_STATIC_MAX_D + 1
    votes = torch.zeros(64, dtype=torch.uint8, device=DEV)      # never read: the call must fail first
    out = torch.zeros(16, dtype=torch.int32, device=DEV)
    rc = lib.mv_select_static(None, ctypes.c_void_p(votes.data_ptr()), 4, d, 8, ctypes.c_void_p(out.data_ptr()), None)
    assert rc == B.MV_ERR_TOO_LARGE
    assert "MV_SELECT_STATIC_MAX_D" in B.status_string(rc)
    rc = lib.mv_select_static(None, None, 4, 1000, 8, ctypes.c_void_p(out.data_ptr()), None)
    assert rc == B.MV_ERR_INVALID_ARG
    torch.cuda.synchronize()
