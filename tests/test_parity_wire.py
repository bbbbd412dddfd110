"""GPU parity of the wire formats (Section 4.3) against the CPU oracle: position streams bit for bit,
decoded positions index for index, quantiser codes bit for bit, interval means within 1e-6 relative
(binary64 sums accumulated in a different order, rounded once to binary32)."""
import numpy as np
import pytest
import torch

from oracle import wire_oracle as W
from paper_2011_06495_b200 import binding as B
from paper_2011_06495_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MEAN_REL_TOL = 1e-6


def gpu_encode(idx_np, d, Bk):
    K = idx_np.shape[0]
    nbits = B.pos_stream_bits(d, Bk, K)
    words = torch.full(((nbits + 31) // 32,), -1, dtype=torch.int32, device=DEV)      # must be fully overwritten
    idx = torch.from_numpy(idx_np.astype(np.int32)).to(DEV)
    B.mv_pos_encode(idx, d, Bk, words)
    torch.cuda.synchronize()
    return words, nbits


def gpu_decode(words, nbits, d, Bk, cap):
    idx = torch.full((max(cap, 1),), -7, dtype=torch.int32, device=DEV)[:cap]
    result = torch.full((4,), -1, dtype=torch.int64, device=DEV)
    ws = torch.empty(B.pos_decode_workspace_bytes(nbits, Bk), dtype=torch.uint8, device=DEV)
    B.mv_pos_decode(words, nbits, d, Bk, idx, result, ws)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), result.cpu().numpy()


def random_support(rng, d, K):
    return np.sort(rng.choice(d, size=K, replace=False)).astype(np.int32)


@pytest.mark.parametrize("d,Bk,K", [
    (12, 4, 3), (1, 1, 0), (1, 1, 1), (37, 1, 37), (37, 37, 0), (1000, 100, 10), (5000, 128, 5000),
    (100_003, 100, 1000), (100_003, 7, 31_000), (1_000_000, 1000, 1000), (1_000_000, 64, 200_000),
    (3_000_017, 100_000, 30_000), (2_000_000, 2_000_000, 999), (1 << 20, 1 << 20, 1 << 20)])
def test_position_stream_matches_the_oracle(d, Bk, K):
    rng = np.random.default_rng(d * 31 + Bk * 7 + K)
    idx = random_support(rng, d, K)
    words, nbits = gpu_encode(idx, d, Bk)
    assert nbits == W.position_stream_bits(d, Bk, K)
    if d <= 1_000_000 or K <= 31_000:                  # the oracle writes bit by bit in Python
        want = W.encode_positions(idx, d, Bk)
        got = words.cpu().numpy().view(np.uint32)
        assert np.array_equal(got, want)
    got_idx, result = gpu_decode(words, nbits, d, Bk, K)
    assert result.tolist()[:3] == [K, (d + Bk - 1) // Bk, 0]
    assert np.array_equal(got_idx, idx)


def test_clustered_and_edge_positions():
    """All positions in one block, the first and the last coordinate, a ragged last block."""
    d, Bk = 100_003, 100
    for idx in (np.arange(4200, 4300), np.array([0, d - 1]), np.arange(d - 3, d), np.arange(0, d, 100), np.arange(99, d, 100)):
        idx = idx.astype(np.int32)
        words, nbits = gpu_encode(idx, d, Bk)
        assert np.array_equal(words.cpu().numpy().view(np.uint32), W.encode_positions(idx, d, Bk))
        got_idx, result = gpu_decode(words, nbits, d, Bk, idx.size)
        assert result.tolist()[:3] == [idx.size, 1001, 0] and np.array_equal(got_idx, idx)


def test_encoder_skips_entries_that_are_not_coordinates():
    """A list padded with -1 (what mv_select_rs leaves when fewer than K coordinates hold a vote), or
    holding an index >= d, must write nothing outside the stream: the valid entries land where the
    oracle puts them for the list without the padding, every other bit stays zero."""
    d, Bk = 100_003, 100
    rng = np.random.default_rng(5)
    good = random_support(rng, d, 700)
    for tail in (np.full(300, -1, np.int32), np.array([d, d + 5, 2**31 - 1, -2**31], np.int64).astype(np.int32)):
        padded = np.concatenate([good, tail]).astype(np.int32)
        guard = torch.full((4096,), 0x5A5A5A5A, dtype=torch.int32, device=DEV)      # the stream sits in the middle
        nbits = B.pos_stream_bits(d, Bk, padded.size)
        nw = (nbits + 31) // 32
        words = guard[1024:1024 + nw]
        assert nw < 2048
        B.mv_pos_encode(torch.from_numpy(padded).to(DEV), d, Bk, words)
        torch.cuda.synchronize()
        g = guard.cpu().numpy().view(np.uint32)
        assert np.all(g[:1024] == 0x5A5A5A5A) and np.all(g[1024 + nw:] == 0x5A5A5A5A), "wrote outside the stream"
        want = W.encode_positions(good, d, Bk)
        got = g[1024:1024 + nw]
        assert np.array_equal(got[:want.size], want) and not got[want.size:].any()


def test_decoder_reads_an_oracle_stream_and_reports_malformed_ones():
    d, Bk, K = 50_000, 128, 3000
    rng = np.random.default_rng(5)
    idx = random_support(rng, d, K)
    want = W.encode_positions(idx, d, Bk)
    nbits = W.position_stream_bits(d, Bk, K)
    words = torch.from_numpy(want.view(np.int32)).to(DEV)
    got_idx, result = gpu_decode(words, nbits, d, Bk, K)
    assert result.tolist()[:3] == [K, 391, 0] and np.array_equal(got_idx, idx)
    # idx too small: the prefix is written, the count is the full one, bit 8 is set
    got_idx, result = gpu_decode(words, nbits, d, Bk, 100)
    assert result[0] == K and result[2] == 8 and np.array_equal(got_idx, idx[:100])
    # a stream cut inside its last position token: truncated token and a missing block
    cut = nbits - 1 - (d + Bk - 1) // Bk + int(idx[-1]) // Bk          # last bit of the last token
    got_idx, result = gpu_decode(words, cut, d, Bk, K)
    assert result[2] & 1 and result[2] & 2
    # an offset beyond the block size (block size 100 has 7 offset bits: offsets 100..127 are invalid)
    bad = W.encode_positions(np.array([127], dtype=np.int32), 1000, 128)
    got_idx, result = gpu_decode(torch.from_numpy(bad.view(np.int32)).to(DEV), W.position_stream_bits(1000, 128, 1), 1000, 100, 4)
    assert result[2] & 4


def test_mask_of_a_step_round_trips():
    """The shared mask of a real step (clustered by layer scale) through encode and decode."""
    w = WL.scaled(WL.resnet_like("c2"), 1_000_003, K=10_000, steps=1)
    grads = WL.gradients(w, 0, DEV)
    err = WL.initial_err(w, DEV)
    ctx = B.MvContext(w.N, w.d, w.K, device=DEV)
    out_idx = torch.empty(w.K, dtype=torch.int32, device=DEV)
    out_val = torch.empty(w.K, dtype=torch.float32, device=DEV)
    ctx.mv_sparse_step(grads, err, out_idx, out_val)
    torch.cuda.synchronize()
    idx = out_idx.cpu().numpy()
    words, nbits = gpu_encode(idx, w.d, 100)
    assert np.array_equal(words.cpu().numpy().view(np.uint32), W.encode_positions(idx, w.d, 100))
    got_idx, result = gpu_decode(words, nbits, w.d, 100, w.K)
    assert result[2] == 0 and np.array_equal(got_idx, idx)
    # and its values through the 4-bit quantiser
    check_quantizer(out_val.cpu().numpy(), 4)


def check_quantizer(v_np, q):
    K = v_np.shape[0]
    v = torch.from_numpy(v_np).to(DEV)
    total = B.quant_stream_words(K, q)
    words = torch.full((total,), -1, dtype=torch.int32, device=DEV)
    rng_out = torch.full((2,), -1.0, dtype=torch.float32, device=DEV)
    ws = torch.empty(B.quant_workspace_bytes(q), dtype=torch.uint8, device=DEV)
    B.mv_quantize(v, q, words, ws, rng_out)
    out = torch.full((max(K, 1),), 7.0, dtype=torch.float32, device=DEV)[:K]
    B.mv_dequantize(words, K, q, out)
    torch.cuda.synchronize()
    codes, means, vmax, vmin = W.quantize(v_np, q)
    got_words = words.cpu().numpy().view(np.uint32)
    assert rng_out.cpu().numpy().tolist() == [float(vmax), float(vmin)]
    nw = (K * q + 31) // 32
    got_codes, got_means = W.unpack_values(got_words, K, q) if K <= 200_000 else (None, got_words[nw:].view(np.float32))
    want_words = W.pack_values(codes, means, q) if K <= 200_000 else None
    if want_words is not None:
        assert np.array_equal(got_words[:nw], want_words[:nw]), "code bits differ"
        assert np.array_equal(got_codes, codes)
    np.testing.assert_allclose(got_means, means, rtol=MEAN_REL_TOL, atol=0)
    L = 1 << (q - 1)
    want_rec = W.dequantize(codes, got_means, q)               # same table: the lookup itself is exact
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want_rec.view(np.uint32))
    return got_words


@pytest.mark.parametrize("q", [1, 2, 3, 4, 5, 8])
@pytest.mark.parametrize("K", [1, 7, 33, 1000, 111_739])
def test_quantizer_matches_the_oracle(q, K):
    rng = np.random.default_rng(q * 1000 + K)
    v = (rng.standard_normal(K) * 10.0 ** rng.uniform(-4, 0, K)).astype(np.float32)
    check_quantizer(v, q)


def test_quantizer_special_inputs():
    check_quantizer(np.zeros(50, np.float32), 4)
    check_quantizer(np.full(50, -2.5, np.float32), 4)
    check_quantizer(np.array([0, 3, -3, 0, -0.0], np.float32), 3)
    check_quantizer(np.array([8, -2, 1, -0.5, 3, 0], np.float32), 2)
    check_quantizer(np.zeros(0, np.float32), 4)
    # magnitudes sitting exactly on the boundaries: ratio 2^8 with L = 8 gives alpha = 2 and b_l = 2^-l exactly
    v = np.array([1.0, 0.5, 0.25, 0.125, 2.0 ** -4, 2.0 ** -5, 2.0 ** -6, 2.0 ** -7, 2.0 ** -8, 0.3, -0.5, -0.0078125],
                 np.float32)
    words = check_quantizer(v, 4)
    codes, _ = W.unpack_values(words, v.size, 4)
    assert (codes[:9] & 7).tolist() == [0, 0, 1, 2, 3, 4, 5, 6, 7]          # a boundary value joins the larger interval
    # denormals and a huge dynamic range
    check_quantizer(np.array([1e-45, 3e38, -1e-20, 5.0, 1e-39], np.float32), 5)


def test_quantizer_large_vector_means():
    rng = np.random.default_rng(11)
    K = 1_342_177
    v = (rng.standard_normal(K) * 10.0 ** rng.uniform(-4, 0, K)).astype(np.float32)
    check_quantizer(v, 4)
