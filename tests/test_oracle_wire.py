"""Pins for the wire-format oracle: the paper's own bit budgets (Section 2.1 formulas, the worked
numbers in the text and the bit-budget columns of Table 1), a hand-written bit stream, round trips,
and closed-form properties of the quantiser."""
import math

import numpy as np
import pytest

from oracle import wire_oracle as W


# ---------------------------------------------------------------- the paper's numbers
def test_load_formulas_match_the_papers_worked_numbers():
    d = 11_173_962
    q_val, q_loc, q = W.load_bits(d, 1e-2, 32)
    # "when phi = 10^-2, 9 bits are required to represent the position of each non-zero value"
    assert math.ceil(q_loc / (1e-2 * d)) == 9
    assert abs(q_val / d - 0.32) < 1e-12                         # Table 1, SSGD-MV: q_val = 3.2e-1
    # Table 1 compression factors: 32 / (q_loc + q_val) per parameter with the 9-bit position budget
    assert round(32 / (0.09 + 0.32)) == 78                       # SSGD-MV x78
    assert round(32 / (0.045 + 0.16)) == 156                     # -L2 x156
    assert round(32 / (0.0225 + 0.08)) == 312                    # -L4 x312
    assert round(32 / (0.01125 + 0.04)) == 624                   # -L8 x624
    assert round(32 / (0.003 + 0.005)) == 4000                   # AD-L8-Q x4000
    # add-drop: phi_ad = 1e-3 -> 12 bits per position, a fifth of the positions -> 2.4 bits (Section 3)
    assert math.ceil(math.log2(1000) + 2) == 12
    assert abs(12 * (2 * 1e-3 / 1e-2) - 2.4) < 1e-12
    assert round(32 / (0.024 + 0.32)) == 93                      # SSGD-MV-AD uplink x93
    assert abs(q - (q_val + q_loc)) < 1e-6                       # Eq. 15 = Eq. 13 + Eq. 14


def test_stream_length_is_eq_14_when_block_is_a_power_of_two():
    """K = phi*d non-zeros, blocks of 1/phi = 2^w coordinates: exactly d*phi*(log2(1/phi) + 2) bits."""
    for w in (4, 6, 7):
        B, nblocks = 1 << w, 1000
        d, K = B * nblocks, nblocks
        assert W.position_stream_bits(d, B, K) == K * (w + 2)
        assert abs(W.load_bits(d, 1.0 / B)[1] - K * (w + 2)) < 1e-6
    # phi = 1e-2: blocks of 100 need 7 offset bits -> the paper's 9 bits per position
    assert W.offset_width(100) + 2 == 9
    assert W.offset_width(128) + 2 == 9 and W.offset_width(64) + 2 == 8      # "phi in [1/64, 1/128]: 9 bits suffice"


# ---------------------------------------------------------------- hand-written stream
def test_hand_written_stream():
    # d = 12, blocks of 4 (2 offset bits); non-zeros at 1, 3 (block 0), none (block 1), 8 (block 2)
    # tokens: 1 01 | 1 11 | 0 || 0 || 1 00 | 0   ->  bits in stream order:
    want_bits = [1, 0, 1, 1, 1, 1, 0, 0, 1, 0, 0, 0]
    words = W.encode_positions([1, 3, 8], 12, 4)
    got_bits = [(int(words[t >> 5]) >> (t & 31)) & 1 for t in range(len(want_bits))]
    assert got_bits == want_bits and W.position_stream_bits(12, 4, 3) == 12
    assert W.decode_positions(words, 12, 12, 4).tolist() == [1, 3, 8]


@pytest.mark.parametrize("seed", range(6))
def test_round_trip(seed):
    rng = np.random.default_rng(seed)
    d = int(rng.integers(1, 5000))
    B = int(rng.choice([1, 2, 3, 7, 16, 100, 128, 1000]))
    K = int(rng.integers(0, min(d, 400) + 1))
    idx = np.sort(rng.choice(d, size=K, replace=False)).astype(np.int32)
    words = W.encode_positions(idx, d, B)
    nbits = W.position_stream_bits(d, B, K)
    assert words.size == (nbits + 31) // 32
    assert np.array_equal(W.decode_positions(words, nbits, d, B), idx)
    # every bit beyond the stream is zero, and the number of one-tokens equals K
    tail = [(int(words[t >> 5]) >> (t & 31)) & 1 for t in range(nbits, words.size * 32)]
    assert not any(tail)


# ---------------------------------------------------------------- quantiser
def test_quantizer_boundaries_are_geometric():
    b = W.quantizer_boundaries(8.0, 0.5, 4)                 # L = 8, ratio 16 -> alpha = 16^(1/8) = sqrt(2)
    assert len(b) == 9 and b[0] == 8.0
    np.testing.assert_allclose(b, 8.0 / np.sqrt(2.0) ** np.arange(9), rtol=1e-14)
    np.testing.assert_allclose(b[-1], 0.5, rtol=1e-13)


def test_quantize_small_example():
    # q = 2: L = 2 intervals, alpha = sqrt(16) = 4, inner boundary 8/4 = 2
    v = np.array([8.0, -2.0, 1.0, -0.5, 3.0, 0.0], dtype=np.float32)
    codes, means, vmax, vmin = W.quantize(v, 2)
    assert (vmax, vmin) == (8.0, 0.5)
    # magnitudes >= 2 -> interval 0 (8, 2, 3); below -> interval 1 (1, 0.5, 0); sign in bit 1
    assert codes.tolist() == [0, 0 | 2, 1, 1 | 2, 0, 1]
    assert means.tolist() == [np.float32(13 / 3), np.float32(0.5)]
    assert W.dequantize(codes, means, 2).tolist() == [np.float32(13 / 3), -np.float32(13 / 3), 0.5, -0.5,
                                                      np.float32(13 / 3), 0.5]


@pytest.mark.parametrize("q", [2, 3, 4, 5])
def test_quantizer_properties(q):
    rng = np.random.default_rng(q)
    v = (rng.standard_normal(5000) * 10.0 ** rng.uniform(-3, 0, 5000)).astype(np.float32)
    codes, means, vmax, vmin = W.quantize(v, q)
    L = 1 << (q - 1)
    a = np.abs(v)
    assert vmax == a.max() and vmin == a[a > 0].min()
    idx = codes & (L - 1)
    assert np.array_equal((codes >> (q - 1)) & 1, np.signbit(v).astype(np.uint8))
    assert idx[np.argmax(a)] == 0 and idx[np.argmin(np.where(a > 0, a, np.inf))] == L - 1
    # interval index is monotone in the magnitude, every value lies within a factor alpha of its
    # interval's mean, and the means decrease with the index
    order = np.argsort(-a, kind="stable")
    assert np.all(np.diff(idx[order].astype(int)) >= 0)
    alpha = (float(vmax) / float(vmin)) ** (1.0 / L)
    rec = np.abs(W.dequantize(codes, means, q))
    assert np.all(rec <= a * alpha * (1 + 1e-6)) and np.all(rec >= a / alpha * (1 - 1e-6))
    used = np.unique(idx)
    assert np.all(np.diff(means[used]) < 0)
    # the reconstruction keeps the mean magnitude of every interval (that is what mu_l is)
    for l in used:
        np.testing.assert_allclose(rec[idx == l].astype(np.float64).mean(), a[idx == l].astype(np.float64).mean(), rtol=1e-6)


def test_quantizer_degenerate_inputs():
    """No non-zero value, or a single magnitude: every code is interval 0 and the round trip is exact
    on the non-zero entries (zeros come back as the common magnitude, as for any value of interval 0)."""
    for v in (np.zeros(7, np.float32), np.full(5, -3.0, np.float32), np.array([0, 2, -2, 0], np.float32)):
        codes, means, vmax, vmin = W.quantize(v, 4)
        assert np.all((codes & 7) == 0) and vmax == vmin == np.abs(v).max()
        rec = W.dequantize(codes, means, 4)
        nz = v != 0
        assert np.array_equal(rec[nz], v[nz]) if nz.all() else np.all(np.sign(rec[nz]) == np.sign(v[nz]))
        assert np.array_equal((codes >> 3) & 1, np.signbit(v).astype(np.uint8))


def test_value_stream_layout():
    # q = 3: codes 5, 2, 7 -> bits 101 010 111 low bit first: stream bits 1,0,1, 0,1,0, 1,1,1 -> 0b111010101
    means = np.array([4, 3, 2, 1], dtype=np.float32)
    words = W.pack_values(np.array([5, 2, 7], dtype=np.uint8), means, 3)
    assert words.size == 1 + 4 and int(words[0]) == 0b111010101
    assert words[1:].view(np.float32).tolist() == [4, 3, 2, 1]
    codes, m = W.unpack_values(words, 3, 3)
    assert codes.tolist() == [5, 2, 7] and m.tolist() == [4, 3, 2, 1]
    rng = np.random.default_rng(0)
    for q in (1, 2, 5, 8):
        c = rng.integers(0, 1 << q, size=77).astype(np.uint8)
        mu = rng.random(1 << (q - 1)).astype(np.float32)
        cc, mm = W.unpack_values(W.pack_values(c, mu, q), 77, q)
        assert np.array_equal(cc, c) and np.array_equal(mm, mu)
