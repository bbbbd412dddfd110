"""CPU oracle for the wire formats of Section 4.3 and the load formulas of Section 2.1.

TEST INFRASTRUCTURE ONLY (see mv_oracle.py); plain Python/numpy, no code shared with the CUDA library.

Sparse position code ("Sparse representation"): the d coordinates are cut into blocks of B
coordinates (the paper's 1/phi); inside a block every non-zero position is sent as a '1' bit
followed by its offset within the block on w = ceil(log2 B) bits, and a single '0' bit closes the
block.  With K = phi*d non-zeros and d*phi blocks that is log2(1/phi) + 2 bits per non-zero (Eq. 14).
Readings where the paper is silent: offsets are written most significant bit first; stream bit t is
bit (t mod 32) of 32-bit word t div 32; positions inside a block are sent in ascending order; a last
block shorter than B is closed like any other; unused bits of the last word are zero.

Fractional quantiser ("Quantized representation", Eq. 18): for a value vector v and a bit budget q,
L = 2**(q-1) geometric intervals between v_max and v_min (the largest and the smallest non-zero
magnitude), alpha = (v_max/v_min)**(1/L), interval l = [v_max/alpha**l, v_max/alpha**(l-1)]; a value
is sent as the index of its interval on q-1 bits plus a sign bit, and the receiver replaces it by
the mean magnitude mu_l of the values that fell into that interval.
Readings: alpha is obtained by q-1 successive square roots of v_max/v_min and the inner boundaries
b_l = b_(l-1)/alpha (b_0 = v_max) by successive divisions, all in binary64, so that both sides get
the same boundaries; a magnitude a has code #{l in 1..L-1 : a < b_l} (a boundary value belongs to
the interval of the larger magnitudes; zeros land in the last interval); the code byte is
index | sign << (q-1); mu_l is the binary64 mean rounded to binary32, 0 for an empty interval;
if there is no non-zero value, or v_max == v_min, every value gets code 0.
"""
from __future__ import annotations

import math

import numpy as np


# ----------------------------------------------------------------------------- load formulas (Eq. 13-15)
def load_bits(d: int, phi: float, q: int = 32):
    """(Q_val, Q_loc, Q) of Eq. 13, 14, 15 for one direction."""
    q_val = q * phi * d
    q_loc = d * phi * (math.log2(1.0 / phi) + 2.0)
    return q_val, q_loc, q_val + q_loc


def offset_width(B: int) -> int:
    return 0 if B <= 1 else int(math.ceil(math.log2(B)))


def position_stream_bits(d: int, B: int, K: int) -> int:
    """Exact length of the position stream: K tokens of 1 + w bits and one closing bit per block."""
    return K * (1 + offset_width(B)) + (d + B - 1) // B


# ----------------------------------------------------------------------------- position code
def encode_positions(idx, d: int, B: int) -> np.ndarray:
    """Bit stream (uint32 words) of an ascending index list, written token by token."""
    w = offset_width(B)
    bits = []
    idx = [int(j) for j in idx]
    k = 0
    for blk in range((d + B - 1) // B):
        while k < len(idx) and idx[k] // B == blk:
            o = idx[k] - blk * B
            bits.append(1)
            bits.extend((o >> (w - 1 - i)) & 1 for i in range(w))      # most significant bit first
            k += 1
        bits.append(0)
    assert k == len(idx)
    words = np.zeros((len(bits) + 31) // 32, dtype=np.uint32)
    for t, b in enumerate(bits):
        if b:
            words[t >> 5] |= np.uint32(1 << (t & 31))
    return words


def decode_positions(words: np.ndarray, nbits: int, d: int, B: int) -> np.ndarray:
    """The receiver's cursor walk described in the paper."""
    w = offset_width(B)
    get = lambda t: (int(words[t >> 5]) >> (t & 31)) & 1
    out, blk, t = [], 0, 0
    while t < nbits:
        if get(t):
            o = 0
            for i in range(w):
                o = (o << 1) | get(t + 1 + i)
            out.append(blk * B + o)
            t += 1 + w
        else:
            blk += 1
            t += 1
    return np.array(out, dtype=np.int32)


# ----------------------------------------------------------------------------- fractional quantiser
def quantizer_boundaries(vmax: float, vmin: float, q: int) -> np.ndarray:
    """b_0 .. b_L in binary64: b_0 = vmax, b_l = b_(l-1) / alpha, alpha = (vmax/vmin)**(1/L) by q-1 square roots."""
    L = 1 << (q - 1)
    alpha = np.float64(vmax) / np.float64(vmin)
    for _ in range(q - 1):
        alpha = np.sqrt(alpha)
    b = np.empty(L + 1, dtype=np.float64)
    b[0] = np.float64(vmax)
    for l in range(1, L + 1):
        b[l] = b[l - 1] / alpha
    return b


def quantize(v: np.ndarray, q: int):
    """Returns (codes uint8[K], means float32[L], vmax, vmin)."""
    v = np.asarray(v, dtype=np.float32)
    a = np.abs(v)
    L = 1 << (q - 1)
    nz = a[a > 0]
    codes = np.zeros(v.shape[0], dtype=np.uint8)
    if nz.size and nz.max() > nz.min():
        vmax, vmin = np.float32(nz.max()), np.float32(nz.min())
        b = quantizer_boundaries(float(vmax), float(vmin), q)
        a64 = a.astype(np.float64)
        for l in range(1, L):
            codes += (a64 < b[l]).astype(np.uint8)
    else:
        vmax = vmin = np.float32(nz.max()) if nz.size else np.float32(0)
    means = np.zeros(L, dtype=np.float32)
    for l in range(L):
        sel = a[codes == l]
        if sel.size:
            means[l] = np.float32(sel.astype(np.float64).sum() / sel.size)
    sign = np.signbit(v).astype(np.uint8)
    return (codes | (sign << (q - 1))).astype(np.uint8), means, vmax, vmin


def dequantize(codes: np.ndarray, means: np.ndarray, q: int) -> np.ndarray:
    L = 1 << (q - 1)
    mag = means[codes & (L - 1)]
    return np.where((codes >> (q - 1)) & 1, -mag, mag).astype(np.float32)


def pack_values(codes: np.ndarray, means: np.ndarray, q: int) -> np.ndarray:
    """Value stream: code k on stream bits [k q, k q + q) (low bit first), then the L means from the next word on."""
    K = codes.shape[0]
    nw = (K * q + 31) // 32
    words = np.zeros(nw + means.shape[0], dtype=np.uint32)
    for k in range(K):
        for i in range(q):
            if (int(codes[k]) >> i) & 1:
                t = k * q + i
                words[t >> 5] |= np.uint32(1 << (t & 31))
    words[nw:] = means.astype(np.float32).view(np.uint32)
    return words


def unpack_values(words: np.ndarray, K: int, q: int):
    nw = (K * q + 31) // 32
    codes = np.zeros(K, dtype=np.uint8)
    for k in range(K):
        c = 0
        for i in range(q):
            t = k * q + i
            c |= ((int(words[t >> 5]) >> (t & 31)) & 1) << i
        codes[k] = c
    return codes, words[nw:nw + (1 << (q - 1))].view(np.float32).copy()
