/*
 * mv_wire.h -- C ABI of the wire formats that carry a sparse mask and its values
 * (Section 4.3 of arXiv 2011.06495, "Sparse representation" and "Quantized representation").
 *
 * Position stream.  The d coordinates are cut into blocks of B coordinates (the paper's 1/phi).
 * Within a block every selected coordinate is a '1' bit followed by its offset inside the block
 * on w = ceil(log2 B) bits; one '0' bit closes each block.  K selected coordinates therefore take
 * K (1 + w) + ceil(d / B) bits, the log2(1/phi) + 2 bits per position of Eq. 14 when K = d / B.
 * Fixed here where the paper is silent: offsets go most significant bit first, positions inside
 * a block ascend, stream bit t is bit (t mod 32) of 32-bit word (t div 32), a short last block is
 * closed like the others and the unused bits of the last word are zero.
 *
 * Value stream (fractional quantiser, Eq. 18).  With q bits per value, L = 2^(q-1) geometric
 * intervals between v_max and v_min (largest and smallest non-zero magnitude),
 * alpha = (v_max / v_min)^(1/L), boundaries b_0 = v_max, b_l = b_(l-1) / alpha.  A value is sent as
 * the number of inner boundaries b_1..b_(L-1) that its magnitude lies strictly below (q-1 bits)
 * with its sign bit above, value k occupying stream bits [k q, k q + q); the L interval means
 * mu_0..mu_(L-1) (binary32) follow from the next 32-bit word on, so the stream has
 * ceil(K q / 32) + L words.  alpha comes from q-1 successive binary64 square roots and the
 * boundaries from successive binary64 divisions; comparisons are made in binary64.  If no value is
 * non-zero or v_max == v_min every index is 0.  Inputs must be finite.
 *
 * Memory and errors follow mv_sparse.h: DEVICE pointers owned by the caller unless said
 * otherwise, nothing is allocated, work is enqueued on `stream` (a cudaStream_t, NULL = default
 * stream) without synchronising the host, status codes are MV_OK / MV_ERR_* and argument checks
 * happen before anything is enqueued.
 */
#ifndef MV_WIRE_H
#define MV_WIRE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* w = ceil(log2 B), 0 for B = 1 (host arithmetic only). */
int mv_pos_offset_bits(int64_t B);

/* Exact stream length in bits for K positions out of d with block size B (host arithmetic only);
 * -1 for arguments out of range. */
int64_t mv_pos_stream_bits(int64_t d, int64_t B, int64_t K);

/* Bytes of scratch mv_pos_decode needs for a stream of nbits bits. */
size_t mv_pos_decode_workspace_bytes(int64_t nbits, int64_t B);

/* Encodes an ascending index list (Section 4.3, sender side).
 *   idx   [K] int32 in   strictly ascending, 0 <= idx < d (as mv_sparse_step writes it); an entry
 *                        outside [0, d) -- such as the -1 padding mv_select_rs leaves when fewer than K
 *                        coordinates hold a vote -- is skipped and writes nothing (the stream is then
 *                        the one of the list without it only if such entries come last)
 *   words [ceil(mv_pos_stream_bits / 32)] uint32 out, fully overwritten
 * Limits: 1 <= d < 2^31, 1 <= B <= d, 0 <= K <= d. */
int mv_pos_encode(void* stream, const int32_t* idx, int64_t K, int64_t d, int64_t B, uint32_t* words);

/* Decodes a position stream (Section 4.3, the receiver's cursor walk, done segment-parallel).
 *   words   [ceil(nbits / 32)] uint32 in
 *   idx     [cap] int32 out: the first min(count, cap) positions, ascending
 *   result  [4] int64 out (device): [0] positions found, [1] blocks closed,
 *           [2] 0 if the stream is well formed (it ends on a token boundary, closes exactly
 *               ceil(d/B) blocks, every position is < d, count <= cap), else a non-zero bit set:
 *               1 truncated token, 2 block count, 4 position out of range, 8 idx too small;
 *           [3] reserved
 *   workspace  mv_pos_decode_workspace_bytes(nbits, B) bytes, 16-byte aligned */
int mv_pos_decode(void* stream, const uint32_t* words, int64_t nbits, int64_t d, int64_t B, int32_t* idx,
                  int64_t cap, int64_t* result, void* workspace, size_t workspace_bytes);

/* Words of the value stream: ceil(K q / 32) + 2^(q-1) (host arithmetic only); -1 if out of range. */
int64_t mv_quant_stream_words(int64_t K, int q);

/* Bytes of scratch mv_quantize needs. */
size_t mv_quant_workspace_bytes(int q);

/* Quantises K values (Eq. 18).  1 <= q <= 8, 0 <= K < 2^31.
 *   v      [K] float in
 *   words  [mv_quant_stream_words(K, q)] uint32 out, fully overwritten
 *   range  [2] float out, may be NULL: v_max, v_min (both 0 when no value is non-zero)
 * The interval means are binary64 sums (accumulated in no fixed order) divided by the count and
 * rounded once to binary32; an empty interval has mean 0. */
int mv_quantize(void* stream, const float* v, int64_t K, int q, uint32_t* words, float* range,
                void* workspace, size_t workspace_bytes);

/* Receiver side: out[k] = +-mu_(index k). */
int mv_dequantize(void* stream, const uint32_t* words, int64_t K, int q, float* out);

#ifdef __cplusplus
}
#endif
#endif /* MV_WIRE_H */
