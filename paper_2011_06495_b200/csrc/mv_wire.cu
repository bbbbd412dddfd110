// mv_wire.cu -- wire formats of a sparse mask and its values for sm_100a (Section 4.3 of arXiv 2011.06495).
//
// Position stream ("Sparse representation"): '1' + w offset bits per selected coordinate, one '0' per
// block of B coordinates.  The encoder is one thread per position: the token of the k-th position
// starts at bit k (1 + w) + (its block number), because exactly that many closing bits precede it.
// The decoder cannot know where tokens start without walking the stream, so it walks it in three
// small kernels: every 512-bit segment is parsed once for each of the w + 1 ways a token can
// straddle its left edge, a single block chains the per-segment results (which entry state is the
// real one, how many positions and blocks precede the segment), and the segments are then parsed
// once more, in parallel, writing the positions.
//
// Value stream ("Quantized representation", Eq. 18): magnitude range by atomic max on the bit
// patterns, boundaries by one thread in binary64 (successive square roots and divisions, so that
// any IEEE host gets the same numbers), then one thread per 32-bit word of the output stream:
// it classifies the few values that overlap its word by binary search over the boundaries and adds
// the magnitudes whose first bit lies in its word to the per-interval sums.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mv_sparse.h"
#include "../../include/mv_wire.h"

namespace {

constexpr int SEG_BITS = 512;        // decoder segment
constexpr int LINK_TILE = 256;       // segments chained per shared-memory tile
constexpr int LINK_CHUNK = 8;        // consecutive segments composed by one thread; LINK_TILE / LINK_CHUNK = 32 chunks
constexpr int QBINS = 128;           // 2^(8-1): most intervals a byte-wide code can name

__host__ __device__ inline int offset_bits(int64_t B) {
  int w = 0;
  while ((int64_t(1) << w) < B) ++w;
  return w;
}

__device__ __forceinline__ uint64_t window(const uint32_t* words, int64_t nwords, int64_t t) {
  int64_t i = t >> 5;
  uint32_t lo = i < nwords ? __ldg(words + i) : 0u;
  uint32_t hi = i + 1 < nwords ? __ldg(words + i + 1) : 0u;
  return ((uint64_t(hi) << 32) | lo) >> (t & 31);
}

// ------------------------------------------------------------------------------------------ position encoder
// An entry that is not a coordinate (negative, e.g. the -1 padding of a short list, or >= d), or whose token
// would not fit the stream, is skipped: nothing is written outside `words`.
__global__ void k_pos_encode(const int32_t* __restrict__ idx, int64_t K, uint32_t B, int w, uint32_t d, int64_t nbits,
                             uint32_t* __restrict__ words) {
  int64_t k = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (k >= K) return;
  const int32_t ji = idx[k];
  if (ji < 0 || uint32_t(ji) >= d) return;
  uint32_t j = uint32_t(ji);
  uint32_t blk = j / B, o = j - blk * B;
  int64_t pos = k * (1 + w) + blk;
  if (pos + 1 + w > nbits) return;
  uint64_t token = 1u | (w ? (uint64_t(__brev(o) >> (32 - w)) << 1) : 0u);     // offset bits, most significant first
  uint64_t val = token << (pos & 31);
  atomicOr(words + (pos >> 5), uint32_t(val));
  if (val >> 32) atomicOr(words + (pos >> 5) + 1, uint32_t(val >> 32));
}

// ------------------------------------------------------------------------------------------ position decoder
// map entry: exit state (6 bits) | positions (13 bits) | closed blocks (13 bits)
//
// Both parsing kernels stage their segments' words in shared memory first (coalesced), one padding
// word per segment so that threads walking different segments hit different banks.
constexpr int SEG_WORDS = SEG_BITS / 32;
constexpr int SCAN_SEGS = 32;        // segments per block of k_pos_scan (times w + 1 threads)
constexpr int EMIT_SEGS = 32;        // segments (= threads) per block of k_pos_emit

__device__ __forceinline__ int padded(int i) { return i + i / SEG_WORDS; }

__device__ __forceinline__ void stage_words(const uint32_t* __restrict__ words, int64_t nwords, int64_t first, int count,
                                            uint32_t* sw) {
  for (int i = threadIdx.x; i < count; i += blockDim.x) sw[padded(i)] = first + i < nwords ? __ldg(words + first + i) : 0u;
  __syncthreads();
}

__global__ void k_pos_scan(const uint32_t* __restrict__ words, int64_t nbits, int w, int64_t nseg, uint32_t* __restrict__ map) {
  __shared__ uint32_t sw[SCAN_SEGS * (SEG_WORDS + 1) + 2];
  const int64_t seg0 = int64_t(blockIdx.x) * SCAN_SEGS;
  stage_words(words, (nbits + 31) >> 5, seg0 * SEG_WORDS, SCAN_SEGS * SEG_WORDS, sw);
  const int ls = threadIdx.x / (w + 1);
  const int r = threadIdx.x - ls * (w + 1);          // bits of a '1' token already consumed left of the segment
  const int64_t seg = seg0 + ls;
  if (ls >= SCAN_SEGS || seg >= nseg) return;
  const int e = int(min(int64_t(SEG_BITS), nbits - seg * SEG_BITS));      // segment-local end
  const int base = ls * SEG_BITS;
  int t = r ? (1 + w - r) : 0;
  uint32_t n1 = 0, n0 = 0;
  while (t < e) {
    uint32_t rest = sw[padded((base + t) >> 5)] >> (t & 31);          // this word from bit t on
    if (rest & 1u) { ++n1; t += 1 + w; }
    else {                                                             // a run of closing bits, up to the word's or the segment's end
      int z = min(min(rest ? __ffs(int(rest)) - 1 : 32, 32 - (t & 31)), e - t);
      n0 += z; t += z;
    }
  }
  uint32_t out = t > e ? uint32_t((1 + w) - (t - e)) : 0u;
  map[seg * (w + 1) + r] = (out << 26) | (n1 << 13) | n0;
}

// Chains the segments.  A segment's map is a function from entry state to (exit state, counts); the
// chain is the composition of these functions from the left.  Per tile of 256 segments: 32 (w + 1)
// threads each compose 8 consecutive maps from one entry state, thread 0 walks the 32 composed
// chunks with the real state, and one thread per segment replays at most 7 maps inside its chunk.
__device__ __forceinline__ void link_step(const uint32_t* tile, int w, int seg, uint32_t& st, int64_t& b1, int64_t& b0) {
  uint32_t m = tile[seg * (w + 1) + st];
  st = m >> 26; b1 += (m >> 13) & 8191u; b0 += m & 8191u;
}

__global__ void __launch_bounds__(1024) k_pos_link(const uint32_t* __restrict__ map, int w, int64_t nseg, int64_t nblocks,
                                                    int64_t cap, uint32_t* __restrict__ ent_state, int64_t* __restrict__ ent_b1,
                                                    int64_t* __restrict__ ent_b0, int64_t* __restrict__ result) {
  extern __shared__ uint32_t tile[];                 // LINK_TILE * (w + 1) map entries
  constexpr int NCHUNK = LINK_TILE / LINK_CHUNK;
  __shared__ uint32_t c_st[NCHUNK * 32], c_n1[NCHUNK * 32], c_n0[NCHUNK * 32];     // composed chunk maps [chunk][entry state]
  __shared__ uint32_t e_st[NCHUNK + 1];
  __shared__ int64_t e_b1[NCHUNK + 1], e_b0[NCHUNK + 1];                             // entries of the chunks; [NCHUNK] carries on
  if (threadIdx.x == 0) { e_st[NCHUNK] = 0; e_b1[NCHUNK] = 0; e_b0[NCHUNK] = 0; }
  for (int64_t base = 0; base < nseg; base += LINK_TILE) {
    const int cnt = int(min(int64_t(LINK_TILE), nseg - base));
    for (int i = threadIdx.x; i < cnt * (w + 1); i += blockDim.x) tile[i] = map[base * (w + 1) + i];
    __syncthreads();
    if (int(threadIdx.x) < NCHUNK * (w + 1)) {
      const int chunk = threadIdx.x / (w + 1), r = threadIdx.x - chunk * (w + 1);
      uint32_t st = r;
      int64_t n1 = 0, n0 = 0;
      for (int sgm = chunk * LINK_CHUNK; sgm < min(cnt, (chunk + 1) * LINK_CHUNK); ++sgm) link_step(tile, w, sgm, st, n1, n0);
      c_st[chunk * 32 + r] = st; c_n1[chunk * 32 + r] = uint32_t(n1); c_n0[chunk * 32 + r] = uint32_t(n0);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t st = e_st[NCHUNK];
      int64_t b1 = e_b1[NCHUNK], b0 = e_b0[NCHUNK];
      for (int c = 0; c < NCHUNK; ++c) {
        e_st[c] = st; e_b1[c] = b1; e_b0[c] = b0;
        b1 += c_n1[c * 32 + st]; b0 += c_n0[c * 32 + st]; st = c_st[c * 32 + st];
      }
      e_st[NCHUNK] = st; e_b1[NCHUNK] = b1; e_b0[NCHUNK] = b0;
    }
    __syncthreads();
    if (int(threadIdx.x) < cnt) {
      const int chunk = threadIdx.x / LINK_CHUNK;
      uint32_t st = e_st[chunk];
      int64_t b1 = e_b1[chunk], b0 = e_b0[chunk];
      for (int sgm = chunk * LINK_CHUNK; sgm < int(threadIdx.x); ++sgm) link_step(tile, w, sgm, st, b1, b0);
      ent_state[base + threadIdx.x] = st; ent_b1[base + threadIdx.x] = b1; ent_b0[base + threadIdx.x] = b0;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    result[0] = e_b1[NCHUNK]; result[1] = e_b0[NCHUNK];
    // the emit kernel may add bit 4; it runs after this kernel on the same stream
    result[2] = (e_st[NCHUNK] ? 1 : 0) | (e_b0[NCHUNK] != nblocks ? 2 : 0) | (e_b1[NCHUNK] > cap ? 8 : 0);
    result[3] = 0;
  }
}

__global__ void __launch_bounds__(EMIT_SEGS) k_pos_emit(const uint32_t* __restrict__ words, int64_t nbits, int64_t d, uint32_t B, int w,
                                                         int64_t nseg, const uint32_t* __restrict__ ent_state,
                                                         const int64_t* __restrict__ ent_b1, const int64_t* __restrict__ ent_b0,
                                                         int32_t* __restrict__ idx, int64_t cap, int64_t* result) {
  __shared__ uint32_t sw[EMIT_SEGS * (SEG_WORDS + 1) + 4];
  const int64_t seg0 = int64_t(blockIdx.x) * EMIT_SEGS;
  // two more words than the segments hold: a token that starts in a segment may end in the next one
  stage_words(words, (nbits + 31) >> 5, seg0 * SEG_WORDS, EMIT_SEGS * SEG_WORDS + 2, sw);
  const int64_t seg = seg0 + threadIdx.x;
  if (seg >= nseg) return;
  const int r = int(ent_state[seg]);
  int64_t k = ent_b1[seg], blk = ent_b0[seg];
  const int e = int(min(int64_t(SEG_BITS), nbits - seg * SEG_BITS));
  const int64_t left = nbits - seg * SEG_BITS;       // stream bits from the segment start on
  const int base = threadIdx.x * SEG_BITS;
  int t = r ? (1 + w - r) : 0;
  bool bad = false;
  while (t < e) {
    int i = (base + t) >> 5;
    uint64_t x = ((uint64_t(sw[padded(i + 1)]) << 32) | sw[padded(i)]) >> (t & 31);
    if (x & 1u) {
      if (t + 1 + w > left) break;                                    // truncated token: reported by the link kernel
      uint32_t o = w ? (__brev(uint32_t(x >> 1)) >> (32 - w)) : 0u;
      int64_t j = blk * int64_t(B) + o;
      if (o >= B || j >= d) bad = true;
      else if (k < cap) idx[k] = int32_t(j);
      ++k; t += 1 + w;
    } else {                                                           // a run of closing bits
      int z = min(x ? __ffsll((long long)x) - 1 : 64, min(32 - (t & 31) + 32, e - t));
      blk += z; t += z;
    }
  }
  if (bad) atomicOr(reinterpret_cast<unsigned long long*>(result + 2), 4ull);
}

// ------------------------------------------------------------------------------------------ quantiser
struct QScratch {
  uint32_t max_bits;        // largest magnitude bit pattern (0 when every value is zero)
  uint32_t inv_min_bits;    // ~(smallest non-zero magnitude bit pattern), 0 when there is none
  uint32_t degenerate;
  uint32_t pad;
  double bounds[QBINS];     // b_1 .. b_(L-1) at [1 .. L-1]
  double sums[QBINS];
  unsigned long long cnts[QBINS];
};

__global__ void k_q_range(const float* __restrict__ v, int64_t K, QScratch* q) {
  uint32_t mx = 0, imn = 0;
  for (int64_t k = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; k < K; k += int64_t(gridDim.x) * blockDim.x) {
    uint32_t b = __float_as_uint(v[k]) & 0x7fffffffu;
    mx = max(mx, b);
    if (b) imn = max(imn, ~b);
  }
  for (int o = 16; o; o >>= 1) {
    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    imn = max(imn, __shfl_xor_sync(0xffffffffu, imn, o));
  }
  if ((threadIdx.x & 31) == 0) {
    if (mx) atomicMax(&q->max_bits, mx);
    if (imn) atomicMax(&q->inv_min_bits, imn);
  }
}

__global__ void k_q_bounds(QScratch* q, int qbits, float* __restrict__ range) {
  float vmax = __uint_as_float(q->max_bits);
  float vmin = q->inv_min_bits ? __uint_as_float(~q->inv_min_bits) : 0.0f;
  if (q->max_bits == 0) vmin = 0.0f;
  bool deg = q->max_bits == 0 || vmax == vmin;
  if (deg) vmin = vmax;
  q->degenerate = deg ? 1u : 0u;
  if (range) { range[0] = vmax; range[1] = vmin; }
  if (deg) return;
  int L = 1 << (qbits - 1);
  double alpha = double(vmax) / double(vmin);
  for (int i = 0; i < qbits - 1; ++i) alpha = sqrt(alpha);
  double b = double(vmax);
  for (int l = 1; l < L; ++l) { b = b / alpha; q->bounds[l] = b; }
}

__device__ __forceinline__ uint32_t classify(double a, const double* sb, int L) {
  // boundaries decrease with l, so {l : a < b_l} is a prefix of 1..L-1; find its length
  uint32_t lo = 0, hi = uint32_t(L - 1);          // answer in [lo, hi]
  while (lo < hi) {
    uint32_t mid = (lo + hi + 1) >> 1;
    if (a < sb[mid]) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__global__ void __launch_bounds__(256) k_q_codes(const float* __restrict__ v, int64_t K, int qbits, QScratch* q,
                                                  uint32_t* __restrict__ words, int64_t nw) {
  __shared__ double sb[QBINS];
  __shared__ double ssum[QBINS];
  __shared__ uint32_t scnt[QBINS];
  const int L = 1 << (qbits - 1);
  const int R = QBINS >> (qbits - 1);              // copies of every interval's accumulator, to spread the atomics
  const bool deg = q->degenerate != 0;
  if (threadIdx.x < QBINS) {
    sb[threadIdx.x] = (threadIdx.x >= 1 && threadIdx.x < L && !deg) ? q->bounds[threadIdx.x] : 0.0;
    ssum[threadIdx.x] = 0.0; scnt[threadIdx.x] = 0;
  }
  __syncthreads();
  int64_t wd = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (wd < nw) {
    int64_t bit0 = wd * 32;
    int64_t k_lo = bit0 / qbits, k_hi = min(K - 1, (bit0 + 31) / qbits);
    uint32_t word = 0;
    for (int64_t k = k_lo; k <= k_hi; ++k) {
      float x = v[k];
      float a = fabsf(x);
      uint32_t c = deg ? 0u : classify(double(a), sb, L);
      uint32_t code = c | ((__float_as_uint(x) >> 31) << (qbits - 1));
      int64_t first = k * qbits;
      if (first >= bit0) {
        word |= code << (first - bit0);
        int slot = int(c) * R + int(threadIdx.x & (R - 1));
        atomicAdd(&ssum[slot], double(a));
        atomicAdd(&scnt[slot], 1u);
      } else {
        word |= code >> (bit0 - first);
      }
    }
    words[wd] = word;
  }
  __syncthreads();
  if (threadIdx.x < QBINS && scnt[threadIdx.x]) {
    atomicAdd(&q->sums[threadIdx.x / R], ssum[threadIdx.x]);
    atomicAdd(&q->cnts[threadIdx.x / R], (unsigned long long)scnt[threadIdx.x]);
  }
}

__global__ void k_q_means(const QScratch* q, int qbits, uint32_t* __restrict__ means) {
  int l = threadIdx.x;
  if (l < (1 << (qbits - 1))) {
    unsigned long long c = q->cnts[l];
    means[l] = __float_as_uint(c ? float(q->sums[l] / double(c)) : 0.0f);
  }
}

__global__ void __launch_bounds__(256) k_dequant(const uint32_t* __restrict__ words, int64_t K, int qbits, int64_t nw,
                                                  float* __restrict__ out) {
  __shared__ float mu[QBINS];
  const int L = 1 << (qbits - 1);
  if (threadIdx.x < L) mu[threadIdx.x] = __uint_as_float(words[nw + threadIdx.x]);
  __syncthreads();
  int64_t k = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (k >= K) return;
  uint32_t code = uint32_t(window(words, nw, k * qbits)) & ((1u << qbits) - 1u);
  float m = mu[code & (L - 1)];
  out[k] = (code >> (qbits - 1)) ? -m : m;
}

inline bool misaligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int cuda_ok() { return cudaGetLastError() == cudaSuccess ? MV_OK : MV_ERR_CUDA; }

struct DecodeLayout { size_t map, state, b1, b0, total; int64_t nseg; };
inline DecodeLayout decode_layout(int64_t nbits, int w) {
  DecodeLayout L;
  L.nseg = (nbits + SEG_BITS - 1) / SEG_BITS;
  size_t o = 0;
  L.map = o;   o = align_up(o + size_t(L.nseg) * (w + 1) * 4, 16);
  L.state = o; o = align_up(o + size_t(L.nseg) * 4, 16);
  L.b1 = o;    o = align_up(o + size_t(L.nseg) * 8, 16);
  L.b0 = o;    o = align_up(o + size_t(L.nseg) * 8, 16);
  L.total = o ? o : 16;
  return L;
}

}  // namespace

extern "C" {

int mv_pos_offset_bits(int64_t B) { return B < 1 ? -1 : offset_bits(B); }

int64_t mv_pos_stream_bits(int64_t d, int64_t B, int64_t K) {
  if (d < 1 || d >= (int64_t(1) << 31) || B < 1 || B > d || K < 0 || K > d) return -1;
  return K * (1 + offset_bits(B)) + (d + B - 1) / B;
}

size_t mv_pos_decode_workspace_bytes(int64_t nbits, int64_t B) {
  if (nbits < 0 || B < 1) return 0;
  return decode_layout(nbits, offset_bits(B)).total;
}

int mv_pos_encode(void* stream, const int32_t* idx, int64_t K, int64_t d, int64_t B, uint32_t* words) {
  int64_t nbits = mv_pos_stream_bits(d, B, K);
  if (nbits < 0 || !words || (K > 0 && !idx) || misaligned(words, 4) || misaligned(idx, 4)) return MV_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(words, 0, size_t((nbits + 31) / 32) * 4, st) != cudaSuccess) return MV_ERR_CUDA;
  if (K > 0) k_pos_encode<<<unsigned((K + 255) / 256), 256, 0, st>>>(idx, K, uint32_t(B), offset_bits(B), uint32_t(d), nbits, words);
  return cuda_ok();
}

int mv_pos_decode(void* stream, const uint32_t* words, int64_t nbits, int64_t d, int64_t B, int32_t* idx, int64_t cap,
                  int64_t* result, void* workspace, size_t workspace_bytes) {
  if (d < 1 || d >= (int64_t(1) << 31) || B < 1 || B > d || nbits < 0 || cap < 0 || !result || (nbits > 0 && !words) ||
      (cap > 0 && !idx) || misaligned(result, 8) || misaligned(workspace, 16))
    return MV_ERR_INVALID_ARG;
  const int w = offset_bits(B);
  DecodeLayout L = decode_layout(nbits, w);
  if (!workspace || workspace_bytes < L.total) return MV_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* base = static_cast<char*>(workspace);
  uint32_t* map = reinterpret_cast<uint32_t*>(base + L.map);
  uint32_t* ent_state = reinterpret_cast<uint32_t*>(base + L.state);
  int64_t* ent_b1 = reinterpret_cast<int64_t*>(base + L.b1);
  int64_t* ent_b0 = reinterpret_cast<int64_t*>(base + L.b0);
  int64_t nblocks = (d + B - 1) / B;
  if (L.nseg > 0)
    k_pos_scan<<<unsigned((L.nseg + SCAN_SEGS - 1) / SCAN_SEGS), SCAN_SEGS * (w + 1), 0, st>>>(words, nbits, w, L.nseg, map);
  k_pos_link<<<1, (LINK_TILE / LINK_CHUNK) * (w + 1) > LINK_TILE ? (LINK_TILE / LINK_CHUNK) * (w + 1) : LINK_TILE, size_t(LINK_TILE) * (w + 1) * 4, st>>>(map, w, L.nseg, nblocks, cap, ent_state, ent_b1, ent_b0, result);
  if (L.nseg > 0)
    k_pos_emit<<<unsigned((L.nseg + EMIT_SEGS - 1) / EMIT_SEGS), EMIT_SEGS, 0, st>>>(words, nbits, d, uint32_t(B), w, L.nseg, ent_state,
                                                                                  ent_b1, ent_b0, idx, cap, result);
  return cuda_ok();
}

int64_t mv_quant_stream_words(int64_t K, int q) {
  if (q < 1 || q > 8 || K < 0 || K >= (int64_t(1) << 31)) return -1;
  return (K * q + 31) / 32 + (int64_t(1) << (q - 1));
}

size_t mv_quant_workspace_bytes(int q) { return (q < 1 || q > 8) ? 0 : align_up(sizeof(QScratch), 16); }

int mv_quantize(void* stream, const float* v, int64_t K, int q, uint32_t* words, float* range, void* workspace,
                size_t workspace_bytes) {
  int64_t total = mv_quant_stream_words(K, q);
  if (total < 0 || !words || (K > 0 && !v) || misaligned(v, 4) || misaligned(words, 4) || misaligned(range, 4) ||
      misaligned(workspace, 16))
    return MV_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < sizeof(QScratch)) return MV_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  QScratch* qs = static_cast<QScratch*>(workspace);
  int64_t nw = (K * q + 31) / 32;
  if (cudaMemsetAsync(qs, 0, sizeof(QScratch), st) != cudaSuccess) return MV_ERR_CUDA;
  if (K > 0) {
    unsigned blocks = unsigned(min(int64_t(148 * 8), (K + 255) / 256));
    k_q_range<<<blocks, 256, 0, st>>>(v, K, qs);
  }
  k_q_bounds<<<1, 1, 0, st>>>(qs, q, range);
  if (nw > 0) k_q_codes<<<unsigned((nw + 255) / 256), 256, 0, st>>>(v, K, q, qs, words, nw);
  k_q_means<<<1, QBINS, 0, st>>>(qs, q, words + nw);
  return cuda_ok();
}

int mv_dequantize(void* stream, const uint32_t* words, int64_t K, int q, float* out) {
  if (mv_quant_stream_words(K, q) < 0 || !words || (K > 0 && !out) || misaligned(words, 4) || misaligned(out, 4))
    return MV_ERR_INVALID_ARG;
  if (K == 0) return MV_OK;
  int64_t nw = (K * q + 31) / 32;
  k_dequant<<<unsigned((K + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(words, K, q, nw, out);
  return cuda_ok();
}

}  // extern "C"
