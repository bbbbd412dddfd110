// Majority-vote sparse DSGD step (Algorithm 1 of arXiv 2011.06495) for sm_100a.
//
// N workers are the rows of one N x d array.  A step is a short sequence of kernels on
// one stream, with no host synchronisation and no device allocation:
//
//   sample     k_sample_hist                  a strided sample of |grads+err| per worker gives a
//                                             lower bound tau_n on the K-th largest magnitude key
//   stream     k_acc_compact                  the one pass over N x d: acc = err + grads written in
//                                             place, elements with key >= tau_n compacted per chunk
//   select     k_select_cluster               a thread-block cluster per worker: exact K-th key T_n of the
//                                             candidates (histograms in shared memory, merged through
//                                             distributed shared memory), or of the full row for a worker
//                                             whose candidate count missed [K, cap]; tie order per chunk
//                                             for workers whose threshold ties are only partly kept; all
//                                             CTAs first clear the bit masks and the vote bytes
//   pick       k_set_bits                     every pick sets its bit in the worker's mask and adds one
//                                             to its coordinate's vote byte (L2 atomics)
//   mask       k_vote_hist, k_vote_write      counting select over vote values 0..N: per-chunk vote
//                                             histograms, v*, output offsets; then supp(M) ascending
//   lists      k_chunk_popc, k_scan_sel, k_lists   ascending per-worker index lists from the masks (side stream)
//   aggregate  k_gather                       mean on the shared mask, residual zeroed in place
//
// With threshold tracking the sample is skipped after the first call: while a call resolves its
// K-th key, the same counts locate a slightly larger rank, and that key is the next call's tau_n.
// MV_MODE_GENERAL (no sampling) fuses a full radix histogram into the first pass instead and uses the
// grid-wide select kernels k_hist<1..3>, k_count, k_set_bits and the bit-sliced vote count k_votes.
// The variants select in "list mode" over explicit (key, index) lists: add-drop voting (k_ad_fill,
// a cluster per list, k_ad_apply; Algorithm 2) and random selection proportional to the votes
// (k_rs_fill, the grid-wide select kernels over its one long list; Algorithm 1, second variant).  A rank that holds only some of the workers gets
// binary64 partial sums from k_gather and finishes with k_finish_mean.
//
// The magnitude order is the order of key(x) = bits(x) & 0x7fffffff; ties go to the lowest index.
#include <cuda_runtime.h>
#include <cooperative_groups.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <math.h>
#include <mutex>
#include <new>

#include "../../include/mv_sparse.h"

namespace {

constexpr int CH = 4096;             // coordinates per chunk (row-relative, so chunks are mask-word aligned)
constexpr int WPC = CH / 32;         // mask words per chunk
constexpr int TPB = 256;             // threads per CTA of the chunk kernels
constexpr int SB_BINS = 8192;        // sample histogram: top 13 bits of the 31-bit key
constexpr int SB_SHIFT = 18;
constexpr int H1_BINS = 2048;        // radix digits of the 31-bit key: 11 + 10 + 10 bits
constexpr int H2_BINS = 1024;
constexpr int H3_BINS = 1024;
constexpr int WIN_SHIFT = 11;        // the select first counts the candidates in [tau, tau + 2^(11+11)) in H1_BINS bins of 2^11 keys
constexpr int WIN_LIST = 1024;       // most keys of one such bin that the select ranks directly
constexpr unsigned FULL = 0xffffffffu;

struct P {
  int N;
  int nchunks;
  int nc_pad;             // nchunks rounded up to a multiple of 8 (row pitch of chunk_vh)
  uint32_t cap;           // candidate slots per worker
  int force_general;
  int list_mode;          // 1: the rows are plain (key, index) lists to select min(K, length) from (add-drop)
  int apply_rows;         // list mode: rows < apply_rows are "add" lists, the others "drop" lists
  int take_all;           // vote_scan: the "mask" is every coordinate that holds a vote (the union of the workers' masks)
  int no_masks;           // 1: the picks only count votes; the workers' bit masks are neither cleared nor set
  const float* prefetch_acc;  // k_vote_write: if set, the rows whose elements at supp(M) the gather is about to read
  uint32_t* vote_words;   // cluster select: if set, every pick also adds one to its vote byte (four bytes per word)
  uint32_t* apply_bits;   // list mode, optional: the vote masks [apply_rows][W] to update in place instead of
                          // writing the picks to worker_bits
  int64_t d;
  int64_t K;
  int64_t W;              // mask words per row = ceil(d/32)
  uint32_t* samp_hist;    // [N][SB_BINS]
  uint32_t* hist1;        // [N][H1_BINS]
  uint32_t* hist2;        // [N][H2_BINS]
  uint32_t* hist3;        // [N][H3_BINS]
  uint32_t* cand_cnt;     // [N]
  uint32_t* sample_done;  // [N] ticket counters (last CTA of a worker finishes the job)
  uint32_t* count_done;   // [N]
  uint32_t* votes_done;   // [1]
  uint8_t* hot;           // [nc_pad] general mode: 1 if any worker picked a coordinate of the chunk
  uint32_t* vote_hist;    // [256]
  uint32_t* tau;          // [N] candidate threshold of this call
  uint32_t* tau_next;     // [N] threshold proposed for the next call (threshold tracking), or null
  uint32_t track_rank;    // rank, among this call's counted keys, at which the next call's threshold is put
  uint32_t* hist2b;       // [N][H2_BINS] second digit within the first-digit bin of track_rank (if not the K-th key's)
  uint32_t* tstate;       // [N][2] that bin and the rank within it (0 = rank not reached)
  uint32_t* diag_cnt;     // [N] copy of cand_cnt that survives the end-of-step clearing
  uint32_t* wstate;       // [N][8]: b1, rem1, b2, rem2, T, cnt_gt, cnt_eq, need
  uint32_t* thresh;       // [N][3]
  uint32_t* vstate;       // [4]: v*, cnt_gt, cnt_eq, quota
  uint2* cand;            // [N][cap] (key, index)
  uint32_t* chunk_base;   // [N][nchunks]
  uint32_t* chunk_cnt;
  uint32_t* chunk_eq;
  uint32_t* tie_base;
  uint32_t* chunk_sel;    // [N][nchunks] selected elements per chunk
  uint32_t* worker_bits;  // [N][W]
  int32_t* worker_idx;    // [N][K]
  uint8_t* votes;         // [d]
  uint16_t* chunk_vh;     // [N+1][nc_pad]: chunk_vh[v][c] = #{coordinates of chunk c with votes >= v}
  uint32_t* out_base;     // [nchunks]
  uint32_t* tie_take;     // [nchunks]
  uint32_t* dbg;          // checked build (MV_DEBUG): status word that collects MV_DBG_* bits, or null
  uint32_t* fb_total;     // running count of worker selections that went over the full row (or null)
  uint4* zero2_ptr;       // k_set_bits, optional: a region that the kernels after it (the lists of the add-drop and
  uint32_t zero2_vecs;    //   random-selection variants) want cleared, in 16-byte units (a memset between two kernels
                          //   would keep the second from being launched while the first still runs)
  int all_chunks;         // k_votes: visit every chunk, whatever p.hot says
};

// Checked build: a kernel that clamps, skips or falls back says so by setting a bit of the status word
// (never a trap or an assert: the context stays usable and the host reads the word afterwards).
#ifdef MV_DEBUG
#define MV_DBG(ptr, bit)                         \
  do {                                           \
    if ((ptr) != nullptr) atomicOr((ptr), (uint32_t)(bit)); \
  } while (0)
constexpr bool kChecked = true;
#else
#define MV_DBG(ptr, bit) \
  do {                   \
  } while (0)
constexpr bool kChecked = false;
#endif

// Programmatic dependent launch: every kernel first waits for the kernel before it on the stream
// to finish (all of its memory operations visible), then lets the kernel after it be scheduled.
// Launch latency of kernel k+1 is thereby hidden behind the execution of kernel k; the order of
// execution and the memory semantics are those of plain stream order.
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ uint32_t fkey(float x) { return __float_as_uint(x) & 0x7fffffffu; }

// one more vote for coordinate j: the vote bytes are packed four to a word and start out zero
__device__ __forceinline__ void add_vote(uint32_t* __restrict__ vote_words, uint32_t j) {
  atomicAdd(vote_words + (j >> 2), 1u << (8u * (j & 3u)));
}

// this CTA's share of clearing `nwords` 32-bit words at a 16-byte aligned address
__device__ __forceinline__ void zero_share(uint32_t* __restrict__ ptr, size_t nwords, size_t bid, size_t nblocks) {
  const size_t nvec = nwords >> 2;
  const size_t per = (nvec + nblocks - 1) / nblocks;
  const size_t v0 = bid * per, v1 = v0 + per < nvec ? v0 + per : nvec;
  uint4* q = reinterpret_cast<uint4*>(ptr);
  for (size_t i = v0 + threadIdx.x; i < v1; i += blockDim.x) q[i] = make_uint4(0, 0, 0, 0);
  if (bid == 0 && threadIdx.x < (nwords & 3)) ptr[(nvec << 2) + threadIdx.x] = 0u;
}

__device__ __forceinline__ uint32_t lanemask_lt() {
  uint32_t m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

__device__ __forceinline__ bool worker_fast(const P& p, int n) {
  if (p.force_general) return false;
  const uint32_t c = p.cand_cnt[n];
  if (p.list_mode) return c > 0 && c <= p.cap;  // a list that overflowed its room counts as empty
  return c >= (uint32_t)p.K && c <= p.cap;
}

// how many elements worker n selects: K, or in list mode min(K, length of its list)
__device__ __forceinline__ uint32_t worker_K(const P& p, int n) {
  if (!p.list_mode) return (uint32_t)p.K;
  const uint32_t c = p.cand_cnt[n];
  return c < (uint32_t)p.K ? c : (uint32_t)p.K;
}

// ---------------------------------------------------------------------------------------------
// Chunk geometry.  Chunk c of row n covers coordinates [c*CH, min(d, (c+1)*CH)).  Rows start at flat
// element n*d, which need not be a multiple of 4, so the chunk is read as the 16-byte aligned
// float4 "slots" that overlap it: slot s starts at flat element fa + 4*s, i.e. at coordinate
// j0 - h + 4*s.  Slots fully inside the chunk use vector accesses, the (at most two) partial ones
// scalar accesses restricted to the chunk's own elements.  A full chunk has 1024 slots when h == 0
// and 1025 otherwise; slot 1024 is handled by thread 255 after all others ("extra").
// ---------------------------------------------------------------------------------------------
struct Geom {
  size_t fa;
  int j0, jend, h, nslots;
};

__device__ __forceinline__ Geom chunk_geom(int n, int c, int64_t d) {
  Geom g;
  const size_t r0 = (size_t)n * (size_t)d;
  g.j0 = c * CH;
  const int64_t je = (int64_t)g.j0 + CH;
  g.jend = (int)(je < d ? je : d);
  const size_t f0 = r0 + (size_t)g.j0;
  g.fa = f0 & ~(size_t)3;
  g.h = (int)(f0 - g.fa);
  g.nslots = (g.h + (g.jend - g.j0) + 3) >> 2;
  return g;
}

// Thread (warp w, lane l) owns slots w*128 + i*32 + l, i = 0..3: a warp covers 512 consecutive
// coordinates, in index order (i, l, element).  ACC: acc = err + grads is computed and stored to err.
// t = the thread's position among the 256 that share the chunk.
template <bool ACC>
__device__ __forceinline__ void load_keys(const Geom& g, const float* __restrict__ grads, float* __restrict__ err,
                                          uint32_t (&key)[4][4], uint32_t (&vm)[4], int t = threadIdx.x) {
  const int warp = t >> 5, lane = t & 31;
  float4 ev[4], gv[4];
  int kind[4];
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const int s = warp * 128 + i * 32 + lane;
    const int jf = g.j0 - g.h + 4 * s;
    kind[i] = 0;
    if (s < g.nslots) kind[i] = (jf >= g.j0 && jf + 3 < g.jend) ? 2 : 1;
    if (kind[i] == 2) {
      const size_t f = g.fa + 4 * (size_t)s;
      ev[i] = __ldcs(reinterpret_cast<const float4*>(err + f));
      if (ACC) gv[i] = __ldcs(reinterpret_cast<const float4*>(grads + f));
    }
  }
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const int s = warp * 128 + i * 32 + lane;
    const int jf = g.j0 - g.h + 4 * s;
    const size_t f = g.fa + 4 * (size_t)s;
    vm[i] = 0;
    key[i][0] = key[i][1] = key[i][2] = key[i][3] = 0;
    if (kind[i] == 2) {
      float4 a = ev[i];
      if (ACC) {
        a.x = __fadd_rn(ev[i].x, gv[i].x);
        a.y = __fadd_rn(ev[i].y, gv[i].y);
        a.z = __fadd_rn(ev[i].z, gv[i].z);
        a.w = __fadd_rn(ev[i].w, gv[i].w);
        __stcs(reinterpret_cast<float4*>(err + f), a);
      }
      key[i][0] = fkey(a.x);
      key[i][1] = fkey(a.y);
      key[i][2] = fkey(a.z);
      key[i][3] = fkey(a.w);
      vm[i] = 0xF;
    } else if (kind[i] == 1) {
#pragma unroll
      for (int e = 0; e < 4; e++) {
        const int j = jf + e;
        if (j >= g.j0 && j < g.jend) {
          float a = err[f + e];
          if (ACC) {
            a = __fadd_rn(a, grads[f + e]);
            err[f + e] = a;
          }
          key[i][e] = fkey(a);
          vm[i] |= 1u << e;
        }
      }
    }
  }
}

// Slot 1024 (exists only when the chunk is full and h != 0); call from one thread.
template <bool ACC>
__device__ __forceinline__ void load_extra(const Geom& g, const float* __restrict__ grads, float* __restrict__ err,
                                           uint32_t (&key)[4], uint32_t& vm) {
  vm = 0;
  key[0] = key[1] = key[2] = key[3] = 0;
  if (g.nslots > 1024) {
    const int jf = g.j0 - g.h + 4096;
    const size_t f = g.fa + 4096;
#pragma unroll
    for (int e = 0; e < 4; e++) {
      const int j = jf + e;
      if (j >= g.j0 && j < g.jend) {
        float a = err[f + e];
        if (ACC) {
          a = __fadd_rn(a, grads[f + e]);
          err[f + e] = a;
        }
        key[e] = fkey(a);
        vm |= 1u << e;
      }
    }
  }
}

// Ordered rank helper: m is this lane's 4-bit element mask for one iteration.  rank0 = number of
// set bits in lower lanes (all four elements), total = set bits in the whole warp.
__device__ __forceinline__ void iter_ranks(uint32_t m, uint32_t lt, uint32_t& rank0, uint32_t& total) {
  const uint32_t b0 = __ballot_sync(FULL, m & 1u);
  const uint32_t b1 = __ballot_sync(FULL, m & 2u);
  const uint32_t b2 = __ballot_sync(FULL, m & 4u);
  const uint32_t b3 = __ballot_sync(FULL, m & 8u);
  rank0 = __popc(b0 & lt) + __popc(b1 & lt) + __popc(b2 & lt) + __popc(b3 & lt);
  total = __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
}

__device__ __forceinline__ uint32_t ge_mask(const uint32_t (&k)[4], uint32_t t) {
  return (k[0] >= t ? 1u : 0u) | (k[1] >= t ? 2u : 0u) | (k[2] >= t ? 4u : 0u) | (k[3] >= t ? 8u : 0u);
}
__device__ __forceinline__ uint32_t gt_mask(const uint32_t (&k)[4], uint32_t t) {
  return (k[0] > t ? 1u : 0u) | (k[1] > t ? 2u : 0u) | (k[2] > t ? 4u : 0u) | (k[3] > t ? 8u : 0u);
}
__device__ __forceinline__ uint32_t eq_mask(const uint32_t (&k)[4], uint32_t t) {
  return (k[0] == t ? 1u : 0u) | (k[1] == t ? 2u : 0u) | (k[2] == t ? 4u : 0u) | (k[3] == t ? 8u : 0u);
}

// Finds the bin holding the rank-th largest element of a histogram (rank counted from the top,
// 1-based): the largest bin b with sum(hist[b..]) >= rank, and rem = rank - sum(hist[b+1..]).
// All NT threads of the CTA call it; if the histogram holds fewer than rank elements, bin = rem = 0.
template <int NB, int NT>
__device__ void block_pick(const uint32_t* __restrict__ hist, uint32_t rank, uint32_t& bin, uint32_t& rem) {
  constexpr int PER = NB / NT;
  __shared__ uint32_t s_wsum[NT / 32];
  __shared__ uint32_t s_res[2];
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  uint32_t loc[PER];
  uint32_t sum = 0;
#pragma unroll
  for (int k = 0; k < PER; k++) {
    loc[k] = __ldcg(hist + t * PER + k);
    sum += loc[k];
  }
  if (t == 0) {
    s_res[0] = 0;
    s_res[1] = 0;
  }
  uint32_t x = sum;  // inclusive suffix sum within the warp
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t y = __shfl_down_sync(FULL, x, off);
    if (lane + off < 32) x += y;
  }
  if (lane == 0) s_wsum[warp] = x;
  __syncthreads();
  uint32_t above = x - sum;
  for (int w = warp + 1; w < NT / 32; w++) above += s_wsum[w];
  if (above < rank && rank <= above + sum) {
    bool done = false;
#pragma unroll
    for (int k = PER - 1; k >= 0; k--) {
      if (!done) {
        if (above + loc[k] >= rank) {
          s_res[0] = (uint32_t)(t * PER + k);
          s_res[1] = rank - above;
          done = true;
        } else {
          above += loc[k];
        }
      }
    }
  }
  __syncthreads();
  bin = s_res[0];
  rem = s_res[1];
  __syncthreads();
}

// block_pick for two ranks of the same histogram in one sweep (same contract for each rank).
template <int NB, int NT>
__device__ void block_pick2(const uint32_t* __restrict__ hist, uint32_t rank_a, uint32_t rank_b, uint32_t& bin_a,
                            uint32_t& rem_a, uint32_t& bin_b, uint32_t& rem_b) {
  constexpr int PER = NB / NT;
  __shared__ uint32_t s_wsum[NT / 32];
  __shared__ uint32_t s_res[4];
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  uint32_t loc[PER];
  uint32_t sum = 0;
#pragma unroll
  for (int k = 0; k < PER; k++) {
    loc[k] = __ldcg(hist + t * PER + k);
    sum += loc[k];
  }
  if (t < 4) s_res[t] = 0;
  uint32_t x = sum;  // inclusive suffix sum within the warp
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t y = __shfl_down_sync(FULL, x, off);
    if (lane + off < 32) x += y;
  }
  if (lane == 0) s_wsum[warp] = x;
  __syncthreads();
  uint32_t above0 = x - sum;
  for (int w = warp + 1; w < NT / 32; w++) above0 += s_wsum[w];
#pragma unroll
  for (int which = 0; which < 2; which++) {
    const uint32_t rank = which ? rank_b : rank_a;
    uint32_t above = above0;
    if (above < rank && rank <= above + sum) {
      bool done = false;
#pragma unroll
      for (int k = PER - 1; k >= 0; k--) {
        if (!done) {
          if (above + loc[k] >= rank) {
            s_res[2 * which] = (uint32_t)(t * PER + k);
            s_res[2 * which + 1] = rank - above;
            done = true;
          } else {
            above += loc[k];
          }
        }
      }
    }
  }
  __syncthreads();
  bin_a = s_res[0];
  rem_a = s_res[1];
  bin_b = s_res[2];
  rem_b = s_res[3];
  __syncthreads();
}

// Exclusive prefix sum over the threads of a CTA (NT = 256 or 1024); `total` gets the CTA sum.
template <int NT>
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* s_w /*NT/32 + 1*/, uint32_t& total) {
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  uint32_t x = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t y = __shfl_up_sync(FULL, x, off);
    if (lane >= off) x += y;
  }
  __syncthreads();  // protects s_w against a previous use
  if (lane == 31) s_w[warp] = x;
  __syncthreads();
  uint32_t base = 0;
  uint32_t tot = 0;
  for (int w = 0; w < NT / 32; w++) {
    const uint32_t sw = s_w[w];
    if (w < warp) base += sw;
    tot += sw;
  }
  total = tot;
  return base + x - v;
}

// ticket: true in every thread of the last CTA of the grid to call it (all threads must call)
__device__ __forceinline__ bool last_cta(uint32_t* counter, uint32_t total) {
  __shared__ uint32_t s_last_flag;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last_flag = (atomicAdd(counter, 1u) == total - 1) ? 1u : 0u;
  __syncthreads();
  const bool last = s_last_flag != 0;
  if (last) __threadfence();
  return last;
}

// ---------------------------------------------------------------------------------------------
// sample: histogram of the top 13 key bits over evenly spaced 32-element lines of each row; the
// last CTA of a worker to finish turns it into tau_n = lower edge of the bin that holds the
// rank-th largest sampled key (a ticket counter, no waiting)
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512) k_sample_hist(P p, const float* __restrict__ grads,
                                                     const float* __restrict__ err, uint32_t U, uint32_t L, int all,
                                                     uint32_t rank) {
  pdl_enter();
  __shared__ uint32_t sh[SB_BINS];
  __shared__ uint32_t s_last;
  const int n = blockIdx.y;
  for (int b = threadIdx.x; b < SB_BINS; b += 512) sh[b] = 0;
  __syncthreads();
  const size_t r0 = (size_t)n * (size_t)p.d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t u0 = (blockIdx.x * 16u + warp) * 8u; u0 < U; u0 += gridDim.x * 128u) {
    float a[8];
    bool ok[8];
#pragma unroll
    for (int q = 0; q < 8; q++) {  // sixteen loads in flight per lane
      const uint32_t u = u0 + q;
      ok[q] = false;
      a[q] = 0.f;
      if (u < U) {
        const uint32_t line = all ? u : u * L;  // L = line stride
        const int64_t j = (int64_t)line * 32 + lane;
        if (j < p.d) {
          ok[q] = true;
          a[q] = __fadd_rn(__ldcs(err + r0 + j), __ldcs(grads + r0 + j));
        }
      }
    }
#pragma unroll
    for (int q = 0; q < 8; q++)
      if (ok[q]) atomicAdd(&sh[fkey(a[q]) >> SB_SHIFT], 1u);
  }
  __syncthreads();
  uint32_t* gh = p.samp_hist + (size_t)n * SB_BINS;
  for (int b = threadIdx.x; b < SB_BINS; b += 512) {
    const uint32_t v = sh[b];
    if (v) atomicAdd(&gh[b], v);
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = (atomicAdd(&p.sample_done[n], 1u) == gridDim.x - 1) ? 1u : 0u;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  uint32_t bin, rem;
  block_pick<SB_BINS, 512>(gh, rank, bin, rem);
  if (threadIdx.x == 0) p.tau[n] = bin << SB_SHIFT;
}

// ---------------------------------------------------------------------------------------------
// stream: acc = err + grads in place; elements with key >= tau_n appended, in index order, to the
// chunk's own run of the worker's candidate buffer (one global atomic per chunk that has any)
// ---------------------------------------------------------------------------------------------
// Writes this thread's candidates at CTA-local positions off + (ordered rank) through `put(pos, entry)`.
template <typename PUT>
__device__ __forceinline__ void emit_candidates(const Geom& g, const uint32_t (&key)[4][4], const uint32_t (&cm)[4],
                                                const uint32_t (&xkey)[4], uint32_t xcm, const uint32_t* s_w, PUT put) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint32_t off = 0;
  for (int w = 0; w < warp; w++) off += s_w[w];
  const uint32_t lt = lanemask_lt();
#pragma unroll
  for (int i = 0; i < 4; i++) {
    uint32_t rank0, tot;
    iter_ranks(cm[i], lt, rank0, tot);
    if (cm[i]) {
      const int jf = g.j0 - g.h + 4 * (warp * 128 + i * 32 + lane);
#pragma unroll
      for (int e = 0; e < 4; e++)
        if (cm[i] & (1u << e)) put(off + rank0 + __popc(cm[i] & ((1u << e) - 1u)), make_uint2(key[i][e], (uint32_t)(jf + e)));
    }
    off += tot;
  }
  if (threadIdx.x == TPB - 1 && xcm) {
    uint32_t xoff = 0;
    for (int w = 0; w < 8; w++) xoff += s_w[w];
    const int jf = g.j0 - g.h + 4096;
#pragma unroll
    for (int e = 0; e < 4; e++)
      if (xcm & (1u << e)) put(xoff + __popc(xcm & ((1u << e) - 1u)), make_uint2(xkey[e], (uint32_t)(jf + e)));
  }
}

__global__ void __launch_bounds__(TPB, 4) k_acc_compact(P p, const float* __restrict__ grads, float* __restrict__ err) {
  pdl_enter();
  constexpr uint32_t QCAP = 1024;  // candidates of a chunk staged in shared memory (more: written directly)
  __shared__ uint32_t s_w[9];
  __shared__ uint32_t s_base;
  __shared__ uint2 s_q[QCAP];
  const int n = blockIdx.y, c = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const Geom g = chunk_geom(n, c, p.d);
  const uint32_t tau = p.tau[n];
  uint32_t key[4][4], vm[4], cm[4];
  load_keys<true>(g, grads, err, key, vm);
  uint32_t xkey[4] = {0, 0, 0, 0}, xcm = 0;
  if (threadIdx.x == TPB - 1) {
    uint32_t xvm;
    load_extra<true>(g, grads, err, xkey, xvm);
    xcm = xvm & ge_mask(xkey, tau);
  }
  uint32_t wsum = 0;
#pragma unroll
  for (int i = 0; i < 4; i++) {
    cm[i] = vm[i] & ge_mask(key[i], tau);
    wsum += __popc(cm[i]);
  }
  wsum = __reduce_add_sync(FULL, wsum);
  if (lane == 0) s_w[warp] = wsum;
  if (threadIdx.x == TPB - 1) s_w[8] = __popc(xcm);
  __syncthreads();
  uint32_t total = 0;
#pragma unroll
  for (int w = 0; w < 9; w++) total += s_w[w];
  // the chunk's run in the worker's candidate buffer: one reservation per chunk that has any,
  // issued now and consumed after the staging, so that its round trip overlaps with it
  uint32_t base_r = 0;
  if (threadIdx.x == 0) {
    if (total) base_r = atomicAdd(&p.cand_cnt[n], total);
    p.chunk_cnt[(size_t)n * p.nchunks + c] = total;
    if (total == 0) p.chunk_base[(size_t)n * p.nchunks + c] = 0;
  }
  if (total == 0) return;  // uniform over the CTA
  uint2* out = p.cand + (size_t)n * p.cap;
  if (total <= QCAP) {
    // stage in index order, then copy out coalesced: whole sectors instead of 8-byte pieces
    emit_candidates(g, key, cm, xkey, xcm, s_w, [&](uint32_t pos, uint2 v) { s_q[pos] = v; });
    if (threadIdx.x == 0) {
      s_base = base_r;
      p.chunk_base[(size_t)n * p.nchunks + c] = base_r;
    }
    __syncthreads();
    const uint32_t base = s_base;
    for (uint32_t i = threadIdx.x; i < total; i += TPB) {
      if (base + i < p.cap) out[base + i] = s_q[i];
      else MV_DBG(p.dbg, MV_DBG_CAND_OVERFLOW);
    }
  } else {
    if (threadIdx.x == 0) {
      s_base = base_r;
      p.chunk_base[(size_t)n * p.nchunks + c] = base_r;
    }
    __syncthreads();
    const uint32_t base = s_base;
    const uint32_t cap = p.cap;
    emit_candidates(g, key, cm, xkey, xcm, s_w, [&](uint32_t pos, uint2 v) {
      if (base + pos < cap) out[base + pos] = v;
      else MV_DBG(p.dbg, MV_DBG_CAND_OVERFLOW);
    });
  }
}

// ---------------------------------------------------------------------------------------------
// exact K-th key by radix select (11 + 10 + 10 bits).  Pass q first resolves digit q-1 from the
// previous pass's histogram (every CTA repeats that small scan; CTA 0 records it), then counts
// digit q among the elements whose higher digits match.
// ---------------------------------------------------------------------------------------------
template <int PASS>
__device__ __forceinline__ uint32_t resolve_prefix(const P& p, int n, uint32_t& track_bin) {
  uint32_t* ws = p.wstate + (size_t)n * 8;
  track_bin = 0xffffffffu;  // no second tracked bin unless pass 2 finds one
  if (PASS == 2) {
    uint32_t b1, rem1;
    if (p.tau_next == nullptr) {
      block_pick<H1_BINS, TPB>(p.hist1 + (size_t)n * H1_BINS, worker_K(p, n), b1, rem1);
    } else {
      // threshold tracking: the next call's candidate threshold is put at rank K + margin among the
      // keys counted in this call (the candidates, or the whole row).  This pass finds the first
      // digit of that rank; the second digit is counted alongside the K-th key's.
      uint32_t tb, trem;
      block_pick2<H1_BINS, TPB>(p.hist1 + (size_t)n * H1_BINS, worker_K(p, n), p.track_rank, b1, rem1, tb, trem);
      if (blockIdx.x == 0 && threadIdx.x == 0) {
        p.tstate[n * 2 + 0] = tb;
        p.tstate[n * 2 + 1] = trem;
      }
      if (trem != 0 && tb != b1) track_bin = tb;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      ws[0] = b1;
      ws[1] = rem1;
    }
    return b1;
  }
  if (PASS == 3) {
    const uint32_t b1 = ws[0], rem1 = ws[1];
    uint32_t b2, rem2;
    // threshold tracking: CTA 0 also settles the next call's threshold (second digit of its rank)
    const bool settle = p.tau_next != nullptr && blockIdx.x == 0;  // CTA-uniform
    uint32_t tb = 0, trem = 0, tb2 = 0, trem2 = 0;
    if (settle) {
      tb = p.tstate[n * 2 + 0];
      trem = p.tstate[n * 2 + 1];
    }
    if (settle && trem != 0 && tb == b1) {  // the usual case: both ranks in the same first-digit bin
      block_pick2<H2_BINS, TPB>(p.hist2 + (size_t)n * H2_BINS, rem1, trem, b2, rem2, tb2, trem2);
    } else {
      block_pick<H2_BINS, TPB>(p.hist2 + (size_t)n * H2_BINS, rem1, b2, rem2);
      if (settle && trem != 0) block_pick<H2_BINS, TPB>(p.hist2b + (size_t)n * H2_BINS, trem, tb2, trem2);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      ws[2] = b2;
      ws[3] = rem2;
      if (settle) {
        uint32_t next = (tb << 20) | (tb2 << 10);
        if (trem == 0) {
          // The counted keys (c candidates, all >= tau) do not reach the rank: go below tau by linear
          // extrapolation in key space from the two ranks that are known, (K, K-th key) and (c, tau),
          // with a quarter to spare; at least 2^10 and at most half a first-digit bin per call.
          const uint32_t tau = p.tau[n], c = p.cand_cnt[n], K = worker_K(p, n);
          const uint32_t t21 = (b1 << 20) | (b2 << 10);
          const float slope = (t21 > tau && c >= K) ? (float)(t21 - tau) / (float)(c - K + 1u) : 0.f;
          float drop = 1.25f * slope * (float)(p.track_rank > c ? p.track_rank - c : 1u);
          drop = fminf(fmaxf(drop, 1024.f), 524288.f);
          next = tau > (uint32_t)drop ? tau - (uint32_t)drop : 0u;
        }
        p.tau_next[n] = next;
      }
    }
    return (b1 << 10) | b2;
  }
  return 0;
}

// Last digit: T_n, cnt_gt, cnt_eq and the tie quota `need` (how many elements equal to T_n are
// kept); every thread gets T, need and cnt_eq, CTA 0 records them.
__device__ __forceinline__ uint32_t resolve_threshold(const P& p, int n, uint32_t& need, uint32_t& cnt_eq) {
  uint32_t* ws = p.wstate + (size_t)n * 8;
  const uint32_t b1 = ws[0], b2 = ws[2], rem2 = ws[3];
  uint32_t b3, rem3;
  block_pick<H3_BINS, TPB>(p.hist3 + (size_t)n * H3_BINS, rem2, b3, rem3);
  const uint32_t T = (b1 << 20) | (b2 << 10) | b3;
  cnt_eq = __ldcg(p.hist3 + (size_t)n * H3_BINS + b3);
  need = rem3;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    const uint32_t cnt_gt = worker_K(p, n) - rem3;
    ws[4] = T;
    ws[5] = cnt_gt;
    ws[6] = cnt_eq;
    ws[7] = rem3;
    p.thresh[n * 3 + 0] = T;
    p.thresh[n * 3 + 1] = cnt_gt;
    p.thresh[n * 3 + 2] = cnt_eq;
  }
  return T;
}

template <int PASS>
__device__ __forceinline__ void hist_add(uint32_t* sh, uint32_t key, uint32_t prefix, uint32_t* sh2, uint32_t track_bin) {
  if (PASS == 1) {
    atomicAdd(&sh[key >> 20], 1u);
  } else if (PASS == 2) {
    if ((key >> 20) == prefix) atomicAdd(&sh[(key >> 10) & 1023u], 1u);
    else if ((key >> 20) == track_bin) atomicAdd(&sh2[(key >> 10) & 1023u], 1u);
  } else {
    if ((key >> 10) == prefix) atomicAdd(&sh[key & 1023u], 1u);
  }
}

template <int PASS>
__device__ __forceinline__ uint32_t* hist_of(const P& p, int n) {
  if (PASS == 1) return p.hist1 + (size_t)n * H1_BINS;
  if (PASS == 2) return p.hist2 + (size_t)n * H2_BINS;
  return p.hist3 + (size_t)n * H3_BINS;
}

// Histogram pass PASS for worker blockIdx.y.  A worker whose candidate count landed in [K, cap]
// ("fast") is counted over its candidate buffer; any other worker over its full row (read back
// from err, which holds acc by now).  FUSED (PASS 1 only) instead reads grads and err, writes acc
// and counts every element: the first pass when sampling is switched off.
template <int PASS, bool FUSED>
__global__ void __launch_bounds__(TPB) k_hist(P p, const float* __restrict__ grads, float* __restrict__ err) {
  pdl_enter();
  constexpr int NB = PASS == 1 ? H1_BINS : H2_BINS;
  __shared__ uint32_t sh[NB];
  const int n = blockIdx.y;
  const bool fast = !FUSED && worker_fast(p, n);
  if (p.list_mode && !fast) return;  // empty list
  __shared__ uint32_t sh2[PASS == 2 ? H2_BINS : 1];
  uint32_t track_bin;
  const uint32_t prefix = resolve_prefix<PASS>(p, n, track_bin);
  for (int b = threadIdx.x; b < NB; b += TPB) sh[b] = 0;
  if (PASS == 2 && track_bin != 0xffffffffu)
    for (int b = threadIdx.x; b < H2_BINS; b += TPB) sh2[b] = 0;
  __syncthreads();
  if (fast) {
    const uint32_t cnt = p.cand_cnt[n];
    const uint2* cd = p.cand + (size_t)n * p.cap;
    const uint32_t stride = gridDim.x * TPB;
    const uint32_t lane = threadIdx.x & 31;
    for (uint32_t b0 = blockIdx.x * TPB + (threadIdx.x & ~31u); b0 < cnt; b0 += 4 * stride) {  // warp-uniform
      uint32_t k[4];
#pragma unroll
      for (int q = 0; q < 4; q++) {
        const uint32_t i = b0 + q * stride + lane;
        k[q] = i < cnt ? __ldcg(&cd[i].x) : 0u;
      }
#pragma unroll
      for (int q = 0; q < 4; q++) {
        if (b0 + q * stride >= cnt) break;  // warp-uniform
        if (b0 + q * stride + lane < cnt) hist_add<PASS>(sh, k[q], prefix, sh2, track_bin);
      }
    }
  } else {
    for (int c = blockIdx.x; c < p.nchunks; c += gridDim.x) {
      const Geom g = chunk_geom(n, c, p.d);
      uint32_t key[4][4], vm[4];
      load_keys<FUSED>(g, grads, err, key, vm);
      if (FUSED && threadIdx.x < WPC) {  // the worker's mask starts out empty
        const int64_t wi = (int64_t)c * WPC + threadIdx.x;
        if (wi < p.W) p.worker_bits[(size_t)n * p.W + wi] = 0u;
      }
#pragma unroll
      for (int i = 0; i < 4; i++)
#pragma unroll
        for (int e = 0; e < 4; e++)
          if (vm[i] & (1u << e)) hist_add<PASS>(sh, key[i][e], prefix, sh2, track_bin);
      if (threadIdx.x == TPB - 1) {
        uint32_t xkey[4], xvm;
        load_extra<FUSED>(g, grads, err, xkey, xvm);
#pragma unroll
        for (int e = 0; e < 4; e++)
          if (xvm & (1u << e)) hist_add<PASS>(sh, xkey[e], prefix, sh2, track_bin);
      }
    }
  }
  __syncthreads();
  uint32_t* gh = hist_of<PASS>(p, n);
  for (int b = threadIdx.x; b < NB; b += TPB) {
    const uint32_t v = sh[b];
    if (v) atomicAdd(&gh[b], v);
  }
  if (PASS == 2 && track_bin != 0xffffffffu) {
    uint32_t* gh2 = p.hist2b + (size_t)n * H2_BINS;
    for (int b = threadIdx.x; b < H2_BINS; b += TPB) {
      const uint32_t v = sh2[b];
      if (v) atomicAdd(&gh2[b], v);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// order: per worker, the number of threshold ties before each chunk (tie_base); a tie is kept if
// its rank in index order is below the worker's quota
// ---------------------------------------------------------------------------------------------
template <int NT>
__device__ void chunk_scan(const P& p, int n) {
  __shared__ uint32_t s_w[NT / 32 + 1];
  const int per = (p.nchunks + NT - 1) / NT;
  const int c0 = min(p.nchunks, (int)threadIdx.x * per), c1 = min(p.nchunks, c0 + per);
  const size_t rb = (size_t)n * p.nchunks;
  uint32_t esum = 0;
  for (int c = c0; c < c1; c++) esum += __ldcg(p.chunk_eq + rb + c);
  uint32_t tot;
  uint32_t run = block_excl_scan<NT>(esum, s_w, tot);
  for (int c = c0; c < c1; c++) {
    p.tie_base[rb + c] = run;
    run += __ldcg(p.chunk_eq + rb + c);
  }
}

// Resolves T_n for every worker.  A worker that keeps only part of its threshold ties also needs
// the ties per chunk: counted from its candidates, or from its full row; the last CTA of the worker
// to finish turns the counts into running offsets.
__global__ void __launch_bounds__(TPB) k_count(P p, float* __restrict__ err) {
  pdl_enter();
  __shared__ uint32_t s_e[TPB / 32];
  const int n = blockIdx.y;
  if (p.list_mode && !worker_fast(p, n)) return;  // empty list
  uint32_t need, cnt_eq;
  const uint32_t T = resolve_threshold(p, n, need, cnt_eq);
  if (need >= cnt_eq) return;  // every tie is kept: no order needed (uniform over the worker's CTAs)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (worker_fast(p, n)) {
    const uint2* cd = p.cand + (size_t)n * p.cap;
    for (int c = blockIdx.x * (TPB / 32) + warp; c < p.nchunks; c += gridDim.x * (TPB / 32)) {
      const size_t ci = (size_t)n * p.nchunks + c;
      const uint32_t cnt = p.chunk_cnt[ci], base = p.chunk_base[ci];
      uint32_t eq = 0;
      for (uint32_t i = lane; i < cnt; i += 32) eq += __ldcg(&cd[base + i].x) == T;
      eq = __reduce_add_sync(FULL, eq);
      if (lane == 0) p.chunk_eq[ci] = eq;
    }
  } else {
    for (int c = blockIdx.x; c < p.nchunks; c += gridDim.x) {
      const Geom g = chunk_geom(n, c, p.d);
      uint32_t key[4][4], vm[4];
      load_keys<false>(g, nullptr, err, key, vm);
      uint32_t eq = 0;
#pragma unroll
      for (int i = 0; i < 4; i++) eq += __popc(vm[i] & eq_mask(key[i], T));
      if (threadIdx.x == TPB - 1) {
        uint32_t xkey[4], xvm;
        load_extra<false>(g, nullptr, err, xkey, xvm);
        eq += __popc(xvm & eq_mask(xkey, T));
      }
      eq = __reduce_add_sync(FULL, eq);
      __syncthreads();
      if (lane == 0) s_e[warp] = eq;
      __syncthreads();
      if (threadIdx.x == 0) {
        uint32_t te = 0;
        for (int w = 0; w < TPB / 32; w++) te += s_e[w];
        p.chunk_eq[(size_t)n * p.nchunks + c] = te;
      }
    }
  }
  if (last_cta(p.count_done + n, gridDim.x)) chunk_scan<TPB>(p, n);
}

// v* = the vote value of the K-th most voted coordinate; then per chunk the output offset and the
// number of v*-ties it may keep (lowest index first).  Run by the last CTA that finished the
// per-chunk vote histograms; all NT threads of that CTA call it.
template <int NT>
__device__ void vote_scan(const P& p) {
  __shared__ uint32_t s_w[NT / 32 + 1];
  __shared__ uint32_t s_v[4];
  __shared__ uint32_t s_h[256];
  for (int v = threadIdx.x; v <= p.N; v += NT) s_h[v] = v ? __ldcg(p.vote_hist + v) : 0u;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t voted = 0;
    for (int v = 1; v <= p.N; v++) voted += s_h[v];
    s_h[0] = (uint32_t)p.d - voted;  // coordinates nobody voted for
    uint32_t acc = 0, vstar = 0, cgt = 0, ceq = 0, total = (uint32_t)p.K;
    if (p.take_all) {  // every voted coordinate: "votes >= 1", all ties at one vote kept
      vstar = 1;
      ceq = s_h[1];
      cgt = voted - ceq;
      total = voted;
    } else {
      for (int v = p.N; v >= 0; v--) {
        const uint32_t h = s_h[v];
        if (acc + h >= (uint32_t)p.K) {
          vstar = (uint32_t)v;
          cgt = acc;
          ceq = h;
          break;
        }
        acc += h;
      }
    }
    s_v[0] = vstar;
    s_v[1] = total;
    s_v[3] = total - cgt;
    p.vstate[0] = vstar;
    p.vstate[1] = cgt;
    p.vstate[2] = ceq;
    p.vstate[3] = total - cgt;
  }
  __syncthreads();
  const uint32_t vstar = s_v[0], quota = s_v[3], n_out = s_v[1];
  // Tiles of NT*8 chunks, a thread taking 8 neighbouring chunks of a tile (one 16-byte load per
  // count array); the loads of TB tiles are issued together, then every tile costs two block scans.
  // ecarry / scarry: v*-ties seen and outputs placed in the tiles before.
  const uint16_t* hge = p.chunk_vh + (size_t)vstar * p.nc_pad;                                   // votes >= v*
  const uint16_t* hgt = (int)vstar < p.N ? p.chunk_vh + (size_t)(vstar + 1) * p.nc_pad : nullptr;  // votes > v*
  constexpr int TB = 4;
  uint32_t ecarry = 0, scarry = 0;
  for (int c00 = 0; c00 < p.nc_pad; c00 += NT * 8 * TB) {  // uniform over the CTA
    uint4 av[TB], gv[TB];
#pragma unroll
    for (int k = 0; k < TB; k++) {
      const int c = c00 + (k * NT + (int)threadIdx.x) * 8;
      av[k] = make_uint4(0, 0, 0, 0);
      gv[k] = make_uint4(0, 0, 0, 0);
      if (c < p.nc_pad) {
        av[k] = __ldcg(reinterpret_cast<const uint4*>(hge + c));
        if (hgt) gv[k] = __ldcg(reinterpret_cast<const uint4*>(hgt + c));
      }
    }
#pragma unroll
    for (int k = 0; k < TB; k++) {
      if (c00 + k * NT * 8 >= p.nc_pad) break;  // uniform over the CTA
      const int c = c00 + (k * NT + (int)threadIdx.x) * 8;
      const uint32_t aw[4] = {av[k].x, av[k].y, av[k].z, av[k].w}, gw[4] = {gv[k].x, gv[k].y, gv[k].z, gv[k].w};
      uint32_t eqv[8], gtv[8], esum = 0, gsum = 0;
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const uint32_t ge = (aw[q >> 1] >> (16 * (q & 1))) & 0xffffu, gt = (gw[q >> 1] >> (16 * (q & 1))) & 0xffffu;
        const bool in = c + q < p.nchunks;
        eqv[q] = in ? ge - gt : 0u;
        gtv[q] = in ? gt : 0u;
        esum += eqv[q];
        gsum += gtv[q];
      }
      uint32_t etot, stot;
      const uint32_t epre = ecarry + block_excl_scan<NT>(esum, s_w, etot);
      const uint32_t taken_before = epre < quota ? epre : quota;           // ties kept in earlier chunks
      const uint32_t taken_here = min(epre + esum, quota) - taken_before;  // ties kept in this thread's chunks
      const uint32_t spre = scarry + block_excl_scan<NT>(gsum + taken_here, s_w, stot);
      // eight neighbouring chunks per thread: their results go out as 16-byte stores (the arrays are
      // padded to whole groups of eight; the slot after the last chunk holds K, the end of the output)
      uint32_t run = epre, srun = spre, tk[8], ob[8];
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const uint32_t take = run >= quota ? 0u : min(eqv[q], quota - run);
        tk[q] = take;
        ob[q] = c + q == p.nchunks ? n_out : srun;
        run += eqv[q];
        srun += gtv[q] + take;
      }
      if (c < p.nc_pad) {
        uint4* tt = reinterpret_cast<uint4*>(p.tie_take + c);
        uint4* oo = reinterpret_cast<uint4*>(p.out_base + c);
        tt[0] = make_uint4(tk[0], tk[1], tk[2], tk[3]);
        tt[1] = make_uint4(tk[4], tk[5], tk[6], tk[7]);
        oo[0] = make_uint4(ob[0], ob[1], ob[2], ob[3]);
        oo[1] = make_uint4(ob[4], ob[5], ob[6], ob[7]);
      }
      ecarry += etot;
      scarry += stot;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) p.out_base[p.nchunks] = n_out;  // sentinel: end of the last chunk
}

// s_vh[v] (v >= 1) holds how many coordinates of chunk c got exactly v votes.  Stores, per chunk,
// the cumulative counts cum[v] = #{votes >= v} (v = 0..N) and adds the exact counts to the global
// histogram.  All threads of the CTA call it.
__device__ __forceinline__ void store_vote_hist_impl(const P& p, int c, uint32_t* s_vh) {
  for (int t = threadIdx.x; t <= p.N; t += blockDim.x) {
    const int64_t rem = p.d - (int64_t)c * CH;
    const uint32_t valid = (uint32_t)(rem < CH ? rem : CH);
    uint32_t ge = 0;  // coordinates with votes >= max(t, 1)
    for (int v = max(t, 1); v <= p.N; v++) ge += s_vh[v];
    uint32_t exact;
    if (t == 0) {
      exact = valid - ge;
      ge = valid;
    } else {
      exact = s_vh[t];
    }
    p.chunk_vh[(size_t)t * p.nc_pad + c] = (uint16_t)ge;
    if (exact && t > 0) atomicAdd(&p.vote_hist[t], exact);  // the zero-vote count is derived later
  }
}

// ---------------------------------------------------------------------------------------------
// vote.  (1) k_set_bits: every worker's candidate buffer is walked flat (balanced however the
// candidates cluster); a thread takes 8 consecutive candidates, which are index-sorted within a
// chunk's run and so mostly share a mask word, merges their bits and ORs each word into the
// worker's global bit mask (zeroed by the streaming pass).  (2) k_tie_bits: workers that keep only
// part of their threshold ties add those, lowest index first.  (3) k_votes: one CTA per chunk adds
// the N masks bit-sliced (8 counter planes per 32-coordinate word) into the vote count.
// ---------------------------------------------------------------------------------------------
// Puts the picked bits `bits` of mask word w of row n where they belong: into the row's bit mask, or
// (add-drop, in-place update) into the vote mask, set for an "add" row and cleared for a "drop" row.
__device__ __forceinline__ void put_bits(const P& p, int n, uint32_t w, uint32_t bits) {
  if (p.no_masks) return;
  if (kChecked && (int64_t)w >= p.W) {
    MV_DBG(p.dbg, MV_DBG_INTERNAL);
    return;
  }
  if (p.apply_bits == nullptr) {
    atomicOr(p.worker_bits + (size_t)n * p.W + w, bits);
  } else if (n < p.apply_rows) {
    atomicOr(p.apply_bits + (size_t)n * p.W + w, bits);
  } else {
    atomicAnd(p.apply_bits + (size_t)(n - p.apply_rows) * p.W + w, ~bits);
  }
}

// The picks of a worker whose K-th key was found over its full row, read off the row itself (err holds acc):
// every element above T_n, and the threshold ties -- all of them, or (ordered = !all_ties) those whose rank in
// index order over the whole row, tie_base[chunk] + rank inside the chunk, is below `need`.  The calling CTA has
// NSUB x 256 threads; each group of 256 takes one chunk at a time: chunks c_first + sub, + c_stride, ...
// All threads of the CTA must call it (it synchronises the CTA).
template <int NSUB>
__device__ __forceinline__ void fullrow_picks(const P& p, int n, float* __restrict__ err, uint32_t T, uint32_t need,
                                              bool all_ties, int c_first, int c_stride, uint32_t (*s_we)[9]) {
  uint32_t* bits_row = p.worker_bits + (size_t)n * p.W;
  const int sub = threadIdx.x >> 8, t = threadIdx.x & 255;
  const int warp = t >> 5, lane = t & 31;
  const uint32_t lt = lanemask_lt();
  for (int c0 = c_first; c0 < p.nchunks; c0 += c_stride) {  // uniform over the CTA
    const int c = c0 + sub;
    const bool valid = c < p.nchunks;
    Geom g = chunk_geom(n, valid ? c : 0, p.d);
    uint32_t key[4][4], vm[4], em[4], sm[4];
    uint32_t xkey[4] = {0, 0, 0, 0}, xvm = 0, xem = 0, xsm = 0;
    if (valid) {
      load_keys<false>(g, nullptr, err, key, vm, t);
      if (t == TPB - 1) {
        load_extra<false>(g, nullptr, err, xkey, xvm);
        xem = xvm & eq_mask(xkey, T);
      }
    } else {
#pragma unroll
      for (int i = 0; i < 4; i++) {
        vm[i] = 0;
        key[i][0] = key[i][1] = key[i][2] = key[i][3] = 0;
      }
    }
#pragma unroll
    for (int i = 0; i < 4; i++) em[i] = vm[i] & eq_mask(key[i], T);
    if (all_ties) {
#pragma unroll
      for (int i = 0; i < 4; i++) sm[i] = (vm[i] & gt_mask(key[i], T)) | em[i];
      if (t == TPB - 1) xsm = (xvm & gt_mask(xkey, T)) | xem;
    } else {
      // keep the threshold ties whose rank (in index order, over the whole row) is below `need`
      uint32_t weq = 0;
#pragma unroll
      for (int i = 0; i < 4; i++) weq += __popc(em[i]);
      weq = __reduce_add_sync(FULL, weq);
      __syncthreads();  // previous chunk's readers of s_we are done
      if (lane == 0) s_we[sub][warp] = weq;
      if (t == TPB - 1) s_we[sub][8] = __popc(xem);
      __syncthreads();
      const uint32_t tb = valid ? p.tie_base[(size_t)n * p.nchunks + c] : 0u;
      uint32_t eoff = tb;
      for (int w = 0; w < warp; w++) eoff += s_we[sub][w];
#pragma unroll
      for (int i = 0; i < 4; i++) {
        uint32_t rank0, tot;
        iter_ranks(em[i], lt, rank0, tot);
        uint32_t take = 0;
#pragma unroll
        for (int e = 0; e < 4; e++) {
          if (em[i] & (1u << e)) {
            const uint32_t r = eoff + rank0 + __popc(em[i] & ((1u << e) - 1u));
            if (r < need) take |= 1u << e;
          }
        }
        sm[i] = (vm[i] & gt_mask(key[i], T)) | take;
        eoff += tot;
      }
      if (t == TPB - 1) {
        uint32_t xoff = tb;
        for (int w = 0; w < 8; w++) xoff += s_we[sub][w];
        uint32_t take = 0;
#pragma unroll
        for (int e = 0; e < 4; e++) {
          if (xem & (1u << e)) {
            const uint32_t r = xoff + __popc(xem & ((1u << e) - 1u));
            if (r < need) take |= 1u << e;
          }
        }
        xsm = (xvm & gt_mask(xkey, T)) | take;
      }
    }
    bool any = false;
#pragma unroll
    for (int i = 0; i < 4; i++) {
      if (sm[i]) {
        any = true;
        const int jf = g.j0 - g.h + 4 * (warp * 128 + i * 32 + lane);
#pragma unroll
        for (int e = 0; e < 4; e++)
          if (sm[i] & (1u << e)) {
            if (!p.no_masks) atomicOr(bits_row + ((uint32_t)(jf + e) >> 5), 1u << ((uint32_t)(jf + e) & 31u));
            if (p.vote_words) add_vote(p.vote_words, (uint32_t)(jf + e));
          }
      }
    }
    if (xsm) {
      any = true;
      const int jf = g.j0 - g.h + 4096;
#pragma unroll
      for (int e = 0; e < 4; e++)
        if (xsm & (1u << e)) {
          if (!p.no_masks) atomicOr(bits_row + ((uint32_t)(jf + e) >> 5), 1u << ((uint32_t)(jf + e) & 31u));
          if (p.vote_words) add_vote(p.vote_words, (uint32_t)(jf + e));
        }
    }
    if (any && valid) p.hot[c] = 1;  // same value from every thread
  }
}

__global__ void __launch_bounds__(TPB) k_set_bits(P p, float* __restrict__ err) {
  pdl_enter();
  __shared__ uint32_t s_we[1][9];
  if (p.zero2_ptr != nullptr) {
    const uint32_t nthreads = gridDim.x * gridDim.y * TPB;
    for (uint32_t i = (blockIdx.y * gridDim.x + blockIdx.x) * TPB + threadIdx.x; i < p.zero2_vecs; i += nthreads)
      p.zero2_ptr[i] = make_uint4(0, 0, 0, 0);
  }
  const int n = blockIdx.y;
  const bool fast = worker_fast(p, n);
  if (p.list_mode && !fast) {  // empty list
    if (kChecked && blockIdx.x == 0 && threadIdx.x == 0 && p.cand_cnt[n] > p.cap) MV_DBG(p.dbg, MV_DBG_LIST_OVERFLOW);
    return;
  }
  if (!fast && !p.force_general && blockIdx.x == 0 && threadIdx.x == 0) {
    MV_DBG(p.dbg, MV_DBG_FALLBACK);
    if (p.fb_total != nullptr) atomicAdd(p.fb_total, 1u);
  }
  const uint32_t* ws = p.wstate + (size_t)n * 8;
  const uint32_t T = ws[4], need = ws[7];
  const bool all_ties = need >= ws[6];
  if (blockIdx.x == 0 && threadIdx.x == 0) p.diag_cnt[n] = p.cand_cnt[n];
  if (!fast) {
    // full-row worker: its picks are read off the row itself (err holds acc), chunk by chunk
    fullrow_picks<1>(p, n, err, T, need, all_ties, blockIdx.x, gridDim.x, s_we);
    return;
  }
  const uint32_t cnt = p.cand_cnt[n];
  const uint2* cd = p.cand + (size_t)n * p.cap;  // cap is a multiple of 8: rows are 64-byte aligned
  for (uint32_t i0 = (blockIdx.x * TPB + threadIdx.x) * 8u; i0 < cnt; i0 += gridDim.x * TPB * 8u) {
    uint4 v[4];
#pragma unroll
    for (int q = 0; q < 4; q++) v[q] = __ldcg(reinterpret_cast<const uint4*>(cd + i0) + q);
    uint32_t curw = 0xffffffffu, acc = 0;
#pragma unroll
    for (int q = 0; q < 8; q++) {
      const uint32_t key = (q & 1) ? v[q >> 1].z : v[q >> 1].x;
      const uint32_t j = (q & 1) ? v[q >> 1].w : v[q >> 1].y;
      const bool sel = i0 + q < cnt && (key > T || (key == T && all_ties));
      if (kChecked && sel && (int64_t)j >= p.d) MV_DBG(p.dbg, MV_DBG_PICK_RANGE);
      if (sel && (int64_t)j < p.d) {
        const uint32_t w = j >> 5;
        if (w != curw) {
          if (acc) put_bits(p, n, curw, acc);
          curw = w;
          acc = 0;
        }
        acc |= 1u << (j & 31u);
        if (p.vote_words) add_vote(p.vote_words, j);
      }
    }
    if (acc) put_bits(p, n, curw, acc);
  }
  // a worker that keeps only part of its threshold ties adds them chunk by chunk, lowest index first
  if (all_ties) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t lt = lanemask_lt();
  for (int c = blockIdx.x * (TPB / 32) + warp; c < p.nchunks; c += gridDim.x * (TPB / 32)) {
    const size_t ci = (size_t)n * p.nchunks + c;
    const uint32_t ccnt = p.chunk_cnt[ci];
    uint32_t run = p.tie_base[ci];
    if (ccnt == 0 || run >= need) continue;
    const uint2* cc = cd + p.chunk_base[ci];
    for (uint32_t i0 = 0; i0 < ccnt && run < need; i0 += 32) {
      const uint32_t i = i0 + lane;
      uint2 kv = make_uint2(0, 0);
      bool eq = false;
      if (i < ccnt) {
        kv = __ldcg(cc + i);
        eq = kv.x == T;
      }
      const uint32_t eb = __ballot_sync(FULL, eq);
      if (eq && run + __popc(eb & lt) < need && (int64_t)kv.y < p.d) {
        put_bits(p, n, kv.y >> 5, 1u << (kv.y & 31u));
        if (p.vote_words) add_vote(p.vote_words, kv.y);
      }
      run += __popc(eb);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// select + vote bits in one kernel: a thread-block cluster per worker.  The cluster's CTAs split the
// worker's candidate buffer, keep their keys in shared memory, count each radix digit (11 + 10 + 10
// bits) into a local shared-memory histogram and, after a cluster barrier, read one another's
// histograms through distributed shared memory; every CTA thus resolves the digit by itself and no
// histogram leaves the SMs.  With T_n known the same CTAs set the worker's mask bits.  A worker whose
// candidate count missed [K, cap] is counted over its full row by the same cluster, and a worker that
// keeps only part of its threshold ties orders them per chunk as k_count / k_set_bits do.
// Every condition under which a cluster barrier is reached depends only on values that all CTAs of
// the cluster compute alike (the candidate count and the merged histograms).
// ---------------------------------------------------------------------------------------------
namespace cg = cooperative_groups;

// CL = CTAs of the cluster that serves one worker: 8 (the portable maximum), or 4 when there are so many
// workers that clusters of 8 would not all be resident at once
constexpr int ST = 1024;        // threads per CTA
constexpr int SK_KEYS = 32768;  // candidate keys a CTA keeps in shared memory between the digit passes

// block_pick2 over a histogram in shared memory, ST threads; rank 0 = not asked (bin = rem = 0)
template <int NB>
__device__ void smem_pick2(const uint32_t* s_hist, uint32_t rank_a, uint32_t rank_b, uint32_t& bin_a, uint32_t& rem_a,
                           uint32_t& bin_b, uint32_t& rem_b) {
  constexpr int PER = NB / ST;
  __shared__ uint32_t s_wsum[ST / 32];
  __shared__ uint32_t s_res[4];
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  uint32_t loc[PER];
  uint32_t sum = 0;
#pragma unroll
  for (int k = 0; k < PER; k++) {
    loc[k] = s_hist[t * PER + k];
    sum += loc[k];
  }
  if (t < 4) s_res[t] = 0;
  uint32_t x = sum;  // inclusive suffix sum within the warp
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t y = __shfl_down_sync(FULL, x, off);
    if (lane + off < 32) x += y;
  }
  if (lane == 0) s_wsum[warp] = x;
  __syncthreads();
  uint32_t above0 = x - sum;
  for (int w = warp + 1; w < ST / 32; w++) above0 += s_wsum[w];
#pragma unroll
  for (int which = 0; which < 2; which++) {
    const uint32_t rank = which ? rank_b : rank_a;
    uint32_t above = above0;
    if (above < rank && rank <= above + sum) {
      bool done = false;
#pragma unroll
      for (int k = PER - 1; k >= 0; k--) {
        if (!done) {
          if (above + loc[k] >= rank) {
            s_res[2 * which] = (uint32_t)(t * PER + k);
            s_res[2 * which + 1] = rank - above;
            done = true;
          } else {
            above += loc[k];
          }
        }
      }
    }
  }
  __syncthreads();
  bin_a = s_res[0];
  rem_a = s_res[1];
  bin_b = s_res[2];
  rem_b = s_res[3];
  __syncthreads();
}

// s_out[b] = sum over the cluster's CTAs of their s_local[b]
template <int NB, int CL>
__device__ __forceinline__ void cluster_merge(cg::cluster_group& cluster, uint32_t* s_local, uint32_t* s_out) {
  const uint32_t* peer[CL];
#pragma unroll
  for (int r = 0; r < CL; r++) peer[r] = cluster.map_shared_rank(s_local, r);
  for (int b = threadIdx.x; b < NB; b += ST) {
    uint32_t v[CL];
#pragma unroll
    for (int r = 0; r < CL; r++) v[r] = peer[r][b];
    uint32_t sum = 0;
#pragma unroll
    for (int r = 0; r < CL; r++) sum += v[r];
    s_out[b] = sum;
  }
  __syncthreads();
}

// f(key) for every element of the chunks of row n that fall to CTA `rank` of the cluster: four
// chunks at a time, 256 threads each
template <int CL, typename F>
__device__ __forceinline__ void cluster_row_keys(const P& p, int n, float* __restrict__ err, uint32_t rank, F f) {
  const int sub = threadIdx.x >> 8, t = threadIdx.x & 255;
  for (int c = (int)rank * 4 + sub; c < p.nchunks; c += CL * 4) {
    const Geom g = chunk_geom(n, c, p.d);
    uint32_t key[4][4], vm[4];
    load_keys<false>(g, nullptr, err, key, vm, t);
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
      for (int e = 0; e < 4; e++)
        if (vm[i] & (1u << e)) f(key[i][e]);
    if (t == TPB - 1) {
      uint32_t xkey[4], xvm;
      load_extra<false>(g, nullptr, err, xkey, xvm);
#pragma unroll
      for (int e = 0; e < 4; e++)
        if (xvm & (1u << e)) f(xkey[e]);
    }
  }
}

template <int CL>
__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(ST, 1) k_select_cluster(P p, float* __restrict__ err, int zero_first, int n_select) {
  pdl_enter();
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ uint32_t s_keys[];       // [SK_KEYS]
  __shared__ uint32_t s_h[3][H1_BINS];       // this CTA's digit counts; pass 2: [0,1024) K-th key's bin, [1024,2048) tracked bin
  __shared__ uint32_t s_m[H1_BINS];          // the same counts summed over the cluster
  __shared__ uint32_t s_te[4][9];
  __shared__ uint32_t s_ws[ST / 32];
  __shared__ uint32_t s_res3[3];
  __shared__ uint32_t s_hw[H1_BINS];         // window counts of this CTA's slice
  {
    // The workers' bit masks and the vote count start out empty.  They are cleared here, by all CTAs
    // of the grid together, and not in the streaming pass: what is written now is still in L2 when
    // the picks arrive as atomics (k_set_bits), whereas lines cleared before the row streamed through
    // would each have to come back from DRAM.  Clusters beyond the workers' only clear.
    // Clusters zero_first and up take part: all of them, or only the extra ones when those are many.
    if ((int)blockIdx.y >= zero_first) {
      const size_t nblocks = (size_t)gridDim.x * (gridDim.y - zero_first);
      const size_t bid = (size_t)(blockIdx.y - zero_first) * gridDim.x + blockIdx.x;
      if (!p.no_masks) zero_share(p.worker_bits, (size_t)p.N * (size_t)p.W, bid, nblocks);
      if (p.vote_words != nullptr) zero_share(p.vote_words, (size_t)p.nchunks * (CH / 4), bid, nblocks);
    }
  }
  if ((int)blockIdx.y >= n_select) return;  // alike in every CTA of the cluster (n_select: workers selected here)
  const int n = blockIdx.y;
  const uint32_t rank = cluster.block_rank();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int b = tid; b < 3 * H1_BINS; b += ST) (&s_h[0][0])[b] = 0;
  __syncthreads();
  const uint32_t cnt = p.cand_cnt[n];
  const bool fast = worker_fast(p, n);  // alike in every CTA of the cluster
  if (p.list_mode && !fast) return;     // an empty list (or one that overflowed its room) selects nothing
  const uint32_t K = worker_K(p, n);    // list mode: min(K, length of the list)
  const bool tracking = p.tau_next != nullptr;
  const uint2* cd = p.cand + (size_t)n * p.cap;
  // this CTA's slice of the candidate buffer
  const uint32_t per = (cnt + CL - 1) / CL;
  const uint32_t s0 = min(cnt, rank * per);
  const uint32_t len = fast ? min(cnt, s0 + per) - s0 : 0u;

  // ---- the usual case: the K-th key lies in a window of 2^22 keys above tau_n ----
  uint32_t T = 0, need = 0, cnt_eq = 0;
  bool resolved = false;  // alike in every CTA of the cluster
  if (fast && !p.list_mode) {  // (a list has no threshold bound: its keys go straight to the three digits)
    const uint32_t tau = p.tau[n];
    uint32_t wsum = 0;
    for (int b = tid; b < H1_BINS; b += ST) s_hw[b] = 0;
    __syncthreads();
    for (uint32_t l0 = 0; l0 < len; l0 += ST * 8) {  // uniform over the CTA
      uint32_t k[8];
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const uint32_t li = l0 + q * ST + tid;
        k[q] = li < len ? __ldcg(&cd[s0 + li].x) : 0u;
      }
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const uint32_t li = l0 + q * ST + tid;
        if (li < len) {
          if (li < SK_KEYS) s_keys[li] = k[q];
          const uint32_t wb = (k[q] - tau) >> WIN_SHIFT;
          if (wb < (uint32_t)H1_BINS) atomicAdd(&s_hw[wb], 1u);
        }
      }
    }
    cluster.sync();
    {
      const uint32_t* peer[CL];
#pragma unroll
      for (int r = 0; r < CL; r++) peer[r] = cluster.map_shared_rank(s_hw, r);
      for (int b = tid; b < H1_BINS; b += ST) {
        uint32_t v = 0;
#pragma unroll
        for (int r = 0; r < CL; r++) v += peer[r][b];
        s_m[b] = v;
        wsum += v;
      }
    }
    wsum = __reduce_add_sync(FULL, wsum);
    if (lane == 0) s_ws[warp] = wsum;
    __syncthreads();
    uint32_t win_total = 0;
    for (int w = 0; w < ST / 32; w++) win_total += s_ws[w];
    const uint32_t above = cnt - win_total;  // candidates beyond the window
    if (K > above) {
      uint32_t bw, rem, bt, trem_w;
      const uint32_t rt = (tracking && p.track_rank > above && p.track_rank <= cnt) ? p.track_rank - above : 0u;
      smem_pick2<H1_BINS>(s_m, K - above, rt, bw, rem, bt, trem_w);
      // the keys of that bin go to a short list
      uint32_t* lcnt = p.hist3 + (size_t)n * H3_BINS;
      uint32_t* list = p.hist2 + (size_t)n * H2_BINS;
      for (uint32_t li = tid; li < len; li += ST) {
        const uint32_t kk = li < SK_KEYS ? s_keys[li] : __ldcg(&cd[s0 + li].x);
        if (((kk - tau) >> WIN_SHIFT) == bw) {
          const uint32_t at = atomicAdd(lcnt, 1u);
          if (at < (uint32_t)WIN_LIST) list[at] = kk;
          else MV_DBG(p.dbg, MV_DBG_WINDOW_OVERFLOW);
        }
      }
      __threadfence();
      cluster.sync();
      const uint32_t m = __ldcg(lcnt);
      if (m <= (uint32_t)WIN_LIST) {
        resolved = true;
        // rank the list: T_n is its rem-th largest key
        uint32_t mine = 0;
        if ((uint32_t)tid < m) {
          mine = __ldcg(list + tid);
          s_m[tid] = mine;
        }
        __syncthreads();
        if ((uint32_t)tid < m) {
          uint32_t gt = 0, eq = 0;
          for (uint32_t i = 0; i < m; i++) {
            const uint32_t o = s_m[i];
            gt += o > mine;
            eq += o == mine;
          }
          if (gt < rem && rem <= gt + eq) {  // every thread that holds T_n writes the same values
            s_res3[0] = mine;
            s_res3[1] = rem - gt;
            s_res3[2] = eq;
          }
        }
        __syncthreads();
        T = s_res3[0];
        need = s_res3[1];
        cnt_eq = s_res3[2];
        if (tracking && rank == 0 && tid == 0) {
          uint32_t next = tau + (bt << WIN_SHIFT);
          if (trem_w == 0) {
            // the candidates do not reach the tracked rank: go below tau by linear extrapolation in
            // key space from (K, T_n) and (cnt, tau), a quarter to spare, between 2^10 and 2^19 per call
            const float slope = T > tau ? (float)(T - tau) / (float)(cnt - K + 1u) : 0.f;
            float drop = 1.25f * slope * (float)(p.track_rank > cnt ? p.track_rank - cnt : 1u);
            drop = fminf(fmaxf(drop, 1024.f), 524288.f);
            next = tau > (uint32_t)drop ? tau - (uint32_t)drop : 0u;
          }
          p.tau_next[n] = next;
        }
      }
    }
  }
  if (!resolved) {
  // ---- digit 1 ----
  if (fast) {
    for (uint32_t l0 = 0; l0 < len; l0 += ST * 8) {  // uniform over the CTA
      uint32_t k[8];
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const uint32_t li = l0 + q * ST + tid;
        k[q] = li < len ? __ldcg(&cd[s0 + li].x) : 0u;
      }
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const uint32_t li = l0 + q * ST + tid;
        const bool ok = li < len;
        const uint32_t act = __ballot_sync(FULL, ok);
        if (ok) {
          if (li < SK_KEYS) s_keys[li] = k[q];
          // keys just above a threshold share a few leading digits: one shared-memory atomic per
          // distinct digit of the warp instead of one per lane
          const uint32_t bin = k[q] >> 20;
          const uint32_t same = __match_any_sync(act, bin);
          if (lane == __ffs(same) - 1) atomicAdd(&s_h[0][bin], (uint32_t)__popc(same));
        }
      }
    }
  } else {
    cluster_row_keys<CL>(p, n, err, rank, [&](uint32_t key) { atomicAdd(&s_h[0][key >> 20], 1u); });
  }
  cluster.sync();
  cluster_merge<H1_BINS, CL>(cluster, s_h[0], s_m);
  uint32_t b1, rem1, tb, trem;
  smem_pick2<H1_BINS>(s_m, K, tracking ? p.track_rank : 0u, b1, rem1, tb, trem);
  const uint32_t track_bin = (tracking && trem != 0 && tb != b1) ? tb : 0xffffffffu;

  // ---- digit 2 (and, with threshold tracking, the second digit of the tracked rank) ----
  auto add2 = [&](uint32_t key) {
    const uint32_t d1 = key >> 20;
    if (d1 == b1) atomicAdd(&s_h[1][(key >> 10) & 1023u], 1u);
    else if (d1 == track_bin) atomicAdd(&s_h[1][1024u + ((key >> 10) & 1023u)], 1u);
  };
  if (fast) {
    for (uint32_t li = tid; li < len; li += ST) add2(li < SK_KEYS ? s_keys[li] : __ldcg(&cd[s0 + li].x));
  } else {
    cluster_row_keys<CL>(p, n, err, rank, add2);
  }
  cluster.sync();
  cluster_merge<H1_BINS, CL>(cluster, s_h[1], s_m);
  uint32_t b2, rem2, tb2 = 0, trem2 = 0;
  if (tracking && trem != 0 && tb == b1) {  // the usual case: both ranks in the same first-digit bin
    smem_pick2<H2_BINS>(s_m, rem1, trem, b2, rem2, tb2, trem2);
  } else {
    uint32_t u0, u1;
    smem_pick2<H2_BINS>(s_m, rem1, 0u, b2, rem2, u0, u1);
    if (tracking && trem != 0) smem_pick2<H2_BINS>(s_m + 1024, trem, 0u, tb2, trem2, u0, u1);
  }
  if (tracking && rank == 0 && tid == 0) {
    uint32_t next = (tb << 20) | (tb2 << 10);
    if (trem == 0) {
      // the counted keys do not reach the tracked rank: go below tau by linear extrapolation in key
      // space from (K, K-th key) and (cnt, tau), a quarter to spare, between 2^10 and 2^19 per call
      const uint32_t tau = p.tau[n];
      const uint32_t t21 = (b1 << 20) | (b2 << 10);
      const float slope = (t21 > tau && cnt >= K) ? (float)(t21 - tau) / (float)(cnt - K + 1u) : 0.f;
      float drop = 1.25f * slope * (float)(p.track_rank > cnt ? p.track_rank - cnt : 1u);
      drop = fminf(fmaxf(drop, 1024.f), 524288.f);
      next = tau > (uint32_t)drop ? tau - (uint32_t)drop : 0u;
    }
    p.tau_next[n] = next;
  }

  // ---- digit 3 ----
  const uint32_t prefix = (b1 << 10) | b2;
  auto add3 = [&](uint32_t key) {
    if ((key >> 10) == prefix) atomicAdd(&s_h[2][key & 1023u], 1u);
  };
  if (fast) {
    for (uint32_t li = tid; li < len; li += ST) add3(li < SK_KEYS ? s_keys[li] : __ldcg(&cd[s0 + li].x));
  } else {
    cluster_row_keys<CL>(p, n, err, rank, add3);
  }
  cluster.sync();
  cluster_merge<H3_BINS, CL>(cluster, s_h[2], s_m);
  uint32_t b3, u0, u1;
  smem_pick2<H3_BINS>(s_m, rem2, 0u, b3, need, u0, u1);
  cnt_eq = s_m[b3];
  T = (b1 << 20) | (b2 << 10) | b3;
  cluster.sync();  // from here on no CTA reads a peer's shared memory
  }
  if (rank == 0 && tid == 0) {
    uint32_t* ws = p.wstate + (size_t)n * 8;
    ws[4] = T;
    ws[5] = K - need;
    ws[6] = cnt_eq;
    ws[7] = need;
    p.thresh[n * 3 + 0] = T;
    p.thresh[n * 3 + 1] = K - need;
    p.thresh[n * 3 + 2] = cnt_eq;
    p.diag_cnt[n] = cnt;
  }
  const bool all_ties = need >= cnt_eq;  // alike in every CTA of the cluster

  if (fast) {
    // the picks themselves are made by k_set_bits, which follows; a worker that keeps only part of its
    // threshold ties (lowest index first) needs the ties per chunk and their running offsets for that
    if (all_ties) return;
    for (int c = (int)rank * (ST / 32) + warp; c < p.nchunks; c += CL * (ST / 32)) {
      const size_t ci = (size_t)n * p.nchunks + c;
      const uint32_t ccnt = p.chunk_cnt[ci], base = p.chunk_base[ci];
      uint32_t eq = 0;
      for (uint32_t i = lane; i < ccnt; i += 32) eq += __ldcg(&cd[base + i].x) == T;
      eq = __reduce_add_sync(FULL, eq);
      if (lane == 0) p.chunk_eq[ci] = eq;
    }
    __threadfence();
    cluster.sync();
    if (rank == 0) chunk_scan<ST>(p, n);
    return;
  }

  // ---- full-row worker: its picks are read off the row itself by k_set_bits; partly kept ties need
  // the ties per chunk and their running offsets ----
  if (all_ties) return;
  const int sub = tid >> 8, t = tid & 255, w8 = t >> 5;
  for (int c0 = (int)rank * 4; c0 < p.nchunks; c0 += CL * 4) {  // uniform over the CTA
    const int c = c0 + sub;
    const bool valid = c < p.nchunks;
    uint32_t eq = 0;
    if (valid) {
      const Geom g = chunk_geom(n, c, p.d);
      uint32_t key[4][4], vm[4];
      load_keys<false>(g, nullptr, err, key, vm, t);
#pragma unroll
      for (int i = 0; i < 4; i++) eq += __popc(vm[i] & eq_mask(key[i], T));
      if (t == TPB - 1) {
        uint32_t xkey[4], xvm;
        load_extra<false>(g, nullptr, err, xkey, xvm);
        eq += __popc(xvm & eq_mask(xkey, T));
      }
    }
    eq = __reduce_add_sync(FULL, eq);
    if (lane == 0) s_te[sub][w8] = eq;
    __syncthreads();
    if (valid && t == 0) {
      uint32_t te = 0;
      for (int w = 0; w < 8; w++) te += s_te[sub][w];
      p.chunk_eq[(size_t)n * p.nchunks + c] = te;
    }
    __syncthreads();
  }
  __threadfence();
  cluster.sync();
  if (rank == 0) chunk_scan<ST>(p, n);
}

constexpr int VT = 128;  // threads of k_votes: one per mask word of the chunk

// Chunks in which no worker kept a candidate are skipped: their votes, selected counts and vote
// histograms were cleared at the start of the step.  NP = number of counter planes (2^NP > N).
template <int NP>
__global__ void __launch_bounds__(VT) k_votes(P p) {
  pdl_enter();
  __shared__ uint32_t s_vh[256];
  __shared__ uint32_t s_sel[256];
  const int tid = threadIdx.x, lane = tid & 31;
  for (int c = blockIdx.x; c < p.nchunks; c += gridDim.x) {
    if (!p.all_chunks && __ldcg(p.hot + c) == 0) continue;  // uniform over the CTA
    __syncthreads();                       // previous chunk's readers are done
    s_vh[tid] = 0;
    s_vh[tid + VT] = 0;
    s_sel[tid] = 0;
    s_sel[tid + VT] = 0;
    __syncthreads();
    const int64_t jb = (int64_t)c * CH + (int64_t)tid * 32;
    const int64_t wi = (int64_t)c * WPC + tid;
    uint32_t planes[NP];
#pragma unroll
    for (int q = 0; q < NP; q++) planes[q] = 0;
    const bool inb = wi < p.W;
    const uint32_t* col = p.worker_bits + (inb ? wi : 0);
    for (int n0 = 0; n0 < p.N; n0 += 8) {
      uint32_t w[8];
#pragma unroll
      for (int q = 0; q < 8; q++) w[q] = (inb && n0 + q < p.N) ? __ldcg(col + (size_t)(n0 + q) * p.W) : 0u;
#pragma unroll
      for (int q = 0; q < 8; q++) {
        uint32_t carry = w[q];
        if (n0 + q < p.N) {  // uniform
          const uint32_t pc = __reduce_add_sync(FULL, (uint32_t)__popc(carry));
          if (lane == 0 && pc) atomicAdd(&s_sel[n0 + q], pc);
        }
#pragma unroll
        for (int r = 0; r < NP; r++) {
          const uint32_t t2 = planes[r] & carry;
          planes[r] ^= carry;
          carry = t2;
        }
      }
    }
    uint32_t any = 0;
#pragma unroll
    for (int q = 0; q < NP; q++) any |= planes[q];
    // histogram of the vote values of this chunk: for each value v, the coordinates whose bit-sliced
    // counter equals v are one AND over the planes away (no per-coordinate atomics)
    if (__ballot_sync(FULL, any != 0)) {  // warp-uniform
      uint32_t valid = 0xffffffffu;       // coordinates of this word that lie below d
      if (jb >= p.d) valid = 0;
      else if (jb + 32 > p.d) valid = (1u << (uint32_t)(p.d - jb)) - 1u;
      for (int v = 1; v <= p.N; v++) {
        uint32_t m = valid;
#pragma unroll
        for (int q = 0; q < NP; q++) m &= ((v >> q) & 1) ? planes[q] : ~planes[q];
        const uint32_t cnt = __reduce_add_sync(FULL, (uint32_t)__popc(m));
        if (lane == 0 && cnt) atomicAdd(&s_vh[v], cnt);
      }
    }
    // expand the planes into 32 vote bytes per thread: a nibble of plane q becomes bit q of four bytes
    if (jb < p.d) {
      uint32_t wv[8];
#pragma unroll
      for (int g = 0; g < 8; g++) {
        uint32_t x = 0;
        if (any) {
#pragma unroll
          for (int q = 0; q < NP; q++) x |= ((((planes[q] >> (4 * g)) & 0xfu) * 0x00204081u) & 0x01010101u) << q;
        }
        wv[g] = x;
      }
      if (jb + 32 <= p.d) {
        uint4* dst = reinterpret_cast<uint4*>(p.votes + jb);
        dst[0] = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        dst[1] = make_uint4(wv[4], wv[5], wv[6], wv[7]);
      } else {
        for (int b = 0; b < 32 && jb + b < p.d; b++) p.votes[jb + b] = (uint8_t)((wv[b >> 2] >> (8 * (b & 3))) & 0xffu);
      }
    }
    __syncthreads();
    for (int n = tid; n < p.N; n += VT) p.chunk_sel[(size_t)n * p.nchunks + c] = s_sel[n];
    store_vote_hist_impl(p, c, s_vh);
  }
  if (last_cta(p.votes_done, gridDim.x)) vote_scan<VT>(p);
}

// per worker: list offset of every chunk = exclusive prefix of the selected counts
__global__ void __launch_bounds__(1024) k_scan_sel(P p) {
  pdl_enter();
  __shared__ uint32_t s_w[33];
  const int n = blockIdx.x;
  const int per = (p.nchunks + 1023) / 1024;
  const int c0 = min(p.nchunks, (int)threadIdx.x * per), c1 = min(p.nchunks, c0 + per);
  const size_t rb = (size_t)n * p.nchunks;
  uint32_t sum = 0;
  for (int c = c0; c < c1; c++) sum += p.chunk_sel[rb + c];
  uint32_t tot;
  uint32_t run = block_excl_scan<1024>(sum, s_w, tot);
  for (int c = c0; c < c1; c++) {
    const uint32_t v = p.chunk_sel[rb + c];
    p.chunk_sel[rb + c] = run;  // in place: count -> offset
    run += v;
  }
}

// ascending index lists from the bit masks: a warp per (worker, chunk).  In round q lane l owns mask
// word 32*q + l; its set bits are staged in shared memory in order and copied out coalesced.
__global__ void __launch_bounds__(TPB) k_lists(P p) {
  pdl_enter();
  __shared__ uint16_t s_buf[TPB / 32][1024];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = blockIdx.y;
  const int c = blockIdx.x + warp * gridDim.x;  // neighbouring chunks go to different CTAs
  if (c >= p.nchunks) return;
  const uint32_t next = c + 1 < p.nchunks ? p.chunk_sel[(size_t)n * p.nchunks + c + 1] : (uint32_t)p.K;
  uint32_t pos = p.chunk_sel[(size_t)n * p.nchunks + c];
  if (next == pos) return;  // nothing selected in this chunk (warp-uniform)
  uint32_t m[4];
#pragma unroll
  for (int q = 0; q < 4; q++) {
    const int64_t wi = (int64_t)c * WPC + q * 32 + lane;
    m[q] = wi < p.W ? __ldcg(p.worker_bits + (size_t)n * p.W + wi) : 0u;
  }
  int32_t* lst = p.worker_idx + (size_t)n * p.K;
  uint16_t* buf = s_buf[warp];
#pragma unroll
  for (int q = 0; q < 4; q++) {
    const uint32_t pc = __popc(m[q]);
    uint32_t x = pc;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t y = __shfl_up_sync(FULL, x, off);
      if (lane >= off) x += y;
    }
    const uint32_t tot = __shfl_sync(FULL, x, 31);
    uint32_t o = x - pc;
    uint32_t mm = m[q];
    while (mm) {
      const int b = __ffs(mm) - 1;
      mm &= mm - 1;
      buf[o++] = (uint16_t)((q * 32 + lane) * 32 + b);
    }
    __syncwarp();
    for (uint32_t t = lane; t < tot; t += 32) {
      if (pos + t < (uint32_t)p.K) lst[pos + t] = c * CH + (int)buf[t];
      else MV_DBG(p.dbg, MV_DBG_LIST_RANGE);
    }
    __syncwarp();
    pos += tot;
  }
}

// ---------------------------------------------------------------------------------------------
// mask: counting select over the vote values 0..N
// ---------------------------------------------------------------------------------------------
// per-chunk and global histogram of vote values, from a vote vector (stand-alone mv_select)
// `copy` (optional): the votes are also written there (the caller's array, when the count was kept elsewhere).
// A warp per chunk: its 4096 vote bytes are eight 16-byte loads per lane, all in flight together, and
// nothing in a chunk's path waits for another warp; the CTA's eight chunks share one flush of the
// global counts and one ticket.
constexpr int VH_WARPS = TPB / 32;

// Vote counts of chunk c from its 4096 vote bytes, held by a warp as eight 16-byte pieces per lane: stores
// chunk_vh[v][c] = #{votes >= v} for v = 0..N and adds the exact counts #{votes == v}, v >= 1, to s_tot (shared
// memory).  #{votes >= v} comes from byte-wise compares over the lane's registers, summed over the warp: no
// per-coordinate atomics, however the votes crowd.  With N <= 127 a compare of four bytes is one subtraction:
// with bit 7 of every byte set beforehand, (byte | 0x80) - v keeps bit 7 exactly when byte >= v, and no borrow
// leaves its byte; the kept bits are added up per byte lane over the 32 words (at most 32 each) and summed once.
// The count is the same in all lanes, so the loop may stop for the whole warp once it reaches zero (the rows
// above are then written as zeros).  All 32 lanes call it.  (The votes are not needed afterwards: q is changed.)
__device__ __forceinline__ void chunk_vote_counts(const P& p, int c, uint4 (&q)[8], int lane, uint32_t* s_tot) {
  const int64_t remd = p.d - (int64_t)c * CH;
  uint32_t prev = (uint32_t)(remd < CH ? remd : CH);  // #{votes >= 0}: every coordinate of the chunk
  if (lane == 0) p.chunk_vh[c] = (uint16_t)prev;
  const bool narrow = p.N <= 127;
  if (narrow) {
#pragma unroll
    for (int u = 0; u < 8; u++) {
      q[u].x |= 0x80808080u;
      q[u].y |= 0x80808080u;
      q[u].z |= 0x80808080u;
      q[u].w |= 0x80808080u;
    }
  }
  int v = 1;
  for (; v <= p.N; v++) {
    const uint32_t v4 = (uint32_t)v * 0x01010101u;
    uint32_t cnt = 0;
    if (narrow) {
      uint32_t lanes4 = 0;  // four byte-wide counters
#pragma unroll
      for (int u = 0; u < 8; u++) {
        lanes4 += ((q[u].x - v4) & 0x80808080u) >> 7;
        lanes4 += ((q[u].y - v4) & 0x80808080u) >> 7;
        lanes4 += ((q[u].z - v4) & 0x80808080u) >> 7;
        lanes4 += ((q[u].w - v4) & 0x80808080u) >> 7;
      }
      cnt = (lanes4 * 0x01010101u) >> 24;
    } else {
#pragma unroll
      for (int u = 0; u < 8; u++) {
        const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
        for (int i = 0; i < 4; i++)
          if (w[i]) cnt += __popc(__vcmpgeu4(w[i], v4)) >> 3;  // (eight bits per matching byte)
      }
    }
    cnt = __reduce_add_sync(FULL, cnt);
    if (lane == 0) {
      p.chunk_vh[(size_t)v * p.nc_pad + c] = (uint16_t)cnt;
      if (v > 1 && prev != cnt) atomicAdd(&s_tot[v - 1], prev - cnt);  // coordinates with exactly v - 1 votes
    }
    prev = cnt;
    if (cnt == 0) break;
  }
  if (v > p.N) {
    if (lane == 0 && prev) atomicAdd(&s_tot[p.N], prev);  // exactly N votes (or more, if the input breaks its contract)
  } else {
    for (int z = v + 1 + lane; z <= p.N; z += 32) p.chunk_vh[(size_t)z * p.nc_pad + c] = 0;
  }
}

__global__ void __launch_bounds__(TPB) k_vote_hist(P p, const uint8_t* __restrict__ votes, uint8_t* __restrict__ copy) {
  pdl_enter();
  __shared__ uint32_t s_tot[256];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int c = blockIdx.x * VH_WARPS + warp;
  s_tot[tid] = 0;
  __syncthreads();
  if (c < p.nchunks) {
    uint4 q[8];
#pragma unroll
    for (int u = 0; u < 8; u++) {
      const int64_t jb = (int64_t)c * CH + (int64_t)(u * 32 + lane) * 16;
      q[u] = make_uint4(0, 0, 0, 0);
      if (jb + 16 <= p.d) {
        q[u] = __ldcg(reinterpret_cast<const uint4*>(votes + jb));
      } else if (jb < p.d) {  // the row's last, partial 16 bytes
        uint32_t w[4] = {0, 0, 0, 0};
        for (int b = 0; b < 16 && jb + b < p.d; b++) w[b >> 2] |= (uint32_t)__ldcg(votes + jb + b) << (8 * (b & 3));
        q[u] = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
#pragma unroll
    for (int u = 0; u < 8; u++) {
      const int64_t jb = (int64_t)c * CH + (int64_t)(u * 32 + lane) * 16;
      const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
      if (copy != nullptr) {
        if (jb + 16 <= p.d) {
          *reinterpret_cast<uint4*>(copy + jb) = q[u];
        } else {
          for (int b = 0; b < 16 && jb + b < p.d; b++) copy[jb + b] = (uint8_t)((w[b >> 2] >> (8 * (b & 3))) & 0xffu);
        }
      }
    }
    chunk_vote_counts(p, c, q, lane, s_tot);
  }
  __syncthreads();
  if (tid >= 1 && tid <= p.N && s_tot[tid]) atomicAdd(&p.vote_hist[tid], s_tot[tid]);  // the zero-vote count is derived later
  if (last_cta(p.votes_done, gridDim.x)) vote_scan<TPB>(p);
}

// writes supp(M) (ascending) and optionally M as a bit mask
__global__ void __launch_bounds__(TPB) k_vote_write(P p, const uint8_t* __restrict__ votes, int32_t* __restrict__ out_idx,
                                                    uint32_t* __restrict__ mask_bits) {
  pdl_enter();
  __shared__ uint32_t s_w[TPB / 32 + 1];
  const int c = blockIdx.x, tid = threadIdx.x;
  const uint32_t vstar = p.vstate[0];
  const uint32_t take = p.tie_take[c];
  const uint32_t ob = p.out_base[c];
  const int64_t jb = (int64_t)c * CH + (int64_t)tid * 16;
  if (p.out_base[c + 1] == ob) {  // no coordinate of this chunk is in the mask (uniform over the CTA)
    if (mask_bits != nullptr && (tid & 1) == 0) {
      const int64_t wi = (int64_t)c * WPC + (tid >> 1);
      if (wi < p.W) mask_bits[wi] = 0u;
    }
    return;
  }
  uint32_t gm = 0, em = 0;
  if (jb < p.d) {
    if (jb + 16 <= p.d) {
      const uint4 q = *reinterpret_cast<const uint4*>(votes + jb);
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int b = 0; b < 16; b++) {
        const uint32_t v = (w[b >> 2] >> (8 * (b & 3))) & 0xffu;
        gm |= (v > vstar ? 1u : 0u) << b;
        em |= (v == vstar ? 1u : 0u) << b;
      }
    } else {
      for (int b = 0; b < 16 && jb + b < p.d; b++) {
        const uint32_t v = votes[jb + b];
        gm |= (v > vstar ? 1u : 0u) << b;
        em |= (v == vstar ? 1u : 0u) << b;
      }
    }
  }
  uint32_t sm = gm;
  if (take > 0) {  // uniform over the CTA
    uint32_t tot;
    const uint32_t epre = block_excl_scan<TPB>(__popc(em), s_w, tot);
    if (epre < take) {
      const uint32_t room = take - epre;  // keep this thread's first `room` ties
      uint32_t e2 = em, kept = 0, cntk = 0;
      while (e2 && cntk < room) {
        const uint32_t low = e2 & (0u - e2);
        kept |= low;
        e2 ^= low;
        cntk++;
      }
      sm |= kept;
    }
  }
  uint32_t tot;
  uint32_t pos = ob + block_excl_scan<TPB>(__popc(sm), s_w, tot);
  uint32_t s2 = sm;
  while (s2) {
    const int b = __ffs(s2) - 1;
    s2 &= s2 - 1;
    if (pos < (uint32_t)p.K) {
      out_idx[pos] = (int32_t)(jb + b);
      // the gather that follows reads this coordinate of every row, scattered over DRAM: ask for
      // those sectors now, so that they are on their way while this kernel drains and the next starts
      if (p.prefetch_acc != nullptr) {
        const float* a = p.prefetch_acc + (jb + b);
        for (int n = 0; n < p.N; n++) asm volatile("prefetch.global.L2 [%0];" ::"l"(a + (size_t)n * (size_t)p.d));
      }
    }
    else MV_DBG(p.dbg, MV_DBG_OUT_RANGE);
    pos++;
  }
  if (mask_bits != nullptr) {
    const uint32_t other = __shfl_xor_sync(FULL, sm, 1);
    if ((tid & 1) == 0) {
      const int64_t wi = (int64_t)c * WPC + (tid >> 1);
      if (wi < p.W) mask_bits[wi] = sm | (other << 16);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// aggregate: out_val[k] = fl32( (sum_n (double)acc[n][idx[k]]) / N ), then acc[n][idx[k]] = +0
// ---------------------------------------------------------------------------------------------
// One output of the aggregate.  G = lanes that share the coordinate: 1, or 8 (lane g then loads rows g, g + 8,
// ..., so that a coordinate's N scattered loads are in flight together even with many workers).  The sum is the
// same sequence of binary64 additions in worker order either way: with G = 8 the values are passed to it by
// shuffles, so all 32 lanes of a warp must call together (`live` = false for lanes without an output).
template <int G>
__device__ __forceinline__ void gather_at(float* __restrict__ acc, int N, int64_t d, int64_t k, int64_t j, bool live, int g,
                                          float* __restrict__ out_val, double* __restrict__ out_sum,
                                          uint32_t* __restrict__ dbg);

template <int G>
__device__ __forceinline__ void gather_one(float* __restrict__ acc, int N, int64_t d, int64_t k, bool live, int g,
                                           const int32_t* __restrict__ idx, float* __restrict__ out_val,
                                           double* __restrict__ out_sum, uint32_t* __restrict__ dbg) {
  const int64_t j = live ? (int64_t)__ldcg(idx + k) : -1;  // (from L2: the index may have been written by this very kernel)
  gather_at<G>(acc, N, d, k, j, live, g, out_val, out_sum, dbg);
}

// the same for output k whose coordinate j the caller already holds (j = -1 for a lane without an output)
template <int G>
__device__ __forceinline__ void gather_at(float* __restrict__ acc, int N, int64_t d, int64_t k, int64_t j, bool live, int g,
                                          float* __restrict__ out_val, double* __restrict__ out_sum,
                                          uint32_t* __restrict__ dbg) {
  const bool bad = j < 0 || j >= d;
  if (live && bad && g == 0) {
    MV_DBG(dbg, MV_DBG_GATHER_RANGE);
    if (out_sum) out_sum[k] = 0.0;
    else out_val[k] = 0.f;
  }
  if (G == 1 && bad) return;
  float* col = acc + (bad ? 0 : j);
  // all loads before any store: a store to acc followed by a load from acc (another row) would
  // otherwise be kept in program order and serialise the memory latency row by row
  double s = 0.0;
  if (G == 1) {
    for (int n0 = 0; n0 < N; n0 += 16) {
      float v[16];
#pragma unroll
      for (int q = 0; q < 16; q++) v[q] = n0 + q < N ? __ldcg(col + (size_t)(n0 + q) * (size_t)d) : 0.f;
#pragma unroll
      for (int q = 0; q < 16; q++)
        if (n0 + q < N) s += (double)v[q];
    }
    for (int n = 0; n < N; n++) __stcg(col + (size_t)n * (size_t)d, 0.0f);
  } else {
    const int lane = threadIdx.x & 31, gbase = lane - g;
    for (int n0 = 0; n0 < N; n0 += 4 * G) {  // uniform over the warp
      float v[4];
#pragma unroll
      for (int q = 0; q < 4; q++) {
        const int n = n0 + q * G + g;
        v[q] = (!bad && n < N) ? __ldcg(col + (size_t)n * (size_t)d) : 0.f;
      }
#pragma unroll
      for (int q = 0; q < 4; q++) {
        if (n0 + q * G >= N) break;  // (uniform over the warp)
#pragma unroll
        for (int h = 0; h < G; h++) {  // workers n0 + q G + h, in this order
          const float x = __shfl_sync(FULL, v[q], gbase + h);
          if (n0 + q * G + h < N) s += (double)x;
        }
      }
    }
    if (bad) return;
    for (int n = g; n < N; n += G) __stcg(col + (size_t)n * (size_t)d, 0.0f);
    if (g != 0) return;
  }
  // a rank that holds only some of the workers hands back its binary64 partial sum instead
  if (out_sum) out_sum[k] = s;
  else out_val[k] = (float)(s / (double)N);
}

// The last kernel of a whole step also clears the leading scratch region (counters and histograms)
// so that the next step can start without a separate memset; zero_vecs = 0 switches that off.
// G = 8 when K is small: the grid is then eight times larger.
template <int G>
__global__ void __launch_bounds__(TPB) k_gather(float* __restrict__ acc, int N, int64_t d, int64_t K,
                                                const int32_t* __restrict__ idx, float* __restrict__ out_val,
                                                uint4* __restrict__ zero_ptr, uint32_t zero_vecs,
                                                double* __restrict__ out_sum, uint32_t* __restrict__ dbg) {
  pdl_enter();
  for (uint32_t i = blockIdx.x * TPB + threadIdx.x; i < zero_vecs; i += gridDim.x * TPB)
    zero_ptr[i] = make_uint4(0, 0, 0, 0);
  const int64_t t = (int64_t)blockIdx.x * TPB + threadIdx.x;
  const int64_t k = t / G;
  if (G == 1 && k >= K) return;
  gather_one<G>(acc, N, d, k, k < K, (int)(t % G), idx, out_val, out_sum, dbg);
}

// worker-sharded step: mean over all workers from the summed partial sums
__global__ void __launch_bounds__(TPB) k_finish_mean(const double* __restrict__ sum, int64_t K, double n_total,
                                                     float* __restrict__ out_val) {
  const int64_t k = (int64_t)blockIdx.x * TPB + threadIdx.x;
  if (k < K) out_val[k] = (float)(sum[k] / n_total);
}

// SSGD-top-K (the comparison scheme: every worker under its own mask, the server averages what arrives).
// idx[0 .. *n_out) = the union of the workers' masks, ascending.  out_val[k] = fl32( (sum over the workers n whose
// mask holds idx[k], in worker order, of (double) acc[n][idx[k]]) / N ); those workers' residual becomes +0 there.
// Entries from *n_out up to `capacity` are set to -1 / 0.  Also clears the leading scratch region like k_gather.
__global__ void __launch_bounds__(TPB) k_union_gather(float* __restrict__ acc, int N, int64_t d, int64_t W,
                                                      const uint32_t* __restrict__ bits, int32_t* __restrict__ idx,
                                                      const uint32_t* __restrict__ n_out, float* __restrict__ out_val,
                                                      int64_t capacity, int32_t* __restrict__ count,
                                                      uint4* __restrict__ zero_ptr, uint32_t zero_vecs) {
  pdl_enter();
  for (uint32_t i = blockIdx.x * TPB + threadIdx.x; i < zero_vecs; i += gridDim.x * TPB)
    zero_ptr[i] = make_uint4(0, 0, 0, 0);
  const int64_t k = (int64_t)blockIdx.x * TPB + threadIdx.x;
  const int64_t U = (int64_t)__ldcg(n_out);
  if (k == 0) *count = (int32_t)(U < capacity ? U : capacity);
  if (k >= capacity) return;
  if (k >= U) {
    idx[k] = -1;
    out_val[k] = 0.f;
    return;
  }
  const int64_t j = __ldcg(idx + k);
  if (j < 0 || j >= d) {
    out_val[k] = 0.f;
    return;
  }
  const uint32_t bit = 1u << (uint32_t)(j & 31);
  const uint32_t* wcol = bits + (j >> 5);
  float* col = acc + j;
  double s = 0.0;
  for (int n0 = 0; n0 < N; n0 += 16) {
    uint32_t has = 0;
    float v[16];
#pragma unroll
    for (int q = 0; q < 16; q++)
      if (n0 + q < N && (__ldcg(wcol + (size_t)(n0 + q) * (size_t)W) & bit)) has |= 1u << q;
#pragma unroll
    for (int q = 0; q < 16; q++) v[q] = (has >> q) & 1u ? __ldcg(col + (size_t)(n0 + q) * (size_t)d) : 0.f;
#pragma unroll
    for (int q = 0; q < 16; q++)
      if ((has >> q) & 1u) s += (double)v[q];
#pragma unroll
    for (int q = 0; q < 16; q++)
      if ((has >> q) & 1u) __stcg(col + (size_t)(n0 + q) * (size_t)d, 0.0f);
  }
  out_val[k] = (float)(s / (double)N);
}

// ---------------------------------------------------------------------------------------------
// add-drop voting (Algorithm 2): from this step's top-K masks M_n and the previous vote masks Mt_n,
//   k_ad_fill   lists, per worker, the coordinates of  M_n & ~Mt_n  (with their keys) and of
//               Mt_n & ~M_n  (with inverted keys), in index order per chunk;
//   k_hist<1..3>, k_count, k_set_bits (list mode, 2N rows) pick the min(K_ad, length) largest of
//               each list -- the largest |acc| to add, the smallest |acc| to drop -- as bit masks;
//   k_ad_apply  Mt_n <- (Mt_n | add_n) & ~drop_n.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(TPB) k_ad_fill(P p, P a, const uint32_t* __restrict__ prev_bits,
                                                 const float* __restrict__ acc) {
  pdl_enter();
  // a warp per (worker, chunk): lane l owns mask words 4l..4l+3 of the chunk, so lane order is index order
  __shared__ uint32_t s_A[TPB / 32][WPC];    // the chunk's "add" candidates as mask words ...
  __shared__ uint16_t s_rank[TPB / 32][WPC];  // ... and how many of them lie in earlier words
  const int n = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = blockIdx.x * (TPB / 32) + warp;
  if (c >= p.nchunks) return;
  uint32_t A[4], D[4];
  uint32_t pa = 0, pd = 0;
#pragma unroll
  for (int q = 0; q < 4; q++) {
    const int64_t wi = (int64_t)c * WPC + lane * 4 + q;
    uint32_t M = 0, Q = 0;
    if (wi < p.W) {
      M = __ldcg(p.worker_bits + (size_t)n * p.W + wi);
      Q = __ldcg(prev_bits + (size_t)n * p.W + wi);
    }
    A[q] = M & ~Q;
    D[q] = Q & ~M;
    pa += __popc(A[q]);
    pd += __popc(D[q]);
  }
  uint32_t xa = pa, xd = pd;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t ya = __shfl_up_sync(FULL, xa, off), yd = __shfl_up_sync(FULL, xd, off);
    if (lane >= off) {
      xa += ya;
      xd += yd;
    }
  }
  const uint32_t tota = __shfl_sync(FULL, xa, 31), totd = __shfl_sync(FULL, xd, 31);
  uint32_t ba = 0, bd = 0;
  if (lane == 0) {
    const size_t ca = (size_t)n * p.nchunks + c, cd = (size_t)(p.N + n) * p.nchunks + c;
    if (tota) ba = atomicAdd(&a.cand_cnt[n], tota);
    if (totd) bd = atomicAdd(&a.cand_cnt[p.N + n], totd);
    a.chunk_base[ca] = ba;
    a.chunk_cnt[ca] = tota;
    a.chunk_base[cd] = bd;
    a.chunk_cnt[cd] = totd;
  }
  if ((tota | totd) == 0) return;
  ba = __shfl_sync(FULL, ba, 0);
  bd = __shfl_sync(FULL, bd, 0);
  const float* row = acc + (size_t)n * (size_t)p.d;
  uint2* la = a.cand + (size_t)n * a.cap;
  uint2* ld = a.cand + (size_t)(p.N + n) * a.cap;
  uint32_t posa = ba + xa - pa, posd = bd + xd - pd;
  // The keys of the "add" candidates: M_n is a subset of the worker's candidate buffer when the
  // worker went through it, so the chunk's run there already holds (key, index) for every one of
  // them, in index order: no need to gather acc.  A full-row worker gathers, like the drop list.
  const bool from_run = tota != 0 && worker_fast(p, n);  // warp-uniform
  if (from_run) {
    uint32_t r = xa - pa;
#pragma unroll
    for (int q = 0; q < 4; q++) {
      s_A[warp][lane * 4 + q] = A[q];
      s_rank[warp][lane * 4 + q] = (uint16_t)r;
      r += __popc(A[q]);
    }
    __syncwarp();
    const size_t ci = (size_t)n * p.nchunks + c;
    const uint32_t rcnt = p.chunk_cnt[ci];
    const uint2* run = p.cand + (size_t)n * p.cap + p.chunk_base[ci];
    for (uint32_t i = lane; i < rcnt; i += 32) {
      const uint2 kv = __ldcg(run + i);
      const uint32_t o = kv.y - (uint32_t)c * CH;  // offset within the chunk
      if (o >= (uint32_t)CH) {                      // cannot happen for a well-formed run
        MV_DBG(p.dbg, MV_DBG_INTERNAL);
        continue;
      }
      const uint32_t w = s_A[warp][o >> 5], bit = o & 31u;
      if ((w >> bit) & 1u) {
        const uint32_t pos = ba + s_rank[warp][o >> 5] + __popc(w & ((1u << bit) - 1u));
        if (pos < a.cap) la[pos] = kv;
        else MV_DBG(p.dbg, MV_DBG_LIST_OVERFLOW);
      }
    }
  }
#pragma unroll
  for (int q = 0; q < 4; q++) {
    const int64_t j0 = ((int64_t)c * WPC + lane * 4 + q) * 32;
    uint32_t m = from_run ? 0u : A[q];
    while (m) {
      const int b = __ffs(m) - 1;
      m &= m - 1;
      const int64_t j = j0 + b;
      if (j < p.d && posa < a.cap) la[posa] = make_uint2(fkey(row[j]), (uint32_t)j);
      else MV_DBG(p.dbg, MV_DBG_LIST_OVERFLOW);
      posa++;
    }
    m = D[q];
    while (m) {
      const int b = __ffs(m) - 1;
      m &= m - 1;
      const int64_t j = j0 + b;
      if (j < p.d && posd < a.cap) ld[posd] = make_uint2(0x7fffffffu - fkey(row[j]), (uint32_t)j);  // smallest first
      else MV_DBG(p.dbg, MV_DBG_LIST_OVERFLOW);
      posd++;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// random selection (SSGD-MV-RS: Algorithm 1 with the S_rand-weighted line).  Coordinate j with
// v_j > 0 votes rings at time E_j / v_j, E_j = -ln u_j, u_j = (x_j + 1/2) / 2^32, x_j the first word
// of Philox4x32-10 (key = seed, counter = (j, 0, draw)); the K earliest ring times are a draw of
// "sample proportionally to the votes until K distinct indices" (exponential clocks, Efraimidis and
// Spirakis).  Everything that decides an index is a fixed sequence of IEEE operations: the
// logarithm below uses binary64 +, *, / only, the ring time is one binary64 division rounded once
// to binary32, equal times go to the lowest index.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t philox4x32_10_first(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                        uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; r++) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c0;
}

__device__ __forceinline__ double neg_log_u(uint32_t x) {
  const unsigned long long v = 2ull * x + 1ull;  // u = v / 2^33
  int e = 63 - __clzll((long long)v);
  double m = __dmul_rn((double)v, __longlong_as_double((long long)(1023 - e) << 52));  // v * 2^-e: [1, 2), exact
  if (m > 1.4142135623730951) {
    m = __dmul_rn(m, 0.5);
    e += 1;
  }
  const double s = __ddiv_rn(__dadd_rn(m, -1.0), __dadd_rn(m, 1.0));
  const double z = __dmul_rn(s, s);
  double poly = 1.0 / 23.0;
#pragma unroll
  for (int k = 21; k >= 1; k -= 2) poly = __dadd_rn(__dmul_rn(poly, z), 1.0 / (double)k);
  const double logm = __dmul_rn(__dmul_rn(2.0, s), poly);
  return __dsub_rn(__dmul_rn((double)(33 - e), 0.6931471805599453), logm);
}

// A CTA per chunk: thread t owns coordinates 16t .. 16t+15 of the chunk, so thread order is index
// order.  Voted coordinates are first compacted, in index order, into shared memory; the threads
// then share them out evenly (the generator and the logarithm are the expensive part, and only about
// one coordinate in ten holds a vote) and append them to the single list `a` (row 0) as
// (0x7fffffff - ring time bits, index): the list-mode select then keeps the K largest keys, i.e. the
// K earliest times.
__global__ void __launch_bounds__(TPB) k_rs_fill(P p, P a, const uint8_t* __restrict__ votes, uint32_t seed_lo,
                                                 uint32_t seed_hi, uint32_t draw_lo, uint32_t draw_hi,
                                                 int32_t* __restrict__ fill_idx) {
  pdl_enter();
  // the index list starts out as all -1 (entries that no selected coordinate fills stay so)
  for (int64_t i = (int64_t)blockIdx.x * TPB + threadIdx.x; i < p.K; i += (int64_t)gridDim.x * TPB) fill_idx[i] = -1;
  __shared__ uint32_t s_w[TPB / 32 + 1];
  __shared__ uint32_t s_base;
  __shared__ uint16_t s_off[CH];  // offset of the coordinate within the chunk
  __shared__ uint8_t s_v[CH];     // its votes
  const int c = blockIdx.x;
  const int64_t j0 = (int64_t)c * CH + threadIdx.x * 16;
  uint8_t v[16];
  if (j0 + 16 <= p.d) {
    const uint4 q = __ldcg(reinterpret_cast<const uint4*>(votes + j0));
    const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 16; i++) v[i] = (uint8_t)(w4[i >> 2] >> (8 * (i & 3)));
  } else {
#pragma unroll
    for (int i = 0; i < 16; i++) v[i] = j0 + i < p.d ? votes[j0 + i] : (uint8_t)0;
  }
  uint32_t cnt = 0;
#pragma unroll
  for (int i = 0; i < 16; i++) cnt += v[i] != 0;
  uint32_t total;
  uint32_t pos = block_excl_scan<TPB>(cnt, s_w, total);
  if (threadIdx.x == 0) {
    const uint32_t base = total ? atomicAdd(&a.cand_cnt[0], total) : 0u;
    s_base = base;
    a.chunk_base[c] = base;
    a.chunk_cnt[c] = total;
  }
  if (total == 0) return;  // uniform over the CTA
#pragma unroll
  for (int i = 0; i < 16; i++) {
    if (v[i] == 0) continue;
    s_off[pos] = (uint16_t)(threadIdx.x * 16 + i);
    s_v[pos] = v[i];
    pos++;
  }
  __syncthreads();
  const uint32_t base = s_base;
  for (uint32_t i = threadIdx.x; i < total; i += TPB) {
    const uint32_t j = (uint32_t)((int64_t)c * CH + s_off[i]);
    const uint32_t x = philox4x32_10_first(j, 0u, draw_lo, draw_hi, seed_lo, seed_hi);
    const double t = __ddiv_rn(neg_log_u(x), (double)s_v[i]);
    const uint32_t tb = __float_as_uint(__double2float_rn(t));
    if (base + i < a.cap) a.cand[base + i] = make_uint2(0x7fffffffu - tb, j);
    else MV_DBG(p.dbg, MV_DBG_LIST_OVERFLOW);
  }
}

// selected coordinates per chunk of bit-mask row blockIdx.y (a warp per chunk)
__global__ void __launch_bounds__(TPB) k_chunk_popc(const uint32_t* __restrict__ bits, int64_t W, int nchunks,
                                                    uint32_t* __restrict__ chunk_sel) {
  pdl_enter();
  const int c = blockIdx.x * (TPB / 32) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (c >= nchunks) return;
  bits += (size_t)blockIdx.y * (size_t)W;
  chunk_sel += (size_t)blockIdx.y * (size_t)nchunks;
  uint32_t s = 0;
#pragma unroll
  for (int q = 0; q < 4; q++) {
    const int64_t wi = (int64_t)c * WPC + q * 32 + lane;
    if (wi < W) s += __popc(__ldcg(bits + wi));
  }
  s = __reduce_add_sync(FULL, s);
  if (lane == 0) chunk_sel[c] = s;
}

__global__ void __launch_bounds__(TPB) k_ad_apply(uint32_t* __restrict__ prev_bits, const uint32_t* __restrict__ ad_bits,
                                                  uint32_t* __restrict__ add_out, uint32_t* __restrict__ drop_out,
                                                  size_t words /* N*W */) {
  pdl_enter();
  for (size_t i = (size_t)blockIdx.x * TPB + threadIdx.x; i < words; i += (size_t)gridDim.x * TPB) {
    const uint32_t add = __ldcg(ad_bits + i), drop = __ldcg(ad_bits + words + i);
    prev_bits[i] = (prev_bits[i] | add) & ~drop;
    if (add_out) add_out[i] = add;
    if (drop_out) drop_out[i] = drop;
  }
}

#include "mv_tail.cuh"
#include "mv_small.cuh"
static_assert(F_RADIX <= SB_BINS, "the three-digit counts live in the sample histogram's rows");

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
struct Layout {
  int nchunks;
  int64_t W;
  uint32_t cap;
  size_t dbg;         // header, at the start of the workspace whatever the sizes: word 0 the checked build's status
  size_t fb_total;    // word, word 1 the running count of full-row selections, word 2 set for good once a bounded
  size_t abort_flag;  // device-side wait has given up (MV_ERR_TIMEOUT)
  size_t tail_words;  // [16] grid barrier, exit ticket and flags of the single-kernel tail (in the cleared region)
  size_t zero_off;    // start of ...
  size_t zero_bytes;  // ... the region that is clear at the start of every vote
  size_t samp_hist, hist1, hist2, hist2b, hist3, cand_cnt, sample_done, count_done, votes_done, hot, vote_hist;
  size_t tau, tau_alt, tstate, diag_cnt, wstate, thresh, vstate, cand, chunk_base, chunk_cnt, chunk_eq, tie_base, chunk_sel;
  size_t worker_bits, worker_idx, votes, chunk_vh, out_base, tie_take;
  size_t votes_alt;   // rows that fit one CTA (d <= SMALL_MAX_D): the second vote array of the single-kernel step ...
  size_t small_state; // ... and its two vote histograms [2][256] and two barrier words (at [512] and [528])
  // add-drop voting: the select state once more, for 2N lists of at most ad_cap entries
  uint32_t ad_cap;
  size_t ad_zero, ad_zero_bytes;  // cleared at the start of every add-drop vote
  size_t ad_hist1, ad_hist2, ad_hist3, ad_cnt, ad_count_done, ad_bits;
  size_t rs_chunk_sel;  // [nchunks] random selection: selected coordinates per chunk, then their offsets
  size_t ad_wstate, ad_thresh, ad_diag, ad_cand, ad_chunk_base, ad_chunk_cnt, ad_chunk_eq, ad_tie_base;
  size_t total;
};

bool sizes_ok(int N, int64_t d, int64_t K) {
  return N >= 1 && N <= 255 && d >= 1 && d < ((int64_t)1 << 31) - 8192 && K >= 1 && K <= d;
}

size_t take(size_t& off, size_t bytes) {
  const size_t at = off;
  off += (bytes + 255) & ~(size_t)255;
  return at;
}

Layout make_layout(int N, int64_t d, int64_t K) {
  Layout L;
  L.nchunks = (int)((d + CH - 1) / CH);
  L.W = (d + 31) / 32;
  int64_t cap = 4 * K + 4096;
  if (cap > d) cap = d;
  L.cap = (uint32_t)((cap + 7) & ~(int64_t)7);  // multiple of 8: every worker's buffer is 64-byte aligned
  size_t off = 0;
  const size_t n = (size_t)N, nc = (size_t)L.nchunks;
  L.dbg = take(off, 12);
  L.fb_total = L.dbg + 4;
  L.abort_flag = L.dbg + 8;
  L.zero_off = off;
  L.samp_hist = take(off, n * SB_BINS * 4);
  L.hist1 = take(off, n * H1_BINS * 4);
  L.hist2 = take(off, n * H2_BINS * 4);
  L.hist3 = take(off, n * H3_BINS * 4);
  L.hist2b = take(off, n * H2_BINS * 4);
  L.cand_cnt = take(off, n * 4);
  L.sample_done = take(off, n * 4);
  L.count_done = take(off, n * 4);
  L.hot = take(off, (size_t)((L.nchunks + 7) & ~7));
  L.votes_done = take(off, 4);
  L.vote_hist = take(off, 256 * 4);
  L.tail_words = take(off, 16 * 4);
  L.zero_bytes = off - L.zero_off;
  L.tau = take(off, n * 4);
  L.tau_alt = take(off, n * 4);
  L.tstate = take(off, n * 2 * 4);
  L.diag_cnt = take(off, n * 4);
  L.wstate = take(off, n * 8 * 4);
  L.thresh = take(off, n * 3 * 4);
  L.vstate = take(off, 4 * 4);
  L.cand = take(off, n * (size_t)L.cap * 8);
  L.chunk_base = take(off, n * nc * 4);
  L.chunk_cnt = take(off, n * nc * 4);
  L.chunk_eq = take(off, n * nc * 4);
  L.tie_base = take(off, n * nc * 4);
  L.chunk_sel = take(off, n * nc * 4);
  L.worker_bits = take(off, n * (size_t)L.W * 4);
  L.worker_idx = take(off, n * (size_t)K * 4);
  L.votes = take(off, nc * CH);
  L.chunk_vh = take(off, (size_t)(((L.nchunks + 7) & ~7)) * (n + 1) * 2);
  L.out_base = take(off, (nc + 1) * 4);
  L.tie_take = take(off, nc * 4);
  L.votes_alt = take(off, d <= SMALL_MAX_D ? nc * CH : 0);
  L.small_state = take(off, d <= SMALL_MAX_D ? (512 + 32) * 4 : 0);
  {
    const size_t m = 2 * n;
    L.ad_cap = (uint32_t)((K + 7) & ~(int64_t)7);
    L.ad_zero = off;
    L.ad_hist1 = take(off, m * H1_BINS * 4);
    L.ad_hist2 = take(off, m * H2_BINS * 4);
    L.ad_hist3 = take(off, m * H3_BINS * 4);
    L.ad_cnt = take(off, m * 4);
    L.ad_count_done = take(off, m * 4);
    L.ad_bits = take(off, m * (size_t)L.W * 4);
    L.ad_zero_bytes = off - L.ad_zero;
    L.ad_wstate = take(off, m * 8 * 4);
    L.ad_thresh = take(off, m * 3 * 4);
    L.ad_diag = take(off, m * 4);
    L.ad_cand = take(off, m * (size_t)L.ad_cap * 8);
    L.rs_chunk_sel = take(off, nc * 4);
    L.ad_chunk_base = take(off, m * nc * 4);
    L.ad_chunk_cnt = take(off, m * nc * 4);
    L.ad_chunk_eq = take(off, m * nc * 4);
    L.ad_tie_base = take(off, m * nc * 4);
  }
  L.total = off;
  return L;
}

bool aligned16(const void* q) { return ((uintptr_t)q & 15u) == 0; }

}  // namespace

struct mv_ctx {
  cudaStream_t stream;
  char* ws;
  size_t ws_bytes;
  int mode;
  int launches;
  // optional CUDA-event timing of the streaming pass (ring of event pairs)
  int timing;                // 0 = off, n = record on every n-th call
  int timing_calls;          // calls seen since timing was switched on
  bool timing_now;           // this call records
  int timed;                 // pairs recorded since the last read
  cudaEvent_t ev[2 * 64];
  bool ev_made;
  // index lists are written on a side stream, concurrently with mask selection and aggregation
  cudaStream_t side;
  cudaEvent_t ev_fork, ev_join, ev_zero;
  int side_state;  // 0 = not tried, 1 = ready, -1 = unavailable
  bool join_pending;
  // optional per-launch timing of one call: pev[i] is recorded after the i-th launch (pev[0] before the first)
  int phase_timing;
  cudaEvent_t pev[48];
  bool pev_made;
  size_t clean_bytes;  // bytes from the start of the cleared region known to be zero (left so by the previous whole step)
  int sms;             // multiprocessors of the workspace's device (0 = not asked yet)
  int cta_budget;      // the largest multiple of 8 CTAs that is not above sms: one CTA per SM for the cluster select
  bool dbg_ready;      // the workspace's header has been cleared once
  int tail_state;      // single-kernel tail: 0 = not tried, 1 = usable on this device, -1 = not
  int tail_mode;       // (mv_set_tail_kernel) 0 = never, 1 = where it pays, 2 = wherever it can run
  int small_state;     // single-kernel small step: 0 = not tried, 1 = usable on this device, -1 = not
  bool small_ready;    // the vote array that the next small step of size (small_N, small_d, small_K) uses is known to be zero
  int small_N;
  int64_t small_d, small_K;
  int small_flip;      // which of the two holds the next call's votes
  int tail_pdl;        // -1: the runtime refused a cooperative launch with programmatic stream serialisation
  // remembered for mv_read_diag
  int last_N;
  int64_t last_d, last_K;
  // threshold tracking (MV_MODE_TRACK): the two tau arrays alternate between "this call" and "next call"
  int tau_flip;       // which array holds the thresholds of the current (or last) call
  bool track_valid;   // the previous call left thresholds for (track_N, track_d, track_K)
  int track_N;
  int64_t track_d, track_K;
};

namespace {

P make_params(const mv_ctx* ctx, const Layout& L, int N, int64_t d, int64_t K) {
  P p;
  char* b = ctx->ws;
  p.N = N;
  p.nchunks = L.nchunks;
  p.nc_pad = (L.nchunks + 7) & ~7;
  p.cap = L.cap;
  p.force_general = ctx->mode == MV_MODE_GENERAL ? 1 : 0;
  p.list_mode = 0;
  p.apply_rows = 0;
  p.no_masks = 0;
  p.take_all = 0;
  p.vote_words = nullptr;
  p.prefetch_acc = nullptr;
  p.apply_bits = nullptr;
  p.d = d;
  p.K = K;
  p.W = L.W;
  p.samp_hist = (uint32_t*)(b + L.samp_hist);
  p.hist1 = (uint32_t*)(b + L.hist1);
  p.hist2 = (uint32_t*)(b + L.hist2);
  p.hist3 = (uint32_t*)(b + L.hist3);
  p.cand_cnt = (uint32_t*)(b + L.cand_cnt);
  p.sample_done = (uint32_t*)(b + L.sample_done);
  p.count_done = (uint32_t*)(b + L.count_done);
  p.votes_done = (uint32_t*)(b + L.votes_done);
  p.hot = (uint8_t*)(b + L.hot);
  p.vote_hist = (uint32_t*)(b + L.vote_hist);
  p.tau = (uint32_t*)(b + (ctx->tau_flip ? L.tau_alt : L.tau));
  p.tau_next = nullptr;
  p.track_rank = 0;
  p.hist2b = (uint32_t*)(b + L.hist2b);
  p.tstate = (uint32_t*)(b + L.tstate);
  p.diag_cnt = (uint32_t*)(b + L.diag_cnt);
  p.wstate = (uint32_t*)(b + L.wstate);
  p.thresh = (uint32_t*)(b + L.thresh);
  p.vstate = (uint32_t*)(b + L.vstate);
  p.cand = (uint2*)(b + L.cand);
  p.chunk_base = (uint32_t*)(b + L.chunk_base);
  p.chunk_cnt = (uint32_t*)(b + L.chunk_cnt);
  p.chunk_eq = (uint32_t*)(b + L.chunk_eq);
  p.tie_base = (uint32_t*)(b + L.tie_base);
  p.chunk_sel = (uint32_t*)(b + L.chunk_sel);
  p.worker_bits = (uint32_t*)(b + L.worker_bits);
  p.worker_idx = (int32_t*)(b + L.worker_idx);
  p.votes = (uint8_t*)(b + L.votes);
  p.chunk_vh = (uint16_t*)(b + L.chunk_vh);
  p.out_base = (uint32_t*)(b + L.out_base);
  p.tie_take = (uint32_t*)(b + L.tie_take);
  p.dbg = kChecked ? (uint32_t*)(b + L.dbg) : nullptr;
  p.fb_total = (uint32_t*)(b + L.fb_total);
  p.zero2_ptr = nullptr;
  p.zero2_vecs = 0;
  p.all_chunks = 0;
  return p;
}

// Properties of the device that holds the workspace, asked for once per context (grid sizes follow
// the number of multiprocessors); the workspace's header (status word, fallback count) is cleared here too.
int device_ready(mv_ctx* ctx) {
  if (ctx->sms == 0) {
    int dev = -1;
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, ctx->ws) == cudaSuccess && at.type == cudaMemoryTypeDevice) dev = at.device;
    else cudaGetLastError();
    if (dev < 0 && cudaGetDevice(&dev) != cudaSuccess) return MV_ERR_CUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return MV_ERR_CUDA;
    ctx->sms = sms;
    ctx->cta_budget = sms >= 8 ? sms - sms % 8 : 8;
  }
  if (!ctx->dbg_ready) {
    if (cudaMemsetAsync(ctx->ws, 0, 12, ctx->stream) != cudaSuccess) return MV_ERR_CUDA;
    ctx->dbg_ready = true;
  }
  return MV_OK;
}

template <typename... KArgs, typename... Args>
cudaError_t launch_smem(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
  return launch_smem(kernel, grid, block, 0, st, args...);
}

// k_select_cluster keeps SK_KEYS keys in dynamic shared memory: above the default limit, so the
// kernel is told once per device
bool cluster_select_ready() {
  static bool done[64] = {false};
  static std::mutex mu;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  std::lock_guard<std::mutex> lock(mu);
  if (!done[dev]) {
    if (cudaFuncSetAttribute(k_select_cluster<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, SK_KEYS * 4) != cudaSuccess ||
        cudaFuncSetAttribute(k_select_cluster<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, SK_KEYS * 4) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    done[dev] = true;
  }
  return true;
}

int per_row_ctas(int N, int want, int budget) {
  int lim = budget / N;
  if (lim < 1) lim = 1;
  if (want < 1) want = 1;
  return want < lim ? want : lim;
}

#define MV_LAUNCH_CHECK()                                                                        \
  do {                                                                                           \
    ctx->launches++;                                                                             \
    if (cudaGetLastError() != cudaSuccess) return MV_ERR_CUDA;                                   \
    if ((ctx->phase_timing == 1 || ctx->phase_timing == 100 + ctx->launches) && ctx->launches < 48) \
      cudaEventRecord(ctx->pev[ctx->launches], ctx->stream);                                     \
  } while (0)

// sample size and rank for the threshold estimate
void sample_plan(int64_t d, int64_t K, uint32_t& U, uint32_t& L, int& all, uint32_t& rank) {
  // sample size: d/256, but large enough that about 100 sampled elements lie above the K-th key
  // (the bound's slack is a few standard deviations of that count), within [32 Ki, 1 Mi]
  int64_t S = d / 256;
  const int64_t s_min = (int64_t)(100.0 * (double)d / (double)K);
  if (S < s_min) S = s_min;
  if (S < 32768) S = 32768;
  if (S > (1 << 20)) S = 1 << 20;
  if (d <= 2 * S) {
    all = 1;
    U = (uint32_t)((d + 31) / 32);
    L = U;
    rank = (uint32_t)K;
    return;
  }
  all = 0;
  U = (uint32_t)(S / 32);
  L = (uint32_t)((d / 32) / U);  // line stride (>= 2): lines 0, L, 2L, ... are sampled
  const double Sn = (double)U * 32.0;
  const double m = Sn * (double)K / (double)d;
  double r = ceil(m + 6.0 * sqrt(m) + 8.0);
  if (r > Sn) r = Sn;
  rank = (uint32_t)r;
}

bool side_ready(mv_ctx* ctx) {
  if (ctx->side_state == 0) {
    ctx->side_state = -1;
    if (cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking) == cudaSuccess) {
      if (cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) == cudaSuccess) {
        if (cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) == cudaSuccess) {
          if (cudaEventCreateWithFlags(&ctx->ev_zero, cudaEventDisableTiming) == cudaSuccess)
            ctx->side_state = 1;
          else
            cudaEventDestroy(ctx->ev_join);
        }
        if (ctx->side_state != 1) cudaEventDestroy(ctx->ev_fork);
      }
      if (ctx->side_state != 1) cudaStreamDestroy(ctx->side);
    }
  }
  return ctx->side_state == 1;
}

// the caller's stream waits for the side stream's work of this call
int join_side(mv_ctx* ctx) {
  if (ctx->join_pending) {
    ctx->join_pending = false;
    if (cudaStreamWaitEvent(ctx->stream, ctx->ev_join, 0) != cudaSuccess) return MV_ERR_CUDA;
  }
  return MV_OK;
}

// steps a1-a3: accumulate, per-worker top-K, votes
// `topk_only`: stop once the workers' bit masks are set (no vote count, no index lists); everything
// then stays on the caller's stream
// `need_hist` = false: the per-chunk vote histograms and offsets are not wanted (the caller selects by other means)
// `want_lists` = false: the ascending per-worker index lists are not wanted (nothing later in a step reads them)
// `want_masks` = false: nor are the workers' bit masks (unless the lists, which are built from them, are)
// `stream_only`: stop after the streaming pass (the single-kernel tail follows); *p_out gets the parameters as
// completed here (thresholds of this and the next call, vote array)
int vote_impl(mv_ctx* ctx, P p, const Layout& L, const float* grads, float* err, bool topk_only = false,
              bool need_hist = true, bool want_lists = true, bool want_masks = true, bool stream_only = false,
              P* p_out = nullptr) {
  cudaStream_t st = ctx->stream;
  const int N = p.N;
  const int SMS = ctx->sms, CTA_BUDGET = ctx->cta_budget;
  ctx->timing_now = ctx->timing > 0 && (ctx->timing_calls++ % ctx->timing) == 0;
  if (ctx->clean_bytes < L.zero_bytes && cudaMemsetAsync(ctx->ws + L.zero_off, 0, L.zero_bytes, st) != cudaSuccess)
    return MV_ERR_CUDA;
  ctx->clean_bytes = 0;  // dirty from here on, until a whole step's last kernel has cleared it again
  ctx->small_ready = false;  // (the vote array is about to be written)
  // general mode: per-chunk outputs of the vote count start out cleared (only chunks with picks are
  // visited later); cleared on the side stream, concurrently with the first pass
  cudaStream_t zs = st;
  if (p.force_general && !topk_only && ctx->phase_timing != 1 && side_ready(ctx) &&
      cudaEventRecord(ctx->ev_fork, st) == cudaSuccess && cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0) == cudaSuccess)
    zs = ctx->side;
  if (p.force_general && !topk_only) {
    const size_t nc = (size_t)p.nchunks;
    cudaError_t e = cudaMemsetAsync(p.votes, 0, (size_t)p.d, zs);
    if (e == cudaSuccess) e = cudaMemsetAsync(p.chunk_sel, 0, (size_t)N * nc * 4, zs);
    if (e == cudaSuccess) e = cudaMemsetAsync(p.chunk_vh, 0, (size_t)(N + 1) * (size_t)p.nc_pad * 2, zs);
    if (e != cudaSuccess) return MV_ERR_CUDA;
    if (zs != st && cudaEventRecord(ctx->ev_zero, zs) != cudaSuccess) return MV_ERR_CUDA;
  }
  // CTAs per worker of the select kernels: enough for a full-row pass, not more than the candidates need
  const int gh = p.force_general ? per_row_ctas(N, p.nchunks, SMS * 8)
                                 : per_row_ctas(N, (int)((p.cap + TPB * 8 - 1) / (TPB * 8)), SMS * 2);
  if (!p.force_general) {
    // threshold tracking: the previous call on this context, if it had the same N, d and K, left a
    // threshold per worker in the other tau array; this call reads it instead of sampling and
    // leaves its own proposal in the array it does not read
    const bool track = ctx->mode == MV_MODE_TRACK;
    const bool tracked = track && ctx->track_valid && ctx->track_N == N && ctx->track_d == p.d && ctx->track_K == p.K;
    if (tracked) ctx->tau_flip ^= 1;
    p.tau = (uint32_t*)(ctx->ws + (ctx->tau_flip ? L.tau_alt : L.tau));
    if (track) {
      p.tau_next = (uint32_t*)(ctx->ws + (ctx->tau_flip ? L.tau : L.tau_alt));
      const double r = ceil((double)p.K * 1.35 + 6.0 * sqrt((double)p.K) + 8.0);
      p.track_rank = (uint32_t)(r < (double)p.d ? r : (double)p.d);
      ctx->track_valid = true;
      ctx->track_N = N;
      ctx->track_d = p.d;
      ctx->track_K = p.K;
    }
    if (!tracked) {
      uint32_t U, Ls, rank;
      int all;
      sample_plan(p.d, p.K, U, Ls, all, rank);
      const int gs = per_row_ctas(N, (int)((U + 127) / 128), SMS * 2);
      launch_k(k_sample_hist, dim3(dim3(gs, N)), dim3(512), st, p, grads, err, U, Ls, all, rank);
      MV_LAUNCH_CHECK();
    }
    // the votes are counted while the picks are made, in the workspace's vote array (whole chunks long)
    uint8_t* const ws_votes = (uint8_t*)(ctx->ws + L.votes);
    p.vote_words = topk_only ? nullptr : (uint32_t*)ws_votes;
    // Nothing reads the workers' bit masks when neither they nor the index lists are an output of the call
    // (a whole step): the picks then only count votes
    p.no_masks = (!topk_only && !want_lists && !want_masks) ? 1 : 0;
    if (ctx->timing_now) cudaEventRecord(ctx->ev[2 * (ctx->timed % 64)], st);
    launch_k(k_acc_compact, dim3(dim3(p.nchunks, N)), dim3(TPB), st, p, grads, err);
    MV_LAUNCH_CHECK();
    if (ctx->timing_now) cudaEventRecord(ctx->ev[2 * (ctx->timed++ % 64) + 1], st);
    if (stream_only) {
      if (p_out) *p_out = p;
      return MV_OK;
    }
    if (!cluster_select_ready()) return MV_ERR_CUDA;
    // a cluster per worker resolves T_n, sets the worker's mask bits and adds its votes
    // (with few workers, extra clusters that only help clearing fill the GPU)
    // (candidate buffers of more than 2^20 entries per worker are more than a cluster's 4 or 8 SMs
    // should walk, above all when the workers are few: those go through the grid-wide select kernels
    // and the clusters only clear)
    const bool wide = p.cap > (1u << 20);
    const int nsel = wide ? 0 : N;
    const int cl = nsel * 8 <= CTA_BUDGET ? 8 : 4;                              // one CTA per SM: keep all clusters resident if possible
    const int zc = nsel * cl < CTA_BUDGET ? (CTA_BUDGET - nsel * cl) / cl : 0;  // clusters that only clear
    // the extra clusters clear alone if that does not take them longer than the select takes (measured:
    // about 450 KB per CTA); otherwise every CTA of the grid clears a share first
    const size_t clear_bytes = (p.no_masks ? 0 : (size_t)N * (size_t)p.W * 4) + (topk_only ? 0 : (size_t)p.nchunks * CH);
    const int zero_first = (nsel > 0 && zc * cl >= 32 && clear_bytes / (size_t)(zc * cl) <= 450 * 1024) ? nsel : 0;
    if (cl == 8) launch_smem(k_select_cluster<8>, dim3(dim3(8, nsel + zc)), dim3(ST), SK_KEYS * 4, st, p, err, zero_first, nsel);
    else launch_smem(k_select_cluster<4>, dim3(dim3(4, nsel + zc)), dim3(ST), SK_KEYS * 4, st, p, err, zero_first, nsel);
    MV_LAUNCH_CHECK();
    if (wide) {
      launch_k(k_hist<1, false>, dim3(dim3(gh, N)), dim3(TPB), st, p, nullptr, err);
      MV_LAUNCH_CHECK();
      launch_k(k_hist<2, false>, dim3(dim3(gh, N)), dim3(TPB), st, p, nullptr, err);
      MV_LAUNCH_CHECK();
      launch_k(k_hist<3, false>, dim3(dim3(gh, N)), dim3(TPB), st, p, nullptr, err);
      MV_LAUNCH_CHECK();
      launch_k(k_count, dim3(dim3(gh, N)), dim3(TPB), st, p, err);
      MV_LAUNCH_CHECK();
    }
    // the picks: mask bits and votes, from the candidates (or the row), by the whole GPU
    launch_k(k_set_bits, dim3(dim3(per_row_ctas(N, (int)((p.cap + TPB * 16 - 1) / (TPB * 16)), SMS * 4), N)), dim3(TPB), st, p,
             err);
    MV_LAUNCH_CHECK();
    if (topk_only) return MV_OK;
    // vote histograms per chunk, v* and the output offsets (the caller's vote array gets its copy here)
    if (need_hist || p.votes != ws_votes) {
      launch_k(k_vote_hist, dim3((p.nchunks + VH_WARPS - 1) / VH_WARPS), dim3(TPB), st, p, (const uint8_t*)ws_votes,
               p.votes != ws_votes ? p.votes : (uint8_t*)nullptr);
      MV_LAUNCH_CHECK();
    }
  } else {
    if (ctx->timing_now) cudaEventRecord(ctx->ev[2 * (ctx->timed % 64)], st);
    launch_k(k_hist<1, true>, dim3(dim3(gh, N)), dim3(TPB), st, p, grads, err);
    MV_LAUNCH_CHECK();
    if (ctx->timing_now) cudaEventRecord(ctx->ev[2 * (ctx->timed++ % 64) + 1], st);
  }
  if (p.force_general) {
    launch_k(k_hist<2, false>, dim3(dim3(gh, N)), dim3(TPB), st, p, nullptr, err);
    MV_LAUNCH_CHECK();
    launch_k(k_hist<3, false>, dim3(dim3(gh, N)), dim3(TPB), st, p, nullptr, err);
    MV_LAUNCH_CHECK();
    launch_k(k_count, dim3(dim3(gh, N)), dim3(TPB), st, p, err);
    MV_LAUNCH_CHECK();
    launch_k(k_set_bits, dim3(dim3(gh, N)), dim3(TPB), st, p, err);
    MV_LAUNCH_CHECK();
  }
  if (topk_only) return MV_OK;
  if (p.force_general) {
    if (zs != st && cudaStreamWaitEvent(st, ctx->ev_zero, 0) != cudaSuccess) return MV_ERR_CUDA;
    const dim3 gv(p.nchunks < SMS * 8 ? p.nchunks : SMS * 8);
    if (N < 4) launch_k(k_votes<2>, gv, dim3(VT), st, p);
    else if (N < 16) launch_k(k_votes<4>, gv, dim3(VT), st, p);
    else if (N < 64) launch_k(k_votes<6>, gv, dim3(VT), st, p);
    else launch_k(k_votes<8>, gv, dim3(VT), st, p);
    MV_LAUNCH_CHECK();
  }
  if (!want_lists) return MV_OK;
  // the index lists feed nothing later in the step: write them on the side stream
  cudaStream_t ls = st;
  if (ctx->phase_timing != 1 && side_ready(ctx) && cudaEventRecord(ctx->ev_fork, st) == cudaSuccess &&
      cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0) == cudaSuccess)
    ls = ctx->side;
  if (!p.force_general) {  // selected coordinates per (worker, chunk), which the general vote count leaves behind
    launch_k(k_chunk_popc, dim3(dim3((p.nchunks + TPB / 32 - 1) / (TPB / 32), N)), dim3(TPB), ls,
             (const uint32_t*)p.worker_bits, p.W, p.nchunks, p.chunk_sel);
    MV_LAUNCH_CHECK();
  }
  launch_k(k_scan_sel, dim3(N), dim3(1024), ls, p);
  MV_LAUNCH_CHECK();
  launch_k(k_lists, dim3(dim3((p.nchunks + TPB / 32 - 1) / (TPB / 32), N)), dim3(TPB), ls, p);
  MV_LAUNCH_CHECK();
  if (ls != st) {
    if (cudaEventRecord(ctx->ev_join, ls) != cudaSuccess) return MV_ERR_CUDA;
    ctx->join_pending = true;
  }
  return MV_OK;
}

// step a4; `have_hist`: chunk_vh / vote_hist were already filled by k_build_votes
int select_impl(mv_ctx* ctx, P p, const Layout& L, const uint8_t* votes, bool have_hist, int32_t* out_idx,
                uint32_t* mask_bits) {
  cudaStream_t st = ctx->stream;
  if (!have_hist) {
    ctx->clean_bytes = 0;
    ctx->small_ready = false;  // (this call's layout may put its scratch where a small step keeps its state)
    if (cudaMemsetAsync(ctx->ws + L.votes_done, 0, L.zero_off + L.zero_bytes - L.votes_done, st) != cudaSuccess)
      return MV_ERR_CUDA;
    launch_k(k_vote_hist, dim3((p.nchunks + VH_WARPS - 1) / VH_WARPS), dim3(TPB), st, p, votes, (uint8_t*)nullptr);
    MV_LAUNCH_CHECK();
  }
  launch_k(k_vote_write, dim3(p.nchunks), dim3(TPB), st, p, votes, out_idx, mask_bits);
  MV_LAUNCH_CHECK();
  return MV_OK;
}

// steps a5-a6
int aggregate_impl(mv_ctx* ctx, float* acc, int N, int64_t d, int64_t K, const int32_t* idx, float* out_val,
                   size_t clear_bytes, double* out_sum = nullptr) {
  const Layout L0 = make_layout(1, 1, 1);  // (the cleared region starts at the same offset for every size)
  uint4* const zp = (uint4*)(ctx->ws + L0.zero_off);
  uint32_t* const dbg = kChecked ? (uint32_t*)(ctx->ws + L0.dbg) : (uint32_t*)nullptr;
  // few coordinates, several workers: eight lanes per coordinate keep the scattered loads in flight together
  if (K <= 65536 && N >= 4)
    launch_k(k_gather<8>, dim3((unsigned)((K * 8 + TPB - 1) / TPB)), dim3(TPB), ctx->stream, acc, N, d, K, idx, out_val, zp,
             (uint32_t)(clear_bytes / 16), out_sum, dbg);
  else
    launch_k(k_gather<1>, dim3((unsigned)((K + TPB - 1) / TPB)), dim3(TPB), ctx->stream, acc, N, d, K, idx, out_val, zp,
             (uint32_t)(clear_bytes / 16), out_sum, dbg);
  MV_LAUNCH_CHECK();
  if (clear_bytes) ctx->clean_bytes = clear_bytes;
  return MV_OK;
}

// dynamic shared memory of the tail kernel: the candidate keys of a CTA's slice, later the output offsets
// (nchunks + 1 words) and tie quotas (16 bits each) of all chunks
size_t tail_smem_bytes(int nc_pad) {
  const size_t table = ((size_t)nc_pad + 8) * 4 + (size_t)nc_pad * 2;
  return table > (size_t)SK_KEYS * 4 ? table : (size_t)SK_KEYS * 4;
}

// The single-kernel tail needs a cooperative launch with one CTA of FT threads per multiprocessor and shared
// memory for the largest table; asked once per context.
bool tail_ready(mv_ctx* ctx) {
  if (ctx->tail_state == 0) {
    ctx->tail_state = -1;
    int dev = -1, coop = 0, per_sm = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess &&
        coop != 0 &&
        cudaFuncSetAttribute(k_tail, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tail_smem_bytes(F_MAXCH)) == cudaSuccess &&
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_tail, FT, tail_smem_bytes(F_MAXCH)) == cudaSuccess && per_sm >= 1)
      ctx->tail_state = 1;
    else
      cudaGetLastError();
  }
  return ctx->tail_state == 1;
}

// Do this call's steps after the streaming pass run as the single kernel?  It can when the mode is not the general
// one, every worker gets a CTA of its own and the chunks' output offsets fit its shared-memory table.  It pays
// (measured: some microseconds per step) when there are many picks to make and outputs to gather, K >= 2^16; with
// a small K the steps are all latency, and the separate kernels, each launched while its predecessor still runs,
// are as fast or faster.
bool tail_usable(mv_ctx* ctx, const Layout& L, int N, int64_t K) {
  if (ctx->tail_mode == 0 || (ctx->tail_mode == 1 && K < 65536)) return false;
  return ctx->mode != MV_MODE_GENERAL && N <= ctx->sms && ((L.nchunks + 7) & ~7) <= F_MAXCH && tail_ready(ctx);
}

// steps a2 (from the candidates on) to a6 as one cooperative kernel; p: the parameters as vote_impl completed them
int tail_impl(mv_ctx* ctx, const P& p, const Layout& L, float* err, int32_t* out_idx, float* out_val) {
  char* b = ctx->ws;
  TailArgs a;
  a.err = err;
  a.out_idx = out_idx;
  a.out_val = out_val;
  a.words = (uint32_t*)(b + L.tail_words);
  a.abort_flag = (uint32_t*)(b + L.abort_flag);
  a.radix = (uint32_t*)(b + L.samp_hist);  // (N x SB_BINS words, free once the thresholds are known; F_RADIX <= SB_BINS)
  a.zero_ptr = (uint4*)(b + L.zero_off);
  a.zero_vecs = (uint32_t)((L.votes_done - L.zero_off) / 16);
  a.last_zero = (uint32_t*)(b + L.votes_done);
  a.last_zero_words = (uint32_t)((L.zero_off + L.zero_bytes - L.votes_done) / 4);
  a.spin_limit = 1u << 21;
  a.dbg = p.dbg;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)ctx->sms);
  cfg.blockDim = dim3(FT);
  cfg.dynamicSmemBytes = tail_smem_bytes(p.nc_pad);
  cfg.stream = ctx->stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  // launched early like the other kernels (it waits for the streaming pass at its start) if the runtime takes a
  // cooperative launch that way; otherwise as a plain cooperative launch
  cfg.numAttrs = ctx->tail_pdl >= 0 ? 2 : 1;
  cudaError_t le = cudaLaunchKernelEx(&cfg, k_tail, p, a);
  if (le != cudaSuccess && cfg.numAttrs == 2) {
    cudaGetLastError();
    ctx->tail_pdl = -1;
    cfg.numAttrs = 1;
    le = cudaLaunchKernelEx(&cfg, k_tail, p, a);
  }
  if (le != cudaSuccess) {
    cudaGetLastError();
    return MV_ERR_CUDA;
  }
#ifdef MV_TAIL_STAMPS
  {
    static bool told = false;
    if (!told) {
      told = true;
      fprintf(stderr, "tail kernel launched with %d attribute(s)\n", (int)cfg.numAttrs);
    }
  }
#endif
  MV_LAUNCH_CHECK();
  ctx->clean_bytes = L.zero_bytes;
  return MV_OK;
}

bool small_ready_dev(mv_ctx* ctx) {
  if (ctx->small_state == 0) {
    ctx->small_state = -1;
    int dev = -1, coop = 0, per_sm = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess &&
        coop != 0 &&
        cudaFuncSetAttribute(k_small, cudaFuncAttributeMaxDynamicSharedMemorySize, SK_KEYS * 4) == cudaSuccess &&
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_small, FT, SK_KEYS * 4) == cudaSuccess && per_sm >= 1)
      ctx->small_state = 1;
    else
      cudaGetLastError();
  }
  return ctx->small_state == 1;
}

// rows that fit a CTA's shared memory: the whole step as one kernel, a CTA per worker
bool small_usable(mv_ctx* ctx, int N, int64_t d) {
  return ctx->tail_mode != 0 && ctx->mode != MV_MODE_GENERAL && d <= SMALL_MAX_D && N <= ctx->sms && small_ready_dev(ctx);
}

int small_impl(mv_ctx* ctx, const P& p, const Layout& L, const float* grads, float* err, int32_t* out_idx, float* out_val) {
  char* b = ctx->ws;
  cudaStream_t st = ctx->stream;
  // the kernel keeps its vote bytes, vote histogram and barrier word in two copies that alternate; both are cleared
  // here the first time (and after any other call that used the vote array), from then on by the kernel itself
  const size_t vbytes = (size_t)L.nchunks * CH;
  if (!ctx->small_ready || ctx->small_N != p.N || ctx->small_d != p.d || ctx->small_K != p.K) {
    if (cudaMemsetAsync(b + L.votes, 0, vbytes, st) != cudaSuccess) return MV_ERR_CUDA;
    if (cudaMemsetAsync(b + L.votes_alt, 0, vbytes, st) != cudaSuccess) return MV_ERR_CUDA;
    if (cudaMemsetAsync(b + L.small_state, 0, (512 + 32) * 4, st) != cudaSuccess) return MV_ERR_CUDA;
    ctx->small_flip = 0;
  }
  uint32_t* const sst = (uint32_t*)(b + L.small_state);
  const int f = ctx->small_flip;
  SmallArgs a;
  a.grads = grads;
  a.err = err;
  a.out_idx = out_idx;
  a.out_val = out_val;
  a.votes_now = (uint32_t*)(b + (f ? L.votes_alt : L.votes));
  a.votes_next = (uint32_t*)(b + (f ? L.votes : L.votes_alt));
  a.hist_now = sst + (f ? 256 : 0);
  a.hist_next = sst + (f ? 0 : 256);
  a.bar_now = sst + 512 + (f ? 16 : 0);
  a.bar_next = sst + 512 + (f ? 0 : 16);
  a.abort_flag = (uint32_t*)(b + L.abort_flag);
  a.spin_limit = 1u << 21;
  a.dbg = p.dbg;
  // threshold tracking as in the streaming path: a call that follows one of the same size reads the bounds that
  // call left and leaves its own in the other array
  const bool track = ctx->mode == MV_MODE_TRACK;
  const bool tracked = track && ctx->track_valid && ctx->track_N == p.N && ctx->track_d == p.d && ctx->track_K == p.K;
  if (tracked) ctx->tau_flip ^= 1;
  a.tau_in = tracked ? (const uint32_t*)(b + (ctx->tau_flip ? L.tau_alt : L.tau)) : nullptr;
  a.tau_out = track ? (uint32_t*)(b + (ctx->tau_flip ? L.tau : L.tau_alt)) : nullptr;
  {
    const double r = ceil((double)p.K * 1.35 + 6.0 * sqrt((double)p.K) + 8.0);
    a.track_rank = (uint32_t)(r < (double)p.d ? r : (double)p.d);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)p.N);
  cfg.blockDim = dim3(FT);
  cfg.dynamicSmemBytes = SK_KEYS * 4;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  // launched early (the kernel waits for its predecessor on the stream at its start) if the runtime takes a
  // cooperative launch that way; otherwise as a plain cooperative launch
  cfg.numAttrs = ctx->tail_pdl >= 0 ? 2 : 1;
  cudaError_t le = cudaLaunchKernelEx(&cfg, k_small, p, a);
  if (le != cudaSuccess && cfg.numAttrs == 2) {
    cudaGetLastError();
    ctx->tail_pdl = -1;
    cfg.numAttrs = 1;
    le = cudaLaunchKernelEx(&cfg, k_small, p, a);
  }
  if (le != cudaSuccess) {
    cudaGetLastError();
    return MV_ERR_CUDA;
  }
  MV_LAUNCH_CHECK();
  ctx->small_flip ^= 1;
  ctx->small_ready = true;  // (the kernel cleared the array that the next call votes in)
  ctx->small_N = p.N;
  ctx->small_d = p.d;
  ctx->small_K = p.K;
  ctx->track_valid = track;
  ctx->track_N = p.N;
  ctx->track_d = p.d;
  ctx->track_K = p.K;
  return MV_OK;
}

// has a bounded device-side wait given up on this context?  (reads the workspace header; the stream must be idle)
int abort_status(mv_ctx* ctx) {
  if (!ctx->dbg_ready) return MV_OK;
  uint32_t flag = 0;
  if (cudaMemcpyAsync(&flag, ctx->ws + 8, 4, cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess) return MV_ERR_CUDA;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return MV_ERR_CUDA;
  return flag != 0 ? MV_ERR_TIMEOUT : MV_OK;
}

bool overlap(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
  return x < y + nb && y < x + na;
}

int check_common(const mv_ctx* ctx, int N, int64_t d, int64_t K, Layout& L) {
  if (ctx == nullptr) return MV_ERR_INVALID_ARG;
  if (!sizes_ok(N, d, K)) return MV_ERR_INVALID_ARG;
  L = make_layout(N, d, K);
  if (ctx->ws_bytes < L.total) return MV_ERR_WORKSPACE;
  return MV_OK;
}

}  // namespace

extern "C" {

size_t mv_workspace_bytes(int N, int64_t d, int64_t K) {
  if (!sizes_ok(N, d, K)) return 0;
  return make_layout(N, d, K).total;
}

int mv_create(mv_ctx** out, void* stream, void* workspace, size_t workspace_bytes) {
  if (out == nullptr) return MV_ERR_INVALID_ARG;
  *out = nullptr;
  if (workspace == nullptr || ((uintptr_t)workspace & 255u) != 0) return MV_ERR_INVALID_ARG;
  mv_ctx* c = new (std::nothrow) mv_ctx;
  if (c == nullptr) return MV_ERR_INVALID_ARG;
  c->stream = (cudaStream_t)stream;
  c->ws = (char*)workspace;
  c->ws_bytes = workspace_bytes;
  c->mode = MV_MODE_AUTO;
  c->tau_flip = 0;
  c->track_valid = false;
  c->launches = 0;
  c->clean_bytes = 0;
  c->sms = 0;
  c->cta_budget = 8;
  c->dbg_ready = false;
  c->tail_state = 0;
  c->tail_mode = 1;
  c->tail_pdl = 0;
  c->small_state = 0;
  c->small_ready = false;
  c->small_d = 0;
  c->small_flip = 0;
  c->timing = 0;
  c->timing_calls = 0;
  c->timing_now = false;
  c->timed = 0;
  c->ev_made = false;
  c->phase_timing = 0;
  c->pev_made = false;
  c->side = nullptr;
  c->side_state = 0;
  c->join_pending = false;
  c->last_N = 0;
  c->last_d = 0;
  c->last_K = 0;
  *out = c;
  return MV_OK;
}

int mv_destroy(mv_ctx* ctx) {
  if (ctx == nullptr) return MV_ERR_INVALID_ARG;
  if (ctx->ev_made)
    for (int i = 0; i < 2 * 64; i++) cudaEventDestroy(ctx->ev[i]);
  if (ctx->pev_made)
    for (int i = 0; i < 48; i++) cudaEventDestroy(ctx->pev[i]);
  if (ctx->side_state == 1) {
    cudaEventDestroy(ctx->ev_fork);
    cudaEventDestroy(ctx->ev_join);
    cudaEventDestroy(ctx->ev_zero);
    cudaStreamDestroy(ctx->side);
  }
  delete ctx;
  return MV_OK;
}

int mv_set_kernel_timing(mv_ctx* ctx, int enable) {
  if (ctx == nullptr) return MV_ERR_INVALID_ARG;
  if (enable && !ctx->ev_made) {
    for (int i = 0; i < 2 * 64; i++)
      if (cudaEventCreate(&ctx->ev[i]) != cudaSuccess) return MV_ERR_CUDA;
    ctx->ev_made = true;
  }
  ctx->timing = enable > 0 ? enable : 0;
  ctx->timing_calls = 0;
  ctx->timed = 0;
  return MV_OK;
}

int mv_set_phase_timing(mv_ctx* ctx, int enable) {
  if (ctx == nullptr) return MV_ERR_INVALID_ARG;
  if (enable && !ctx->pev_made) {
    for (int i = 0; i < 48; i++)
      if (cudaEventCreate(&ctx->pev[i]) != cudaSuccess) return MV_ERR_CUDA;
    ctx->pev_made = true;
  }
  ctx->phase_timing = enable > 0 ? enable : 0;  // 1: every launch; 100 + i: only the start and launch i
  return MV_OK;
}

int mv_read_phase_times(mv_ctx* ctx, float* ms, int capacity, int* count) {
  if (ctx == nullptr || ms == nullptr || count == nullptr || !ctx->pev_made) return MV_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return MV_ERR_CUDA;
  if (ctx->phase_timing >= 100) {  // single probe: time from the start of the call to the end of launch i
    const int i = ctx->phase_timing - 100;
    if (i < 1 || i > ctx->launches || i > 47 || capacity < 1) return MV_ERR_INVALID_ARG;
    if (cudaEventElapsedTime(&ms[0], ctx->pev[0], ctx->pev[i]) != cudaSuccess) return MV_ERR_CUDA;
    *count = 1;
    return MV_OK;
  }
  int n = ctx->launches < 47 ? ctx->launches : 47;
  if (n > capacity) n = capacity;
  for (int i = 0; i < n; i++)
    if (cudaEventElapsedTime(&ms[i], ctx->pev[i], ctx->pev[i + 1]) != cudaSuccess) return MV_ERR_CUDA;
  *count = n;
  return MV_OK;
}

int mv_read_kernel_timing(mv_ctx* ctx, float* total_ms, int* launches) {
  if (ctx == nullptr || total_ms == nullptr || launches == nullptr || !ctx->ev_made) return MV_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return MV_ERR_CUDA;
  const int cnt = ctx->timed < 64 ? ctx->timed : 64;
  float sum = 0.f;
  for (int i = 0; i < cnt; i++) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->ev[2 * i], ctx->ev[2 * i + 1]) != cudaSuccess) return MV_ERR_CUDA;
    sum += ms;
  }
  *total_ms = sum;
  *launches = cnt;
  ctx->timed = 0;
  return MV_OK;
}

int mv_set_tail_kernel(mv_ctx* ctx, int enable) {
  if (ctx == nullptr) return MV_ERR_INVALID_ARG;
  if (enable < 0 || enable > 2) return MV_ERR_INVALID_ARG;
  ctx->tail_mode = enable;
  return MV_OK;
}

int mv_set_mode(mv_ctx* ctx, int mode) {
  if (ctx == nullptr || (mode != MV_MODE_AUTO && mode != MV_MODE_GENERAL && mode != MV_MODE_TRACK))
    return MV_ERR_INVALID_ARG;
  ctx->mode = mode;
  ctx->track_valid = false;
  return MV_OK;
}

int mv_vote(mv_ctx* ctx, const float* grads, float* err, int N, int64_t d, int64_t K, int32_t* worker_idx,
            uint32_t* worker_bits, uint8_t* votes, uint32_t* thresh) {
  Layout L;
  const int rc = check_common(ctx, N, d, K, L);
  if (rc != MV_OK) return rc;
  if (grads == nullptr || err == nullptr || !aligned16(grads) || !aligned16(err)) return MV_ERR_INVALID_ARG;
  const size_t nb = (size_t)N * (size_t)d * 4;
  if (overlap(grads, nb, err, nb)) return MV_ERR_INVALID_ARG;
  if ((worker_idx && !aligned16(worker_idx)) || (worker_bits && !aligned16(worker_bits)) ||
      (votes && !aligned16(votes)) || (thresh && !aligned16(thresh)))
    return MV_ERR_INVALID_ARG;
  if (const int rd = device_ready(ctx)) return rd;
  ctx->launches = 0;
  if (ctx->phase_timing) cudaEventRecord(ctx->pev[0], ctx->stream);
  P p = make_params(ctx, L, N, d, K);
  if (worker_idx) p.worker_idx = worker_idx;
  if (worker_bits) p.worker_bits = worker_bits;
  if (votes) p.votes = votes;
  if (thresh) p.thresh = thresh;
  ctx->last_N = N;
  ctx->last_d = d;
  ctx->last_K = K;
  const int rc2 = vote_impl(ctx, p, L, grads, err, false, true, worker_idx != nullptr, worker_bits != nullptr);
  const int rc3 = join_side(ctx);
  return rc2 != MV_OK ? rc2 : rc3;
}

int mv_select(mv_ctx* ctx, const uint8_t* votes, int N, int64_t d, int64_t K, int32_t* out_idx, uint32_t* mask_bits) {
  Layout L;
  const int rc = check_common(ctx, N, d, K, L);
  if (rc != MV_OK) return rc;
  if (votes == nullptr || out_idx == nullptr || !aligned16(votes) || !aligned16(out_idx)) return MV_ERR_INVALID_ARG;
  if (mask_bits && !aligned16(mask_bits)) return MV_ERR_INVALID_ARG;
  if (const int rd = device_ready(ctx)) return rd;
  ctx->launches = 0;
  if (ctx->phase_timing) cudaEventRecord(ctx->pev[0], ctx->stream);
  P p = make_params(ctx, L, N, d, K);
  return select_impl(ctx, p, L, votes, false, out_idx, mask_bits);
}

int mv_aggregate(mv_ctx* ctx, float* acc, int N, int64_t d, int64_t K, const int32_t* idx, float* out_val) {
  Layout L;
  const int rc = check_common(ctx, N, d, K, L);
  if (rc != MV_OK) return rc;
  if (acc == nullptr || idx == nullptr || out_val == nullptr || !aligned16(acc) || !aligned16(idx) || !aligned16(out_val))
    return MV_ERR_INVALID_ARG;
  if (const int rd = device_ready(ctx)) return rd;
  ctx->launches = 0;
  if (ctx->phase_timing) cudaEventRecord(ctx->pev[0], ctx->stream);
  return aggregate_impl(ctx, acc, N, d, K, idx, out_val, 0);
}

int mv_aggregate_partial(mv_ctx* ctx, float* acc, int N_local, int64_t d, int64_t K, const int32_t* idx,
                         double* out_sum) {
  Layout L;
  const int rc = check_common(ctx, N_local, d, K, L);
  if (rc != MV_OK) return rc;
  if (acc == nullptr || idx == nullptr || out_sum == nullptr || !aligned16(acc) || !aligned16(idx) || !aligned16(out_sum))
    return MV_ERR_INVALID_ARG;
  if (const int rd = device_ready(ctx)) return rd;
  ctx->launches = 0;
  if (ctx->phase_timing) cudaEventRecord(ctx->pev[0], ctx->stream);
  return aggregate_impl(ctx, acc, N_local, d, K, idx, nullptr, 0, out_sum);
}

int mv_finish_mean(void* stream, const double* sum, int64_t K, int N_total, float* out_val) {
  if (sum == nullptr || out_val == nullptr || K < 1 || N_total < 1 || !aligned16(sum) || !aligned16(out_val))
    return MV_ERR_INVALID_ARG;
  k_finish_mean<<<(unsigned)((K + TPB - 1) / TPB), TPB, 0, (cudaStream_t)stream>>>(sum, K, (double)N_total, out_val);
  return cudaGetLastError() == cudaSuccess ? MV_OK : MV_ERR_CUDA;
}

int mv_sparse_step(mv_ctx* ctx, const float* grads, float* err, int N, int64_t d, int64_t K, int32_t* out_idx,
                   float* out_val) {
  Layout L;
  int rc = check_common(ctx, N, d, K, L);
  if (rc != MV_OK) return rc;
  if (grads == nullptr || err == nullptr || out_idx == nullptr || out_val == nullptr) return MV_ERR_INVALID_ARG;
  if (!aligned16(grads) || !aligned16(err) || !aligned16(out_idx) || !aligned16(out_val)) return MV_ERR_INVALID_ARG;
  const size_t nb = (size_t)N * (size_t)d * 4;
  if (overlap(grads, nb, err, nb)) return MV_ERR_INVALID_ARG;
  if (const int rd = device_ready(ctx)) return rd;
  ctx->launches = 0;
  if (ctx->phase_timing) cudaEventRecord(ctx->pev[0], ctx->stream);
  P p = make_params(ctx, L, N, d, K);
  ctx->last_N = N;
  ctx->last_d = d;
  ctx->last_K = K;
  if (small_usable(ctx, N, d)) {
    P ps = p;
    return small_impl(ctx, ps, L, grads, err, out_idx, out_val);
  }
  if (tail_usable(ctx, L, N, K)) {
    // two kernels: the streaming pass, then everything else (select, picks, votes, shared mask, aggregate) in one
    P pt = p;
    rc = vote_impl(ctx, p, L, grads, err, false, true, false, false, true, &pt);
    if (rc == MV_OK) rc = tail_impl(ctx, pt, L, err, out_idx, out_val);
    return rc;
  }
  rc = vote_impl(ctx, p, L, grads, err, false, true, false, false);  // (the workers' lists and masks are no output of the step)
  p.prefetch_acc = err;
  if (rc == MV_OK) rc = select_impl(ctx, p, L, p.votes, true, out_idx, nullptr);
  if (rc == MV_OK) rc = aggregate_impl(ctx, err, N, d, K, out_idx, out_val, L.zero_bytes);
  const int rcj = join_side(ctx);
  return rc != MV_OK ? rc : rcj;
}

int mv_topk_union_step(mv_ctx* ctx, const float* grads, float* err, int N, int64_t d, int64_t K, int32_t* out_idx,
                       float* out_val, int64_t capacity, int32_t* count) {
  Layout L;
  int rc = check_common(ctx, N, d, K, L);
  if (rc != MV_OK) return rc;
  if (grads == nullptr || err == nullptr || out_idx == nullptr || out_val == nullptr || count == nullptr)
    return MV_ERR_INVALID_ARG;
  if (!aligned16(grads) || !aligned16(err) || !aligned16(out_idx) || !aligned16(out_val) || ((uintptr_t)count & 3u) != 0)
    return MV_ERR_INVALID_ARG;
  const int64_t most = (int64_t)N * K < d ? (int64_t)N * K : d;  // the union cannot hold more
  if (capacity < most || capacity >= ((int64_t)1 << 31)) return MV_ERR_INVALID_ARG;
  const size_t nb = (size_t)N * (size_t)d * 4;
  if (overlap(grads, nb, err, nb)) return MV_ERR_INVALID_ARG;
  if (const int rd = device_ready(ctx)) return rd;
  ctx->launches = 0;
  if (ctx->phase_timing) cudaEventRecord(ctx->pev[0], ctx->stream);
  P p = make_params(ctx, L, N, d, K);
  p.take_all = 1;
  ctx->last_N = N;
  ctx->last_d = d;
  ctx->last_K = K;
  // the workers' masks (kept in the workspace), the votes, and the offsets of all voted coordinates
  rc = vote_impl(ctx, p, L, grads, err, false, true, false, true);
  if (rc != MV_OK) return rc;
  P w = p;
  w.K = capacity;  // room of the list that k_vote_write fills
  rc = select_impl(ctx, w, L, p.votes, true, out_idx, nullptr);
  if (rc != MV_OK) return rc;
  launch_k(k_union_gather, dim3((unsigned)((capacity + TPB - 1) / TPB)), dim3(TPB), ctx->stream, err, N, d, L.W,
           (const uint32_t*)p.worker_bits, out_idx, (const uint32_t*)(p.out_base + p.nchunks), out_val, capacity, count,
           (uint4*)(ctx->ws + L.zero_off), (uint32_t)(L.zero_bytes / 16));
  MV_LAUNCH_CHECK();
  ctx->clean_bytes = L.zero_bytes;
  return join_side(ctx);
}

int mv_ad_step(mv_ctx* ctx, const float* grads, float* err, uint32_t* prev_bits, int N, int64_t d, int64_t K,
               int64_t K_ad, int32_t* out_idx, float* out_val, uint32_t* add_bits, uint32_t* drop_bits, uint8_t* msum) {
  Layout L;
  int rc = check_common(ctx, N, d, K, L);
  if (rc != MV_OK) return rc;
  if (K_ad < 1 || K_ad > K) return MV_ERR_INVALID_ARG;
  if (grads == nullptr || err == nullptr || prev_bits == nullptr || out_idx == nullptr || out_val == nullptr)
    return MV_ERR_INVALID_ARG;
  if (!aligned16(grads) || !aligned16(err) || !aligned16(prev_bits) || !aligned16(out_idx) || !aligned16(out_val))
    return MV_ERR_INVALID_ARG;
  if ((add_bits && !aligned16(add_bits)) || (drop_bits && !aligned16(drop_bits)) || (msum && !aligned16(msum)))
    return MV_ERR_INVALID_ARG;
  const size_t nb = (size_t)N * (size_t)d * 4;
  if (overlap(grads, nb, err, nb)) return MV_ERR_INVALID_ARG;
  if (const int rd = device_ready(ctx)) return rd;
  ctx->launches = 0;
  if (ctx->phase_timing) cudaEventRecord(ctx->pev[0], ctx->stream);
  cudaStream_t st = ctx->stream;
  P p = make_params(ctx, L, N, d, K);
  ctx->last_N = N;
  ctx->last_d = d;
  ctx->last_K = K;
  char* b = ctx->ws;
  // without add/drop outputs the picks update the vote masks in place (set for add, clear for drop);
  // otherwise they are materialised as 2N masks first and applied by k_ad_apply
  const bool direct = add_bits == nullptr && drop_bits == nullptr;
  // this step's top-K masks M_n (kept in the workspace); err now holds acc
  rc = vote_impl(ctx, p, L, grads, err, true);
  if (rc != MV_OK) return rc;
  // the add and drop selections: 2N lists through the select kernels in list mode
  P a = p;
  a.N = 2 * N;
  a.K = K_ad;
  a.cap = L.ad_cap;
  a.list_mode = 1;
  a.force_general = 0;
  a.hist1 = (uint32_t*)(b + L.ad_hist1);
  a.hist2 = (uint32_t*)(b + L.ad_hist2);
  a.hist3 = (uint32_t*)(b + L.ad_hist3);
  a.cand_cnt = (uint32_t*)(b + L.ad_cnt);
  a.count_done = (uint32_t*)(b + L.ad_count_done);
  a.worker_bits = (uint32_t*)(b + L.ad_bits);
  a.wstate = (uint32_t*)(b + L.ad_wstate);
  a.thresh = (uint32_t*)(b + L.ad_thresh);
  a.diag_cnt = (uint32_t*)(b + L.ad_diag);
  a.cand = (uint2*)(b + L.ad_cand);
  a.chunk_base = (uint32_t*)(b + L.ad_chunk_base);
  a.chunk_cnt = (uint32_t*)(b + L.ad_chunk_cnt);
  a.chunk_eq = (uint32_t*)(b + L.ad_chunk_eq);
  a.tie_base = (uint32_t*)(b + L.ad_tie_base);
  a.apply_rows = N;
  a.apply_bits = direct ? prev_bits : nullptr;
  // (the list state is cleared by a memset here, not by the picks kernel as in the random-selection step: measured,
  // the step is 4 us faster this way -- the memset keeps the list fill from being launched while the picks still run)
  if (cudaMemsetAsync(b + L.ad_zero, 0, direct ? L.ad_bits - L.ad_zero : L.ad_zero_bytes, st) != cudaSuccess)
    return MV_ERR_CUDA;
  launch_k(k_ad_fill, dim3(dim3((p.nchunks + TPB / 32 - 1) / (TPB / 32), N)), dim3(TPB), st, p, a,
           (const uint32_t*)prev_bits, (const float*)err);
  MV_LAUNCH_CHECK();
  const int ga = per_row_ctas(2 * N, (int)((a.cap + TPB * 8 - 1) / (TPB * 8)), ctx->sms * 2);
  if (a.cap <= (1u << 20) && cluster_select_ready()) {
    // a cluster per list finds the key of its K_ad-th entry (three radix digits; nothing is cleared here)
    const int rows = 2 * N;
    if (rows * 8 <= ctx->cta_budget) launch_smem(k_select_cluster<8>, dim3(dim3(8, rows)), dim3(ST), SK_KEYS * 4, st, a, err, rows, rows);
    else launch_smem(k_select_cluster<4>, dim3(dim3(4, rows)), dim3(ST), SK_KEYS * 4, st, a, err, rows, rows);
    MV_LAUNCH_CHECK();
  } else {
    launch_k(k_hist<1, false>, dim3(dim3(ga, 2 * N)), dim3(TPB), st, a, nullptr, err);
    MV_LAUNCH_CHECK();
    launch_k(k_hist<2, false>, dim3(dim3(ga, 2 * N)), dim3(TPB), st, a, nullptr, err);
    MV_LAUNCH_CHECK();
    launch_k(k_hist<3, false>, dim3(dim3(ga, 2 * N)), dim3(TPB), st, a, nullptr, err);
    MV_LAUNCH_CHECK();
    launch_k(k_count, dim3(dim3(ga, 2 * N)), dim3(TPB), st, a, err);
    MV_LAUNCH_CHECK();
  }
  launch_k(k_set_bits, dim3(dim3(ga, 2 * N)), dim3(TPB), st, a, err);
  MV_LAUNCH_CHECK();
  if (!direct) {
    const size_t words = (size_t)N * (size_t)p.W;
    launch_k(k_ad_apply, dim3((unsigned)((words + TPB * 4 - 1) / (TPB * 4))), dim3(TPB), st, prev_bits,
             (const uint32_t*)a.worker_bits, add_bits, drop_bits, words);
    MV_LAUNCH_CHECK();
  }
  // votes of the updated masks (= the server's running sum, Eq. 16), shared mask, aggregate
  P v = p;
  v.worker_bits = prev_bits;
  if (msum) v.votes = msum;
  if (cudaMemsetAsync(p.hot, 1, (size_t)p.nc_pad, st) != cudaSuccess) return MV_ERR_CUDA;  // every chunk may hold votes
  {
    const dim3 gv(p.nchunks < ctx->sms * 8 ? p.nchunks : ctx->sms * 8);
    if (N < 4) launch_k(k_votes<2>, gv, dim3(VT), st, v);
    else if (N < 16) launch_k(k_votes<4>, gv, dim3(VT), st, v);
    else if (N < 64) launch_k(k_votes<6>, gv, dim3(VT), st, v);
    else launch_k(k_votes<8>, gv, dim3(VT), st, v);
  }
  MV_LAUNCH_CHECK();
  // Fewer than K coordinates may hold a vote here (v* = 0).  k_votes visited every chunk, so its
  // per-chunk counts include the unvoted coordinates and its scan is valid in that case too.
  rc = select_impl(ctx, v, L, v.votes, true, out_idx, nullptr);
  if (rc != MV_OK) return rc;
  return aggregate_impl(ctx, err, N, d, K, out_idx, out_val, L.zero_bytes);
}

}  // extern "C" (reopened below)

namespace {

// P for the add-drop / random-selection lists: the select state once more, over `rows` lists
P list_params(const mv_ctx* ctx, const Layout& L, const P& p, int rows, int64_t K_list, uint32_t cap) {
  char* b = ctx->ws;
  P a = p;
  a.N = rows;
  a.K = K_list;
  a.cap = cap;
  a.list_mode = 1;
  a.force_general = 0;
  a.tau_next = nullptr;
  a.hist1 = (uint32_t*)(b + L.ad_hist1);
  a.hist2 = (uint32_t*)(b + L.ad_hist2);
  a.hist3 = (uint32_t*)(b + L.ad_hist3);
  a.cand_cnt = (uint32_t*)(b + L.ad_cnt);
  a.count_done = (uint32_t*)(b + L.ad_count_done);
  a.worker_bits = (uint32_t*)(b + L.ad_bits);
  a.wstate = (uint32_t*)(b + L.ad_wstate);
  a.thresh = (uint32_t*)(b + L.ad_thresh);
  a.diag_cnt = (uint32_t*)(b + L.ad_diag);
  a.cand = (uint2*)(b + L.ad_cand);
  a.chunk_base = (uint32_t*)(b + L.ad_chunk_base);
  a.chunk_cnt = (uint32_t*)(b + L.ad_chunk_cnt);
  a.chunk_eq = (uint32_t*)(b + L.ad_chunk_eq);
  a.tie_base = (uint32_t*)(b + L.ad_tie_base);
  a.apply_rows = 0;
  a.apply_bits = nullptr;
  a.zero2_ptr = nullptr;
  a.zero2_vecs = 0;
  return a;
}

// bytes of list state that a random selection wants clear: the select state and one row of mask words (whole 16-byte units)
size_t rs_zero_bytes(const Layout& L, int64_t W) { return (((L.ad_bits - L.ad_zero) + (size_t)W * 4) + 15) & ~(size_t)15; }

// S_rand-weighted: voted coordinates with their ring times into one list, the K earliest through the
// list-mode select into a bit mask, the mask into an ascending index list
// `cleared`: the list state was cleared by the picks kernel of the step that calls (p.zero2_ptr)
int rs_select_impl(mv_ctx* ctx, const P& p, const Layout& L, const uint8_t* votes, uint64_t seed, uint64_t draw,
                   int32_t* out_idx, uint32_t* mask_bits, bool cleared = false) {
  cudaStream_t st = ctx->stream;
  char* b = ctx->ws;
  // The list regions written here sit at offsets of this call's own (N, d, K): they may overlap the
  // region that a whole step of another size left cleared, so nothing counts as clean from here on
  // (a whole step that follows gets the zeros back from its last kernel).
  ctx->clean_bytes = 0;
  ctx->small_ready = false;
  // one list that can hold every voted coordinate (at most min(d, N K) of them)
  const uint64_t room = (uint64_t)2 * (uint64_t)p.N * (uint64_t)L.ad_cap;
  P a = list_params(ctx, L, p, 1, p.K, (uint32_t)(room < 0xfffffff8ull ? room : 0xfffffff8ull));
  if (!cleared && cudaMemsetAsync(b + L.ad_zero, 0, rs_zero_bytes(L, p.W), st) != cudaSuccess) return MV_ERR_CUDA;
  launch_k(k_rs_fill, dim3(p.nchunks), dim3(TPB), st, p, a, votes, (uint32_t)seed, (uint32_t)(seed >> 32), (uint32_t)draw,
           (uint32_t)(draw >> 32), out_idx);
  MV_LAUNCH_CHECK();
  uint64_t most = (uint64_t)p.N * (uint64_t)p.K;
  if (most > (uint64_t)p.d) most = (uint64_t)p.d;
  const int ga = per_row_ctas(1, (int)((most + TPB * 8 - 1) / (TPB * 8)), ctx->sms * 2);
  launch_k(k_hist<1, false>, dim3(dim3(ga, 1)), dim3(TPB), st, a, nullptr, nullptr);
  MV_LAUNCH_CHECK();
  launch_k(k_hist<2, false>, dim3(dim3(ga, 1)), dim3(TPB), st, a, nullptr, nullptr);
  MV_LAUNCH_CHECK();
  launch_k(k_hist<3, false>, dim3(dim3(ga, 1)), dim3(TPB), st, a, nullptr, nullptr);
  MV_LAUNCH_CHECK();
  launch_k(k_count, dim3(dim3(ga, 1)), dim3(TPB), st, a, nullptr);
  MV_LAUNCH_CHECK();
  launch_k(k_set_bits, dim3(dim3(ga, 1)), dim3(TPB), st, a, nullptr);
  MV_LAUNCH_CHECK();
  P r = a;
  r.list_mode = 0;
  r.chunk_sel = (uint32_t*)(b + L.rs_chunk_sel);
  r.worker_idx = out_idx;
  launch_k(k_chunk_popc, dim3((p.nchunks + TPB / 32 - 1) / (TPB / 32)), dim3(TPB), st, (const uint32_t*)a.worker_bits, p.W,
           p.nchunks, r.chunk_sel);
  MV_LAUNCH_CHECK();
  launch_k(k_scan_sel, dim3(1), dim3(1024), st, r);
  MV_LAUNCH_CHECK();
  launch_k(k_lists, dim3(dim3((p.nchunks + TPB / 32 - 1) / (TPB / 32), 1)), dim3(TPB), st, r);
  MV_LAUNCH_CHECK();
  if (mask_bits &&
      cudaMemcpyAsync(mask_bits, a.worker_bits, (size_t)p.W * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return MV_ERR_CUDA;
  return MV_OK;
}

}  // namespace

extern "C" {

int mv_select_rs(mv_ctx* ctx, const uint8_t* votes, int N, int64_t d, int64_t K, uint64_t seed, uint64_t draw,
                 int32_t* out_idx, uint32_t* mask_bits) {
  Layout L;
  const int rc = check_common(ctx, N, d, K, L);
  if (rc != MV_OK) return rc;
  if (votes == nullptr || out_idx == nullptr || !aligned16(votes) || !aligned16(out_idx)) return MV_ERR_INVALID_ARG;
  if (mask_bits && !aligned16(mask_bits)) return MV_ERR_INVALID_ARG;
  if (const int rd = device_ready(ctx)) return rd;
  ctx->launches = 0;
  if (ctx->phase_timing) cudaEventRecord(ctx->pev[0], ctx->stream);
  const P p = make_params(ctx, L, N, d, K);
  return rs_select_impl(ctx, p, L, votes, seed, draw, out_idx, mask_bits);
}

int mv_rs_step(mv_ctx* ctx, const float* grads, float* err, int N, int64_t d, int64_t K, uint64_t seed, uint64_t draw,
               int32_t* out_idx, float* out_val) {
  Layout L;
  int rc = check_common(ctx, N, d, K, L);
  if (rc != MV_OK) return rc;
  if (grads == nullptr || err == nullptr || out_idx == nullptr || out_val == nullptr) return MV_ERR_INVALID_ARG;
  if (!aligned16(grads) || !aligned16(err) || !aligned16(out_idx) || !aligned16(out_val)) return MV_ERR_INVALID_ARG;
  const size_t nb = (size_t)N * (size_t)d * 4;
  if (overlap(grads, nb, err, nb)) return MV_ERR_INVALID_ARG;
  if (const int rd = device_ready(ctx)) return rd;
  ctx->launches = 0;
  if (ctx->phase_timing) cudaEventRecord(ctx->pev[0], ctx->stream);
  P p = make_params(ctx, L, N, d, K);
  ctx->last_N = N;
  ctx->last_d = d;
  ctx->last_K = K;
  // (the picks kernel also clears the list state of the selection that follows)
  p.zero2_ptr = (uint4*)(ctx->ws + L.ad_zero);
  p.zero2_vecs = (uint32_t)(rs_zero_bytes(L, L.W) / 16);
  rc = vote_impl(ctx, p, L, grads, err, false, false, false, false);  // the random selection reads the votes themselves
  p.zero2_ptr = nullptr;
  // the union of N top-K sets holds at least K coordinates, so the mask is always full
  if (rc == MV_OK) rc = rs_select_impl(ctx, p, L, p.votes, seed, draw, out_idx, nullptr, true);
  if (rc == MV_OK) rc = aggregate_impl(ctx, err, N, d, K, out_idx, out_val, L.zero_bytes);
  const int rcj = join_side(ctx);
  return rc != MV_OK ? rc : rcj;
}

int mv_sparse_step_host(mv_ctx* ctx, const float* h_grads, int N, int64_t d, int64_t K, int32_t* h_out_idx,
                        float* h_out_val, float* d_grads, float* d_err, int32_t* d_out_idx, float* d_out_val) {
  Layout L;
  int rc = check_common(ctx, N, d, K, L);
  if (rc != MV_OK) return rc;
  if (h_grads == nullptr || h_out_idx == nullptr || h_out_val == nullptr) return MV_ERR_INVALID_ARG;
  if (d_grads == nullptr || d_err == nullptr || d_out_idx == nullptr || d_out_val == nullptr) return MV_ERR_INVALID_ARG;
  if (!aligned16(d_grads) || !aligned16(d_err) || !aligned16(d_out_idx) || !aligned16(d_out_val)) return MV_ERR_INVALID_ARG;
  const size_t nb = (size_t)N * (size_t)d * 4;
  if (overlap(d_grads, nb, d_err, nb)) return MV_ERR_INVALID_ARG;
  if (cudaMemcpyAsync(d_grads, h_grads, nb, cudaMemcpyHostToDevice, ctx->stream) != cudaSuccess) return MV_ERR_CUDA;
  rc = mv_sparse_step(ctx, d_grads, d_err, N, d, K, d_out_idx, d_out_val);
  if (rc != MV_OK) return rc;
  if (cudaMemcpyAsync(h_out_idx, d_out_idx, (size_t)K * 4, cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess)
    return MV_ERR_CUDA;
  if (cudaMemcpyAsync(h_out_val, d_out_val, (size_t)K * 4, cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess)
    return MV_ERR_CUDA;
  return abort_status(ctx);  // (waits for the stream)
}

int mv_read_diag(mv_ctx* ctx, int N, uint32_t* per_worker) {
  if (ctx == nullptr || per_worker == nullptr || N < 1 || N != ctx->last_N) return MV_ERR_INVALID_ARG;
  const Layout L = make_layout(ctx->last_N, ctx->last_d, ctx->last_K);
  uint32_t* cnt = (uint32_t*)malloc((size_t)N * 8);
  if (cnt == nullptr) return MV_ERR_INVALID_ARG;
  uint32_t* tau = cnt + N;
  cudaError_t e = cudaMemcpyAsync(cnt, ctx->ws + L.diag_cnt, (size_t)N * 4, cudaMemcpyDeviceToHost, ctx->stream);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(tau, ctx->ws + (ctx->tau_flip ? L.tau_alt : L.tau), (size_t)N * 4, cudaMemcpyDeviceToHost, ctx->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
  const int ab = e == cudaSuccess ? abort_status(ctx) : MV_ERR_CUDA;
  if (ab != MV_OK) {
    free(cnt);
    return ab;
  }
  for (int n = 0; n < N; n++) {
    const bool general = ctx->mode == MV_MODE_GENERAL || cnt[n] < (uint32_t)ctx->last_K || cnt[n] > L.cap;
    per_worker[n * 4 + 0] = cnt[n];
    per_worker[n * 4 + 1] = ctx->mode == MV_MODE_GENERAL ? 0u : tau[n];
    per_worker[n * 4 + 2] = general ? 1u : 0u;
    per_worker[n * 4 + 3] = 0u;
  }
  free(cnt);
  return MV_OK;
}

int mv_last_launches(const mv_ctx* ctx) { return ctx ? ctx->launches : 0; }

int mv_fallback_count(mv_ctx* ctx, uint32_t* total) {
  if (ctx == nullptr || total == nullptr) return MV_ERR_INVALID_ARG;
  *total = 0;
  if (!ctx->dbg_ready) return MV_OK;  // no call yet
  if (cudaMemcpyAsync(total, ctx->ws + 4, 4, cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess) return MV_ERR_CUDA;
  return abort_status(ctx);  // (waits for the stream)
}

int mv_debug_build(void) { return kChecked ? 1 : 0; }

int mv_debug_status(mv_ctx* ctx, int* device_status) {
  if (ctx == nullptr || device_status == nullptr) return MV_ERR_INVALID_ARG;
  *device_status = 0;
  if (!kChecked || !ctx->dbg_ready) return MV_OK;  // an unchecked build sets no bits; no call yet: nothing to read
  uint32_t word = 0;
  if (cudaMemcpyAsync(&word, ctx->ws, 4, cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess) return MV_ERR_CUDA;
  if (cudaMemsetAsync(ctx->ws, 0, 4, ctx->stream) != cudaSuccess) return MV_ERR_CUDA;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return MV_ERR_CUDA;
  *device_status = (int)word;
  return abort_status(ctx);
}

// ---------------------------------------------------------------------------------------------
// mv_select_static: the shared-mask selection with its scratch in a fixed device array
// ---------------------------------------------------------------------------------------------
}  // extern "C" (reopened below)

namespace {

constexpr int64_t STATIC_MAX_D = (int64_t)MV_SELECT_STATIC_MAX_D;
constexpr int STATIC_MAX_CHUNKS = (int)((STATIC_MAX_D + CH - 1) / CH);
// fixed layout inside the array (offsets in bytes, each a multiple of 256)
constexpr size_t ST_VOTES_DONE = 0;                                   // ticket counter, must start at zero
constexpr size_t ST_VOTE_HIST = 256;                                  // 256 counters, must start at zero
constexpr size_t ST_VSTATE = ST_VOTE_HIST + 256 * 4;
constexpr size_t ST_OUT_BASE = ST_VSTATE + 256;
constexpr size_t ST_TIE_TAKE = ST_OUT_BASE + (((size_t)STATIC_MAX_CHUNKS + 1) * 4 + 255) / 256 * 256;
constexpr size_t ST_CHUNK_VH = ST_TIE_TAKE + ((size_t)STATIC_MAX_CHUNKS * 4 + 255) / 256 * 256;
constexpr size_t ST_TOTAL = ST_CHUNK_VH + (size_t)256 * STATIC_MAX_CHUNKS * 2;

// Lives in the module's image on every GPU that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_select_scratch[ST_TOTAL];

// In host code the name g_select_scratch is only a handle for the runtime, not a device address:
// the address a kernel can use is asked for once per device and remembered here.
constexpr int MAX_DEVICES = 64;
unsigned char* g_select_scratch_addr[MAX_DEVICES] = {nullptr};

int select_scratch_address(unsigned char** out) {
  static std::mutex mu;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return MV_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  if (g_select_scratch_addr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_select_scratch) != cudaSuccess || ptr == nullptr) return MV_ERR_CUDA;
    g_select_scratch_addr[dev] = (unsigned char*)ptr;
  }
  *out = g_select_scratch_addr[dev];
  return MV_OK;
}

}  // namespace

extern "C" {

int mv_select_static(void* stream, const uint8_t* votes, int N, int64_t d, int64_t K, int32_t* out_idx,
                     uint32_t* mask_bits) {
  if (!sizes_ok(N, d, K)) return MV_ERR_INVALID_ARG;
  if (d > STATIC_MAX_D) return MV_ERR_TOO_LARGE;
  if (votes == nullptr || out_idx == nullptr || !aligned16(votes) || !aligned16(out_idx)) return MV_ERR_INVALID_ARG;
  if (mask_bits && !aligned16(mask_bits)) return MV_ERR_INVALID_ARG;
  unsigned char* base = nullptr;
  const int rc = select_scratch_address(&base);
  if (rc != MV_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  P p = {};
  p.N = N;
  p.nchunks = (int)((d + CH - 1) / CH);
  p.nc_pad = (p.nchunks + 7) & ~7;
  p.d = d;
  p.K = K;
  p.W = (d + 31) / 32;
  p.votes_done = (uint32_t*)(base + ST_VOTES_DONE);
  p.vote_hist = (uint32_t*)(base + ST_VOTE_HIST);
  p.vstate = (uint32_t*)(base + ST_VSTATE);
  p.out_base = (uint32_t*)(base + ST_OUT_BASE);
  p.tie_take = (uint32_t*)(base + ST_TIE_TAKE);
  p.chunk_vh = (uint16_t*)(base + ST_CHUNK_VH);
  // the array keeps whatever the last call left: the ticket and the vote histogram start at zero
  if (cudaMemsetAsync(base, 0, ST_VSTATE, st) != cudaSuccess) return MV_ERR_CUDA;
  if (launch_k(k_vote_hist, dim3((p.nchunks + VH_WARPS - 1) / VH_WARPS), dim3(TPB), st, p, votes, (uint8_t*)nullptr) != cudaSuccess)
    return MV_ERR_CUDA;
  if (launch_k(k_vote_write, dim3(p.nchunks), dim3(TPB), st, p, votes, out_idx, mask_bits) != cudaSuccess)
    return MV_ERR_CUDA;
  if (cudaGetLastError() != cudaSuccess) return MV_ERR_CUDA;
  return MV_OK;
}

const char* mv_status_string(int status) {
  switch (status) {
    case MV_OK: return "ok";
    case MV_ERR_INVALID_ARG: return "invalid argument (null or misaligned pointer, size out of range, or grads overlapping err)";
    case MV_ERR_WORKSPACE: return "workspace smaller than mv_workspace_bytes(N, d, K)";
    case MV_ERR_CUDA: return "the CUDA runtime reported an error";
    case MV_ERR_TIMEOUT: return "a bounded wait between the CTAs of a kernel gave up; results of this context are not valid";
    case MV_ERR_TOO_LARGE: return "d exceeds MV_SELECT_STATIC_MAX_D, the size the built-in scratch array of mv_select_static was compiled for";
    default: return "unknown status";
  }
}

}  // extern "C"
