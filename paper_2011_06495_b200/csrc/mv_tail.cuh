// mv_tail.cuh -- everything of a whole step that follows the streaming pass, as ONE persistent kernel.
// (Included by mv_sparse.cu inside its anonymous namespace, after the helpers it uses.)
//
// After the streaming pass every worker has its candidate buffer; what is left of Algorithm 1 is short,
// strictly ordered work: T_n per worker (S_top, Eq. 6), the votes (Eq. 9, inner sum), the K most voted
// coordinates (Eq. 9, outer S_top), the mean on them and the residual (Eq. 8, error update).  As separate
// kernels each of these steps pays a drain, a refill and a single-CTA follow-up; here one CTA per
// multiprocessor stays resident and the steps are separated by grid barriers instead:
//
//   clear the votes | window histogram of the candidates          -- barrier 1
//   bin of the K-th key, its keys to a short list                  -- barrier 2
//   rank the list: T_n       [a crowded bin (very large K): its keys counted one by one, +1 barrier]
//                            [rare: three radix digits, +3 barriers, over the candidates or the full row]
//   picks: one vote per selected coordinate                        -- barrier 3
//                            [rare: threshold ties kept only in part, ordered by index, +2 barriers]
//   vote histogram per chunk and over the vector                   -- barrier 4
//   v*, output offsets (every CTA for itself), supp(M), gather, mean, residual zeros; scratch cleared
//
// The kernel is launched cooperatively (all CTAs are resident together, so a barrier always completes);
// every barrier wait is bounded all the same: a CTA that gives up sets a sticky flag, every CTA that sees
// the flag leaves, and the host reports MV_ERR_TIMEOUT.  Every barrier is reached under conditions that
// are the same for all CTAs of the grid (flags are read only after a barrier that follows their writes).

#ifdef MV_TAIL_STAMPS  // profiling build only: phase boundaries of CTA 0 by the global timer, printed now and then
#include <stdio.h>
__device__ unsigned g_stamp_calls;
#define TAIL_STAMP(i)                                                        \
  do {                                                                       \
    if (threadIdx.x == 0) {                                                  \
      unsigned long long t_;                                                 \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                 \
      stamps[i] = t_;                                                        \
    }                                                                        \
  } while (0)
#else
#define TAIL_STAMP(i) \
  do {                \
  } while (0)
#endif

constexpr int FT = 1024;         // threads per CTA of the tail kernel (== ST: smem_pick2 and chunk_scan<ST> are shared)
constexpr int F_MAXCH = 32768;   // most chunks (padded to eight) whose output offsets fit the shared-memory table
constexpr int F_RADIX = 7168;    // per worker: 2048 + 2048 + 1024 counters of the three-digit route, 2048 of the second count

struct TailArgs {
  float* err;               // [N][d] acc on entry, the residual on exit
  int32_t* out_idx;         // [K]
  float* out_val;           // [K]
  uint32_t* words;          // [16] in the cleared region: 0 barrier arrivals, 1 exit ticket, 2 bit 0 "a worker needs the
                            //      three-digit route", bit 1 "a worker counts the keys of its crowded bin a second
                            //      time", 3 "a worker keeps its threshold ties only in part"
  uint32_t* abort_flag;     // workspace header: set for good when a barrier wait gave up
  uint32_t* radix;          // [N][F_RADIX] digit counts of the three-digit route
  uint4* zero_ptr;          // start of the scratch region that must be clear when the next step starts
  uint32_t zero_vecs;       // its part, in 16-byte units, that all CTAs clear together at the end
  uint32_t* last_zero;      // the rest of it (vote histogram, ticket, these words): cleared by the last CTA out
  uint32_t last_zero_words;
  uint32_t spin_limit;      // polls after which a barrier wait gives up
  uint32_t* dbg;
};

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* q) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(q) : "memory");
  return v;
}

// Grid barrier on a counter that only grows during a launch (it is zero at the start and put back to zero by
// the last CTA to leave the kernel).  Returns false, in all threads of the CTA, if the wait was given up.
struct GridBar {
  uint32_t* ctr;
  uint32_t* abort_flag;
  uint32_t nblocks, target, limit;
};

__device__ __forceinline__ bool grid_barrier(GridBar& b) {
  __shared__ uint32_t s_bar_ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    b.target += b.nblocks;
    __threadfence();
    atomicAdd(b.ctr, 1u);
    uint32_t ok = ld_acquire(b.abort_flag) == 0u ? 1u : 0u, spins = 0u;  // (a wait given up earlier: leave at once)
    while (ok && ld_acquire(b.ctr) < b.target) {
      if (ld_acquire(b.abort_flag) != 0u) {
        ok = 0u;
        break;
      }
      if (++spins > b.limit) {
        atomicExch(b.abort_flag, 1u);
        ok = 0u;
        break;
      }
      __nanosleep(40);
    }
    __threadfence();
    s_bar_ok = ok;
  }
  __syncthreads();
  return s_bar_ok != 0u;
}

// sum over the CTA (FT threads); s_w: FT / 32 words
__device__ __forceinline__ uint32_t block_sum_ft(uint32_t v, uint32_t* s_w) {
  v = __reduce_add_sync(FULL, v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = v;
  __syncthreads();
  uint32_t tot = 0;
  for (int w = 0; w < FT / 32; w++) tot += s_w[w];
  return tot;
}

// s_local's non-zero counts are added to the worker's global counts
__device__ __forceinline__ void flush_counts(const uint32_t* s_local, uint32_t* __restrict__ g, int nbins) {
  for (int bb = threadIdx.x; bb < nbins; bb += FT) {
    const uint32_t v = s_local[bb];
    if (v) atomicAdd(&g[bb], v);
  }
}

// f(key) for every element of the chunks of row n that fall to CTA `rank` of `gsz`: four chunks at a time,
// 256 threads each
template <typename F>
__device__ __forceinline__ void tail_row_keys(const P& p, int n, float* __restrict__ err, int rank, int gsz, F f) {
  const int sub = threadIdx.x >> 8, t = threadIdx.x & 255;
  for (int c = rank * 4 + sub; c < p.nchunks; c += gsz * 4) {
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

// next call's candidate threshold when the counted keys do not reach the tracked rank: go below tau by linear
// extrapolation in key space from (K, key_K) and (cnt, tau), a quarter to spare, between 2^10 and 2^19 per call
__device__ __forceinline__ uint32_t tau_below(uint32_t tau, uint32_t key_K, uint32_t cnt, uint32_t K, uint32_t track_rank) {
  const float slope = (key_K > tau && cnt >= K) ? (float)(key_K - tau) / (float)(cnt - K + 1u) : 0.f;
  float drop = 1.25f * slope * (float)(track_rank > cnt ? track_rank - cnt : 1u);
  drop = fminf(fmaxf(drop, 1024.f), 524288.f);
  return tau > (uint32_t)drop ? tau - (uint32_t)drop : 0u;
}

__global__ void __launch_bounds__(FT, 1) k_tail(P p, TailArgs a) {
  extern __shared__ uint32_t dsm[];      // max(SK_KEYS, 1.5 nc_pad + 8) words: the slice's keys | vote-histogram scratch |
                                         // output offsets and tie quotas of all chunks
  __shared__ uint32_t s_hw[H1_BINS];     // this CTA's counts (window, then one radix digit at a time)
  __shared__ uint32_t s_m[H1_BINS];      // the worker's counts: all CTAs of its group together
  __shared__ uint32_t s_ws[FT / 32];
  __shared__ uint32_t s_res3[3];
  __shared__ uint32_t s_we[4][9];
  __shared__ uint32_t s_hv[256];
  __shared__ uint32_t s_vs[4];
  __shared__ uint32_t s_sw[FT / 32 + 1];
  __shared__ uint32_t s_lastout;
#ifdef MV_TAIL_STAMPS
  unsigned long long stamps[16];
#endif
#ifdef MV_TAIL_STAMPS
  unsigned long long t_begin_;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_begin_));
#endif
  pdl_enter();
#ifdef MV_TAIL_STAMPS
  if (threadIdx.x == 0) {
    unsigned long long t_;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));
    p.out_base[4 * blockIdx.x] = (uint32_t)t_begin_;
    p.out_base[4 * blockIdx.x + 1] = (uint32_t)t_;
  }
#endif
  uint32_t* s_keys = dsm;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, b = blockIdx.x;
  GridBar bar;
  bar.ctr = a.words;
  bar.abort_flag = a.abort_flag;
  bar.nblocks = (uint32_t)G;
  bar.target = 0u;
  bar.limit = a.spin_limit;

  TAIL_STAMP(0);
  // ---- the votes start out empty (cleared now, so that they are still in L2 when the picks arrive) ----
  zero_share(p.vote_words, (size_t)p.nchunks * (CH / 4), (size_t)b, (size_t)G);

  // ---- worker n is served by a group of gsz CTAs (N <= G); CTAs beyond the groups idle until the vote histogram ----
  const int gsz = G / p.N;
  const int n = b / gsz, rank = b % gsz;
  const bool has = n < p.N;
  const uint32_t K = (uint32_t)p.K;
  const bool tracking = p.tau_next != nullptr;
  uint32_t cnt = 0, s0 = 0, len = 0, tau = 0;
  bool fast = false;
  const uint2* cd = p.cand;
  uint32_t* R1 = a.radix;
  if (has) {
    cnt = p.cand_cnt[n];
    fast = worker_fast(p, n);
    tau = p.tau[n];
    cd = p.cand + (size_t)n * p.cap;
    const uint32_t per = (cnt + gsz - 1) / gsz;
    s0 = min(cnt, (uint32_t)rank * per);
    len = fast ? min(cnt, s0 + per) - s0 : 0u;
    R1 = a.radix + (size_t)n * F_RADIX;
    for (int i = rank * FT + tid; i < F_RADIX; i += gsz * FT) R1[i] = 0u;
  }
  uint32_t* R2 = R1 + 2048;
  uint32_t* R3 = R1 + 4096;
  uint32_t* R4 = R1 + 5120;  // the worker's second count: keys of bin bw by their low WIN_SHIFT bits
  uint32_t* gh = p.hist1 + (size_t)(has ? n : 0) * H1_BINS;   // the worker's window counts
  uint32_t* lcnt = p.hist3 + (size_t)(has ? n : 0) * H3_BINS;  // length of its short list ...
  uint32_t* list = p.hist2 + (size_t)(has ? n : 0) * H2_BINS;  // ... of the keys in the bin of rank K
  uint32_t* lidx = p.hist2b + (size_t)(has ? n : 0) * H2_BINS; // ... and their coordinates

  // ---- window histogram: candidates within 2^22 of tau_n, in 2048 bins of 2^11 keys ----
  const bool idx_kept = len <= (uint32_t)(SK_KEYS / 2);  // the slice's coordinates fit beside its keys: the picks need no second read
  if (has && fast) {
    for (int bb = tid; bb < H1_BINS; bb += FT) s_hw[bb] = 0;
    __syncthreads();
    for (uint32_t l0 = 0; l0 < len; l0 += FT * 8) {  // uniform over the CTA
      uint2 k[8];
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const uint32_t li = l0 + q * FT + tid;
        k[q] = li < len ? __ldcg(&cd[s0 + li]) : make_uint2(0u, 0u);
      }
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const uint32_t li = l0 + q * FT + tid;
        if (li < len) {
          if (li < SK_KEYS) s_keys[li] = k[q].x;
          if (idx_kept) s_keys[SK_KEYS / 2 + li] = k[q].y;  // (a slice of at most SK_KEYS / 2 keeps its coordinates too)
          const uint32_t wb = (k[q].x - tau) >> WIN_SHIFT;
          if (wb < (uint32_t)H1_BINS) atomicAdd(&s_hw[wb], 1u);
        }
      }
    }
    __syncthreads();
    flush_counts(s_hw, gh, H1_BINS);
  }
  TAIL_STAMP(1);
  if (!grid_barrier(bar)) return;  // 1
  TAIL_STAMP(2);

  // ---- the bin that holds rank K; its keys go to the worker's short list.  A bin too crowded for that (rows so
  // long that many elements share every magnitude near the threshold) is counted a second time, key by key ----
  bool will_resolve = false, lvl2 = false;
  uint32_t bw = 0, rem = 0, bt = 0, trem_w = 0;
  if (has && fast) {
    uint32_t wsum = 0;
    for (int bb = tid; bb < H1_BINS; bb += FT) {
      const uint32_t v = __ldcg(&gh[bb]);
      s_m[bb] = v;
      wsum += v;
    }
    const uint32_t win_total = block_sum_ft(wsum, s_ws);
    const uint32_t above = cnt - win_total;  // candidates beyond the window
    if (K > above) {                         // alike in all CTAs of the group
      const uint32_t rt = (tracking && p.track_rank > above && p.track_rank <= cnt) ? p.track_rank - above : 0u;
      smem_pick2<H1_BINS>(s_m, K - above, rt, bw, rem, bt, trem_w);
      if (s_m[bw] <= (uint32_t)WIN_LIST) {
        will_resolve = true;
        for (uint32_t li = tid; li < len; li += FT) {
          const uint32_t kk = li < SK_KEYS ? s_keys[li] : __ldcg(&cd[s0 + li].x);
          if (((kk - tau) >> WIN_SHIFT) == bw) {
            const uint32_t at = atomicAdd(lcnt, 1u);
            if (at < (uint32_t)WIN_LIST) {
              list[at] = kk;
              lidx[at] = idx_kept ? s_keys[SK_KEYS / 2 + li] : __ldcg(&cd[s0 + li].y);
            } else {
              MV_DBG(a.dbg, MV_DBG_INTERNAL);
            }
          }
        }
      } else {
        lvl2 = true;
        if (rank == 0 && tid == 0) MV_DBG(a.dbg, MV_DBG_WINDOW_OVERFLOW);
        __syncthreads();
        for (int bb = tid; bb < H1_BINS; bb += FT) s_hw[bb] = 0;
        __syncthreads();
        for (uint32_t li = tid; li < len; li += FT) {
          const uint32_t kk = li < SK_KEYS ? s_keys[li] : __ldcg(&cd[s0 + li].x);
          if (((kk - tau) >> WIN_SHIFT) == bw) atomicAdd(&s_hw[(kk - tau) & ((1u << WIN_SHIFT) - 1u)], 1u);
        }
        __syncthreads();
        flush_counts(s_hw, R4, 1 << WIN_SHIFT);
        if (tid == 0) atomicOr(a.words + 2, 2u);
      }
    }
  }
  bool need_slow = has && !will_resolve && !lvl2;  // a full-row worker, or a K-th key outside the window
  if (need_slow && tid == 0) atomicOr(a.words + 2, 1u);
  TAIL_STAMP(3);
  if (!grid_barrier(bar)) return;  // 2
  TAIL_STAMP(4);

  uint32_t T = 0, need = 0, cnt_eq = 0;
  uint32_t flags2 = 0;  // the detours that some worker of the grid needs (written before barrier 2, so alike in every CTA)
  if (will_resolve) {
    // rank the list: T_n is its rem-th largest key
    // (the list holds every candidate whose key equals T_n, with its coordinate: a thread that holds such a tie
    // also learns how many ties precede it in index order, which settles the ties without any pass of its own)
    // (the list's length, its entries -- slot tid exists whatever the length -- and the flags are asked for together)
    uint32_t mine = __ldcg(list + tid), myidx = __ldcg(lidx + tid), tie_lt = 0;
    const uint32_t m = __ldcg(lcnt);
    flags2 = ld_acquire(a.words + 2);
    if (m <= 96u) {  // a short list: every key against every key (alike in all threads)
      if ((uint32_t)tid < m) {
        s_m[tid] = mine;
        s_hw[tid] = myidx;
      }
      __syncthreads();
      if ((uint32_t)tid < m) {
        uint32_t gt = 0, eq = 0;
        for (uint32_t i = 0; i < m; i++) {
          const uint32_t o = s_m[i];
          gt += o > mine;
          if (o == mine) {
            eq++;
            tie_lt += s_hw[i] < myidx ? 1u : 0u;
          }
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
      // ties kept only in part: the `need` lowest coordinates among them vote here (one CTA of the group does it)
      if (need < cnt_eq && rank == 0 && (uint32_t)tid < m && mine == T && tie_lt < need) {
        if ((int64_t)myidx < p.d) add_vote(p.vote_words, myidx);
        else MV_DBG(a.dbg, MV_DBG_PICK_RANGE);
      }
    } else {
      // a longer list (the pairwise count grows with its square): the list's keys all lie in bin bw, so their low
      // WIN_SHIFT bits tell them apart; one counter per key value, and the rem-th largest is read off the counts
      __syncthreads();
      for (int bb = tid; bb < H1_BINS; bb += FT) s_hw[bb] = 0;
      if (tid == 0) s_res3[0] = 0;
      __syncthreads();
      if ((uint32_t)tid < m) atomicAdd(&s_hw[(mine - tau) & ((1u << WIN_SHIFT) - 1u)], 1u);
      __syncthreads();
      uint32_t b2, u0, u1;
      smem_pick2<H1_BINS>(s_hw, rem, 0u, b2, need, u0, u1);
      T = tau + (bw << WIN_SHIFT) + b2;
      cnt_eq = s_hw[b2];
      if (need < cnt_eq && rank == 0) {  // alike in all threads: the ties, by coordinate, among themselves
        const bool tie = (uint32_t)tid < m && mine == T;
        if (tie) s_m[atomicAdd(&s_res3[0], 1u)] = myidx;
        __syncthreads();
        if (tie) {
          for (uint32_t i = 0; i < cnt_eq; i++) tie_lt += s_m[i] < myidx ? 1u : 0u;
          if (tie_lt < need) {
            if ((int64_t)myidx < p.d) add_vote(p.vote_words, myidx);
            else MV_DBG(a.dbg, MV_DBG_PICK_RANGE);
          }
        }
      }
    }
    if (tracking && rank == 0 && tid == 0)
      p.tau_next[n] = trem_w != 0 ? tau + (bt << WIN_SHIFT) : tau_below(tau, T, cnt, K, p.track_rank);
  }

  // ---- the second count (the same decision in every CTA of the grid: the flag was written before barrier 2): the
  // worker's keys of bin bw, one counter per key, give T_n, cnt_eq and need directly; ties kept only in part go to
  // the short list with their coordinates, and the lowest coordinates among them vote ----
  bool tie_listed = will_resolve;  // the worker's partly kept ties (if any) are settled through the short list
  if (!will_resolve) flags2 = ld_acquire(a.words + 2);
  if ((flags2 & 2u) != 0u) {
    bool list_ties = false;
    if (lvl2) {
      for (int bb = tid; bb < H1_BINS; bb += FT) s_m[bb] = __ldcg(&R4[bb]);
      __syncthreads();
      uint32_t b2, u0, u1;
      smem_pick2<H1_BINS>(s_m, rem, 0u, b2, need, u0, u1);
      T = tau + (bw << WIN_SHIFT) + b2;
      cnt_eq = s_m[b2];
      if (need < cnt_eq) {
        if (cnt_eq <= (uint32_t)WIN_LIST) {
          list_ties = true;
          for (uint32_t li = tid; li < len; li += FT) {
            const uint32_t kk = li < SK_KEYS ? s_keys[li] : __ldcg(&cd[s0 + li].x);
            if (kk == T) {
              const uint32_t at = atomicAdd(lcnt, 1u);
              if (at < (uint32_t)WIN_LIST) lidx[at] = __ldcg(&cd[s0 + li].y);
              else MV_DBG(a.dbg, MV_DBG_INTERNAL);
            }
          }
        } else {  // more equal keys than the list holds: their order comes from the per-chunk route below
          lvl2 = false;
        }
      }
      if (tracking && rank == 0 && tid == 0)
        p.tau_next[n] = trem_w != 0 ? tau + (bt << WIN_SHIFT) : tau_below(tau, T, cnt, K, p.track_rank);
    }
    if (!grid_barrier(bar)) return;  // +1
    if (list_ties) {
      tie_listed = true;
      const uint32_t m = min(__ldcg(lcnt), (uint32_t)WIN_LIST);
      uint32_t myidx = 0;
      if ((uint32_t)tid < m) {
        myidx = __ldcg(lidx + tid);
        s_hw[tid] = myidx;
      }
      __syncthreads();
      if (rank == 0 && (uint32_t)tid < m) {
        uint32_t tie_lt = 0;
        for (uint32_t i = 0; i < m; i++) tie_lt += s_hw[i] < myidx ? 1u : 0u;
        if (tie_lt < need) {
          if ((int64_t)myidx < p.d) add_vote(p.vote_words, myidx);
          else MV_DBG(a.dbg, MV_DBG_PICK_RANGE);
        }
      }
    } else if (lvl2) {
      tie_listed = true;  // (every tie is kept, or none is left open)
    }
  }

  // ---- rare: three radix digits (11 + 10 + 10 bits) for the workers that are not resolved yet, over their
  // candidates or, for a worker whose candidate count missed [K, cap], over its full row.  Whether this part
  // runs is the same for the whole grid (the flag was written before barrier 2). ----
  if ((flags2 & 1u) != 0u) {
    uint32_t b1 = 0, rem1 = 0, tb = 0, trem = 0, b2 = 0, rem2 = 0, tb2 = 0, trem2 = 0;
    auto slice_keys = [&](auto f) {
      if (fast) {
        for (uint32_t li = tid; li < len; li += FT) f(li < SK_KEYS ? s_keys[li] : __ldcg(&cd[s0 + li].x));
      } else {
        tail_row_keys(p, n, a.err, rank, gsz, f);
      }
    };
    // digit 1
    if (need_slow) {
      for (int bb = tid; bb < H1_BINS; bb += FT) s_hw[bb] = 0;
      __syncthreads();
      slice_keys([&](uint32_t key) { atomicAdd(&s_hw[key >> 20], 1u); });
      __syncthreads();
      flush_counts(s_hw, R1, H1_BINS);
    }
    if (!grid_barrier(bar)) return;  // +1
    // digit 2 (and, with threshold tracking, the second digit of the tracked rank)
    if (need_slow) {
      for (int bb = tid; bb < H1_BINS; bb += FT) {
        s_m[bb] = __ldcg(&R1[bb]);
        s_hw[bb] = 0;
      }
      __syncthreads();
      smem_pick2<H1_BINS>(s_m, K, tracking ? p.track_rank : 0u, b1, rem1, tb, trem);
      const uint32_t track_bin = (tracking && trem != 0 && tb != b1) ? tb : 0xffffffffu;
      slice_keys([&](uint32_t key) {
        const uint32_t d1 = key >> 20;
        if (d1 == b1) atomicAdd(&s_hw[(key >> 10) & 1023u], 1u);
        else if (d1 == track_bin) atomicAdd(&s_hw[1024u + ((key >> 10) & 1023u)], 1u);
      });
      __syncthreads();
      flush_counts(s_hw, R2, H1_BINS);
    }
    if (!grid_barrier(bar)) return;  // +2
    // digit 3
    if (need_slow) {
      for (int bb = tid; bb < H1_BINS; bb += FT) {
        s_m[bb] = __ldcg(&R2[bb]);
        s_hw[bb] = 0;
      }
      __syncthreads();
      uint32_t u0, u1;
      if (tracking && trem != 0 && tb == b1) {  // the usual case: both ranks in the same first-digit bin
        smem_pick2<H2_BINS>(s_m, rem1, trem, b2, rem2, tb2, trem2);
      } else {
        smem_pick2<H2_BINS>(s_m, rem1, 0u, b2, rem2, u0, u1);
        if (tracking && trem != 0) smem_pick2<H2_BINS>(s_m + 1024, trem, 0u, tb2, trem2, u0, u1);
      }
      if (tracking && rank == 0 && tid == 0)
        p.tau_next[n] = trem != 0 ? ((tb << 20) | (tb2 << 10)) : tau_below(tau, (b1 << 20) | (b2 << 10), cnt, K, p.track_rank);
      const uint32_t prefix = (b1 << 10) | b2;
      slice_keys([&](uint32_t key) {
        if ((key >> 10) == prefix) atomicAdd(&s_hw[key & 1023u], 1u);
      });
      __syncthreads();
      flush_counts(s_hw, R3, H3_BINS);
    }
    if (!grid_barrier(bar)) return;  // +3
    if (need_slow) {
      for (int bb = tid; bb < H3_BINS; bb += FT) s_m[bb] = __ldcg(&R3[bb]);
      __syncthreads();
      uint32_t b3, u0, u1;
      smem_pick2<H3_BINS>(s_m, rem2, 0u, b3, need, u0, u1);
      cnt_eq = s_m[b3];
      T = (b1 << 20) | (b2 << 10) | b3;
    }
  }
  if (has && rank == 0 && tid == 0) {
    uint32_t* ws = p.wstate + (size_t)n * 8;
    ws[4] = T;
    ws[5] = K - need;
    ws[6] = cnt_eq;
    ws[7] = need;
    p.thresh[n * 3 + 0] = T;
    p.thresh[n * 3 + 1] = K - need;
    p.thresh[n * 3 + 2] = cnt_eq;
    p.diag_cnt[n] = cnt;
    if (!fast) {
      MV_DBG(a.dbg, MV_DBG_FALLBACK);
      if (p.fb_total != nullptr) atomicAdd(p.fb_total, 1u);
    }
  }
  const bool all_ties = need >= cnt_eq;  // alike in all CTAs of the group
  const bool ties_open = !all_ties && !tie_listed;  // partly kept ties that still have to be put in index order

  TAIL_STAMP(5);
  // ---- picks: every selected coordinate gets one more vote.  A worker that keeps only part of its threshold
  // ties (lowest index first) votes for the keys above T_n now and counts its ties per chunk; the ties follow. ----
  if (has) {
    if (fast) {
      for (uint32_t l0 = 0; l0 < len; l0 += FT * 4) {  // (four candidates in flight per thread)
        uint2 kv[4];
#pragma unroll
        for (int q = 0; q < 4; q++) {
          const uint32_t li = l0 + q * FT + tid;
          kv[q] = make_uint2(0u, 0u);
          if (li < len) kv[q] = idx_kept ? make_uint2(s_keys[li], s_keys[SK_KEYS / 2 + li]) : __ldcg(&cd[s0 + li]);
        }
#pragma unroll
        for (int q = 0; q < 4; q++) {
          if (l0 + q * FT + tid < len && (kv[q].x > T || (kv[q].x == T && all_ties))) {
            if ((int64_t)kv[q].y < p.d) add_vote(p.vote_words, kv[q].y);
            else MV_DBG(a.dbg, MV_DBG_PICK_RANGE);
          }
        }
      }
      if (ties_open) {
        for (int c = rank * (FT / 32) + warp; c < p.nchunks; c += gsz * (FT / 32)) {
          const size_t ci = (size_t)n * p.nchunks + c;
          const uint32_t ccnt = p.chunk_cnt[ci], base = p.chunk_base[ci];
          uint32_t eq = 0;
          for (uint32_t i = lane; i < ccnt; i += 32) eq += __ldcg(&cd[base + i].x) == T;
          eq = __reduce_add_sync(FULL, eq);
          if (lane == 0) p.chunk_eq[ci] = eq;
        }
      }
    } else if (all_ties) {
      fullrow_picks<4>(p, n, a.err, T, need, true, rank * 4, gsz * 4, s_we);
    } else {
      const int sub = tid >> 8, t = tid & 255, w8 = t >> 5;
      for (int c0 = rank * 4; c0 < p.nchunks; c0 += gsz * 4) {  // uniform over the CTA
        const int c = c0 + sub;
        const bool valid = c < p.nchunks;
        uint32_t eq = 0;
        if (valid) {
          const Geom g = chunk_geom(n, c, p.d);
          uint32_t key[4][4], vm[4];
          load_keys<false>(g, nullptr, a.err, key, vm, t);
#pragma unroll
          for (int i = 0; i < 4; i++) eq += __popc(vm[i] & eq_mask(key[i], T));
          if (t == TPB - 1) {
            uint32_t xkey[4], xvm;
            load_extra<false>(g, nullptr, a.err, xkey, xvm);
            eq += __popc(xvm & eq_mask(xkey, T));
          }
        }
        eq = __reduce_add_sync(FULL, eq);
        if (lane == 0) s_we[sub][w8] = eq;
        __syncthreads();
        if (valid && t == 0) {
          uint32_t te = 0;
          for (int w = 0; w < 8; w++) te += s_we[sub][w];
          p.chunk_eq[(size_t)n * p.nchunks + c] = te;
        }
        __syncthreads();
      }
    }
    if (ties_open && tid == 0) atomicOr(a.words + 3, 1u);
  }
  TAIL_STAMP(6);
  if (!grid_barrier(bar)) return;  // 3
  TAIL_STAMP(7);

  // ---- rare: the partly kept ties, in index order (again the same decision in every CTA of the grid) ----
  if (ld_acquire(a.words + 3) != 0u) {
    if (has && ties_open && rank == 0) chunk_scan<ST>(p, n);  // running tie count before every chunk
    if (!grid_barrier(bar)) return;  // +1
    if (has && ties_open) {
      if (fast) {
        const uint32_t lt = lanemask_lt();
        for (int c = rank * (FT / 32) + warp; c < p.nchunks; c += gsz * (FT / 32)) {
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
            if (eq && run + __popc(eb & lt) < need && (int64_t)kv.y < p.d) add_vote(p.vote_words, kv.y);
            run += __popc(eb);
          }
        }
      } else {
        fullrow_picks<4>(p, n, a.err, T, need, false, rank * 4, gsz * 4, s_we);
      }
    }
    if (!grid_barrier(bar)) return;  // +2
  }

  TAIL_STAMP(8);
  // ---- vote histogram: per chunk the counts #{votes >= v}, over the vector the exact counts; a warp per chunk ----
  {
    uint32_t* s_tot = dsm;               // the CTA's exact counts per vote value
    __syncthreads();                      // (the keys are not needed any more)
    if (tid < 256) s_tot[tid] = 0;
    __syncthreads();
    for (int c = warp * G + b; c < p.nchunks; c += G * (FT / 32)) {  // neighbouring chunks go to different CTAs
      uint4 q[8];
#pragma unroll
      for (int u = 0; u < 8; u++) {
        const int64_t jb = (int64_t)c * CH + (int64_t)(u * 32 + lane) * 16;
        q[u] = jb < p.d ? __ldcg(reinterpret_cast<const uint4*>(p.votes + jb)) : make_uint4(0, 0, 0, 0);
      }
      chunk_vote_counts(p, c, q, lane, s_tot);
    }
    __syncthreads();
    if (tid >= 1 && tid <= p.N && s_tot[tid]) atomicAdd(&p.vote_hist[tid], s_tot[tid]);
  }
  TAIL_STAMP(9);
  if (!grid_barrier(bar)) return;  // 4
  TAIL_STAMP(10);

  // ---- v* = vote count of the K-th most voted coordinate (every CTA for itself: N + 1 numbers) ----
  for (int v = tid; v < 256; v += FT) s_hv[v] = (v >= 1 && v <= p.N) ? __ldcg(p.vote_hist + v) : 0u;
  __syncthreads();
  if (tid == 0) {
    uint32_t voted = 0;
    for (int v = 1; v <= p.N; v++) voted += s_hv[v];
    s_hv[0] = (uint32_t)p.d - voted;  // coordinates nobody voted for
    uint32_t acc = 0, vstar = 0, cgt = 0, ceq = 0;
    for (int v = p.N; v >= 0; v--) {
      const uint32_t h = s_hv[v];
      if (acc + h >= K) {
        vstar = (uint32_t)v;
        cgt = acc;
        ceq = h;
        break;
      }
      acc += h;
    }
    s_vs[0] = vstar;
    s_vs[1] = cgt;
    s_vs[2] = ceq;
    s_vs[3] = K - cgt;
    if (b == 0) {
      p.vstate[0] = vstar;
      p.vstate[1] = cgt;
      p.vstate[2] = ceq;
      p.vstate[3] = K - cgt;
    }
  }
  __syncthreads();
  const uint32_t vstar = s_vs[0], quota = s_vs[3];

  // ---- output offset of every chunk and the v*-ties it keeps (lowest index first): a scan over the chunks' counts
  // in tiles of 8 FT chunks, thread t taking chunks 8t .. 8t+7 of the tile; every CTA computes the whole table, in
  // shared memory (ecarry / scarry: v*-ties seen and outputs placed in the tiles before) ----
  uint32_t* s_ob = dsm;                                                  // [nc_pad + 8]: nchunks + 1 offsets
  uint16_t* s_tk = reinterpret_cast<uint16_t*>(dsm + p.nc_pad + 8);      // [nc_pad]
  {
    const uint16_t* hge = p.chunk_vh + (size_t)vstar * p.nc_pad;                                    // votes >= v*
    const uint16_t* hgt = (int)vstar < p.N ? p.chunk_vh + (size_t)(vstar + 1) * p.nc_pad : nullptr;  // votes > v*
    uint32_t ecarry = 0, scarry = 0;
    for (int c0 = 0; c0 < p.nc_pad; c0 += FT * 8) {  // uniform over the CTA
      const int c = c0 + tid * 8;
      uint4 av = make_uint4(0, 0, 0, 0), gv = make_uint4(0, 0, 0, 0);
      if (c < p.nc_pad) {
        av = __ldcg(reinterpret_cast<const uint4*>(hge + c));
        if (hgt) gv = __ldcg(reinterpret_cast<const uint4*>(hgt + c));
      }
      const uint32_t aw[4] = {av.x, av.y, av.z, av.w}, gw[4] = {gv.x, gv.y, gv.z, gv.w};
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
      const uint32_t epre = ecarry + block_excl_scan<FT>(esum, s_sw, etot);
      const uint32_t taken_before = epre < quota ? epre : quota;           // ties kept in earlier chunks
      const uint32_t taken_here = min(epre + esum, quota) - taken_before;  // ties kept in this thread's chunks
      const uint32_t spre = scarry + block_excl_scan<FT>(gsum + taken_here, s_sw, stot);
      uint32_t run = epre, srun = spre;
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const uint32_t take = run >= quota ? 0u : min(eqv[q], quota - run);
        if (c + q < p.nchunks) {
          s_ob[c + q] = srun;
          s_tk[c + q] = (uint16_t)take;
        }
        run += eqv[q];
        srun += gtv[q] + take;
      }
      ecarry += etot;
      scarry += stot;
    }
    if (tid == 0) s_ob[p.nchunks] = K;
  }
  __syncthreads();

  TAIL_STAMP(11);
  // ---- supp(M), ascending: a warp per chunk that holds outputs, the chunks dealt out over all warps of the grid.
  // Lane l owns the chunk's coordinates [128 l, 128 l + 128), so lane order is index order and one scan over the
  // lanes places the outputs (a second one, only in a chunk that keeps part of its v*-ties, places those) ----
  {
    const uint32_t vs4 = vstar * 0x01010101u;
    for (int c = warp * G + b; c < p.nchunks; c += G * (FT / 32)) {
      const uint32_t ob = s_ob[c];
      if (s_ob[c + 1] == ob) continue;  // no coordinate of this chunk is in the mask
      const uint32_t tk = s_tk[c];
      const int64_t jl = (int64_t)c * CH + (int64_t)lane * 128;  // the lane's first coordinate
      uint4 qv[8];
#pragma unroll
      for (int u = 0; u < 8; u++) {
        const int64_t jb = jl + 16 * u;
        qv[u] = jb < p.d ? __ldcg(reinterpret_cast<const uint4*>(p.votes + jb)) : make_uint4(0, 0, 0, 0);
      }
      // one bit per coordinate: votes > v*, votes == v* (byte compares give 0xff per hit; a multiply gathers one bit
      // of each of the four bytes); coordinates at or beyond d are left out
      uint32_t gm[4] = {0, 0, 0, 0}, em[4] = {0, 0, 0, 0};
#pragma unroll
      for (int u = 0; u < 8; u++) {
        const uint32_t w[4] = {qv[u].x, qv[u].y, qv[u].z, qv[u].w};
        if (vstar == 0u || (w[0] | w[1] | w[2] | w[3]) != 0u) {
          uint32_t g16 = 0, e16 = 0;
#pragma unroll
          for (int i = 0; i < 4; i++) {
            g16 |= (((__vcmpgtu4(w[i], vs4) & 0x01010101u) * 0x01020408u) >> 24) << (4 * i);
            e16 |= (((__vcmpeq4(w[i], vs4) & 0x01010101u) * 0x01020408u) >> 24) << (4 * i);
          }
          const int64_t left = p.d - (jl + 16 * u);  // bytes of this piece that are coordinates
          const uint32_t inb = left >= 16 ? 0xffffu : (left <= 0 ? 0u : (1u << (int)left) - 1u);
          gm[u >> 1] |= (g16 & inb) << (16 * (u & 1));
          em[u >> 1] |= (e16 & inb) << (16 * (u & 1));
        }
      }
      if (tk > 0) {  // uniform over the warp: the chunk's first tk v*-ties, in index order, are kept
        const uint32_t pe = __popc(em[0]) + __popc(em[1]) + __popc(em[2]) + __popc(em[3]);
        uint32_t x = pe;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const uint32_t y = __shfl_up_sync(FULL, x, off);
          if (lane >= off) x += y;
        }
        const uint32_t before = x - pe;
        uint32_t room = before < tk ? tk - before : 0u;
#pragma unroll
        for (int i = 0; i < 4; i++) {
          uint32_t e2 = em[i];
          while (e2 && room) {
            const uint32_t low = e2 & (0u - e2);
            gm[i] |= low;
            e2 ^= low;
            room--;
          }
        }
      }
      const uint32_t ps = __popc(gm[0]) + __popc(gm[1]) + __popc(gm[2]) + __popc(gm[3]);
      uint32_t x = ps;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t y = __shfl_up_sync(FULL, x, off);
        if (lane >= off) x += y;
      }
      uint32_t pos = ob + x - ps;
#pragma unroll
      for (int i = 0; i < 4; i++) {
        uint32_t sm = gm[i];
        while (sm) {
          const int bb = __ffs(sm) - 1;
          sm &= sm - 1;
          if (pos < K) a.out_idx[pos] = (int32_t)(jl + 32 * i + bb);
          else MV_DBG(a.dbg, MV_DBG_OUT_RANGE);
          pos++;
        }
      }
    }
  }
  TAIL_STAMP(12);
  if (!grid_barrier(bar)) return;  // 5

  // ---- aggregate on the shared mask and zero the residual there: every CTA an equal share of the K outputs ----
  {
    const uint32_t lo = (uint32_t)((uint64_t)b * K / (uint64_t)G), hi = (uint32_t)((uint64_t)(b + 1) * K / (uint64_t)G);
    const uint32_t m = hi - lo;
    if (m * 8u <= (uint32_t)FT) {  // few outputs: eight lanes share a coordinate's N rows
      const uint32_t kk = (uint32_t)tid >> 3;
      gather_one<8>(a.err, p.N, p.d, (int64_t)lo + kk, kk < m, tid & 7, a.out_idx, a.out_val, nullptr, a.dbg);
    } else {
      for (uint32_t k = lo + tid; k < hi; k += FT) gather_one<1>(a.err, p.N, p.d, (int64_t)k, true, 0, a.out_idx, a.out_val, nullptr, a.dbg);
    }
  }

  TAIL_STAMP(13);
  // ---- leave the scratch region clear for the next step; the last CTA out clears what the others used to the end ----
  for (uint32_t i = (uint32_t)b * FT + tid; i < a.zero_vecs; i += (uint32_t)G * FT) a.zero_ptr[i] = make_uint4(0, 0, 0, 0);
#ifdef MV_TAIL_STAMPS
  if (threadIdx.x == 0) {
    unsigned long long t_;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));
    p.out_base[4 * blockIdx.x + 2] = (uint32_t)t_;
    p.out_base[4 * blockIdx.x + 3] = (uint32_t)(stamps[9] - stamps[8]);  // this CTA's vote-histogram phase
  }
#endif
  __threadfence();
  __syncthreads();
  if (tid == 0) s_lastout = (atomicAdd(a.words + 1, 1u) == (uint32_t)G - 1u) ? 1u : 0u;
  __syncthreads();
  if (s_lastout) {
    __threadfence();
    for (uint32_t i = tid; i < a.last_zero_words; i += FT) a.last_zero[i] = 0u;
  }
#ifdef MV_TAIL_STAMPS
  TAIL_STAMP(14);
  if (s_lastout && threadIdx.x == 0 && (atomicAdd(&g_stamp_calls, 1u) % 97u) == 96u) {
    uint32_t b0 = 0xffffffffu, b1 = 0, w0 = 0xffffffffu, w1 = 0, e0 = 0xffffffffu, e1 = 0;
    for (int i = 0; i < G; i++) {
      const uint32_t tb = __ldcg(p.out_base + 4 * i), tw = __ldcg(p.out_base + 4 * i + 1), te = __ldcg(p.out_base + 4 * i + 2);
      b0 = min(b0, tb); b1 = max(b1, tb); w0 = min(w0, tw); w1 = max(w1, tw); e0 = min(e0, te); e1 = max(e1, te);
    }
    {
      uint32_t hmin = 0xffffffffu, hmax = 0, hsum = 0, harg = 0;
      for (int i = 0; i < G; i++) {
        const uint32_t h = __ldcg(p.out_base + 4 * i + 3);
        hmin = min(hmin, h); hsum += h;
        if (h > hmax) { hmax = h; harg = i; }
      }
      printf("hist phase per cta: min %.1f avg %.1f max %.1f us (cta %u)\n", hmin * 1e-3, hsum * 1e-3 / G, hmax * 1e-3, harg);
    }
    printf("ctas: first start 0, last start %.1f, wait over %.1f .. %.1f, first end %.1f, last end %.1f us\n", (b1 - b0) * 1e-3,
           (w0 - b0) * 1e-3, (w1 - b0) * 1e-3, (e0 - b0) * 1e-3, (e1 - b0) * 1e-3);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0 && (g_stamp_calls % 97u) == 0u) {
    printf("tail stamps us:");
    for (int i = 1; i <= 14; i++) printf(" %.1f", (double)(stamps[i] - stamps[i - 1]) * 1e-3);
    printf("\n");
  }
#endif
}
