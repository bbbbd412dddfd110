// mv_small.cuh -- a whole step as ONE kernel for rows that fit a CTA's shared memory (d <= 32768).
// (Included by mv_sparse.cu inside its anonymous namespace, after mv_tail.cuh.)
//
// A problem this small is all launch latency when it runs as a sequence of kernels.  Here worker n is CTA n:
// it reads its row once (acc = err + grads, written in place), keeps the d magnitude keys in shared memory,
// finds its exact K-th key there and votes.  The K-th key is found from a lower bound tau on it -- carried from the
// previous call (threshold tracking) or read off a 256-key sample -- by counting the keys >= tau in 2048 equal
// bins between tau and the row's largest key and ranking the keys of the bin that holds rank K directly; the
// leading bits of a magnitude key are mostly exponent, so a plain radix digit over all keys piles thousands of
// shared-memory atomics on a handful of counters, and the three-digit radix select is kept only as the fallback
// for a bound that turns out too high and for a crowded bin (heavy ties).  After the
// only grid barrier every CTA reads the d vote bytes, finds v* and the output positions for itself, writes its
// share of supp(M), gathers the mean there and zeroes the residual.  The vote bytes, the vote histogram (kept up
// to date by the votes themselves: every vote is an atomic add that returns the count before it) and the barrier
// word alternate between two copies from call to call: the copy not in use is cleared for the next call while
// this one runs, so no barrier and no exit ticket is spent on clearing.  Launched cooperatively; the barrier
// wait is bounded like those of the tail.

constexpr int SMALL_MAX_D = SK_KEYS;  // 32768 keys of shared memory

struct SmallArgs {
  const float* grads;
  float* err;
  int32_t* out_idx;
  float* out_val;
  // Three pieces of state alternate between two copies from call to call; this call finds its copy all zero and
  // clears the other one, which the previous call used and the next call will use:
  uint32_t* votes_now;    // the vote bytes, four to a word (whole chunks long)
  uint32_t* votes_next;
  uint32_t* hist_now;     // [256] coordinates per vote count (bins 1..N)
  uint32_t* hist_next;
  uint32_t* bar_now;      // arrivals at the grid barrier
  uint32_t* bar_next;
  uint32_t* abort_flag;
  uint32_t spin_limit;
  uint32_t* dbg;
  const uint32_t* tau_in;  // [N] lower bounds on the K-th keys left by the previous call, or null (then a sample gives them)
  uint32_t* tau_out;       // [N] bounds for the next call (threshold tracking), or null
  uint32_t track_rank;     // the next call's bound is put at this rank among the keys >= tau
};

constexpr int SMALL_SAMPLE = 256;  // keys sampled per row when no bound is carried

__global__ void __launch_bounds__(FT, 1) k_small(P p, SmallArgs a) {
#ifdef MV_TAIL_STAMPS
  unsigned long long stamps[16];
#endif
  TAIL_STAMP(0);
  pdl_enter();
  extern __shared__ uint32_t s_key[];  // [d] the row's magnitude keys
  __shared__ uint32_t s_h[H1_BINS];
  __shared__ uint32_t s_list[WIN_LIST];
  __shared__ uint32_t s_samp[SMALL_SAMPLE];
  __shared__ uint32_t s_sw[FT / 32 + 1];
  __shared__ uint32_t s_hv[256];
  __shared__ uint32_t s_vs[4];
  __shared__ uint32_t s_res[4];
  __shared__ uint32_t s_lcnt, s_ccnt;
  const int tid = threadIdx.x;
  const int G = gridDim.x, n = blockIdx.x;  // G == N
  const int d = (int)p.d;
  const uint32_t K = (uint32_t)p.K;
  GridBar bar;
  bar.ctr = a.bar_now;
  bar.abort_flag = a.abort_flag;
  bar.nblocks = (uint32_t)G;
  bar.target = 0u;
  bar.limit = a.spin_limit;

  const uint32_t tau_carried = a.tau_in != nullptr ? __ldcg(a.tau_in + n) : 0u;  // (asked for now, needed after the row)
  // ---- accumulate (Algorithm 1, error feedback): the row once through; its keys stay in shared memory ----
  uint32_t kmax = 0;  // the row's largest key
  {
    const float* grow = a.grads + (size_t)n * (size_t)d;
    float* erow = a.err + (size_t)n * (size_t)d;
    for (int j0 = 0; j0 < d; j0 += FT * 8) {  // (eight loads of each array in flight per thread)
      float e[8], g[8];
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int j = j0 + q * FT + tid;
        e[q] = j < d ? __ldcs(erow + j) : 0.f;
        g[q] = j < d ? __ldcs(grow + j) : 0.f;
      }
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int j = j0 + q * FT + tid;
        if (j < d) {
          const float v = __fadd_rn(e[q], g[q]);
          erow[j] = v;
          const uint32_t k = fkey(v);
          s_key[j] = k;
          kmax = max(kmax, k);
        }
      }
    }
    kmax = __reduce_max_sync(FULL, kmax);
    if ((tid & 31) == 0) s_sw[tid >> 5] = kmax;
    __syncthreads();  // (the keys are in shared memory from here on)
    for (int w = 0; w < FT / 32; w++) kmax = max(kmax, s_sw[w]);
    __syncthreads();
  }
  TAIL_STAMP(1);
  // ---- S_top (Eq. 6): the exact K-th key T_n, with cnt_eq = #{keys == T_n} and need = how many of those are kept.
  // Up to two tries with a lower bound tau (the carried one, then the sampled one): count the keys >= tau in
  // H1_BINS equal bins over [tau, kmax], find the bin of rank K (and, with tracking, of the next call's rank), rank
  // that bin's keys directly.  A try gives up, alike in all threads, when fewer than K keys reach tau or when the
  // bin is too crowded to rank; then three radix digits (11 + 10 + 10 bits) over all keys settle it. ----
  uint32_t T = 0, need = 0, cnt_eq = 0;
  bool resolved = false, tried = false;
  for (int attempt = a.tau_in != nullptr ? 0 : 1; attempt < 2 && !resolved; attempt++) {
    if (tried) __syncthreads();  // (the try before this one is over in every thread)
    tried = true;
    uint32_t tau = 0;
    if (attempt == 0) {
      tau = tau_carried;
    } else {
      // the r-th largest of S evenly spaced keys, r a few standard deviations beyond the expected rank S K / d
      const int S = d < SMALL_SAMPLE ? d : SMALL_SAMPLE;
      const float m = (float)S * (float)K / (float)d;
      const uint32_t r = (uint32_t)ceilf(m + 6.f * sqrtf(m) + 8.f);
      if (r < (uint32_t)S) {
        uint32_t mine = 0;
        if (tid < S) {
          mine = s_key[(int)(((int64_t)tid * d) / S)];
          s_samp[tid] = mine;
        }
        __syncthreads();
        if (tid < S) {
          uint32_t gt = 0, eq = 0;
          for (int i = 0; i < S; i++) {
            const uint32_t o = s_samp[i];
            gt += o > mine;
            eq += o == mine;
          }
          if (gt < r && r <= gt + eq) s_res[0] = mine;  // (every thread that holds that key writes the same value)
        }
        __syncthreads();
        tau = s_res[0];
        __syncthreads();
      }
    }
    if (kmax < tau) continue;  // nothing reaches the bound
    const uint32_t span = kmax - tau;
    const int sbits = 32 - __clz(span);
    const int shift = sbits > 11 ? sbits - 11 : 0;  // (span >> shift) < H1_BINS
    for (int bb = tid; bb < H1_BINS; bb += FT) s_h[bb] = 0;
    if (tid == 0) {
      s_lcnt = 0;
      s_ccnt = 0;
    }
    __syncthreads();
    uint32_t c_loc = 0;
    for (int j = tid; j < d; j += FT) {
      const uint32_t k = s_key[j];
      if (k >= tau) {
        c_loc++;
        atomicAdd(&s_h[(k - tau) >> shift], 1u);
      }
    }
    c_loc = __reduce_add_sync(FULL, c_loc);
    if ((tid & 31) == 0 && c_loc) atomicAdd(&s_ccnt, c_loc);
    __syncthreads();
    const uint32_t C = s_ccnt;  // keys >= tau
    if (C < K) continue;        // the bound was too high
    const uint32_t rt = (a.tau_out != nullptr && a.track_rank <= C) ? a.track_rank : 0u;
    uint32_t bw, rem, bt, trem;
    smem_pick2<H1_BINS>(s_h, K, rt, bw, rem, bt, trem);
    for (int j = tid; j < d; j += FT) {
      const uint32_t k = s_key[j];
      if (k >= tau && ((k - tau) >> shift) == bw) {
        const uint32_t at = atomicAdd(&s_lcnt, 1u);
        if (at < (uint32_t)WIN_LIST) s_list[at] = k;
      }
    }
    __syncthreads();
    const uint32_t m = s_lcnt;
    if (m > (uint32_t)WIN_LIST) continue;  // too many keys share the bin of rank K (heavy ties)
    if ((uint32_t)tid < m) {
      const uint32_t mine = s_list[tid];
      uint32_t gt = 0, eq = 0;
      for (uint32_t i = 0; i < m; i++) {
        const uint32_t o = s_list[i];
        gt += o > mine;
        eq += o == mine;
      }
      if (gt < rem && rem <= gt + eq) {  // the rem-th largest key of the bin is T_n
        s_res[0] = mine;
        s_res[1] = rem - gt;
        s_res[2] = eq;
      }
    }
    __syncthreads();
    T = s_res[0];
    need = s_res[1];
    cnt_eq = s_res[2];
    resolved = true;
    if (a.tau_out != nullptr && tid == 0)
      a.tau_out[n] = trem != 0 ? tau + (bt << shift) : tau_below(tau, T, C, K, a.track_rank);
  }
  __syncthreads();
  TAIL_STAMP(2);
  if (!resolved) {
    uint32_t b1, rem1, b2, rem2, b3, u0, u1;
    for (int bb = tid; bb < H1_BINS; bb += FT) s_h[bb] = 0;
    __syncthreads();
    for (int j = tid; j < d; j += FT) atomicAdd(&s_h[s_key[j] >> 20], 1u);
    __syncthreads();
    smem_pick2<H1_BINS>(s_h, K, 0u, b1, rem1, u0, u1);
    for (int bb = tid; bb < H1_BINS; bb += FT) s_h[bb] = 0;
    __syncthreads();
    for (int j = tid; j < d; j += FT) {
      const uint32_t k = s_key[j];
      if ((k >> 20) == b1) atomicAdd(&s_h[(k >> 10) & 1023u], 1u);
    }
    __syncthreads();
    smem_pick2<H2_BINS>(s_h, rem1, 0u, b2, rem2, u0, u1);
    for (int bb = tid; bb < H1_BINS; bb += FT) s_h[bb] = 0;
    __syncthreads();
    const uint32_t prefix = (b1 << 10) | b2;
    for (int j = tid; j < d; j += FT) {
      const uint32_t k = s_key[j];
      if ((k >> 10) == prefix) atomicAdd(&s_h[k & 1023u], 1u);
    }
    __syncthreads();
    smem_pick2<H3_BINS>(s_h, rem2, 0u, b3, need, u0, u1);
    cnt_eq = s_h[b3];
    T = (b1 << 20) | (b2 << 10) | b3;
    // the next call starts an eighth of a binade below this call's K-th key
    if (a.tau_out != nullptr && tid == 0) a.tau_out[n] = T > (1u << 20) ? T - (1u << 20) : 0u;
    __syncthreads();
  }
  TAIL_STAMP(3);
  if (tid == 0) {
    uint32_t* ws = p.wstate + (size_t)n * 8;
    ws[4] = T;
    ws[5] = K - need;
    ws[6] = cnt_eq;
    ws[7] = need;
    p.thresh[n * 3 + 0] = T;
    p.thresh[n * 3 + 1] = K - need;
    p.thresh[n * 3 + 2] = cnt_eq;
    p.diag_cnt[n] = K;  // (no candidate buffer here: reported as "exactly K kept")
  }
  // ---- the votes (Eq. 9, inner sum): keys above T_n, and the `need` lowest-index ties.  Thread t owns the
  // coordinates [t per, (t + 1) per), so thread order is index order.  Every vote is an atomic add that hands back
  // the coordinate's count before it, so the CTA also learns how the vote histogram changes: a coordinate that goes
  // from v to v + 1 votes leaves bin v and enters bin v + 1 (signed changes per bin, summed over the grid before
  // the barrier; the bin of zero votes is derived afterwards) ----
  int* s_hd = reinterpret_cast<int*>(s_h);  // [256] this CTA's changes to the vote histogram
  for (int v = tid; v < 256; v += FT) s_hd[v] = 0;
  {
    const int per = (d + FT - 1) / FT;
    const int j0 = min(d, tid * per), j1 = min(d, j0 + per);
    uint32_t erank = 0;
    if (need < cnt_eq) {  // ties kept only in part (alike in all threads): their rank in index order
      uint32_t eq = 0, etot;
      for (int j = j0; j < j1; j++) eq += s_key[j] == T;
      erank = block_excl_scan<FT>(eq, s_sw, etot);
    } else {
      __syncthreads();  // (s_hd is clear)
    }
    for (int jb = j0; jb < j1; jb += 8) {
      uint32_t old[8], hit = 0;
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int j = jb + q;
        old[q] = 0;
        if (j < j1) {
          const uint32_t k = s_key[j];
          bool take = k > T;
          if (k == T) {
            take = erank < need;
            erank++;
          }
          if (take) {
            hit |= 1u << q;
            old[q] = atomicAdd(a.votes_now + ((uint32_t)j >> 2), 1u << (8u * ((uint32_t)j & 3u)));
          }
        }
      }
#pragma unroll
      for (int q = 0; q < 8; q++) {
        if (hit & (1u << q)) {
          const uint32_t v = (old[q] >> (8u * ((uint32_t)(jb + q) & 3u))) & 0xffu;
          if (v < 255u) atomicAdd(&s_hd[v + 1], 1);
          if (v) atomicSub(&s_hd[v], 1);
        }
      }
    }
    __syncthreads();
    if (tid >= 1 && tid <= p.N && s_hd[tid] != 0) atomicAdd(a.hist_now + tid, (uint32_t)s_hd[tid]);
  }
  TAIL_STAMP(4);
  if (!grid_barrier(bar)) return;  // the only one: all votes are in

  TAIL_STAMP(5);
  // ---- Eq. 9, outer S_top, by every CTA for itself: thread t owns vote bytes [32 t, 32 t + 32) ----
  const uint4* vq = reinterpret_cast<const uint4*>(a.votes_now) + 2 * tid;
  uint4 q0 = make_uint4(0, 0, 0, 0), q1 = q0;
  if (32 * tid < d) {  // (the array is whole chunks long and zero beyond d)
    q0 = __ldcg(vq);
    q1 = __ldcg(vq + 1);
  }
  if (tid < 256) s_hv[tid] = (tid >= 1 && tid <= p.N) ? __ldcg(a.hist_now + tid) : 0u;
  // the arrays of the next call (nobody reads them during this one): its vote bytes, its histogram, its barrier word
  zero_share(a.votes_next, (size_t)p.nchunks * (CH / 4), (size_t)n, (size_t)G);
  if (n == 0 && tid < 256) a.hist_next[tid] = 0u;
  if (n == 0 && tid == 0) *a.bar_next = 0u;
  const uint32_t w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
  __syncthreads();
  if (tid == 0) {
    uint32_t voted = 0;
    for (int v = 1; v <= p.N; v++) voted += s_hv[v];
    s_hv[0] = (uint32_t)d - voted;
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
    s_vs[3] = K - cgt;
    if (n == 0) {
      p.vstate[0] = vstar;
      p.vstate[1] = cgt;
      p.vstate[2] = ceq;
      p.vstate[3] = K - cgt;
    }
  }
  __syncthreads();
  TAIL_STAMP(6);
  const uint32_t vstar = s_vs[0], quota = s_vs[3];
  uint32_t gm = 0, em = 0;  // one bit per coordinate of the thread: votes > v*, votes == v*
  {
    const uint32_t vs4 = vstar * 0x01010101u;
#pragma unroll
    for (int i = 0; i < 8; i++) {
      gm |= (((__vcmpgtu4(w[i], vs4) & 0x01010101u) * 0x01020408u) >> 24) << (4 * i);
      em |= (((__vcmpeq4(w[i], vs4) & 0x01010101u) * 0x01020408u) >> 24) << (4 * i);
    }
    const int left = d - 32 * tid;
    const uint32_t inb = left >= 32 ? 0xffffffffu : (left <= 0 ? 0u : (1u << left) - 1u);
    gm &= inb;
    em &= inb;
  }
  // one scan for both counts (each at most 32768 over the row: sixteen bits apiece): the v*-ties and the
  // coordinates above v* before this thread; the thread's outputs start after those and the ties kept so far
  uint32_t both_tot;
  const uint32_t both = block_excl_scan<FT>(((uint32_t)__popc(em) << 16) | (uint32_t)__popc(gm), s_sw, both_tot);
  const uint32_t epre = both >> 16, gpre = both & 0xffffu;
  uint32_t sm = gm;
  if (epre < quota) {  // keep this thread's first ties while the quota lasts
    uint32_t room = quota - epre, e2 = em;
    while (e2 && room) {
      const uint32_t low = e2 & (0u - e2);
      sm |= low;
      e2 ^= low;
      room--;
    }
  }
  uint32_t pos = gpre + min(epre, quota);
  const uint32_t lo = (uint32_t)((uint64_t)n * K / (uint64_t)G), hi = (uint32_t)((uint64_t)(n + 1) * K / (uint64_t)G);
  int32_t* s_out = reinterpret_cast<int32_t*>(s_key);  // this CTA's outputs [lo, hi) of supp(M) (the keys are done with)
  while (sm) {
    const int bb = __ffs(sm) - 1;
    sm &= sm - 1;
    if (pos >= lo && pos < hi) {
      a.out_idx[pos] = 32 * tid + bb;
      s_out[pos - lo] = 32 * tid + bb;
    }
    pos++;
  }
  __syncthreads();
  TAIL_STAMP(7);
  // ---- Eq. 8 and the error update on those outputs ----
  {
    const uint32_t m = hi - lo;
    if (m * 8u <= (uint32_t)FT) {
      const uint32_t kk = (uint32_t)tid >> 3;
      const bool live = kk < m;
      gather_at<8>(a.err, p.N, p.d, (int64_t)lo + kk, live ? (int64_t)s_out[kk] : -1, live, tid & 7, a.out_val, nullptr, a.dbg);
    } else {
      for (uint32_t k = tid; k < m; k += FT) gather_at<1>(a.err, p.N, p.d, (int64_t)lo + k, (int64_t)s_out[k], true, 0, a.out_val, nullptr, a.dbg);
    }
  }
  TAIL_STAMP(8);
#ifdef MV_TAIL_STAMPS
  TAIL_STAMP(9);
  if (blockIdx.x == 0 && threadIdx.x == 0 && (atomicAdd(&g_stamp_calls, 1u) % 199u) == 198u) {
    printf("small stamps us:");
    for (int i = 1; i <= 9; i++) printf(" %.1f", (double)(stamps[i] - stamps[i - 1]) * 1e-3);
    printf("\n");
  }
#endif
}
