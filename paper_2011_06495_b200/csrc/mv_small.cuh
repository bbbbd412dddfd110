// mv_small.cuh -- a whole step as ONE kernel for rows that fit a CTA's shared memory (d <= 32768).
// (Included by mv_sparse.cu inside its anonymous namespace, after mv_tail.cuh.)
//
// A problem this small is all launch latency when it runs as a sequence of kernels.  Here worker n is CTA n:
// it reads its row once (acc = err + grads, written in place), keeps the d magnitude keys in shared memory,
// finds its exact K-th key there by three radix digits (no sampling, no candidate buffer) and votes.  After the
// only grid barrier every CTA reads the d vote bytes, finds v* and the output positions for itself, writes its
// share of supp(M), gathers the mean there and zeroes the residual.  The vote bytes alternate between two
// arrays from call to call: the one not in use is cleared for the next call while this one runs, so no
// barrier is spent on clearing.  Launched cooperatively; the barrier wait is bounded like those of the tail.

constexpr int SMALL_MAX_D = SK_KEYS;  // 32768 keys of shared memory

struct SmallArgs {
  const float* grads;
  float* err;
  int32_t* out_idx;
  float* out_val;
  uint32_t* votes_now;    // this call's vote bytes, four to a word, all zero at the start (whole chunks long)
  uint32_t* votes_next;   // the other array: cleared here for the next call
  uint32_t* words;        // [16] barrier arrivals, exit ticket (zero at the start, put back to zero at the end)
  uint32_t* abort_flag;
  uint32_t spin_limit;
  uint32_t* dbg;
};

__global__ void __launch_bounds__(FT, 1) k_small(P p, SmallArgs a) {
#ifdef MV_TAIL_STAMPS
  unsigned long long stamps[16];
#endif
  TAIL_STAMP(0);
  pdl_enter();
  extern __shared__ uint32_t s_key[];  // [d] the row's magnitude keys
  __shared__ uint32_t s_h[H1_BINS];
  __shared__ uint32_t s_sw[FT / 32 + 1];
  __shared__ uint32_t s_hv[256];
  __shared__ uint32_t s_vs[4];
  __shared__ uint32_t s_lastout;
  const int tid = threadIdx.x;
  const int G = gridDim.x, n = blockIdx.x;  // G == N
  const int d = (int)p.d;
  const uint32_t K = (uint32_t)p.K;
  GridBar bar;
  bar.ctr = a.words;
  bar.abort_flag = a.abort_flag;
  bar.nblocks = (uint32_t)G;
  bar.target = 0u;
  bar.limit = a.spin_limit;

  // ---- accumulate (Algorithm 1, error feedback): the row once through; its keys stay in shared memory ----
  {
    const float* grow = a.grads + (size_t)n * (size_t)d;
    float* erow = a.err + (size_t)n * (size_t)d;
    for (int j0 = 0; j0 < d; j0 += FT * 4) {
      float e[4], g[4];
#pragma unroll
      for (int q = 0; q < 4; q++) {
        const int j = j0 + q * FT + tid;
        e[q] = j < d ? __ldcs(erow + j) : 0.f;
        g[q] = j < d ? __ldcs(grow + j) : 0.f;
      }
#pragma unroll
      for (int q = 0; q < 4; q++) {
        const int j = j0 + q * FT + tid;
        if (j < d) {
          const float v = __fadd_rn(e[q], g[q]);
          erow[j] = v;
          s_key[j] = fkey(v);
        }
      }
    }
  }
  TAIL_STAMP(1);
  // ---- S_top (Eq. 6): the exact K-th key by three radix digits (11 + 10 + 10 bits) over the keys in shared memory ----
  uint32_t b1, rem1, b2, rem2, b3, need, u0, u1;
  for (int bb = tid; bb < H1_BINS; bb += FT) s_h[bb] = 0;
  __syncthreads();
  for (int j = tid; j < d; j += FT) atomicAdd(&s_h[s_key[j] >> 20], 1u);
  __syncthreads();
  smem_pick2<H1_BINS>(s_h, K, 0u, b1, rem1, u0, u1);
  TAIL_STAMP(2);
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
  TAIL_STAMP(3);
  const uint32_t cnt_eq = s_h[b3];
  const uint32_t T = (b1 << 20) | (b2 << 10) | b3;
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
  // coordinates [t per, (t + 1) per), so thread order is index order ----
  {
    const int per = (d + FT - 1) / FT;
    const int j0 = min(d, tid * per), j1 = min(d, j0 + per);
    uint32_t eq = 0;
    for (int j = j0; j < j1; j++) eq += s_key[j] == T;
    uint32_t etot;
    uint32_t erank = block_excl_scan<FT>(eq, s_sw, etot);
    for (int j = j0; j < j1; j++) {
      const uint32_t k = s_key[j];
      bool take = k > T;
      if (k == T) {
        take = erank < need;
        erank++;
      }
      if (take) add_vote(a.votes_now, (uint32_t)j);
    }
  }
  TAIL_STAMP(4);
  if (!grid_barrier(bar)) return;  // the only one: all votes are in

  TAIL_STAMP(5);
  // ---- the other vote array, for the next call (nobody reads it during this one) ----
  zero_share(a.votes_next, (size_t)p.nchunks * (CH / 4), (size_t)n, (size_t)G);

  // ---- Eq. 9, outer S_top, by every CTA for itself: thread t owns vote bytes [32 t, 32 t + 32) ----
  const uint4* vq = reinterpret_cast<const uint4*>(a.votes_now) + 2 * tid;
  uint4 q0 = make_uint4(0, 0, 0, 0), q1 = q0;
  if (32 * tid < d) {  // (the array is whole chunks long and zero beyond d)
    q0 = __ldcg(vq);
    q1 = __ldcg(vq + 1);
  }
  const uint32_t w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
  for (int v = tid; v < 256; v += FT) s_hv[v] = 0;
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 8; i++) {
    uint32_t x = w[i];
    while (x) {
      const int bb = (__ffs(x) - 1) >> 3;
      atomicAdd(&s_hv[(x >> (8 * bb)) & 0xffu], 1u);
      x &= ~(0xffu << (8 * bb));
    }
  }
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
  uint32_t etot, stot;
  const uint32_t epre = block_excl_scan<FT>(__popc(em), s_sw, etot);
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
  uint32_t pos = block_excl_scan<FT>(__popc(sm), s_sw, stot);
  const uint32_t lo = (uint32_t)((uint64_t)n * K / (uint64_t)G), hi = (uint32_t)((uint64_t)(n + 1) * K / (uint64_t)G);
  while (sm) {  // this CTA writes outputs [lo, hi) of supp(M)
    const int bb = __ffs(sm) - 1;
    sm &= sm - 1;
    if (pos >= lo && pos < hi) a.out_idx[pos] = 32 * tid + bb;
    pos++;
  }
  __syncthreads();
  TAIL_STAMP(7);
  // ---- Eq. 8 and the error update on those outputs ----
  {
    const uint32_t m = hi - lo;
    if (m * 8u <= (uint32_t)FT) {
      const uint32_t kk = (uint32_t)tid >> 3;
      gather_one<8>(a.err, p.N, p.d, (int64_t)lo + kk, kk < m, tid & 7, a.out_idx, a.out_val, nullptr, a.dbg);
    } else {
      for (uint32_t k = lo + tid; k < hi; k += FT) gather_one<1>(a.err, p.N, p.d, (int64_t)k, true, 0, a.out_idx, a.out_val, nullptr, a.dbg);
    }
  }
  TAIL_STAMP(8);
  // ---- the last CTA out puts the barrier words back to zero ----
  __threadfence();
  __syncthreads();
  if (tid == 0) s_lastout = (atomicAdd(a.words + 1, 1u) == (uint32_t)G - 1u) ? 1u : 0u;
  __syncthreads();
  if (s_lastout && tid < 2) a.words[tid] = 0u;
#ifdef MV_TAIL_STAMPS
  TAIL_STAMP(9);
  if (blockIdx.x == 0 && threadIdx.x == 0 && (atomicAdd(&g_stamp_calls, 1u) % 199u) == 198u) {
    printf("small stamps us:");
    for (int i = 1; i <= 9; i++) printf(" %.1f", (double)(stamps[i] - stamps[i - 1]) * 1e-3);
    printf("\n");
  }
#endif
}
