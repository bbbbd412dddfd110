/*
 * mv_sparse.h -- C ABI of the majority-vote sparse DSGD step for NVIDIA B200 (sm_100a).
 *
 * The library computes one iteration of "sparse SGD with majority voting"
 * (Algorithm 1 of arXiv 2011.06495) for N workers held as the rows of one
 * N x d array on a single GPU:
 *
 *   acc_n   = grads_n + err_n                    error feedback      (Algorithm 1, accumulate step)
 *   M_n     = S_top(|acc_n|, K)                  per-worker top-K    (Eq. 6, definition of S_top)
 *   votes   = sum_n M_n                          vote count          (Eq. 9, inner sum)
 *   M       = S_top(votes, K)                    shared mask         (Eq. 9, outer S_top)
 *   out_val = (1/N) sum_n acc_n  on supp(M)      shared-mask mean    (Eq. 8; the 1/N of the text)
 *   err_n   = acc_n - M (x) acc_n                residual            (Algorithm 1, error update)
 *
 * Conventions (the paper leaves them open; they are part of this contract):
 *   - |x| is ordered by key(x) = bits(x) & 0x7fffffff; ties in either S_top go to the
 *     lowest coordinate index, so every result is unique.
 *   - supports are ascending int32 index lists; bit masks are ceil(d/32) uint32 words
 *     per row, bit b of word w standing for coordinate 32*w + b, unused tail bits zero.
 *   - out_val is the mean: binary64 accumulation in worker order, one division by N,
 *     one rounding to binary32.
 *   - the residual is +0.0f on the mask and a bit copy of acc elsewhere.
 *
 * Memory: unless a parameter says "host", every pointer is a DEVICE pointer owned by
 * the caller, row-major and contiguous (row pitch d), 16-byte aligned at its base.
 * The library allocates and frees no device memory: scratch space is the caller's
 * workspace of mv_workspace_bytes() bytes, reused by every call on the context.
 * All work is enqueued on the stream given to mv_create; no call synchronises the
 * host except mv_sparse_step_host and mv_read_diag.  A context is not thread-safe.
 *
 * Limits: 1 <= N <= 255, 1 <= d < 2^31 - 8192, 1 <= K <= d.
 *
 * Errors: every int-returning function returns MV_OK or a negative MV_ERR_* code;
 * argument checks happen before anything is enqueued, so a failed call has no effect.
 */
#ifndef MV_SPARSE_H
#define MV_SPARSE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  MV_OK = 0,
  MV_ERR_INVALID_ARG = -1, /* null or misaligned pointer, N/d/K out of range, grads aliasing err */
  MV_ERR_WORKSPACE = -2,   /* workspace smaller than mv_workspace_bytes(N, d, K) */
  MV_ERR_CUDA = -3,        /* the CUDA runtime refused a launch or a copy */
  MV_ERR_TOO_LARGE = -4,   /* mv_select_static only: d is larger than MV_SELECT_STATIC_MAX_D */
  MV_ERR_TIMEOUT = -5      /* a bounded wait between the CTAs of a kernel gave up (never expected: the kernel that
                              waits is launched so that all its CTAs run together); the results of that call and
                              of later calls on the context are not valid.  Reported by the calls that wait for
                              the stream: mv_sparse_step_host, mv_read_diag, mv_fallback_count, mv_debug_status */
};

enum {
  MV_MODE_AUTO = 0,    /* sampled threshold + single streaming pass, exact multi-pass select as fallback */
  MV_MODE_GENERAL = 1, /* always the exact multi-pass radix select (no sampling) */
  MV_MODE_TRACK = 2    /* as AUTO, but a call that follows one with the same N, d, K on the same context takes
                          its candidate threshold from that call's key histogram instead of sampling: meant
                          for the consecutive steps of one training run, where |acc| changes slowly.  Exact
                          for any input: a worker whose threshold turns out unusable (fewer than K or more
                          than 4K + 4096 candidates) takes the multi-pass select for that call.
                          The carried thresholds belong to the context, not to a buffer: use one context
                          per residual buffer (per training run).  A context that alternates between two
                          residual buffers of the same shape stays exact but hands each the other's
                          thresholds, and whenever those do not fit, the slow route is taken. */
};

/* Bits of the device status word of a checked build (see mv_debug_status).  The first three report a
 * detour that leaves every result exact; the others report an index that was refused. */
enum {
  MV_DBG_CAND_OVERFLOW = 1,   /* streaming pass (S_top candidate filter): a worker had more candidates than its
                                 buffer holds; the surplus was dropped and the worker takes the full-row select */
  MV_DBG_WINDOW_OVERFLOW = 2, /* select (S_top, K-th key): the bin of the K-th key held more than 1024 keys; it was resolved
                                 by a second count over that bin's keys, or by the three-digit radix select */
  MV_DBG_FALLBACK = 4,        /* select: a worker's K-th key was found over its full row (candidate count outside [K, cap]) */
  MV_DBG_LIST_OVERFLOW = 8,   /* add-drop / random selection (Algorithm 2; Algorithm 1, S_rand line): a list outgrew its
                                 room and was treated as empty */
  MV_DBG_PICK_RANGE = 16,     /* picks (Eq. 9, inner sum): a candidate named a coordinate >= d and was skipped */
  MV_DBG_LIST_RANGE = 32,     /* supp(M_n) lists: an entry beyond position K was not written */
  MV_DBG_OUT_RANGE = 64,      /* supp(M) (Eq. 9, outer S_top): an entry beyond position K was not written */
  MV_DBG_GATHER_RANGE = 128,  /* aggregate (Eq. 8): idx[k] outside [0, d); out_val[k] = 0 and the residual is untouched there */
  MV_DBG_INTERNAL = 256       /* an index computed inside a kernel left its array and the access was skipped */
};

typedef struct mv_ctx mv_ctx;

/* Bytes of device scratch needed for a problem of this size (host computation only).
 * Returns 0 if N, d or K is out of range. */
size_t mv_workspace_bytes(int N, int64_t d, int64_t K);

/* Creates a context bound to `stream` (a cudaStream_t, may be NULL for the default
 * stream) and to `workspace` (device memory, 256-byte aligned, owned by the caller,
 * must outlive the context).  Touches no device memory. */
int mv_create(mv_ctx** out, void* stream, void* workspace, size_t workspace_bytes);
int mv_destroy(mv_ctx* ctx);

/* Chooses how the per-worker threshold is found (MV_MODE_*).  Results are identical. */
int mv_set_mode(mv_ctx* ctx, int mode);

/* How mv_sparse_step runs what follows its pass over grads and err (S_top from the candidates on, the votes of
 * Eq. 9, the shared mask, the aggregate of Eq. 8 and the residual): either as the sequence of kernels that mv_vote,
 * mv_select and mv_aggregate use, or as ONE kernel whose CTAs (one per multiprocessor, launched cooperatively) stay
 * resident and meet at grid barriers.  The single kernel can run when the device supports cooperative launches,
 * N is at most the number of multiprocessors, d <= 32768 * 4096 = 2^27 and the mode is not MV_MODE_GENERAL.
 *   enable = 1 (default): the single kernel where it can run and K >= 65536 (many picks and outputs: there it is
 *                         faster), the sequence otherwise;  0: always the sequence;  2: the single kernel wherever
 *                         it can run.
 * The bytes of every result are the same either way.  The barrier waits are bounded: see MV_ERR_TIMEOUT. */
int mv_set_tail_kernel(mv_ctx* ctx, int enable);

/* The whole step (Algorithm 1 from the accumulate line to the aggregate line).
 *   grads   [N*d] in      the workers' model differences / gradients
 *   err     [N*d] in/out  e_n on entry, the new residual e_n on exit
 *   out_idx [K]   out     supp(M), ascending
 *   out_val [K]   out     mean of acc over the workers on supp(M)
 * Equivalent to mv_vote, mv_select, mv_aggregate in that order. */
int mv_sparse_step(mv_ctx* ctx, const float* grads, float* err, int N, int64_t d, int64_t K,
                   int32_t* out_idx, float* out_val);

/* Voting phase, worker side and vote count (Algorithm 1 up to the vote sum; Eq. 6, Eq. 9 inner sum).
 *   err         [N*d]           in/out  e_n on entry, acc_n on exit
 *   worker_idx  [N*K]           out     supp(M_n) ascending, row n at n*K          (may be NULL)
 *   worker_bits [N*ceil(d/32)]  out     M_n as bit masks                           (may be NULL)
 *   votes       [d] uint8       out     votes per coordinate                       (may be NULL)
 *   thresh      [N*3] uint32    out     per worker: K-th largest key T_n, number of keys above
 *                                       it, number of keys equal to it             (may be NULL)
 * An output passed as NULL is not delivered (the masks, votes and thresholds then live in the workspace
 * only; the ascending lists are not built at all). */
int mv_vote(mv_ctx* ctx, const float* grads, float* err, int N, int64_t d, int64_t K,
            int32_t* worker_idx, uint32_t* worker_bits, uint8_t* votes, uint32_t* thresh);

/* Voting phase, server side (Eq. 9 outer S_top): the K most voted coordinates.
 *   votes     [d] uint8        in   every value must be <= N
 *   out_idx   [K]              out  ascending
 *   mask_bits [ceil(d/32)]     out  the same set as a bit mask (may be NULL) */
int mv_select(mv_ctx* ctx, const uint8_t* votes, int N, int64_t d, int64_t K,
              int32_t* out_idx, uint32_t* mask_bits);

/* One step of majority voting with add-drop (Algorithm 2, MV-AD; the vote update and Eq. 16).
 * Each worker keeps a vote mask from the previous step and changes at most K_ad entries in each
 * direction: it adds the K_ad largest |acc| among its current top-K coordinates that it did not
 * vote for, and drops the K_ad smallest |acc| among its previous votes that are not in its current
 * top-K (fewer if fewer are eligible; ties to the lowest index).  The shared mask is the K
 * coordinates voted for by most workers under the updated masks (the running sum of Eq. 16 is
 * that count), filled up in index order if fewer than K coordinates have a vote.  Aggregation and
 * residual are those of mv_sparse_step.
 *   grads     [N*d] in; err [N*d] in/out (residual); out_idx [K], out_val [K] out
 *   prev_bits [N*ceil(d/32)] in/out  the workers' vote masks; at most K bits per worker and no
 *                                    bits at or beyond d (all-zero masks are a valid start)
 *   K_ad      1 <= K_ad <= K
 *   add_bits, drop_bits [N*ceil(d/32)] out, may be NULL: what each worker added / dropped
 *   msum      [d] uint8 out, may be NULL: votes per coordinate under the updated masks */
int mv_ad_step(mv_ctx* ctx, const float* grads, float* err, uint32_t* prev_bits, int N, int64_t d, int64_t K,
               int64_t K_ad, int32_t* out_idx, float* out_val, uint32_t* add_bits, uint32_t* drop_bits,
               uint8_t* msum);

/* One step of SSGD-top-K, the scheme the paper compares majority voting with (Section 2, first paragraph: every
 * worker sends acc_n (x) S_top(|acc_n|, K), Eq. 6, and the server forms (1/N) sum_n of what it receives, the
 * estimate of Eq. 7; Table 1, row SSGD-top-K).  No consensus: the masks differ from worker to worker, so the
 * aggregate is non-zero on their union, between K and min(d, N K) coordinates.
 *   grads    [N*d] in;  err [N*d] in/out: e_n on entry, acc_n - M_n (x) acc_n on exit (each worker's residual is
 *                       zeroed on its OWN mask)
 *   out_idx  [capacity] out  the union of the workers' masks, ascending; entries from *count on are -1
 *   out_val  [capacity] out  per union coordinate: the binary64 sum, in worker order, over the workers whose mask
 *                            holds it, divided by N (all N workers), rounded once to binary32; 0 from *count on
 *   capacity            >= min(d, N K), else MV_ERR_INVALID_ARG
 *   count    [1] int32 out (DEVICE): the size of the union */
int mv_topk_union_step(mv_ctx* ctx, const float* grads, float* err, int N, int64_t d, int64_t K,
                       int32_t* out_idx, float* out_val, int64_t capacity, int32_t* count);

/* Worker-sharded step (the paper's remark under Eq. 8 that a shared mask lets the values be summed by
 * an all-reduce): when the N workers are spread over several GPUs, each rank runs mv_vote on its
 * N_local rows, the vote counts (uint8 [d]) are summed over the ranks, every rank runs mv_select on
 * the summed votes with N = the total number of workers, mv_aggregate_partial gives the rank's
 * binary64 partial sums on the shared mask (and zeroes its workers' residual there), the partial
 * sums are summed over the ranks and mv_finish_mean divides by the total number of workers and
 * rounds once to binary32.  The two sums over ranks are the caller's collectives; the library only
 * provides the two kernels that a single-GPU step does not need.
 *   out_sum [K] double out: sum over this rank's workers, in worker order, of acc[n][idx[k]]
 *   sum     [K] double in : the sum of all ranks' out_sum;  out_val [K] float out
 * Differences from the single-GPU mean: only the order in which the binary64 terms of different
 * ranks are added (fixed by the collective), i.e. at most a last-bit difference after rounding. */
int mv_aggregate_partial(mv_ctx* ctx, float* acc, int N_local, int64_t d, int64_t K, const int32_t* idx,
                         double* out_sum);
int mv_finish_mean(void* stream, const double* sum, int64_t K, int N_total, float* out_val);

/* Majority voting with random selection (SSGD-MV-RS: Algorithm 1 with the S_rand-weighted line; Section
 * 4.1 words it as "select indices at random using the votes until K unique indices are selected").
 * The shared mask is a draw of successive sampling proportional to the votes, taken with one random
 * number per coordinate (exponential clocks): coordinate j with v_j > 0 votes gets the ring time
 * t_j = E_j / v_j, E_j = -ln((x_j + 1/2) / 2^32), x_j = first output word of Philox4x32-10 with key
 * (seed low, seed high) and counter (j, 0, draw low, draw high); the K smallest t_j win.  So that a
 * CPU statement of the same rule gives the same indices, every deciding operation is fixed: -ln by
 * the binary64 recipe v = 2x+1, e = floor(log2 v), m = v/2^e (halved and e+1 if m > sqrt 2),
 * s = (m-1)/(m+1), ln m = 2s(1 + s^2/3 + ... + s^22/23) by Horner from the 1/23 end,
 * E = (33-e) ln2 - ln m; t_j is one binary64 division rounded once to binary32; equal t_j go to the
 * lowest index.  Coordinates without a vote are never selected; if fewer than K hold a vote, the
 * tail of out_idx is filled with -1.  The same (seed, draw) gives the same mask; use a new `draw`
 * every step.
 *
 * mv_select_rs: votes [d] uint8 in: the count of at most N workers voting for at most K coordinates each
 *              (so at most N K coordinates hold a vote; with more than that nothing is selected and
 *              out_idx is all -1); out_idx [K] out ascending; mask_bits may be NULL.
 * mv_rs_step:  as mv_sparse_step with this selection in place of the K most voted (the union of the
 *              workers' top-K sets always holds at least K coordinates, so out_idx is full). */
int mv_select_rs(mv_ctx* ctx, const uint8_t* votes, int N, int64_t d, int64_t K, uint64_t seed, uint64_t draw,
                 int32_t* out_idx, uint32_t* mask_bits);
int mv_rs_step(mv_ctx* ctx, const float* grads, float* err, int N, int64_t d, int64_t K, uint64_t seed, uint64_t draw,
               int32_t* out_idx, float* out_val);

/* mv_select for callers that cannot hand the library a workspace.  (The paper has no counterpart
 * to this call: it is the same selection as mv_select, packaged differently.)
 *
 * Who needs it: code that runs where device memory may not be allocated -- inside a region that
 * the application has closed to cudaMalloc (a real-time loop, a plug-in whose host forbids
 * allocation after start-up, a process whose memory pool is already fully handed out) -- and that
 * therefore has no buffer of mv_workspace_bytes() to give to mv_create.  This call needs neither a
 * context nor a workspace and calls no allocating routine: its scratch space is an array compiled
 * into the library, about 2.2 MB, which every GPU that loads the library holds until the process
 * ends.  The caller still owns and passes the input and the outputs.
 *
 *   stream    cudaStream_t to enqueue on (NULL = default stream)
 *   votes     [d] uint8        in   every value must be <= N
 *   out_idx   [K]              out  ascending
 *   mask_bits [ceil(d/32)]     out  the same set as a bit mask (may be NULL)
 *
 * Limits: d <= MV_SELECT_STATIC_MAX_D (the array is sized for that; a larger d returns
 * MV_ERR_TOO_LARGE and nothing is enqueued); N and K as for mv_select.
 * First use: the first call on each device looks up the array's device address (with that device
 * current) and remembers it; make that first call outside any stream capture.
 * Sharing: all calls in the process use the one array, which keeps what the previous call left;
 * the call itself clears the parts that must start at zero.  Two calls whose kernels overlap on
 * the GPU (different streams without an ordering between them) would race on the array: order
 * them.  Results are identical to mv_select's. */
#define MV_SELECT_STATIC_MAX_D (1 << 24)
int mv_select_static(void* stream, const uint8_t* votes, int N, int64_t d, int64_t K,
                     int32_t* out_idx, uint32_t* mask_bits);

/* Sparse communication phase (Algorithm 1 from the masked send to the aggregate; Eq. 8).
 *   acc     [N*d] in/out  acc_n on entry, the residual on exit
 *   idx     [K]   in      distinct coordinates in [0, d)
 *   out_val [K]   out     mean over the workers of acc[:, idx[k]] */
int mv_aggregate(mv_ctx* ctx, float* acc, int N, int64_t d, int64_t K, const int32_t* idx, float* out_val);

/* The whole step for a caller whose gradients live in HOST memory (Algorithm 1, same lines
 * as mv_sparse_step).  Copies h_grads (host, ideally pinned) into d_grads, runs the step on
 * the device-resident residual d_err, copies the K indices and values back to the host
 * buffers and waits for the stream before returning.
 *   h_grads [N*d] host in; h_out_idx [K], h_out_val [K] host out;
 *   d_grads [N*d], d_err [N*d], d_out_idx [K], d_out_val [K] device buffers of the caller. */
int mv_sparse_step_host(mv_ctx* ctx, const float* h_grads, int N, int64_t d, int64_t K,
                        int32_t* h_out_idx, float* h_out_val,
                        float* d_grads, float* d_err, int32_t* d_out_idx, float* d_out_val);

/* Diagnostics of the last mv_vote / mv_sparse_step on this context; waits for the stream.
 *   per_worker [N*4] host uint32 out: candidates kept by the streaming pass, sampled
 *   lower bound on the threshold key, 1 if the exact multi-pass select was used, 0 (spare). */
int mv_read_diag(mv_ctx* ctx, int N, uint32_t* per_worker);

/* Running count, since the context's first call, of worker selections (one worker in one call) whose
 * K-th key had to be found over the full row because the candidate threshold of the streaming pass
 * admitted fewer than K or more than 4K + 4096 elements (S_top of Algorithm 1 stays exact either way;
 * this is the slow route).  Counted on the device; the call waits for the stream.  total: host, out. */
int mv_fallback_count(mv_ctx* ctx, uint32_t* total);

/* Optional timing of the streaming pass (the kernel that reads grads and err and writes acc,
 * i.e. the accumulate line of Algorithm 1 fused with the candidate filter of S_top): with
 * every = n >= 1, each n-th mv_vote / mv_sparse_step records a CUDA-event pair around that one
 * kernel on the context's stream (a pair costs a few microseconds of stream time); every = 0
 * switches it off.  mv_read_kernel_timing waits for the stream, returns the summed duration in
 * milliseconds and the number of launches it covers (at most the last 64), and restarts the
 * count.  The first enabling call creates the events. */
int mv_set_kernel_timing(mv_ctx* ctx, int every);
int mv_read_kernel_timing(mv_ctx* ctx, float* total_ms, int* launches);

/* Optional per-launch timing of a whole call, for profiling without an external tool.
 * enable = 1: a CUDA event is recorded before the first and after every kernel launch of each call
 * (the events serialise the kernels, so the parts add up to more than the undisturbed call);
 * mv_read_phase_times then returns, for the last call, the milliseconds between consecutive
 * events: ms[i] covers the i-th kernel in launch order (Algorithm 1's steps in the order listed at
 * the top of this file), at most `capacity` (and 47) values, *count their number.
 * enable = 100 + i: only two events, before the first launch and after the i-th (1-based), which
 * disturbs the call far less; mv_read_phase_times returns that one interval in ms[0].
 * enable = 0: off.  While on, all work of a call stays on the context's stream. */
int mv_set_phase_timing(mv_ctx* ctx, int enable);
int mv_read_phase_times(mv_ctx* ctx, float* ms, int capacity, int* count);

/* Number of kernels the last call on this context enqueued. */
int mv_last_launches(const mv_ctx* ctx);

/* Checked build.  The library can be compiled with -DMV_DEBUG (paper_2011_06495_b200/build.py, debug=True,
 * gives libmvsparse_debug.so): every place where a kernel clamps an index, drops an entry that does not fit
 * or takes the exact but slower route then also sets one of the MV_DBG_* bits in a status word that lives in
 * the first bytes of the context's workspace.  Nothing traps and nothing is asserted: the kernels do what the
 * normal build does, and the context stays usable.  mv_debug_status waits for the context's stream, returns
 * the bits collected since the previous read in *device_status and clears them.  In a normal build it
 * returns MV_OK with *device_status = 0.  mv_debug_build returns 1 for a checked build, else 0.
 * (Steps named by the bits: S_top of Eq. 6 / Algorithm 1 for the candidate, window and fallback bits, the
 * vote sum and the outer S_top of Eq. 9, the aggregate of Eq. 8.) */
int mv_debug_status(mv_ctx* ctx, int* device_status);
int mv_debug_build(void);

const char* mv_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MV_SPARSE_H */
