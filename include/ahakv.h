/* ahakv.h -- C ABI of the B200 (sm_100a) implementation of AhaKV's eviction step.
 *
 * AhaKV (arXiv 2506.03762) evicts KV-cache rows per layer and per head in three
 * steps: an eviction SCORE from the last r queries against all cached keys
 * (Section 4.1-4.3), a budgeted SELECTION (Algorithm 1) and the COMPACTION of the
 * surviving K/V rows (Algorithm 1, generation phase, first line of the loop body).
 *
 * Notation: B sequences, Hq query heads, Hkv KV heads, G = Hq/Hkv, d head dim,
 * n cached tokens, n_total logical tokens seen so far, r observation window,
 * B_r recent window, Bud = B_r + B_s total budget, n_keep = min(n, Bud).
 *
 * Conventions that hold for every entry point unless it says otherwise:
 *  - Every tensor pointer is DEVICE memory owned by the caller.  The library
 *    allocates nothing per call; scratch comes from the caller (`ws`).
 *  - Calls are asynchronous on `stream` and never synchronise.
 *  - Argument errors are found on the host before any launch and returned as a
 *    status; nothing aborts, throws or traps.  No output is written in that case.
 *  - Inputs are row-major with the head dimension contiguous and every row
 *    16-byte aligned.  Default layout is q_obs [B,Hq,r,d], k and v [B,Hkv,n,d];
 *    other layouts are described by element strides (batch, head, token).
 *  - Outputs are dense: score [B,Hkv,n] float32, kept_idx [B,Hkv,n_keep] int32
 *    strictly ascending per (b, KV head), k_out and v_out [B,Hkv,n_keep,d] in the
 *    input dtype, score_out [B,Hkv,n_keep] float32.  Outputs must not alias inputs.
 *  - q_obs holds the queries of the last r positions and k, v the cache, all as
 *    the attention layer uses them (after any positional rotation).
 */
#ifndef AHAKV_H_
#define AHAKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  AHAKV_OK = 0,
  AHAKV_ERR_INVALID_ARG = 1, /* a pointer, size, stride or parameter is wrong            */
  AHAKV_ERR_UNSUPPORTED = 2, /* a legal request this library has no kernel for          */
  AHAKV_ERR_WORKSPACE = 3,   /* ws is null, misaligned or smaller than required          */
  AHAKV_ERR_CUDA = 4,        /* a CUDA runtime call or a launch failed                   */
  AHAKV_ERR_TIMEOUT = 5      /* a bounded device-side wait ran out (see last_device_status) */
} ahakv_status;

typedef enum { AHAKV_F32 = 0, AHAKV_F16 = 1, AHAKV_BF16 = 2 } ahakv_dtype;

typedef enum {
  AHAKV_SCALE_FIXED = 0,         /* lambda = scale for every row; 1/sqrt(d) is the plain softmax of Eq. 1 */
  AHAKV_SCALE_ADAPTIVE_ROW = 1,  /* Eq. 12 per observation row, i = the row's logical position + 1       */
  AHAKV_SCALE_ADAPTIVE_CALL = 2  /* Eq. 12 once, with i = n_total                                         */
} ahakv_scale_mode;

enum {
  AHAKV_FLAG_VALUE_PRIOR = 1,   /* refine the score with Eq. 13-15                                   */
  AHAKV_FLAG_POOL_ZERO_PAD = 2, /* Eq. 13's mean filter divides edge windows by the full width        */
  AHAKV_FLAG_GROUP_MAX = 4      /* pool the query heads of a KV head by maximum instead of mean        */
};

typedef struct CUstream_st* ahakv_stream_t; /* a cudaStream_t; NULL is the legacy default stream */

typedef struct {
  int32_t batch, n_q_heads, n_kv_heads; /* n_q_heads % n_kv_heads == 0                              */
  int32_t head_dim;                     /* 64 or 128                                                */
  int32_t n_ctx;                        /* n: rows currently in k and v, >= 1                       */
  int64_t n_total;                      /* tokens seen so far, >= n_ctx (== n_ctx during prefill)   */
  int32_t obs_window;                   /* r: 1 .. min(n_ctx, 256 / G)                              */
  int32_t recent_window;                /* B_r: 0 .. budget                                         */
  int32_t budget;                       /* Bud >= 1                                                 */
  int32_t dtype;                        /* ahakv_dtype of q_obs, k, v, k_out, v_out                 */
  int32_t scale_mode;                   /* ahakv_scale_mode                                         */
  float scale;                          /* lambda for AHAKV_SCALE_FIXED (> 0)                       */
  int32_t pool_kernel;                  /* odd width >= 1 of Eq. 13's mean filter; 1 = no smoothing */
  uint32_t flags;
  int64_t q_stride[3], k_stride[3], v_stride[3]; /* elements: batch, head, token; all 0 = dense default */
} ahakv_params;

/* Bytes of scratch the other entry points need for these parameters (0 if they are invalid).
 * The pointer handed in as `ws` must be 256-byte aligned.  The scratch holds no state between
 * calls, but two calls that overlap on the GPU must not share it. */
size_t ahakv_workspace_bytes(const ahakv_params* p);

/* Eq. 12 (Section 4.2): lambda = sqrt(2 ln(n_total / budget) / head_dim), natural log, on the host.
 * Returns 1/sqrt(head_dim) when n_total <= budget, where Eq. 12 has no real value. */
double ahakv_lambda(int64_t n_total, int32_t budget, int32_t head_dim);

/* Eviction score (Sections 4.1-4.3; Algorithm 1, Prefill lines 6-10 and Generation line F_t):
 *   a_ij = SG-softmax over the keys row i may see (Eq. 1 with the causal mask, Eq. 9 with
 *          lambda from scale_mode, lambda multiplying the raw dot product q.k),
 *   S_j  = sum of a_ij over the r observation rows (Eq. 5), averaged over the G query heads of
 *          the KV head,
 *   with AHAKV_FLAG_VALUE_PRIOR: S_j *= avgpool(|V|^2)_j / max avgpool(|V|^2) (Eq. 13-15),
 *   with score_prev != NULL: S_j += score_prev_j (Algorithm 1: F_t = ... + F_{t-1}).
 * Observation row i sits at logical position n_total - r + i and sees cache rows 0 .. n - r + i.
 * score_prev: nullable, [B,Hkv,n] float32.  score: [B,Hkv,n] float32 out.
 * v may be NULL when the value prior is off.
 * Resources: for 16-bit inputs and n_ctx >= 128 the scoring kernel is launched cooperatively with one CTA per SM
 * and takes each SM's whole tensor memory (512 columns) and nearly all of its shared memory for its duration.  A
 * kernel of the caller's that allocates tensor memory and runs concurrently on another stream can be held up
 * until it ends, and holds it up the same way: the allocation is the hardware's, and the time it waits does not
 * count against the kernel's own bounded waits.  Do not overlap such kernels with this call. */
ahakv_status ahakv_score(const ahakv_params* p, const void* q_obs, const void* k, const void* v,
                         const float* score_prev, float* score, void* ws, size_t ws_bytes,
                         ahakv_stream_t stream);

/* The same score with the r observation rows at positions of the caller's choice instead of the last r (the
 * paper's Limitations section: the recent rows are one choice of "a constant number of accumulators", a TopK
 * choice of the same number another; which rows to take is the caller's policy, this entry point accumulates
 * whichever it is given).  obs_pos: HOST array of r logical positions, strictly ascending, each inside the cache
 * ([n_total - n_ctx, n_total)); q_obs holds the queries of those positions in that order.  Row i sees the cache
 * rows up to its own position (Eq. 1) and, with AHAKV_SCALE_ADAPTIVE_ROW, takes Eq. 12 at obs_pos[i] + 1 tokens.
 * obs_pos = the last r positions gives ahakv_score exactly. */
ahakv_status ahakv_score_rows(const ahakv_params* p, const int64_t* obs_pos, const void* q_obs, const void* k,
                              const void* v, const float* score_prev, float* score, void* ws, size_t ws_bytes,
                              ahakv_stream_t stream);

/* Accumulation over ALL query rows (Section 4.1, Eq. 2-3: S_j = sum over i >= j of a_ij; the paper's "w/o RA"
 * ablation, and H2O's score when scale_mode is AHAKV_SCALE_FIXED with scale 1/sqrt(d) and the value prior is off).
 * q_all holds a query for every cached row, [B,Hq,n,d] (q_stride describes it otherwise).  The rows are scored
 * obs_window at a time (1 .. 256 / G; ceil(n / obs_window) passes of the kernels of ahakv_score, each over the
 * keys its rows can see), summed, and the value prior and score_prev are applied to the sum.  O(n^2 d) work: this
 * is the cost Recent Accumulation removes.  ws as for ahakv_score with the same parameters.
 * AHAKV_FLAG_GROUP_MAX is not offered here (AHAKV_ERR_UNSUPPORTED). */
ahakv_status ahakv_score_full_causal(const ahakv_params* p, const void* q_all, const void* k, const void* v,
                                     const float* score_prev, float* score, void* ws, size_t ws_bytes,
                                     ahakv_stream_t stream);

/* One generation step of the score (Algorithm 1, Generation: A = q_t K^T, F_t = SGsoftmax(A) + F_{t-1}): the one
 * new query of every head against the n cached keys (the new token's own key is row n - 1), pooled over the
 * query heads of each KV head, plus score_prev (nullable; 0 for the new row).  p->obs_window must be 1.  A
 * kernel of its own: K is read once with 16-byte loads, the G x n logits stay in shared memory, no scratch
 * memory is needed.  It takes G <= 8 (or 12, 16) query heads per KV head and G * n <= 40960 logits, which covers
 * caches held at their budget; larger problems and AHAKV_FLAG_VALUE_PRIOR (Algorithm 1's generation phase has
 * no value prior) get AHAKV_ERR_UNSUPPORTED: use ahakv_score with obs_window 1 for those.
 * q_t: [B,Hq,1,d].  score_prev, score: [B,Hkv,n] float32; they may be the same buffer. */
ahakv_status ahakv_score_step(const ahakv_params* p, const void* q_t, const void* k, const float* score_prev,
                              float* score, ahakv_stream_t stream);

/* Compaction in place (Algorithm 1, Generation: K <- K_S, V <- V_S before the next token): rows kept_idx[t] of k,
 * v (and of score, nullable, [B,Hkv,n]) move to rows t; rows from n_keep on are left as they are.  kept_idx is
 * ascending, so rows before the first evicted index are not touched and only the rest is moved.  One CTA per
 * (sequence, KV head), batches staged in shared memory.  The exception to "outputs must not alias inputs". */
ahakv_status ahakv_compact_inplace(const ahakv_params* p, void* k, void* v, float* score, const int32_t* kept_idx,
                                   ahakv_stream_t stream);

/* One generation step on a cache kept as slots (Algorithm 1, Generation, with K <- K_S, V <- V_S done by bookkeeping
 * instead of by moving rows).  Attention does not depend on the order of the cached rows, and Algorithm 1 uses a
 * token's position only to protect the most recent ones, so the cache of a (sequence, KV head) can be a set of
 * budget + 1 slots with a table of positions: the evicted token's slot is where the next token is written, and no
 * row is ever moved.  Per (sequence, KV head), in one kernel: the new token's key and value rows (k_t, v_t:
 * [B,Hkv,1,d], dense) are copied into slot free_slot[b,h]; the one new query per head (q_t: [B,Hq,1,d]) is scored
 * against all budget + 1 slots exactly as ahakv_score_step does (lambda of Eq. 12 from p->n_total, the number of
 * tokens so far with the new one); score ([B,Hkv,budget+1] float32) becomes F_t = SGsoftmax(A_t) + F_{t-1} in
 * place, the new token starting from zero; pos ([B,Hkv,budget+1] int32, the position of the token in each slot)
 * gets p->n_total - 1 for the new token; and of the slots whose position is below p->n_total - recent_window (the
 * recent window is the last recent_window positions, the new token's included, and is never evicted, so those
 * tokens are all in the cache) the one with the smallest score -- of equal scores the most recent token, which is
 * the token ahakv_select drops when it keeps the lowest indices among ties -- is declared free: pos = -1 there and
 * free_slot[b,h] = its index.  The result is the cache ahakv_score_step + ahakv_select + ahakv_compact_inplace
 * leave, up to the order of the rows.
 * p->n_ctx must be budget + 1 and p->obs_window 1; the limits of ahakv_score_step apply (AHAKV_ERR_UNSUPPORTED
 * otherwise).  k, v: [B,Hkv,budget+1,d] with the strides of p.  A free_slot entry outside [0, budget] leaves that
 * head untouched; a position table in which no slot lies outside the recent window sets free_slot[b,h] = -1.  To
 * start from a cache of budget rows in order: slots 0 .. budget-1 with pos = their positions, free_slot = budget. */
ahakv_status ahakv_step_slots(const ahakv_params* p, const void* q_t, const void* k_t, const void* v_t, void* k, void* v,
                              float* score, int32_t* pos, int32_t* free_slot, ahakv_stream_t stream);

/* Row entropy of the scaled softmax (Section 4.2, Eq. 6): H_i = - sum_j a_ij ln a_ij (natural log) for every
 * observation row of every query head, with a_ij exactly as in ahakv_score (mask, lambda from scale_mode).  A
 * diagnostic: Eq. 10 predicts E[H_i] = ln i - lambda^2 d / 2, and Eq. 12 picks lambda so that this is ln(budget).
 * entropy: [B,Hq,r] float32 out.  ws: ahakv_entropy_workspace_bytes(p) bytes, 256-byte aligned (not the scoring
 * workspace).  Runs on the FP32 pipes (double for float32 inputs); it is not part of the eviction path. */
size_t ahakv_entropy_workspace_bytes(const ahakv_params* p);
ahakv_status ahakv_row_entropy(const ahakv_params* p, const void* q_obs, const void* k, float* entropy, void* ws,
                               size_t ws_bytes, ahakv_stream_t stream);

/* Selection (Algorithm 1: S^r = recent B_r tokens, S^s = TopK(F, B_s), S = S^s U S^r).
 * Keeps rows [n - B_r, n) and the B_s = budget - B_r highest-scoring rows of [0, n - B_r);
 * equal scores are taken lowest index first; the result is ascending.  n <= budget keeps all rows.
 * score: [B,Hkv,n] float32 in.  kept_idx: [B,Hkv,n_keep] int32 out.  ws and ws_bytes are not used (selection
 * works in shared memory) and may be NULL and 0. */
ahakv_status ahakv_select(const ahakv_params* p, const float* score, int32_t* kept_idx, void* ws,
                          size_t ws_bytes, ahakv_stream_t stream);

/* Compaction (Algorithm 1, Generation: K <- K_S, V <- V_S): row t of the outputs is a byte copy of
 * row kept_idx[t] of the inputs.  score / score_out are nullable together and gather the score the
 * same way, so that it can be carried into the next round.  Indices outside [0, n) are an error
 * the caller must not make: they are not checked on the device. */
ahakv_status ahakv_compact(const ahakv_params* p, const void* k, const void* v, const float* score,
                           const int32_t* kept_idx, void* k_out, void* v_out, float* score_out,
                           ahakv_stream_t stream);

/* The whole step for one layer: score, select, compact, queued back to back on `stream` with no host
 * synchronisation in between.  score_prev and score_out are nullable; kept_idx is required. */
ahakv_status ahakv_evict(const ahakv_params* p, const void* q_obs, const void* k, const void* v,
                         const float* score_prev, void* k_out, void* v_out, float* score_out,
                         int32_t* kept_idx, void* ws, size_t ws_bytes, ahakv_stream_t stream);

/* ahakv_evict with a budget of its own for every (sequence, KV head) (Algorithm 1 runs per head; the paper gives
 * every head the same budget, allocators that do not can say so here).  head_budget: [B,Hkv] int32 in device
 * memory, read by the selection kernel; an entry is held to [max(recent_window, 1), p->budget].  Head (b, h) keeps
 * its recent window and the best head_budget[b,h] - recent_window of the rest.  Outputs keep the strides of
 * ahakv_evict (n_keep = min(n_ctx, p->budget) rows a head): a head that keeps fewer fills kept_idx[b,h,t] with -1 from
 * its own count on, and the rows of k_out, v_out and score_out from there on are left as they were.  The scores are
 * those of ahakv_evict: in particular the scale of Eq. 12 is the call's, from p->budget, not one per head.  Tie
 * rule and errors are ahakv_evict's too. */
ahakv_status ahakv_evict_head_budgets(const ahakv_params* p, const int32_t* head_budget, const void* q_obs,
                                      const void* k, const void* v, const float* score_prev, void* k_out, void* v_out,
                                      float* score_out, int32_t* kept_idx, void* ws, size_t ws_bytes,
                                      ahakv_stream_t stream);

/* The whole step for a batch whose sequences differ in length, position and budget (a serving batch).  `p`
 * describes the allocation: p->n_ctx is the token extent of k, v and score_prev (the longest sequence's room),
 * p->budget the largest budget; everything else holds for all sequences.  seqs: HOST array of p->batch entries;
 * sequence b has seqs[b].n_ctx cached rows (obs_window <= n_ctx <= p->n_ctx), has seen seqs[b].n_total tokens and
 * keeps seqs[b].budget rows (recent_window <= budget <= p->budget).  The heads of one sequence share its budget.
 * Layouts: q_obs, k, v as described by p (default [B,Hq,r,d] and [B,Hkv,p->n_ctx,d]; rows past a sequence's n_ctx
 * are not read).  Arrays indexed by token or by kept row are dense per sequence inside the sequence's slot of the
 * full-size array: score_prev for sequence b starts at b * Hkv * p->n_ctx floats and is [Hkv, n_ctx_b] from there;
 * k_out, v_out, score_out and kept_idx start at b * Hkv * keep_max rows (keep_max = min(p->n_ctx, p->budget)) and
 * are [Hkv, min(n_ctx_b, budget_b), ...] from there.  The sequences are queued one after the other on `stream`
 * with the kernels of ahakv_evict, sharing `ws` (sized for p); each gets exactly what ahakv_evict would give it
 * alone.  Nothing is queued if any entry is invalid. */
typedef struct {
  int32_t n_ctx;
  int32_t budget;
  int64_t n_total;
} ahakv_seq;
ahakv_status ahakv_evict_ragged(const ahakv_params* p, const ahakv_seq* seqs, const void* q_obs, const void* k,
                                const void* v, const float* score_prev, void* k_out, void* v_out, float* score_out,
                                int32_t* kept_idx, void* ws, size_t ws_bytes, ahakv_stream_t stream);

/* Reads the status word the kernels of the last call on this workspace left in `ws` (synchronises
 * `stream`).  AHAKV_OK, or AHAKV_ERR_TIMEOUT if a bounded device-side wait gave up, in which case
 * the call's outputs are not valid. */
ahakv_status ahakv_last_device_status(const void* ws, ahakv_stream_t stream);

/* Stage timing, for measurement only (no counterpart in the paper).  While enabled, ahakv_score and
 * ahakv_evict record CUDA events on the caller's stream around each stage: 0 the scoring kernels
 * (logits, SG-softmax, column sums), 1 the |V|^2 stream, 2 the value-prior refinement, 3 selection,
 * 4 compaction.  ahakv_profile_enable(1) creates the events (the only allocation the library ever
 * makes) and clears the totals; ahakv_profile_enable(0) destroys them.  ahakv_profile_read
 * synchronises the device, adds up the milliseconds per stage over the calls made since the last
 * read (at most AHAKV_PROFILE_MAX_CALLS are kept; older ones are dropped), writes them to
 * ms[AHAKV_N_STAGES] and returns the number of calls covered, or -1 when profiling is off. */
enum { AHAKV_N_STAGES = 5, AHAKV_PROFILE_MAX_CALLS = 256 };
ahakv_status ahakv_profile_enable(int on);
int64_t ahakv_profile_read(double* ms);
const char* ahakv_stage_name(int stage);

/* The eviction score for callers that cannot provide scratch memory (this entry point has no
 * counterpart in the paper; it exists for deployment).  Some users of this library cannot allocate
 * device memory where they call it: an inference server whose memory pool was sized at start-up and
 * hands out nothing afterwards, an extension that receives tensors but no allocator, a caller that must
 * not touch cudaMalloc because it synchronises the device and can fail under memory pressure.  For them
 * the library carries its own scratch: a device array of AHAKV_STATIC_WS_BYTES that every GPU holds from
 * the time the library is loaded until the process ends.
 *
 * Computes exactly what ahakv_score computes, with the same kernels; the caller passes inputs and
 * outputs only.  Nothing is allocated or freed, by this call or by anything it calls.
 *  - Limit: ahakv_workspace_bytes(p) must not exceed AHAKV_STATIC_WS_BYTES (ahakv_static_workspace_bytes()
 *    returns it at run time); larger problems get AHAKV_ERR_WORKSPACE and nothing is launched.  8 MiB
 *    covers, for instance, one sequence of 8 KV heads x 16384 tokens (3.5 MiB), 32 heads x 4096 tokens
 *    (2 MiB) or a 16-sequence decode round of 8 KV heads x 2080 tokens (5.3 MiB); 32 heads x 16384
 *    tokens (8.02 MiB) is just over.
 *  - The first call on each device looks up the array's device address (the device must be current, as
 *    for every other call); make that first call before you start capturing a stream.
 *  - All calls on a device share the one array, which keeps whatever the last call left in it.  The call
 *    resets what has to start clean, so calls in sequence are independent; two calls that overlap on the
 *    GPU (different streams) race on the array and must be serialised by the caller.
 *  - ahakv_static_last_device_status(stream) is ahakv_last_device_status for this scratch (it synchronises
 *    `stream`): after a device-side timeout the output is undefined, exactly as in ahakv_score.
 * Parameters are judged exactly as ahakv_score judges them (same status codes). */
#define AHAKV_STATIC_WS_BYTES (8u << 20)
size_t ahakv_static_workspace_bytes(void);
ahakv_status ahakv_static_last_device_status(ahakv_stream_t stream);
ahakv_status ahakv_score_static(const ahakv_params* p, const void* q_obs, const void* k, const void* v,
                                const float* score_prev, float* score, ahakv_stream_t stream);

/* For tests of the failure path only (no counterpart in the paper).  Every wait inside the tensor-core scoring
 * kernel on something another thread, the copy engine, the tensor core or another CTA must deliver is bounded
 * (1 s); when one runs out the kernel records AHAKV_ERR_TIMEOUT in the workspace's status word and winds down
 * without trapping, so the context stays usable.  wait_ms > 0 shortens that limit for the launches that follow
 * (0 restores 1 s); withhold_first_partial != 0 plants the fault that makes a wait run out: the softmax
 * statistics of the first run of the first row block are never published, so whoever merges that row block waits
 * in vain.  While either is set, launches use a second instantiation of the same kernel code that takes the limit
 * and the fault from its arguments; the instantiation every other call runs has neither.  Process-wide; not for
 * production use. */
void ahakv_test_set_wait(int32_t wait_ms, int32_t withhold_first_partial);

/* Number of kernels the library has launched in this process since it was loaded. */
int64_t ahakv_launch_count(void);

const char* ahakv_status_string(ahakv_status s);

#ifdef __cplusplus
}
#endif
#endif /* AHAKV_H_ */
