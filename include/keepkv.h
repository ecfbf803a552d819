/*
 * keepkv.h -- C ABI of the KeepKV hot path for NVIDIA B200 (sm_100a).
 *
 * KeepKV (arXiv 2504.09936) keeps a KV cache within a fixed budget by merging the
 * entries it would otherwise evict into their most similar retained entries, in a
 * way that leaves the current attention output unchanged (Theorem 2).  This
 * library implements the three operations of its decode loop for one attention
 * layer:
 *
 *   keepkv_append            K_t = [K_{t-1}, k_t], V_t = [V_{t-1}, v_t]          (Eq. 2)
 *   keepkv_decode_attention  o = sum p_i s_i v_i / sum p_i s_i                   (Eq. 6)
 *                            and the running score estimate of every entry       (Eq. 8)
 *   keepkv_compress          Algorithm 1: select retained / evicted sets, match
 *                            each evicted key to its most cosine-similar retained
 *                            key, merge with the ZIP equations (Eq. 7, Eq. A.3).
 *
 * Conventions
 *  - Every pointer is DEVICE memory owned by the caller unless its name ends in
 *    `_host`.  The library allocates nothing, holds no state between calls
 *    (one exception: the built-in scratch array of keepkv_decode_attention_static)
 *    and never synchronises: each call validates its arguments on the host, enqueues
 *    kernels on `stream` (a cudaStream_t passed as void*) and returns at once.
 *  - Return value: KEEPKV_OK or a negative keepkv_status.  Nothing is enqueued
 *    when a negative value is returned, except for KEEPKV_ERR_CUDA (a launch
 *    failed part-way; keepkv_last_cuda_error() gives the cudaError_t).
 *  - Problems only the device can see (append into a full cache) are reported by
 *    OR-ing a KEEPKV_DEV_* bit into *status_dev, an int32 the caller zeroes and
 *    reads back when it likes; the offending work item is skipped, never faulted.
 *  - Layouts are dense row-major with the last index fastest.  bf16 is the
 *    storage type of keys, values, queries and outputs; all accumulation is fp32.
 *  - A "unit" is one (sequence b, kv head h) pair, u = b * H_kv + h.  Query head
 *    g of unit u is head h * G + g, G = H_q / H_kv.
 */
#ifndef KEEPKV_H_
#define KEEPKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum keepkv_status {
  KEEPKV_OK = 0,
  KEEPKV_ERR_INVALID_ARG = -1,     /* null pointer, non-positive size, misaligned pointer      */
  KEEPKV_ERR_UNSUPPORTED = -2,     /* d not in {64,128}, G not in {1,2,4,8}, N_cap % 64 != 0 ...  */
  KEEPKV_ERR_CAPACITY = -3,        /* budget + period exceeds N_cap, budget > N_cap             */
  KEEPKV_ERR_WORKSPACE = -4,       /* workspace smaller than keepkv_workspace_bytes             */
  KEEPKV_ERR_CUDA = -5             /* a CUDA runtime/driver call failed                         */
} keepkv_status;

/* bits OR-ed into *status_dev by kernels */
#define KEEPKV_DEV_APPEND_FULL 1   /* keepkv_append: seq_len == N_cap, the token was dropped    */
#define KEEPKV_DEV_TIMEOUT 2       /* a bounded wait inside a kernel ran out                    */
#define KEEPKV_DEV_NOT_STEADY 4    /* keepkv_compress with KEEPKV_FLAG_COMPRESS_STEADY met a unit  */
                                   /* outside the steady-state limits; it was left untouched     */

#define KEEPKV_DEV_POSITIONS 8     /* keepkv_compress_inplace: a unit's position array does not hold its n_sink first */
                                   /* and n_recent last tokens; its result is unspecified                         */

typedef struct keepkv_params {
  int32_t B;                /* sequences                                                       */
  int32_t H_q;              /* query heads                                                     */
  int32_t H_kv;             /* kv heads; G = H_q / H_kv in {1,2,4,8}                           */
  int32_t d;                /* head dimension, 64 or 128                                       */
  int32_t N_cap;            /* allocated entries per unit (stride of the entry axis), % 64 == 0 */
  int32_t period;           /* compression period P, used only to check N_cap >= budget + P    */
  int32_t n_sink;           /* entries always kept at the front (App. B.3: 4)                  */
  int32_t n_recent;         /* entries always kept at the back  (App. B.3: recent window)      */
  float sm_scale;           /* 1/sqrt(d) of Eq. 3                                              */
  float ema_alpha;          /* alpha of Eq. 8, in [0,1); 0 makes the estimate the last score   */
  float merge_threshold;    /* T of Algorithm 1 (paper: 0.8); -INFINITY merges always, +INFINITY never (evict only) */
  float gamma_min;          /* a group is merged only if gamma_min < gamma <= gamma_max, gamma */
  float gamma_max;          /* the key rescale factor of Eq. A.3; (-INF, +INF) = paper as is   */
  int32_t flags;            /* KEEPKV_FLAG_* bits, normally 0                                  */
  int32_t reserved[2];      /* must be zero                                                    */
} keepkv_params;

/* keepkv_compress for a cache in its steady state: the caller promises that every unit evicts at most 128
 * entries and has at most 2048 entries between the sinks and the recent window (a serving loop that
 * compresses every P <= 128 steps back to a fixed budget knows this).  One kernel then does the whole
 * compression instead of the general pipeline's five, with the same bits as result.  A unit that breaks the
 * promise is left untouched (its dst rows, dst.seq_len and outputs are unspecified) and
 * KEEPKV_DEV_NOT_STEADY is raised in *status_dev.  Needs budget > 0. */
#define KEEPKV_FLAG_COMPRESS_STEADY 1

/* keepkv_decode_attention, keepkv_decode_step and their host and static variants: the caller promises that the
 * kernel which precedes this call on the stream (of this library or not) writes none of the arrays of `cache`
 * (K, V, votes, lscore, seq_len) -- a model that calls once per layer, each layer with its own cache, knows this.
 * The launch then reads the lengths and requests its first key / value tiles while that kernel is still
 * finishing (programmatic dependent launch); the queries, the token to append, the workspace and every write wait
 * for it as always, so results are bit-identical.  If the promise is broken (e.g. two consecutive calls on one
 * cache) the call may attend to stale lengths, rows or scores; nothing faults.  Ignored by every other call. */
#define KEEPKV_FLAG_CACHE_IDLE 2

/* One layer's cache.  Rows [seq_len[b], N_cap) of a unit are unspecified. */
typedef struct keepkv_cache {
  void *K;                  /* bf16 [B, H_kv, N_cap, d]  keys k_i              (16-byte aligned) */
  void *V;                  /* bf16 [B, H_kv, N_cap, d]  values v_i            (16-byte aligned) */
  float *votes;             /* fp32 [B, H_kv, N_cap]     Electoral Votes p_i, 1 for a fresh entry */
  float *lscore;            /* fp32 [B, H_kv, N_cap]     ln of the EMA score estimate (Eq. 8);  */
                            /*                           -INFINITY = never scored               */
  int32_t *seq_len;         /* i32  [B]                  valid entries, shared by the kv heads  */
} keepkv_cache;

/* Per-unit counters written by keepkv_compress, [B * H_kv] of them. */
typedef struct keepkv_stats {
  int32_t n_retained;       /* entries kept (= new seq_len)                                    */
  int32_t n_evicted;        /* entries not kept                                                */
  int32_t n_merged;         /* evicted entries folded into a retained one                      */
  int32_t n_below_T;        /* evicted entries whose best cosine did not exceed T              */
  int32_t n_guard_groups;   /* groups rejected by the gamma guard (their members are dropped)  */
  int32_t n_groups;         /* retained entries that had at least one candidate member         */
  int32_t max_group;        /* largest number of members merged into one entry                 */
  int32_t reserved;
} keepkv_stats;

/* Bytes of scratch the calls below need for this shape (a function of B, H_q, H_kv, d, N_cap
 * only).  The same workspace serves decode and compress; calls that share one must not overlap
 * in time.  It must be 256-byte aligned and set up once with keepkv_workspace_init. */
int keepkv_workspace_bytes(const keepkv_params *p, size_t *bytes);

/* Zeroes the arrival counters kept in the workspace (they return to zero after every call). */
int keepkv_workspace_init(const keepkv_params *p, void *ws, size_t ws_bytes, void *stream);

/* Eq. 2.  For every sequence b and kv head h, writes k_new[b,h,:], v_new[b,h,:] (bf16 [B,H_kv,d])
 * to row seq_len[b], sets that entry's votes to 1 (Section 3.3.1: p initialised to 1) and its
 * lscore to -INFINITY, then increments seq_len[b].  A sequence already at N_cap (or whose
 * seq_len[b] is negative) is left unchanged and KEEPKV_DEV_APPEND_FULL is raised in *status_dev. */
int keepkv_append(const keepkv_params *p, const keepkv_cache *cache, const void *k_new, const void *v_new,
                  int32_t *status_dev, void *stream);

/* Eq. 6 (Electoral-Votes attention; Eq. 3 when all votes are 1).  For each query head,
 *   l_i = sm_scale * q . k_i,   o = sum_i p_i e^{l_i} v_i / sum_i p_i e^{l_i},  i < seq_len[b].
 * q, out: bf16 [B, H_q, d].  lse_or_null: fp32 [B, H_q], ln sum_i p_i e^{l_i} (-INF for an empty
 * sequence, whose output is 0).
 * update_scores != 0 also advances Eq. 8 for every entry read: the kv head's score at this step
 * is the mean over its G query heads of e^{l_i}; lscore <- ln(alpha e^{lscore} + (1-alpha) score),
 * or ln(score) for an entry never scored before or when alpha = 0: the first observed score
 * initialises the state, which equals Eq. 8's bias correction S/(1 - alpha^n) counted from the entry's
 * first observation at n = 1 only (from n = 2 on the plain recursion is used, not the corrected form).
 * This is the "attention scores s^t" input of Algorithm 1, produced without materialising them. */
int keepkv_decode_attention(const keepkv_params *p, const keepkv_cache *cache, const void *q, void *out,
                            float *lse_or_null, int update_scores, void *ws, size_t ws_bytes, int32_t *status_dev,
                            void *stream);

/* One decode step on device buffers in ONE launch: keepkv_append of (k_new, v_new) followed by
 * keepkv_decode_attention of q, with exactly their results (the attention sees the fresh entry; with
 * update_scores its score estimate becomes its first observation; lengths grow by one; a sequence already
 * at N_cap keeps its entries, attends to them only, and raises KEEPKV_DEV_APPEND_FULL).  Arguments as for
 * those two calls. */
int keepkv_decode_step(const keepkv_params *p, const keepkv_cache *cache, const void *q, const void *k_new,
                       const void *v_new, void *out, float *lse_or_null, int update_scores, void *ws, size_t ws_bytes,
                       int32_t *status_dev, void *stream);

/* Eq. 8, first case: the score estimate at the end of prefill, from the last W prompt queries
 * (W = w + 1 <= 32).  q_window: bf16 [B, H_q, W, d], oldest query first; query k sits at position
 * seq_len[b] - W + k and, the prompt being causal, scores only the entries at or before it.  For every entry
 * i < seq_len[b] of every kv head
 *   lscore_i <- ln( sum_k alpha^(W-1-k) s_i^k / sum_k alpha^(W-1-k) ),   k over the window queries that see i,
 * with s_i^k the mean over the head's G query heads of exp(sm_scale q_k . k_i); alpha = 0 keeps the last query
 * only.  The division by the accumulated weight is the bias correction of Eq. 8 (1 - alpha^(w+1) for an entry
 * older than the window).  Whatever lscore held before is overwritten; K, V, votes are only read. */
int keepkv_prefill_scores(const keepkv_params *p, const keepkv_cache *cache, const void *q_window, int32_t W,
                          int32_t *status_dev, void *stream);

/* Algorithm 1, out of place: reads `src` (unchanged), writes `dst` (distinct buffers of the same
 * shape).  Per unit, with len = src.seq_len[b] and budget b_b (budget_dev[b] if given, else
 * budget_scalar; likewise n_recent_dev[b] / p->n_recent):
 *   1. key kappa_i = fp32(ln p_i + lscore_i); retained set = first n_sink, last n_recent and the
 *      largest kappa among the rest, equal keys -> lower index; everything else is evicted
 *      (Algorithm 1, selection step; App. B.3).  If the budget is below n_sink + n_recent the recent
 *      window shrinks first.  len <= budget: plain ordered copy.
 *   2. each evicted key takes the retained key of highest cosine similarity as its target,
 *      equal values -> lower slot, and is merged only if that cosine exceeds merge_threshold
 *      (Algorithm 1, similarity and arg-max steps).  The cosine is the fp32 value dot/(sqrtf(n_e)*sqrtf(n_c)) with dot and the
 *      squared norms accumulated by fused multiply-add from 0 over channels 0..d-1.
 *   3. every retained entry with members is rewritten by Eq. A.3 using exp(lscore) as score
 *      estimate: v_r, k_r, p_r = sum of votes, lscore_r = ln(sum p s / sum p) (Algorithm 1, merge step).
 *   4. dst holds the retained entries in ascending source order, dst.seq_len[b] = min(len, b_b).
 * Optional outputs: retained_idx_or_null i32 [B, H_kv, N_cap] (first seq_len entries valid: source
 * index of each dst row); target_or_null i32 [B, H_kv, N_cap] (per source entry: dst slot it was
 * merged into, -1 dropped, -2 retained); stats_or_null [B * H_kv]. */
int keepkv_compress(const keepkv_params *p, const keepkv_cache *src, const keepkv_cache *dst,
                    const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                    int32_t *retained_idx_or_null, int32_t *target_or_null, keepkv_stats *stats_or_null, void *ws,
                    size_t ws_bytes, int32_t *status_dev, void *stream);

/* keepkv_compress with the selection of step 1 driven by the caller's own importance scores (Section 3.4: the
 * method puts no constraint on the token selection, the retained and evicted sets only designate the merging
 * pairs; Section 4.5 combines it with H2O's accumulated attention and PyramidInfer's selection).
 * select_score_or_null: fp32 [B, H_kv, N_cap], larger = more important, must not be NaN; it replaces kappa
 * among the entries between the sinks and the recent window (equal scores -> lower index); votes and lscore
 * still drive the merge of step 3.  NULL makes this keepkv_compress.  Everything else as there. */
int keepkv_compress_scored(const keepkv_params *p, const keepkv_cache *src, const keepkv_cache *dst,
                           const float *select_score_or_null, const int32_t *budget_dev, int32_t budget_scalar,
                           const int32_t *n_recent_dev, int32_t *retained_idx_or_null, int32_t *target_or_null,
                           keepkv_stats *stats_or_null, void *ws, size_t ws_bytes, int32_t *status_dev, void *stream);

/* Algorithm 1 in place, for the periodic mode of Section 1 and any loop that compresses every few steps: "discard
 * (k_e, v_e), (k_c, v_c) and insert (k_r, v_r)" taken literally.  Retained entries stay in their rows, a merged entry
 * overwrites its target's row, and only the retained rows at or beyond the new length move, into the rows of evicted
 * entries below it: a steady-state compression touches O(evicted + merged) rows instead of rewriting the cache.  The
 * price is that the cache is no longer in token order, so the caller keeps three more arrays with it:
 *   pos      i32 [B, H_kv, N_cap]  token position of every row (valid for rows below pos_len[b])
 *   pos_len  i32 [B]               rows whose position is recorded; rows [pos_len[b], seq_len[b]) are the tokens
 *                                  appended since (keepkv_append / keepkv_decode_step), in order
 *   n_seen   i32 [B]               tokens of the sequence that have a recorded position
 * The call first gives the appended rows the positions n_seen[b], n_seen[b] + 1, ...; on return pos_len[b] =
 * seq_len[b] = the new length and n_seen[b] counts them.  To start after keepkv_compress (whose dst is in token
 * order): pos = its retained_idx output, pos_len = its new length, n_seen = the prompt length.
 * Per unit, with len = seq_len[b] and the budget as in keepkv_compress:
 *   1. retained set: the n_sink smallest and the n_recent largest positions, and the largest kappa among the other
 *      rows, equal keys -> lower ROW; (the first n_sink and last n_recent tokens must all be present, which holds as
 *      long as the windows are not enlarged between calls: otherwise KEEPKV_DEV_POSITIONS is raised)
 *   2. every evicted row takes the retained row of highest cosine similarity, equal values -> lower ROW, and is
 *      merged iff that cosine exceeds merge_threshold (the cosine of keepkv_compress);
 *   3. every target with members is rewritten in its row by Eq. A.3, guard as in keepkv_compress;
 *   4. with n = min(len, budget): the retained rows at or above n, in ascending order, move into the evicted rows
 *      below n, in ascending order (K, V, votes, lscore, pos); seq_len[b] = n.
 * On a cache in token order without equal keys or cosines the surviving entries are those of keepkv_compress.
 * Optional outputs: moved_from_or_null i32 [B, H_kv, N_cap] (the row each final row came from), target_or_null
 * i32 [B, H_kv, N_cap] (per row before step 4: row of its target, -1 dropped, -2 retained), stats_or_null. */
int keepkv_compress_inplace(const keepkv_params *p, const keepkv_cache *cache, int32_t *pos, int32_t *pos_len,
                            int32_t *n_seen, const int32_t *budget_dev, int32_t budget_scalar,
                            const int32_t *n_recent_dev, int32_t *moved_from_or_null, int32_t *target_or_null,
                            keepkv_stats *stats_or_null, void *ws, size_t ws_bytes, int32_t *status_dev, void *stream);

/* Prefill compression with the merge policy of Section 3.4 (App. B, Table 3): "merge first, then evict".  Before any
 * eviction, entries of the prompt whose keys are similar enough are merged with each other; the eviction strategy
 * (the selection of keepkv_compress, without any further merging) is applied to the result.
 * `cache` holds the prompt on entry and the compressed cache on return; `scratch` is a second buffer of the same
 * shape (a serving loop's ping-pong partner) whose contents are destroyed.  Per unit, with len = cache.seq_len[b]:
 *   1. every entry e takes its most cosine-similar OTHER entry c(e) (the fixed fp32 cosine of keepkv_compress, equal
 *      values -> lower index);
 *   2. e is merged into c(e) iff that cosine exceeds merge_threshold, c(e) lies before e in the cache, and c(e) is
 *      not itself merged into an earlier entry (the earlier of two entries is the target; no entry is both target
 *      and member; the paper states the policy, not the pairing rule: this is the library's reading);
 *   3. every target is rewritten by Eq. A.3 over its members (votes add up), with the gamma guard of
 *      keepkv_compress: a group the guard rejects loses its members and the target stays as it was;
 *   4. the entries that were not merged away, in source order, form the merged prompt; it is cut to the budget by
 *      step 1 of keepkv_compress (sinks, recent window, largest kappa; kappa from the merged votes and scores),
 *      the evicted entries are dropped.  Because the heads of a sequence share seq_len, the budget of a sequence is
 *      capped by the length of its shortest merged head: cache.seq_len[b] = min(budget_b, min over heads).
 * Optional outputs: retained_idx_or_null i32 [B, H_kv, N_cap] (source index, in the prompt, of each row of the
 * result); stats_or_null [B * H_kv] (n_retained = new length, n_evicted = len - n_retained, n_merged / n_groups /
 * n_guard_groups / max_group of the merge pass, n_below_T = 0).  The similarity search compares all pairs of a
 * unit's entries: 2 len^2 d flop per unit, on the tensor cores. */
int keepkv_compress_merge_first(const keepkv_params *p, const keepkv_cache *cache, const keepkv_cache *scratch,
                                const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                                int32_t *retained_idx_or_null, keepkv_stats *stats_or_null, void *ws, size_t ws_bytes,
                                int32_t *status_dev, void *stream);

/* One decode step driven from HOST memory (the call a serving loop makes): copies q_host,
 * k_new_host, v_new_host (pinned or pageable host memory, shapes as above) into the device
 * staging buffers q_dev/k_new_dev/v_new_dev, runs keepkv_decode_step
 * (update_scores as given) and copies the result from out_dev into out_host, all enqueued on
 * `stream`; the caller synchronises the stream before reading out_host. */
int keepkv_decode_step_host(const keepkv_params *p, const keepkv_cache *cache, const void *q_host,
                            const void *k_new_host, const void *v_new_host, void *out_host, void *q_dev,
                            void *k_new_dev, void *v_new_dev, void *out_dev, int update_scores, void *ws,
                            size_t ws_bytes, int32_t *status_dev, void *stream);

/* The same step for n_layers independent layer caches of one shape in one call: the host arrays carry the
 * layers back to back (q_host, out_host: bf16 [n_layers, B, H_q, d]; k_new_host, v_new_host: bf16
 * [n_layers, B, H_kv, d]; the device staging buffers have the same shapes), and are moved with one copy
 * each per call instead of one per layer -- with a single copy for all three inputs when k_new_host starts where
 * q_host ends and v_new_host where k_new_host ends, and the three staging buffers lie the same way.
 * caches_host: host array of n_layers keepkv_cache structs. */
int keepkv_decode_step_host_layers(const keepkv_params *p, const keepkv_cache *caches_host, int32_t n_layers,
                                   const void *q_host, const void *k_new_host, const void *v_new_host, void *out_host,
                                   void *q_dev, void *k_new_dev, void *v_new_dev, void *out_dev, int update_scores,
                                   void *ws, size_t ws_bytes, int32_t *status_dev, void *stream);

/* The periodic mode of Section 1 keeps the complete KV cache outside the working memory and recompresses from it every
 * period.  These two calls keep that complete cache in HOST memory (K_host, V_host: bf16 [B, H_kv, N_cap, d],
 * seq_len_host: i32 [B], all host pointers; pinned memory makes the load asynchronous).
 * keepkv_complete_append_host is Eq. 2 on the host copy: the step's k_new_host / v_new_host (bf16 [B, H_kv, d]) go
 * to row seq_len_host[b] of every head and the lengths grow by one; a plain host memcpy, no stream involved;
 * KEEPKV_ERR_CAPACITY, with nothing written, if a sequence is full.
 * keepkv_complete_load_host brings the complete cache into a device cache of the same shape, enqueued on `stream`:
 * the first seq_len_host[b] rows of K and V of every unit (one pitched copy per sequence and array), the lengths, and
 * the state of a cache nobody has attended to yet (votes 1, lscore -INFINITY).  The host arrays must stay unchanged
 * until the stream has passed the copies.  What follows is the ordinary path: keepkv_decode_attention with
 * update_scores on the loaded cache scores it with the current query, keepkv_compress cuts it to the budget. */
int keepkv_complete_append_host(const keepkv_params *p, void *K_host, void *V_host, int32_t *seq_len_host,
                                const void *k_new_host, const void *v_new_host);
int keepkv_complete_load_host(const keepkv_params *p, const void *K_host, const void *V_host,
                              const int32_t *seq_len_host, const keepkv_cache *dev, void *stream);

/* No counterpart in the paper: the same operation as keepkv_decode_attention for callers that cannot
 * provide a workspace because they cannot allocate device memory where they call this (code running
 * inside another runtime's memory pool, a serving loop whose buffers were all fixed at start-up, a
 * deployment that forbids cudaMalloc after initialisation).  The split-KV scratch is a fixed array
 * of KEEPKV_STATIC_SCRATCH_BYTES inside the library image; every GPU that loads the library holds
 * it until the process exits.  The call allocates and frees nothing.
 *  - Arguments as keepkv_decode_attention, without ws / ws_bytes; inputs and outputs stay the caller's.
 *  - Shapes whose decode scratch exceeds the array are refused with KEEPKV_ERR_WORKSPACE before
 *    anything is enqueued.  The exact rule, with U = B*H_kv and align256(x) = x rounded up to a multiple
 *    of 256:  align256(4*(U+1)) + align256(1024*(16 + G*d)*4) <= KEEPKV_STATIC_SCRATCH_BYTES
 *    (G = 8, d = 128: the pool takes 4 259 840 bytes, which leaves room for 1 032 191 units).
 *  - Every call clears the 4*(U+1) bytes of arrival counters with a cudaMemsetAsync on `stream` before its
 *    kernel (3.6 MB at the largest admissible U; a few hundred bytes for ordinary batches).
 *  - The first call on each device looks up the array's device address; make that call outside any
 *    stream capture, with the device current that `stream` belongs to.
 *  - All calls on one GPU share the array and find in it whatever the previous call left: the call
 *    itself clears the counters it needs at zero, but two calls that overlap on the GPU (different
 *    streams, or different host threads without ordering) race on it.  Order them on one stream. */
#define KEEPKV_STATIC_SCRATCH_BYTES (8u << 20)
int keepkv_decode_attention_static(const keepkv_params *p, const keepkv_cache *cache, const void *q, void *out,
                                   float *lse_or_null, int update_scores, int32_t *status_dev, void *stream);

/* Test hook, not for production use: process-wide settings of the decode launches that follow (keepkv_decode_attention,
 * keepkv_decode_step, their host and static variants).  spin_limit > 0 replaces the number of polls after which a
 * bounded wait inside the kernel gives up (0 restores the default).  withhold_tile >= 0 makes every CTA announce
 * the tile at that position of its tile sequence without ever issuing its copies, so that the wait for it runs out with
 * nothing in flight: the call then returns normally, KEEPKV_DEV_TIMEOUT is raised in *status_dev and the outputs of
 * that call are unspecified; -1 restores normal operation.  This is how the kernels' timeout path is exercised
 * without faulting or hanging a GPU. */
int keepkv_debug_decode(int spin_limit, int withhold_tile);

/* Human-readable name of a keepkv_status. */
const char *keepkv_status_string(int status);

/* cudaError_t of the most recent KEEPKV_ERR_CUDA on this thread (0 if none). */
int keepkv_last_cuda_error(void);

/* Number of kernels the most recent successful call on this thread enqueued. */
int keepkv_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* KEEPKV_H_ */
