/*
 * lr_verify.h -- C ABI of the step-parallel verification pass of Lookahead
 * Reasoning on one B200 (sm_100a).
 *
 * One verify pass (Algorithm 1, the "in parallel do" block, with token-level
 * speculative decoding running inside every branch) is three device steps:
 *
 *   lr_verify_attention  nested-prefix paged GQA attention of every branch's
 *                        query tokens over  prefix (+) S_1..S_depth (+) own tail
 *   lr_accept_greedy     greedy token-level acceptance over vocab-wide logits
 *   lr_commit            step-level output construction on the paged KV cache
 *
 * Conventions
 *   - Plain C.  No exceptions, no aborts, no device traps.  Every function
 *     returns LR_OK (0) or a negative lr_status; lr_strerror() names it and
 *     lr_last_error() gives the detail message of the calling thread's last
 *     failing call.
 *   - Pointers ending in _h are HOST pointers, pointers ending in _d are DEVICE
 *     pointers on the context's device.  All buffers are owned by the caller;
 *     the library never frees or reallocates them.  The only device memory the
 *     library itself ever uses is inside the caller-provided workspace /
 *     scratch buffers; host-side it owns the opaque lr_ctx / lr_plan objects.
 *   - "stream" is a cudaStream_t passed as void*.  All device work is enqueued
 *     on it and no call synchronises unless its comment says so.
 *   - bf16 tensors are passed as raw pointers to 16-bit words.
 *   - There is no CPU fallback: without a usable sm_100 device every call fails.
 *   - Same inputs and same plan give bit-identical outputs.
 *
 * Data layout
 *   Q, O      [n_q_rows][n_q_heads][head_dim] bf16, rows packed by branch
 *             (branch b owns rows cu_q[b] .. cu_q[b+1]-1, in token order).
 *   K/V pool  [n_pool_pages][n_kv_heads][16][head_dim] bf16; a page holds 16
 *             tokens.  Every span (prefix, segment, tail) starts at token slot 0
 *             of its first page and owns whole pages; the unused slots of its
 *             last page may hold anything (NaN included) and never affect a
 *             result.  A physical page belongs to at most one span.
 *   logits    [n_rows][row_stride] bf16, first `vocab` entries of a row used;
 *             branch b with L_b drafts owns the L_b+1 rows starting at
 *             cu_draft[b] + b: row i scores draft i, row L_b gives the bonus.
 */
#ifndef LR_VERIFY_H_
#define LR_VERIFY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lr_status {
  LR_OK = 0,
  LR_EINVAL = -1,       /* bad argument: null pointer, inconsistent lengths, page id out of range ... */
  LR_EUNSUPPORTED = -2, /* shape or device outside what the kernels implement */
  LR_ECUDA = -3,        /* a CUDA runtime / driver call failed (text in lr_last_error) */
  LR_ETIMEOUT = -4,     /* a bounded device-side wait expired (reported by lr_poll_status) */
  LR_EBOUNDS = -5,      /* a device-side bounds check tripped (reported by lr_poll_status) */
  LR_ENOMEM = -6        /* caller-provided workspace too small / host allocation failed */
} lr_status;

typedef struct lr_ctx lr_ctx;   /* per (device, model geometry) */
typedef struct lr_plan lr_plan; /* per batch structure; reusable across passes and KV pools */

/* Model geometry.  Supported: head_dim 64 or 128, page_size 16,
 * n_q_heads a multiple of n_kv_heads with group size <= 16, vocab >= 1. */
typedef struct lr_model {
  int32_t n_q_heads, n_kv_heads, head_dim, page_size, vocab;
} lr_model;

/*
 * Integer description of one pass; every array is a HOST array of int32 that
 * only needs to live until lr_plan_create returns.
 *
 * Request r owns chain spans req_span_off[r] .. req_span_off[r+1]-1: the first
 * is the shared prefix x_{1:t} (length >= 0), the c-th after it is draft step
 * segment c (length >= 1), c = 1..gamma_r.  Span s holds span_len[s] tokens in
 * page slots span_slot[s] .. span_slot[s]+ceil(len/16)-1 of page_ids[].
 *
 * Branch b (branches of one request are contiguous, br_req non-decreasing)
 * sees the prefix and the first br_depth[b] segments of its request (that is
 * x'_j of Algorithm 1 with j = depth) plus, causally, its private tail of
 * br_own_len[b] tokens (slots from br_own_slot[b]); the LAST q_len_b =
 * cu_q[b+1]-cu_q[b] tail tokens are the queries.  br_n_draft[b] (<= own_len)
 * is L_b, the number of token-level drafts being verified for the branch.
 *
 * Multi-branch (tree) drafting (Section 3, "Multi-Branch Drafting"): with
 * seg_parent != NULL the draft steps of a request form a tree.  For span s of
 * request r, local index c = s - req_span_off[r] >= 1, seg_parent[s] is the
 * local index (0 = the prefix, else 1..c-1) of the step that segment c
 * continues; the entries at prefix spans are ignored.  br_depth[b] is then the
 * local index of the node branch b continues (0 = the prefix alone): the
 * branch sees the prefix and the segments on the way from the prefix to that
 * node, in that order.  The nested chain is the tree with seg_parent = c - 1,
 * and NULL means exactly that.  In tree mode no node may lie more than 8 steps
 * below the prefix (LR_EINVAL otherwise).
 */
typedef struct lr_batch {
  int32_t n_req, n_branch, n_span, n_page_slots;
  const int32_t *req_span_off; /* [n_req+1]   */
  const int32_t *span_len;     /* [n_span]    */
  const int32_t *span_slot;    /* [n_span]    */
  const int32_t *br_req;       /* [n_branch]  */
  const int32_t *br_depth;     /* [n_branch]  0..gamma_r */
  const int32_t *br_own_len;   /* [n_branch]  >= q_len   */
  const int32_t *br_own_slot;  /* [n_branch]  */
  const int32_t *br_n_draft;   /* [n_branch]  0..own_len */
  const int32_t *cu_q;         /* [n_branch+1] query-row offsets, q_len >= 1 */
  const int32_t *page_ids;     /* [n_page_slots] physical page numbers, distinct */
  int64_t n_pool_pages;        /* pages in each of the K and V pools */
  const int32_t *seg_parent;   /* [n_span] or NULL (nested chain); see above */
} lr_batch;

/* Host-only check of a batch description against the rules above (no device
 * needed): LR_OK, or LR_EINVAL with the first violated rule in lr_last_error(). */
int lr_validate_batch(const lr_model *model, const lr_batch *batch_h);

/* ---- context ------------------------------------------------------------ */

/* Creates a context on CUDA device `device` (must be compute capability 10.x).
 * Allocates only host memory.  LR_EUNSUPPORTED for geometry outside the list
 * above or a non-sm_100 device. */
int lr_create(lr_ctx **out, const lr_model *model, int device);
int lr_destroy(lr_ctx *ctx);

/* ---- plan --------------------------------------------------------------- */

/* Bytes of device workspace lr_plan_create needs for this batch (metadata
 * tables, the work list of the attention kernel, split-KV partial results and
 * a status word).  Validates the batch (LR_EINVAL with detail on failure). */
int lr_plan_bytes(const lr_ctx *ctx, const lr_batch *batch_h, size_t *bytes_out);

/* Validates the batch, builds the device-side tables and the attention work
 * partition on the host and enqueues their upload into workspace_d (256-byte
 * aligned, >= lr_plan_bytes) on `stream`.  The host staging copy lives in the
 * plan, so the call does not synchronise.  The plan may be used by any number
 * of later passes over any KV pools with >= batch_h->n_pool_pages pages, on
 * the same stream (or after the upload has completed).  Two passes that use
 * the same plan must not overlap on the device (they share the workspace). */
int lr_plan_create(lr_ctx *ctx, const lr_batch *batch_h, void *workspace_d, size_t workspace_bytes,
                   void *stream, lr_plan **out);
/* Releases the plan (not the workspace, which is the caller's).  The plan's pinned host buffer goes back to its
 * context for the next plan, so destroy every plan before its context.  Contexts and their plans are not
 * thread-safe: one thread at a time per context. */
int lr_plan_destroy(lr_plan *plan);

/* ---- the three steps ---------------------------------------------------- */

/*
 * Nested-prefix verify attention (Algorithm 1, parallel target step generation;
 * Background, "verifies these tokens in a single parallel forward pass").
 * For every branch b, query i, head h:
 *     O = softmax(scale * q K^T) V   over the keys of the prefix, of segments
 *     1..depth_b and of tail tokens 0 .. own_len_b - q_len_b + i   (inclusive),
 * with KV head h / (n_q_heads / n_kv_heads).  softmax_scale <= 0 selects
 * 1/sqrt(head_dim).  out_d: [n_q_rows][n_q_heads][head_dim] bf16.  lse_d
 * (nullable): [n_q_rows][n_q_heads] fp32, natural log of the sum of exp of the
 * scaled scores.  Accumulation and softmax are fp32.
 * Errors: LR_EINVAL (null / misaligned pointers: q, out, pools need 16-byte
 * alignment), LR_ECUDA (launch failure).  Device-side problems (a page id
 * beyond the pool, an expired wait) set the plan's status word; see
 * lr_poll_status.
 */
int lr_verify_attention(lr_plan *plan, const void *q_d, const void *k_pool_d, const void *v_pool_d,
                        void *out_d, float *lse_d, float softmax_scale, void *stream);

/* What lr_verify_attention will launch for this plan (host-side query, no device work).
 *   tensor_core_ok   1 when the shape allows the tcgen05 kernel (head_dim 128, tensor-map coordinates
 *                    within 32 bits, at most 254 branches per request, tails of at most 2047 pages)
 *   path             the current selection (0 automatic, 1 CUDA cores, 2 tensor cores)
 *   uses_tensor_core 1 when the next call would run the tcgen05 kernel
 *   n_cta            CTAs of the tcgen05 kernel (0 on the CUDA-core path)
 *   n_pieces         (CTA, request, KV head, query tiles) work items
 *   n_merge_targets  query tiles whose keys are split over several CTAs and need a merge
 *   n_partial_slots  fp32 partial results those CTAs write
 */
typedef struct lr_plan_info {
  int32_t tensor_core_ok, path, uses_tensor_core, n_cta, n_pieces, n_merge_targets, n_partial_slots;
} lr_plan_info;
int lr_plan_describe(const lr_plan *plan, lr_plan_info *info_out);

/* Selects the attention implementation for later lr_verify_attention calls on
 * this plan: 0 = automatic (tensor-core path when the shape allows it), 1 =
 * force the CUDA-core path (every shape), 2 = force the tensor-core path
 * (LR_EUNSUPPORTED later if the shape does not allow it).  For testing. */
int lr_plan_set_attention_path(lr_plan *plan, int path);

/* Test hook for the device-side bounds checks: overwrites the physical page id of page slot `page_slot`
 * (an index into lr_batch.page_ids) with new_id in every device table of the plan, by patching the plan's host
 * image and uploading it again on `stream`.  No validation of new_id: that is the point.  A kernel that meets
 * an id outside [0, n_pool_pages) reads page 0 in its place and raises LR_EBOUNDS in the status word
 * (lr_poll_status); it never dereferences the id. */
int lr_plan_debug_set_page(lr_plan *plan, int32_t page_slot, int32_t new_id, void *stream);

/* Test hook for the bounded device-side waits: every wait of the tensor-core attention kernels of later
 * lr_verify_attention calls on this plan gives up after `microseconds` (default: one second).  With a limit
 * shorter than a trip to memory a wait expires while its data is still on the way; the CTA then records
 * LR_ETIMEOUT in the status word, lets the copies and products it has in flight finish (bounded again), releases
 * its tensor memory and returns.  The output of such a pass is unspecified; the context stays usable. */
int lr_plan_debug_set_wait_limit(lr_plan *plan, uint32_t microseconds);

/* Test hook that makes one wait run out: the first CTA of the tensor-core attention kernels expects `bytes` more on
 * its first KV stage than its copies deliver, so the barrier of that stage never completes and the waits on it
 * expire after the limit above -- LR_ETIMEOUT through lr_poll_status, nothing worse: the CTA leaves through its
 * abort path, every other CTA finishes normally.  0 switches the hook off.  Set a short limit first. */
int lr_plan_debug_set_phantom_bytes(lr_plan *plan, uint32_t bytes);

/* Bytes of scratch lr_accept_greedy needs for n_rows logits rows.  The scratch
 * must be zero-filled before its first use; every call leaves it zero-filled. */
int lr_accept_scratch_bytes(int32_t n_rows, size_t *bytes_out);

/*
 * Greedy token-level acceptance (Background, "Speculative Decoding": drafts are
 * processed in order, the process halts at the first rejected one and a final
 * token comes from the target's distribution at that position).
 *     t_i    = argmax_v logits[row0_b + i][v]      (lowest index on ties, +0 == -0,
 *                                                   NaN ranks as -inf)
 *     n_b    = max{ n <= L_b : draft[cu_draft[b]+i] == t_i for all i < n }
 *     bonus_b = t_{n_b}
 * A draft id outside [0, vocab) never matches.  n_rows must equal
 * cu_draft[n_branch] + n_branch.  row_argmax_d (nullable) receives every t_i.
 * logits_d must be 16-byte aligned and row_stride_elems a multiple of 8.
 * Calls that share a scratch buffer must not overlap on the device.
 */
int lr_accept_greedy(lr_ctx *ctx, const void *logits_d, int64_t row_stride_elems,
                     const int32_t *draft_ids_d, const int32_t *cu_draft_d, int32_t n_branch, int32_t n_rows,
                     int32_t *n_accept_d, int32_t *bonus_id_d, int32_t *row_argmax_d,
                     void *scratch_d, void *stream);

/*
 * Stochastic token-level acceptance (Background, "Speculative Decoding": a
 * rejection-sampling procedure processes the proposed tokens in order; an
 * accepted token is kept, at the first rejection the process halts and a final
 * token is sampled from the target's distribution), for drafts whose draft
 * distribution is a point mass at the drafted token (prompt-lookup / n-gram
 * drafts, the paper's SD method).  With P_i = softmax(logits[row0_b + i] / T):
 *     draft i is accepted iff u_accept[cu_draft[b] + i] < P_i(d_i)   (= min(1, P/Q));
 *     n_b     = number of drafts accepted before the first rejection;
 *     final_b = inverse-CDF sample with u_final[b] (smallest v whose cumulative
 *               weight exceeds u * total) from P_{n_b} with the rejected token
 *               removed, or from P_{L_b} when every draft was accepted.
 * The uniforms (in [0, 1)) are inputs: the call draws no random numbers.  A draft
 * id outside [0, vocab) has probability 0.  Arithmetic is fp32; a decision whose
 * uniform lies within rounding of its threshold may differ from an exact
 * evaluation.  p_draft_d (nullable, [sum L_b]) receives P_i(d_i) for the drafts
 * up to and including the first rejected one.  Rows, strides and alignment as
 * for lr_accept_greedy; temperature must be > 0; at most 65535 rows per call.
 * scratch_d: lr_accept_sample_scratch_bytes bytes, 8-byte aligned, no initial
 * contents needed; calls sharing it must not overlap on the device.
 */
int lr_accept_sample_scratch_bytes(const lr_ctx *ctx, int32_t n_rows, size_t *bytes_out);
int lr_accept_sample(lr_ctx *ctx, const void *logits_d, int64_t row_stride_elems, const int32_t *draft_ids_d,
                     const int32_t *cu_draft_d, int32_t n_branch, int32_t n_rows, float temperature,
                     const float *u_accept_d, const float *u_final_d, int32_t *n_accept_d, int32_t *final_id_d,
                     float *p_draft_d, void *scratch_d, void *stream);

/*
 * lr_accept_sample with the sampling filters of Section 4, "Setup" (top-p 0.95,
 * and top-k 20 for one model family) applied to the target distribution first.
 * Rank the tokens of a row by P_i, largest first, equal values by index.
 *   top_k > 0: only the first top_k ranks stay, renormalised;
 *   top_p < 1: of those, rank r stays iff the renormalised mass of the ranks
 *              before it is below top_p (the first always stays); renormalised.
 * P'_i is the result (0 outside the kept set), and the rule of
 * lr_accept_sample runs on P'_i: draft i is accepted iff u_accept < P'_i(d_i),
 * the final token comes from P'_{n_b} with the rejected token removed, or from
 * P'_{L_b}.  top_k = 0 and top_p = 1 switch the respective filter off.
 * Masses are rounded to multiples of 2^-40 of the row's largest one and summed
 * as integers: results do not depend on summation order, and the final draw is
 * exact given those masses.  A row whose kept set changes when top_p moves by
 * a few parts in 10^6 may keep one token more or fewer than an exact
 * evaluation.  p_draft_d (nullable, [sum L_b]) receives P'_i(d_i) of every
 * draft; n_kept_d (nullable, [n_rows]) the size of every row's kept set.
 * Rows, strides and alignment as for lr_accept_greedy; temperature > 0,
 * top_k >= 0, 0 < top_p <= 1, else LR_EINVAL.  scratch_d:
 * lr_accept_sample_filtered_scratch_bytes bytes, 8-byte aligned, no initial
 * contents needed; calls sharing it must not overlap on the device.
 */
int lr_accept_sample_filtered_scratch_bytes(const lr_ctx *ctx, int32_t n_rows, size_t *bytes_out);
int lr_accept_sample_filtered(lr_ctx *ctx, const void *logits_d, int64_t row_stride_elems, const int32_t *draft_ids_d,
                              const int32_t *cu_draft_d, int32_t n_branch, int32_t n_rows, float temperature,
                              int32_t top_k, float top_p, const float *u_accept_d, const float *u_final_d,
                              int32_t *n_accept_d, int32_t *final_id_d, float *p_draft_d, int32_t *n_kept_d,
                              void *scratch_d, void *stream);

/*
 * lr_accept_greedy without a caller-provided scratch buffer.  (The paper has no
 * counterpart: this is a packaging variant of the call above, same results.)
 *
 * For callers that cannot obtain device memory at the point of the call: a
 * serving engine that handed every free byte of HBM to its KV cache at start-up,
 * or code running where cudaMalloc is off limits because it synchronises the
 * whole device and may fail late.  The row keys and the ticket counter live in
 * an array built into the library (8 * (LR_ACCEPT_STATIC_MAX_ROWS + 1) bytes on
 * every GPU that loads it, held until the process exits).  The call allocates
 * nothing, neither with cudaMalloc nor through any library.
 *
 *   - n_rows > LR_ACCEPT_STATIC_MAX_ROWS is rejected with LR_EINVAL.
 *   - The first call on a device looks up the array's device address (a
 *     cudaGetSymbolAddress call, made with ctx's device current); make that
 *     first call outside any stream capture, and from one thread only (the
 *     looked-up address is cached without a lock).
 *   - Every call makes ctx's device current for its own duration and puts the
 *     caller's current device back before it returns.
 *   - All calls on one device share the one array.  Each call clears the part
 *     it uses on `stream` before its kernel runs, so leftovers of an earlier
 *     call never matter, but two calls whose device work overlaps in time
 *     (different streams, no dependency between them) race on it.
 * Arguments, results and errors are otherwise those of lr_accept_greedy.
 */
#define LR_ACCEPT_STATIC_MAX_ROWS 4096
int lr_accept_greedy_static(lr_ctx *ctx, const void *logits_d, int64_t row_stride_elems,
                            const int32_t *draft_ids_d, const int32_t *cu_draft_d, int32_t n_branch, int32_t n_rows,
                            int32_t *n_accept_d, int32_t *bonus_id_d, int32_t *row_argmax_d, void *stream);

/*
 * Step-level commit (Algorithm 1, last two lines: j* = index of the first
 * rejected draft step, output = accepted draft steps followed by the decisive
 * target step).  verdict_d: uint8 [sum_r gamma_r], request r's verdicts at
 * req_span_off[r] - r.  Per request r:
 *     n_steps_accepted = j*;  survivor = lowest-numbered branch of depth j*
 *     (-1 if none);  kept_tail = own_len - L + n_accept of the survivor (0 if
 *     none);  committed_len = prefix + segments 1..j* + kept_tail.
 * keep list (CSR by request: keep_off [n_req+1], keep_pages / keep_valid sized
 * n_page_slots): prefix pages, pages of segments 1..j*, the first
 * ceil(kept_tail/16) tail pages of the survivor, each with its number of valid
 * tokens.  free list (free_off, free_pages): pages of segments j*+1..gamma,
 * then the branch tails in branch order (for the survivor only the pages past
 * the kept ones).  keep and free together list every page slot of the request
 * exactly once.  No KV data is moved.
 *
 * With a tree of draft steps (lr_batch.seg_parent; Section 3, "Multi-Branch
 * Drafting") verdict c - 1 of a request says whether segment c agrees with the
 * target step written after the node it continues.  Starting at the prefix the
 * commit moves to the lowest-numbered child whose verdict is set, until no
 * child agrees; n_steps_accepted is the number of moves, survivor the
 * lowest-numbered branch that continues the node reached, the kept segments
 * are those moved through (keep list in that order) and the free list holds
 * every other segment in index order, then the tails as above.
 *
 * At most LR_COMMIT_MAX_REQUESTS requests per pass: a plan of a larger batch is
 * accepted (attention and acceptance have no such limit) but lr_commit on it
 * returns LR_EUNSUPPORTED before anything is launched.
 */
#define LR_COMMIT_MAX_REQUESTS 4096
int lr_commit(lr_plan *plan, const uint8_t *verdict_d, const int32_t *n_accept_d,
              int32_t *n_steps_accepted_d, int32_t *survivor_d, int32_t *committed_len_d,
              int32_t *keep_off_d, int32_t *keep_pages_d, int32_t *keep_valid_d,
              int32_t *free_off_d, int32_t *free_pages_d, void *stream);

/*
 * Compaction of the committed KV (the step after the output construction of
 * Algorithm 1: the accepted draft steps and the decisive target step become the
 * shared context of the next cycle).  Input: the keep lists lr_commit wrote.
 * Token k of request r's committed sequence is moved, in place in the pools, to
 * slot k % 16 of the page keep_pages[keep_off[r] + k / 16].  Outputs per request:
 * new_len = its committed length; n_pages_kept = ceil(new_len / 16): that many
 * leading entries of its keep list now hold the sequence densely, the remaining
 * entries of its keep list are no longer needed by it.  Tokens in front of the
 * request's first partly filled kept page are not touched.  Bytes of the kept
 * pages beyond the sequence are unspecified afterwards; no other page is written.
 * scratch_d: lr_compact_scratch_bytes bytes, 256-byte aligned, no initial
 * contents needed.  Three launches on `stream`; a page id outside the pools sets
 * the plan's status word (LR_EBOUNDS) instead of being dereferenced.  The batch
 * must be the one the plan and the keep lists were made for.  At most
 * LR_COMPACT_MAX_REQUESTS requests per pass (LR_EUNSUPPORTED beyond, before
 * anything is launched or written).
 */
#define LR_COMPACT_MAX_REQUESTS 8192
int lr_compact_scratch_bytes(const lr_plan *plan, size_t *bytes_out);
int lr_compact(lr_plan *plan, const int32_t *keep_off_d, const int32_t *keep_pages_d, const int32_t *keep_valid_d,
               void *k_pool_d, void *v_pool_d, int32_t *new_len_d, int32_t *n_pages_kept_d, void *scratch_d, void *stream);

/* ---- whole pass with host buffers ---------------------------------------- */

/* Host-side inputs and outputs of one pass; every pointer is a HOST pointer
 * (pinned memory makes the copies asynchronous).  The KV pools stay on the
 * device: they are the engine's resident cache, not a per-pass input. */
typedef struct lr_pass_host_io {
  const void *q_h;            /* [n_q_rows][n_q_heads][head_dim] bf16 */
  const void *logits_h;       /* [n_rows][vocab] bf16, dense rows      */
  const int32_t *draft_ids_h; /* [sum L_b]                             */
  const uint8_t *verdict_h;   /* [sum gamma_r]                         */
  void *out_h;                /* [n_q_rows][n_q_heads][head_dim] bf16  */
  int32_t *n_accept_h, *bonus_id_h;                          /* [n_branch] */
  int32_t *n_steps_accepted_h, *survivor_h, *committed_len_h; /* [n_req]   */
  int32_t *keep_off_h, *free_off_h;                           /* [n_req+1] */
  int32_t *keep_pages_h, *keep_valid_h, *free_pages_h;        /* [n_page_slots] */
} lr_pass_host_io;

/* Bytes of device staging lr_verify_pass_host needs for this plan. */
int lr_pass_staging_bytes(const lr_plan *plan, size_t *bytes_out);

/* One whole pass from host buffers: copies Q, logits, draft ids and verdicts to
 * the device staging buffer, runs the three steps, copies every result back and
 * WAITS for the stream.  staging_d: caller-owned device memory of
 * lr_pass_staging_bytes, zero-filled before its first use.  Returns the device
 * status like lr_poll_status. */
int lr_verify_pass_host(lr_plan *plan, const lr_pass_host_io *io, const void *k_pool_d, const void *v_pool_d,
                        void *staging_d, size_t staging_bytes, float softmax_scale, void *stream);

/* ---- status ------------------------------------------------------------- */

/* Waits for `stream`, reads the plan's device status word and clears it.
 * Returns LR_OK, LR_ETIMEOUT or LR_EBOUNDS; *detail_out (nullable) receives a
 * kernel-specific code saying where it happened. */
int lr_poll_status(lr_plan *plan, void *stream, int32_t *detail_out);

/* Number of kernels the library has launched on behalf of this context. */
int64_t lr_launch_count(const lr_ctx *ctx);

const char *lr_strerror(int status);
const char *lr_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* LR_VERIFY_H_ */
