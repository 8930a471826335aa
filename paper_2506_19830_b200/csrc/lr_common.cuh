// Shared declarations of the verify-pass library: host objects, the device view
// of a plan, and small device helpers.  Internal; the public surface is
// include/lr_verify.h.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include <string.h>
#include <string>
#include <vector>

#include "lr_verify.h"

namespace lr {

constexpr int kPage = 16;
constexpr int kMaxTreeDepth = 8;  // deepest node of a draft-step tree (tree mode only; a chain may be longer)

// Device status word layout: [0] = code (0 ok, 1 timeout, 2 bounds), [1] = detail.
enum DevStatus : int { kDevOk = 0, kDevTimeout = 1, kDevBounds = 2 };

// Device view of the integer tables of a batch (all pointers into the plan workspace).
struct DevBatch {
  const int32_t *req_span_off, *span_len, *span_slot;
  const int32_t *br_req, *br_depth, *br_own_len, *br_own_slot, *br_n_draft;
  const int32_t *cu_q, *cu_draft, *page_ids;
  const int32_t *req_br_off;  // [n_req+1] branch range of each request
  const int32_t *span_req;    // [n_span] owning request of each span
  // commit tables.  Request r's chain prefix sums start at index req_span_off[r] + r and have
  // gamma_r + 2 entries: entry c = pages (tokens) of spans 0..c-1.  Its tail prefix sums start at
  // req_br_off[r] + r: entry k = pages of the tails of its first k branches.
  const int32_t *slot_item;   // [n_page_slots] owning span, or n_span + owning branch, or -1
  const int32_t *chain_pg;    // [n_span + n_req]
  const int32_t *chain_tok;   // [n_span + n_req]
  const int32_t *tail_pg;     // [n_branch + n_req]
  const int32_t *compact_stage_off;  // [n_req+1] staging-token range of each request in lr_compact
  // Tree of draft steps.  Spans are numbered in depth-first order per request (prefix 0); span c is seen
  // from node n iff span_tin[c] <= span_tin[n] <= span_last[c] (last = highest number in c's subtree).  On the
  // nested chain tin = c and last = gamma.  Children of span s: child_list[child_off[s] .. child_off[s+1]),
  // local indices in increasing order.
  const int32_t *span_tin, *span_last;  // [n_span]
  const int32_t *child_off, *child_list;  // [n_span+1], [n_span]
  int32_t tree;  // 1 when the batch gave seg_parent
  int32_t n_req, n_branch, n_span, n_page_slots, n_q_rows;
  int32_t n_q_heads, n_kv_heads, head_dim, group;
  int64_t n_pool_pages;
  int32_t *status;  // [2]
};

// ---- tensor-core attention plan (device side) -------------------------------
// A request's *extended chain* is the list of its page slots in the order
// prefix, segments 1..gamma, branch tails; consecutive groups of 8 pages form
// 128-key tiles.  The query rows that share one KV head -- (query token, head in
// group) pairs -- are packed into 128-row M-tiles.  A *group* is (request, KV
// head, one or two M-tiles); its tiles are cut into contiguous *pieces*, one or
// more per CTA.  A CTA runs two independent streams: the two M-tiles of the
// piece, or -- for a piece with one M-tile -- its even and odd tiles.  A
// *target* is one M-tile of one (request, KV head); when several streams
// contribute to a target each writes an fp32 partial and a second kernel merges.
struct TcPage {      // one per extended-chain page
  int32_t page;      // physical page id
  uint32_t meta;     // bits 0-4 valid tokens (0..16), 5-12 and 21-28 (chain pages) first and last depth-first node number that sees it, 13-20 owner branch (local, +1; 0 = chain), 21-31 (tail pages) first tail token index of the page / 16
};
struct TcRow {       // one per query row of the batch
  int32_t depth_branch;  // depth-first number of the branch's node | local branch index << 16
  int32_t limit;         // last tail token the row sees
};
struct TcPiece {
  int32_t req, kv_head;           // page list (index into reqs), KV head
  int32_t mtile0, n_mt;           // first M-tile and how many (1 or 2)
  int32_t tile_begin, tile_end;   // tiles of that page list
  int32_t slot[2];                // per stream: >= 0 partial slot, -1 write the final output, -2 nothing to write
};
struct TcReq {           // one page list: what one group of M-tiles of a request sweeps (pieces index it by `req`)
  int32_t page_off;     // first TcPage of the list
  int32_t n_pages;      // its pages: prefix, the segments and tails some row of the group can see
  int32_t q_row0, n_q;  // query token range of the request
  int32_t n_dense_tiles;  // leading tiles made only of full prefix pages (no masking needed)
  int32_t pad[3];
};
struct TcTarget {
  int32_t req, kv_head, mtile;
  int32_t slot_begin, n_slots;  // partial slots to merge (n_slots >= 2)
  int32_t q_row0, n_q;          // query token range of the request (copied, to spare a dependent load)
  int32_t pad;
};
struct TcCtaHead {    // everything a CTA needs to start, in one 256-byte record (one round trip to memory)
  int32_t piece0, piece1;   // its pieces
  TcPiece first;            // copy of pieces[piece0]
  TcReq first_req;          // copy of reqs[first.req]
  int32_t first_pages[32];  // physical ids of pages 32*c .. 32*c+31 of that request, c = first.tile_begin / 4; -1 = absent
  int32_t pad[14];
};
struct DevTcPlan {
  const TcCtaHead *heads;        // [n_cta]
  const TcPage *pages;
  const TcRow *rows;             // [n_q_rows]
  const TcPiece *pieces;
  const int32_t *cta_piece_off;  // [n_cta+1]
  const TcReq *reqs;
  const TcTarget *targets;
  int32_t n_cta, n_targets;
  int32_t tokens_per_mtile;  // floor(128 / group)
  uint32_t wait_limit_us;    // bound of every device-side wait (test hook: lr_plan_debug_set_wait_limit)
  uint32_t phantom_tx_bytes; // test hook: bytes CTA 0 expects on its first KV stage beyond what its copies deliver
  float *partial_o;          // [n_slots][32 chunks of 4 channels][128 rows][4] fp32, unnormalised
  float *partial_ml;         // [n_slots][128][2] (reference exponent in log2 units, sum)
};

// ---- CTA-pair attention plan (device side) -----------------------------------
// Two CTAs on neighbouring SMs work as one unit: CTA c of the pair owns M-tile mtile0 + c of a piece (its query
// rows, scores, probabilities and output accumulator) and supplies half of every KV tile; one tcgen05.mma with
// cta_group::2 (M = 256) applies the whole tile to both M-tiles.  Pages, rows and requests are described as for the
// single-CTA plan above.
struct PrPiece {
  int32_t req, kv_head;
  int32_t mtile0, n_mt;           // first M-tile and how many (1 or 2: with 1 the second CTA only lends its half of the KV tile)
  int32_t tile_begin, tile_end;   // tiles of the request's extended chain
  int32_t slot[2];                // per CTA of the pair: >= 0 partial slot, -1 write the final output, -2 nothing to write
  int32_t target[2];              // per CTA: merge target (index into targets / counters), -1 when slot < 0
};
struct PrHead {                   // everything a pair needs to start, in one 256-byte record
  int32_t piece0, piece1;
  PrPiece first;
  TcReq first_req;
  int32_t first_pages[32];        // physical ids of pages 32*c .. 32*c+31 of that request, c = first.tile_begin / 4; -1 = absent
  int32_t pad[12];
};
struct DevPairPlan {
  const PrHead *heads;            // [n_pairs]
  const TcPage *pages;
  const TcRow *rows;
  const PrPiece *pieces;
  const TcReq *reqs;
  const TcTarget *targets;
  int32_t n_pairs, n_targets;
  int32_t tokens_per_mtile;
  uint32_t wait_limit_us;         // bound of every device-side wait (test hook: lr_plan_debug_set_wait_limit)
  uint32_t phantom_tx_bytes;      // test hook: bytes CTA 0 of pair 0 expects on its first KV stage beyond what its copies deliver
  float *partial_o;               // [n_slots][32 chunks of 4 channels][128 rows][4] fp32, unnormalised
  float *partial_ml;              // [n_slots][128][2] (reference exponent in log2 units, sum)
  uint32_t *counters;             // [n_targets] arrival tickets of the contributors of a target; zero between launches
};

}  // namespace lr

struct lr_ctx {
  lr_model model;
  int device;
  int sm_count;
  int64_t launches;
  void *tmap_encode;  // cuTensorMapEncodeTiled entry point (driver), resolved lazily
  struct TmapEntry { const void *ptr; int64_t n; int kind; alignas(64) unsigned char map[128]; };
  std::vector<TmapEntry> tmaps;
  // Pinned host buffers of destroyed plans, kept for the next plan: allocating and freeing pinned memory costs
  // far more than building a plan.  `uploaded` is recorded after the buffer's last upload; a new user waits on it.
  struct PinnedBuf { void *ptr; size_t cap; cudaEvent_t uploaded; };
  std::vector<PinnedBuf> pinned_free;
};

struct lr_plan {
  lr_ctx *ctx;
  lr::DevBatch dev;
  lr::DevTcPlan tc;
  lr::DevPairPlan pr;
  bool tc_ok;             // shape allows the tensor-core path
  bool pair_ok;           // shape allows the CTA-pair tensor-core path
  int pr_pieces, pr_partial_slots;
  size_t o_pr_pages, o_pr_heads;
  int n_pr_pages, n_pr_heads;
  int attention_path;     // 0 auto, 1 generic, 2 tensor core (single CTA), 3 tensor core (CTA pairs)
  int tc_pieces, tc_partial_slots;  // for lr_plan_describe
  // where the physical page ids sit in the image (lr_plan_debug_set_page)
  size_t o_page_ids, o_tc_pages, o_tc_heads;
  int n_tc_pages, n_tc_heads;
  std::vector<unsigned char> staging;  // host copy of the uploaded image (kept alive for the async copy)
  void *pinned;           // pinned host image
  size_t pinned_cap;
  void *results_pinned;   // pinned bounce buffer for the integer results of lr_verify_pass_host (allocated on first use)
  size_t results_pinned_cap;
  cudaEvent_t uploaded;   // recorded after the image's upload
  size_t image_bytes;
  void *workspace_d;
  size_t workspace_bytes;
  struct { size_t o_tok_off, o_first_moved, o_staging, bytes; } compact;  // layout of lr_compact's scratch
  // host copies needed at launch time
  int32_t n_rows_logits, n_drafts, n_verdicts;
  std::vector<int32_t> cu_draft_h;
};

namespace lr {

// Byte image of everything lr_plan_create uploads; sections are 256-byte aligned.
struct Image {
  std::vector<unsigned char> bytes;
  size_t add(const void *src, size_t n) {
    size_t off = (bytes.size() + 255) / 256 * 256;
    bytes.resize(off + n);
    if (src && n) memcpy(bytes.data() + off, src, n);
    return off;
  }
};

// Host-side result of planning the tensor-core attention for one batch.
struct TcHostPlan {
  bool ok = false;  // shape supported by the tensor-core path
  size_t o_heads = 0, o_pages = 0, o_rows = 0, o_pieces = 0, o_cta_piece_off = 0, o_reqs = 0, o_targets = 0;  // image offsets
  int n_cta = 0, n_targets = 0, n_pieces = 0, n_partial_slots = 0, tokens_per_mtile = 0, n_pages = 0;
  // scratch region behind the image: (exponent, sum) pairs, then fp32 partial outputs
  size_t s_ml = 0, s_o = 0, scratch_bytes = 0, scratch_zero_bytes = 0;
};
// span_tin / span_last: depth-first interval labels of the spans ([n_span] each, see DevBatch)
int tc_build_host_plan(const lr_ctx *ctx, const lr_batch *b, const int32_t *req_br_off, const int32_t *span_tin,
                       const int32_t *span_last, TcHostPlan &out, Image &img);
void tc_bind_device_plan(const TcHostPlan &h, unsigned char *image_base, unsigned char *scratch_base, lr_plan *p);

// Host-side result of planning the CTA-pair attention for one batch.
struct PairHostPlan {
  bool ok = false;
  size_t o_heads = 0, o_pages = 0, o_rows = 0, o_pieces = 0, o_reqs = 0, o_targets = 0;  // image offsets
  int n_pairs = 0, n_targets = 0, n_pieces = 0, n_partial_slots = 0, tokens_per_mtile = 0, n_pages = 0;
  // scratch region behind the image: ticket counters, (exponent, sum) pairs, fp32 partial outputs
  size_t s_counters = 0, s_ml = 0, s_o = 0, scratch_bytes = 0, scratch_zero_bytes = 0;
};
int pair_build_host_plan(const lr_ctx *ctx, const lr_batch *b, const int32_t *req_br_off, const int32_t *span_tin,
                         const int32_t *span_last, PairHostPlan &out, Image &img);
void pair_bind_device_plan(const PairHostPlan &h, unsigned char *image_base, unsigned char *scratch_base, lr_plan *p);

void set_error(const char *fmt, ...);

// Launch as a programmatic dependent of the kernel before it in the stream: the grid is set up while that kernel
// drains; the kernel itself waits (griddepcontrol.wait) before it touches anything its predecessor wrote.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
int cuda_fail(cudaError_t e, const char *what);

// kernels (each file exposes launchers)
int init_kernels(lr_ctx *ctx);  // per-device function attributes; called by lr_create
int init_commit_kernel();
int init_attn_tc_kernel();
int init_attn_pair_kernel();
int launch_attn_pair(lr_plan *p, const void *q, const void *k, const void *v, void *out, float *lse, float scale,
                     cudaStream_t s);
int launch_attn_generic(lr_plan *p, const void *q, const void *k, const void *v, void *out, float *lse, float scale,
                        cudaStream_t s);
int launch_attn_tc(lr_plan *p, const void *q, const void *k, const void *v, void *out, float *lse, float scale,
                   cudaStream_t s);
int launch_accept(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts, const int32_t *cu_draft,
                  int32_t n_branch, int32_t n_rows, int32_t *n_accept, int32_t *bonus, int32_t *row_argmax,
                  void *scratch, cudaStream_t s);
int launch_accept_static(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts, const int32_t *cu_draft,
                         int32_t n_branch, int32_t n_rows, int32_t *n_accept, int32_t *bonus, int32_t *row_argmax,
                         cudaStream_t s);
size_t accept_sample_scratch_bytes(int32_t vocab, int32_t n_rows);
int launch_accept_sample(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts, const int32_t *cu_draft,
                         int32_t n_branch, int32_t n_rows, float temperature, const float *u_accept, const float *u_final,
                         int32_t *n_accept, int32_t *final_id, float *p_draft, void *scratch, cudaStream_t s);
size_t accept_filtered_scratch_bytes(int32_t n_rows);
int launch_accept_filtered(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts, const int32_t *cu_draft,
                           int32_t n_branch, int32_t n_rows, float temperature, int32_t top_k, float top_p,
                           const float *u_accept, const float *u_final, int32_t *n_accept, int32_t *final_id, float *p_draft,
                           int32_t *n_kept, void *scratch, cudaStream_t s);
int launch_compact(lr_plan *p, const int32_t *keep_off, const int32_t *keep_pages, const int32_t *keep_valid, void *k_pool,
                   void *v_pool, int32_t *new_len, int32_t *n_pages_kept, void *scratch, cudaStream_t s);
int launch_commit(lr_plan *p, const uint8_t *verdict, const int32_t *n_accept, int32_t *n_steps, int32_t *survivor,
                  int32_t *committed, int32_t *keep_off, int32_t *keep_pages, int32_t *keep_valid, int32_t *free_off,
                  int32_t *free_pages, cudaStream_t s);

}  // namespace lr
