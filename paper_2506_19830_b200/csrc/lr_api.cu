// Host side of the C ABI: contexts, batch validation, plan images, launch
// wrappers and the host-buffer pass.  No device memory is allocated here; every
// device byte the library touches lies in caller-provided buffers.
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "lr_common.cuh"

namespace lr {

static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

int cuda_fail(cudaError_t e, const char *what) {
  if (e == cudaSuccess) return LR_OK;
  set_error("%s: %s", what, cudaGetErrorString(e));
  return LR_ECUDA;
}

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int pages_of(int64_t n) { return (int)((n + kPage - 1) / kPage); }

// ---- batch validation --------------------------------------------------------
#define LR_REQUIRE(cond, ...)          \
  do {                                 \
    if (!(cond)) {                     \
      set_error(__VA_ARGS__);          \
      return LR_EINVAL;                \
    }                                  \
  } while (0)

static int validate_batch(const lr_batch *b) {
  LR_REQUIRE(b != nullptr, "null batch");
  LR_REQUIRE(b->n_req >= 1 && b->n_branch >= 1 && b->n_span >= b->n_req && b->n_page_slots >= 1,
             "batch needs at least one request, one branch and one page slot");
  LR_REQUIRE(b->req_span_off && b->span_len && b->span_slot && b->br_req && b->br_depth && b->br_own_len &&
                 b->br_own_slot && b->br_n_draft && b->cu_q && b->page_ids,
             "null table pointer in batch");
  LR_REQUIRE(b->n_pool_pages >= 1 && b->n_pool_pages <= (int64_t)1 << 31, "n_pool_pages out of range");
  LR_REQUIRE(b->req_span_off[0] == 0 && b->req_span_off[b->n_req] == b->n_span, "req_span_off must run from 0 to n_span");
  std::vector<unsigned char> slot_used((size_t)b->n_page_slots, 0);
  auto claim = [&](int64_t first, int64_t len, const char *what, int idx) -> int {
    int n = pages_of(len);
    LR_REQUIRE(first >= 0 && first + n <= b->n_page_slots, "%s %d: page slots [%lld, %lld) outside [0, %d)", what, idx,
               (long long)first, (long long)(first + n), b->n_page_slots);
    for (int i = 0; i < n; ++i) {
      LR_REQUIRE(!slot_used[first + i], "%s %d: page slot %lld is claimed twice", what, idx, (long long)(first + i));
      slot_used[first + i] = 1;
    }
    return LR_OK;
  };
  for (int r = 0; r < b->n_req; ++r) {
    int s0 = b->req_span_off[r], s1 = b->req_span_off[r + 1];
    LR_REQUIRE(s1 > s0, "request %d has no prefix span", r);
    LR_REQUIRE(s1 - s0 - 1 <= 255, "request %d: more than 255 draft step segments", r);
    for (int s = s0; s < s1; ++s) {
      LR_REQUIRE(b->span_len[s] >= (s == s0 ? 0 : 1), "span %d of request %d has length %d", s - s0, r, b->span_len[s]);
      if (int rc = claim(b->span_slot[s], b->span_len[s], "span", s)) return rc;
    }
    if (b->seg_parent) {
      std::vector<int> level((size_t)(s1 - s0), 0);
      for (int c = 1; c < s1 - s0; ++c) {
        const int par = b->seg_parent[s0 + c];
        LR_REQUIRE(par >= 0 && par < c, "request %d: segment %d continues %d, which is not the prefix or an earlier segment", r, c, par);
        level[c] = level[par] + 1;
        LR_REQUIRE(level[c] <= kMaxTreeDepth, "request %d: segment %d lies %d steps below the prefix (tree mode allows %d)", r,
                   c, level[c], kMaxTreeDepth);
      }
    }
  }
  LR_REQUIRE(b->cu_q[0] == 0, "cu_q[0] must be 0");
  for (int i = 0; i < b->n_branch; ++i) {
    int r = b->br_req[i];
    LR_REQUIRE(r >= 0 && r < b->n_req, "branch %d: request %d out of range", i, r);
    LR_REQUIRE(i == 0 || b->br_req[i - 1] <= r, "branches must be grouped by request (br_req non-decreasing)");
    int gamma = b->req_span_off[r + 1] - b->req_span_off[r] - 1;
    LR_REQUIRE(b->br_depth[i] >= 0 && b->br_depth[i] <= gamma, "branch %d: depth %d outside [0, %d]", i, b->br_depth[i], gamma);
    int q_len = b->cu_q[i + 1] - b->cu_q[i];
    LR_REQUIRE(q_len >= 1, "branch %d: q_len %d < 1", i, q_len);
    LR_REQUIRE(b->br_own_len[i] >= q_len, "branch %d: own_len %d < q_len %d", i, b->br_own_len[i], q_len);
    LR_REQUIRE(b->br_n_draft[i] >= 0 && b->br_n_draft[i] <= b->br_own_len[i], "branch %d: n_draft %d outside [0, own_len]", i,
               b->br_n_draft[i]);
    if (int rc = claim(b->br_own_slot[i], b->br_own_len[i], "branch tail", i)) return rc;
  }
  std::vector<unsigned char> page_used((size_t)((b->n_pool_pages + 7) / 8), 0);
  for (int i = 0; i < b->n_page_slots; ++i) {
    if (!slot_used[i]) continue;  // slots no span refers to are ignored
    int64_t p = b->page_ids[i];
    LR_REQUIRE(p >= 0 && p < b->n_pool_pages, "page_ids[%d] = %lld outside the pool of %lld pages", i, (long long)p,
               (long long)b->n_pool_pages);
    LR_REQUIRE(!(page_used[p >> 3] & (1u << (p & 7))), "physical page %lld is referenced by two page slots", (long long)p);
    page_used[p >> 3] |= (unsigned char)(1u << (p & 7));
  }
  return LR_OK;
}

// ---- plan image --------------------------------------------------------------
struct Layout {
  Image img;
  size_t o_req_span_off, o_span_len, o_span_slot, o_br_req, o_br_depth, o_br_own_len, o_br_own_slot, o_br_n_draft, o_cu_q,
      o_cu_draft, o_page_ids, o_req_br_off, o_span_req, o_status, o_slot_item, o_chain_pg, o_chain_tok, o_tail_pg, o_compact_stage_off,
      o_span_tin, o_span_last, o_child_off, o_child_list;
  size_t compact_tokens;
  std::vector<int32_t> cu_draft;
  TcHostPlan tc;
  PairHostPlan pr;
  size_t image_bytes, total_bytes, pair_scratch_off;
};

static int build_layout(const lr_ctx *ctx, const lr_batch *b, Layout &L) {
  if (!ctx) {
    set_error("null context");
    return LR_EINVAL;
  }
  if (int rc = validate_batch(b)) return rc;
  const size_t I = sizeof(int32_t);
  std::vector<int32_t> cu_draft(b->n_branch + 1, 0), req_br_off(b->n_req + 1, 0), span_req(b->n_span, 0);
  for (int i = 0; i < b->n_branch; ++i) {
    cu_draft[i + 1] = cu_draft[i] + b->br_n_draft[i];
    req_br_off[b->br_req[i] + 1]++;
  }
  for (int r = 0; r < b->n_req; ++r) {
    req_br_off[r + 1] += req_br_off[r];
    for (int s = b->req_span_off[r]; s < b->req_span_off[r + 1]; ++s) span_req[s] = r;
  }
  Image &g = L.img;
  L.o_req_span_off = g.add(b->req_span_off, I * (b->n_req + 1));
  L.o_span_len = g.add(b->span_len, I * b->n_span);
  L.o_span_slot = g.add(b->span_slot, I * b->n_span);
  L.o_br_req = g.add(b->br_req, I * b->n_branch);
  L.o_br_depth = g.add(b->br_depth, I * b->n_branch);
  L.o_br_own_len = g.add(b->br_own_len, I * b->n_branch);
  L.o_br_own_slot = g.add(b->br_own_slot, I * b->n_branch);
  L.o_br_n_draft = g.add(b->br_n_draft, I * b->n_branch);
  L.o_cu_q = g.add(b->cu_q, I * (b->n_branch + 1));
  L.o_cu_draft = g.add(cu_draft.data(), I * (b->n_branch + 1));
  L.o_page_ids = g.add(b->page_ids, I * b->n_page_slots);
  L.o_req_br_off = g.add(req_br_off.data(), I * (b->n_req + 1));
  L.o_span_req = g.add(span_req.data(), I * b->n_span);
  {
    std::vector<int32_t> slot_item((size_t)b->n_page_slots, -1), chain_pg((size_t)b->n_span + b->n_req, 0),
        chain_tok((size_t)b->n_span + b->n_req, 0), tail_pg((size_t)b->n_branch + b->n_req, 0);
    for (int r = 0; r < b->n_req; ++r) {
      const int s0 = b->req_span_off[r], s1 = b->req_span_off[r + 1], base = s0 + r;
      for (int s = s0; s < s1; ++s) {
        const int npg = pages_of(b->span_len[s]);
        chain_pg[base + (s - s0) + 1] = chain_pg[base + (s - s0)] + npg;
        chain_tok[base + (s - s0) + 1] = chain_tok[base + (s - s0)] + b->span_len[s];
        for (int k = 0; k < npg; ++k) slot_item[b->span_slot[s] + k] = s;
      }
      const int b0 = req_br_off[r], b1 = req_br_off[r + 1], tb = b0 + r;
      for (int i = b0; i < b1; ++i) {
        const int npg = pages_of(b->br_own_len[i]);
        tail_pg[tb + (i - b0) + 1] = tail_pg[tb + (i - b0)] + npg;
        for (int k = 0; k < npg; ++k) slot_item[b->br_own_slot[i] + k] = b->n_span + i;
      }
    }
    L.o_slot_item = g.add(slot_item.data(), I * slot_item.size());
    L.o_chain_pg = g.add(chain_pg.data(), I * chain_pg.size());
    L.o_chain_tok = g.add(chain_tok.data(), I * chain_tok.size());
    L.o_tail_pg = g.add(tail_pg.data(), I * tail_pg.size());
    // lr_compact: at most the segments and one tail of a request are displaced
    std::vector<int32_t> stage_off((size_t)b->n_req + 1, 0);
    size_t tokens = 0;
    for (int r = 0; r < b->n_req; ++r) {
      stage_off[r] = (int32_t)tokens;
      size_t segs = 0, tail = 0;
      for (int s = b->req_span_off[r] + 1; s < b->req_span_off[r + 1]; ++s) segs += (size_t)b->span_len[s];
      for (int i = req_br_off[r]; i < req_br_off[r + 1]; ++i) tail = std::max(tail, (size_t)b->br_own_len[i]);
      tokens += segs + tail;
      stage_off[r + 1] = (int32_t)tokens;
    }
    L.compact_tokens = tokens;
    L.o_compact_stage_off = g.add(stage_off.data(), I * stage_off.size());
  }
  // depth-first interval labels and child lists of the draft-step trees (a chain when seg_parent is absent)
  std::vector<int32_t> span_tin((size_t)b->n_span, 0), span_last((size_t)b->n_span, 0), child_off((size_t)b->n_span + 1, 0),
      child_list((size_t)b->n_span, 0);
  for (int r = 0; r < b->n_req; ++r) {
    const int s0 = b->req_span_off[r], n = b->req_span_off[r + 1] - s0;
    auto parent_of = [&](int c) { return b->seg_parent ? b->seg_parent[s0 + c] : c - 1; };
    std::vector<int> n_child((size_t)n, 0);
    for (int c = 1; c < n; ++c) n_child[parent_of(c)]++;
    for (int c = 0; c < n; ++c) child_off[s0 + c + 1] = child_off[s0 + c] + n_child[c];
    std::vector<int> fill((size_t)n, 0);
    for (int c = 1; c < n; ++c) {  // increasing c: every list comes out sorted
      const int par = parent_of(c);
      child_list[child_off[s0 + par] + fill[par]++] = c;
    }
    std::vector<int> size((size_t)n, 1);  // subtree sizes: children have larger indices than parents
    for (int c = n - 1; c >= 1; --c) size[parent_of(c)] += size[c];
    // pre-order numbers: a node's number is its parent's + 1 + the subtree sizes of its earlier siblings
    for (int c = 0; c < n; ++c) {
      int next = span_tin[s0 + c] + 1;
      for (int k = child_off[s0 + c]; k < child_off[s0 + c + 1]; ++k) {
        span_tin[s0 + child_list[k]] = next;
        next += size[child_list[k]];
      }
      span_last[s0 + c] = span_tin[s0 + c] + size[c] - 1;
    }
  }
  L.o_span_tin = g.add(span_tin.data(), I * span_tin.size());
  L.o_span_last = g.add(span_last.data(), I * span_last.size());
  L.o_child_off = g.add(child_off.data(), I * child_off.size());
  L.o_child_list = g.add(child_list.data(), I * child_list.size());
  int32_t zero2[2] = {0, 0};
  L.o_status = g.add(zero2, sizeof(zero2));
  L.cu_draft = cu_draft;
  if (int rc = tc_build_host_plan(ctx, b, req_br_off.data(), span_tin.data(), span_last.data(), L.tc, g)) return rc;
  if (int rc = pair_build_host_plan(ctx, b, req_br_off.data(), span_tin.data(), span_last.data(), L.pr, g)) return rc;
  L.image_bytes = align_up(g.bytes.size(), 256);
  L.pair_scratch_off = L.image_bytes + align_up(L.tc.scratch_bytes, 256);
  L.total_bytes = L.pair_scratch_off + align_up(L.pr.scratch_bytes, 256);
  return LR_OK;
}

}  // namespace lr

using namespace lr;

static int check_model(const lr_model *m, const char *who) {
  if (m->n_q_heads < 1 || m->n_kv_heads < 1 || m->vocab < 1) {
    set_error("%s: non-positive model dimension", who);
    return LR_EINVAL;
  }
  if ((m->head_dim != 64 && m->head_dim != 128) || m->page_size != kPage || m->n_q_heads % m->n_kv_heads != 0 ||
      m->n_q_heads / m->n_kv_heads > 16) {
    set_error("%s: unsupported geometry (head_dim %d, page_size %d, heads %d/%d)", who, m->head_dim, m->page_size,
              m->n_q_heads, m->n_kv_heads);
    return LR_EUNSUPPORTED;
  }
  return LR_OK;
}

extern "C" int lr_validate_batch(const lr_model *m, const lr_batch *b) {
  if (!m) {
    set_error("lr_validate_batch: null model");
    return LR_EINVAL;
  }
  if (int rc = check_model(m, "lr_validate_batch")) return rc;
  return validate_batch(b);
}

// ---- context -------------------------------------------------------------------
extern "C" int lr_create(lr_ctx **out, const lr_model *m, int device) {
  if (!out || !m) {
    set_error("lr_create: null argument");
    return LR_EINVAL;
  }
  *out = nullptr;
  if (int rc = check_model(m, "lr_create")) return rc;
  int n_dev = 0;
  if (int rc = cuda_fail(cudaGetDeviceCount(&n_dev), "cudaGetDeviceCount")) return rc;
  if (device < 0 || device >= n_dev) {
    set_error("lr_create: device %d not present (%d devices)", device, n_dev);
    return LR_EINVAL;
  }
  cudaDeviceProp prop;
  if (int rc = cuda_fail(cudaGetDeviceProperties(&prop, device), "cudaGetDeviceProperties")) return rc;
  if (prop.major != 10) {
    set_error("lr_create: device %d is sm_%d%d; this library is built for sm_100a only", device, prop.major, prop.minor);
    return LR_EUNSUPPORTED;
  }
  if (int rc = cuda_fail(cudaSetDevice(device), "cudaSetDevice")) return rc;
  lr_ctx *c = new (std::nothrow) lr_ctx();
  if (!c) return LR_ENOMEM;
  c->model = *m;
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  c->launches = 0;
  c->tmap_encode = nullptr;
  if (int rc = init_commit_kernel()) { delete c; return rc; }
  if (int rc = init_attn_tc_kernel()) { delete c; return rc; }
  if (int rc = init_attn_pair_kernel()) { delete c; return rc; }
  *out = c;
  return LR_OK;
}

extern "C" int lr_destroy(lr_ctx *ctx) {
  if (ctx) {
    for (auto &pb : ctx->pinned_free) {
      cudaEventSynchronize(pb.uploaded);
      cudaEventDestroy(pb.uploaded);
      cudaFreeHost(pb.ptr);
    }
  }
  delete ctx;
  return LR_OK;
}

// A pinned buffer of at least `bytes`: the smallest cached one that fits, else a new one (capacity rounded up to a
// power of two, at least 64 KB, so that the next plan of a similar batch fits too).
static int take_pinned(lr_ctx *ctx, size_t bytes, void **ptr, size_t *cap, cudaEvent_t *ev) {
  int best = -1;
  for (int i = 0; i < (int)ctx->pinned_free.size(); ++i)
    if (ctx->pinned_free[i].cap >= bytes && (best < 0 || ctx->pinned_free[i].cap < ctx->pinned_free[best].cap)) best = i;
  if (best >= 0) {
    lr_ctx::PinnedBuf pb = ctx->pinned_free[best];
    ctx->pinned_free.erase(ctx->pinned_free.begin() + best);
    if (int rc = cuda_fail(cudaEventSynchronize(pb.uploaded), "cudaEventSynchronize(pinned buffer)")) return rc;
    *ptr = pb.ptr; *cap = pb.cap; *ev = pb.uploaded;
    return LR_OK;
  }
  size_t c = 64 << 10;
  while (c < bytes) c <<= 1;
  if (int rc = cuda_fail(cudaMallocHost(ptr, c), "cudaMallocHost(plan image)")) return rc;
  if (int rc = cuda_fail(cudaEventCreateWithFlags(ev, cudaEventDisableTiming), "cudaEventCreate")) {
    cudaFreeHost(*ptr);
    return rc;
  }
  *cap = c;
  return LR_OK;
}

static void give_back_pinned(lr_ctx *ctx, void *ptr, size_t cap, cudaEvent_t ev) {
  if (ctx->pinned_free.size() < 8) {
    ctx->pinned_free.push_back({ptr, cap, ev});
    return;
  }
  cudaEventSynchronize(ev);
  cudaEventDestroy(ev);
  cudaFreeHost(ptr);
}

extern "C" int64_t lr_launch_count(const lr_ctx *ctx) { return ctx ? ctx->launches : 0; }

// ---- plan ----------------------------------------------------------------------
extern "C" int lr_plan_bytes(const lr_ctx *ctx, const lr_batch *b, size_t *bytes_out) {
  if (!bytes_out) {
    set_error("lr_plan_bytes: null bytes_out");
    return LR_EINVAL;
  }
  Layout L;
  if (int rc = build_layout(ctx, b, L)) return rc;
  *bytes_out = L.total_bytes;
  return LR_OK;
}

extern "C" int lr_plan_create(lr_ctx *ctx, const lr_batch *b, void *ws, size_t ws_bytes, void *stream, lr_plan **out) {
  if (!out || !ws) {
    set_error("lr_plan_create: null argument");
    return LR_EINVAL;
  }
  *out = nullptr;
  if (((uintptr_t)ws & 255) != 0) {
    set_error("lr_plan_create: workspace must be 256-byte aligned");
    return LR_EINVAL;
  }
  Layout L;
  if (int rc = build_layout(ctx, b, L)) return rc;
  if (ws_bytes < L.total_bytes) {
    set_error("lr_plan_create: workspace of %zu bytes, %zu needed", ws_bytes, L.total_bytes);
    return LR_ENOMEM;
  }
  if (int rc = cuda_fail(cudaSetDevice(ctx->device), "cudaSetDevice")) return rc;
  lr_plan *p = new (std::nothrow) lr_plan();
  if (!p) return LR_ENOMEM;
  p->ctx = ctx;
  p->pinned = nullptr;
  p->results_pinned = nullptr;
  p->results_pinned_cap = 0;
  p->image_bytes = L.image_bytes;
  p->workspace_d = ws;
  p->workspace_bytes = ws_bytes;
  p->attention_path = 0;
  p->o_page_ids = L.o_page_ids;
  if (int rc = take_pinned(ctx, L.image_bytes, &p->pinned, &p->pinned_cap, &p->uploaded)) {
    delete p;
    return rc;
  }
  memset(p->pinned, 0, L.image_bytes);
  memcpy(p->pinned, L.img.bytes.data(), L.img.bytes.size());
  unsigned char *base = reinterpret_cast<unsigned char *>(ws);
  auto at = [&](size_t off) { return reinterpret_cast<const int32_t *>(base + off); };
  DevBatch &d = p->dev;
  d.req_span_off = at(L.o_req_span_off);
  d.span_len = at(L.o_span_len);
  d.span_slot = at(L.o_span_slot);
  d.br_req = at(L.o_br_req);
  d.br_depth = at(L.o_br_depth);
  d.br_own_len = at(L.o_br_own_len);
  d.br_own_slot = at(L.o_br_own_slot);
  d.br_n_draft = at(L.o_br_n_draft);
  d.cu_q = at(L.o_cu_q);
  d.cu_draft = at(L.o_cu_draft);
  d.page_ids = at(L.o_page_ids);
  d.req_br_off = at(L.o_req_br_off);
  d.span_req = at(L.o_span_req);
  d.slot_item = at(L.o_slot_item);
  d.chain_pg = at(L.o_chain_pg);
  d.chain_tok = at(L.o_chain_tok);
  d.tail_pg = at(L.o_tail_pg);
  d.compact_stage_off = at(L.o_compact_stage_off);
  d.span_tin = at(L.o_span_tin);
  d.span_last = at(L.o_span_last);
  d.child_off = at(L.o_child_off);
  d.child_list = at(L.o_child_list);
  d.tree = b->seg_parent ? 1 : 0;
  {
    size_t off = 0;
    auto take = [&](size_t n) { size_t o = off; off = align_up(off + n, 256); return o; };
    p->compact.o_tok_off = take(sizeof(int32_t) * (size_t)b->n_page_slots);
    p->compact.o_first_moved = take(sizeof(int32_t) * (size_t)b->n_req);
    p->compact.o_staging = take(L.compact_tokens * 2 * (size_t)ctx->model.n_kv_heads * ctx->model.head_dim * 2);
    p->compact.bytes = std::max<size_t>(off, 256);
  }
  d.status = reinterpret_cast<int32_t *>(base + L.o_status);
  d.n_req = b->n_req;
  d.n_branch = b->n_branch;
  d.n_span = b->n_span;
  d.n_page_slots = b->n_page_slots;
  d.n_q_rows = b->cu_q[b->n_branch];
  d.n_q_heads = ctx->model.n_q_heads;
  d.n_kv_heads = ctx->model.n_kv_heads;
  d.head_dim = ctx->model.head_dim;
  d.group = ctx->model.n_q_heads / ctx->model.n_kv_heads;
  d.n_pool_pages = b->n_pool_pages;
  p->cu_draft_h = L.cu_draft;
  p->n_drafts = L.cu_draft[b->n_branch];
  p->n_rows_logits = p->n_drafts + b->n_branch;
  p->n_verdicts = b->n_span - b->n_req;
  tc_bind_device_plan(L.tc, base, base + L.image_bytes, p);
  pair_bind_device_plan(L.pr, base, base + L.pair_scratch_off, p);
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(ws, p->pinned, L.image_bytes, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess && L.tc.scratch_zero_bytes)
    e = cudaMemsetAsync(base + L.image_bytes, 0, L.tc.scratch_zero_bytes, s);
  if (e == cudaSuccess && L.pr.scratch_zero_bytes)
    e = cudaMemsetAsync(base + L.pair_scratch_off, 0, L.pr.scratch_zero_bytes, s);
  if (e == cudaSuccess) e = cudaEventRecord(p->uploaded, s);
  if (e != cudaSuccess) {
    give_back_pinned(ctx, p->pinned, p->pinned_cap, p->uploaded);
    delete p;
    return cuda_fail(e, "plan upload");
  }
  *out = p;
  return LR_OK;
}

extern "C" int lr_plan_destroy(lr_plan *p) {
  if (!p) return LR_OK;
  if (p->pinned) give_back_pinned(p->ctx, p->pinned, p->pinned_cap, p->uploaded);
  if (p->results_pinned) cudaFreeHost(p->results_pinned);
  delete p;
  return LR_OK;
}

extern "C" int lr_plan_set_attention_path(lr_plan *p, int path) {
  if (!p || path < 0 || path > 3) {
    set_error("lr_plan_set_attention_path: bad argument");
    return LR_EINVAL;
  }
  p->attention_path = path;
  return LR_OK;
}

extern "C" int lr_plan_describe(const lr_plan *p, lr_plan_info *info) {
  if (!p || !info) {
    set_error("lr_plan_describe: null argument");
    return LR_EINVAL;
  }
  memset(info, 0, sizeof(*info));
  info->tensor_core_ok = p->tc_ok ? 1 : 0;
  info->path = p->attention_path;
  if (p->attention_path == 3) {
    info->uses_tensor_core = p->pair_ok ? 1 : 0;
    if (p->pair_ok) {
      info->n_cta = 2 * p->pr.n_pairs;
      info->n_pieces = p->pr_pieces;
      info->n_merge_targets = p->pr.n_targets;
      info->n_partial_slots = p->pr_partial_slots;
    }
    return LR_OK;
  }
  info->uses_tensor_core = (p->tc_ok && p->attention_path != 1) ? 1 : 0;
  if (info->uses_tensor_core) {
    info->n_cta = p->tc.n_cta;
    info->n_pieces = p->tc_pieces;
    info->n_merge_targets = p->tc.n_targets;
    info->n_partial_slots = p->tc_partial_slots;
  }
  return LR_OK;
}

extern "C" int lr_plan_debug_set_wait_limit(lr_plan *p, uint32_t microseconds) {
  if (!p || microseconds == 0) {
    set_error("lr_plan_debug_set_wait_limit: bad argument");
    return LR_EINVAL;
  }
  p->tc.wait_limit_us = microseconds;
  p->pr.wait_limit_us = microseconds;
  return LR_OK;
}

extern "C" int lr_plan_debug_set_phantom_bytes(lr_plan *p, uint32_t bytes) {
  if (!p) {
    set_error("lr_plan_debug_set_phantom_bytes: null plan");
    return LR_EINVAL;
  }
  p->tc.phantom_tx_bytes = bytes;
  p->pr.phantom_tx_bytes = bytes;
  return LR_OK;
}

extern "C" int lr_plan_debug_set_page(lr_plan *p, int32_t page_slot, int32_t new_id, void *stream) {
  if (!p || page_slot < 0 || page_slot >= p->dev.n_page_slots) {
    set_error("lr_plan_debug_set_page: bad argument");
    return LR_EINVAL;
  }
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  // the pinned image is the source of the last upload: wait until that copy has read it
  if (int rc = cuda_fail(cudaEventSynchronize(p->uploaded), "cudaEventSynchronize(plan image)")) return rc;
  unsigned char *img = reinterpret_cast<unsigned char *>(p->pinned);
  int32_t *ids = reinterpret_cast<int32_t *>(img + p->o_page_ids);
  const int32_t old_id = ids[page_slot];
  ids[page_slot] = new_id;
  // physical page ids are distinct within a batch, so the old id names this slot in the attention tables too
  TcPage *pages = reinterpret_cast<TcPage *>(img + p->o_tc_pages);
  for (int i = 0; i < p->n_tc_pages; ++i)
    if (pages[i].page == old_id && (pages[i].meta & 31u) != 0u) pages[i].page = new_id;
  TcCtaHead *heads = reinterpret_cast<TcCtaHead *>(img + p->o_tc_heads);
  for (int c = 0; c < p->n_tc_heads; ++c)
    for (int k = 0; k < 32; ++k)
      if (heads[c].first_pages[k] == old_id && heads[c].piece1 > heads[c].piece0) heads[c].first_pages[k] = new_id;
  TcPage *ppages = reinterpret_cast<TcPage *>(img + p->o_pr_pages);
  for (int i = 0; i < p->n_pr_pages; ++i)
    if (ppages[i].page == old_id && (ppages[i].meta & 31u) != 0u) ppages[i].page = new_id;
  PrHead *pheads = reinterpret_cast<PrHead *>(img + p->o_pr_heads);
  for (int c = 0; c < p->n_pr_heads; ++c)
    for (int k = 0; k < 32; ++k)
      if (pheads[c].first_pages[k] == old_id && pheads[c].piece1 > pheads[c].piece0) pheads[c].first_pages[k] = new_id;
  cudaError_t e = cudaMemcpyAsync(p->workspace_d, p->pinned, p->image_bytes, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaEventRecord(p->uploaded, s);
  return cuda_fail(e, "lr_plan_debug_set_page upload");
}

// ---- steps ---------------------------------------------------------------------
extern "C" int lr_verify_attention(lr_plan *p, const void *q, const void *k, const void *v, void *out, float *lse,
                                   float scale, void *stream) {
  if (!p || !q || !k || !v || !out) {
    set_error("lr_verify_attention: null argument");
    return LR_EINVAL;
  }
  if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15) != 0 || ((uintptr_t)lse & 3) != 0) {
    set_error("lr_verify_attention: q, pools and out must be 16-byte aligned");
    return LR_EINVAL;
  }
  if (!(scale > 0.f)) scale = 1.0f / sqrtf((float)p->dev.head_dim);
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (p->attention_path == 3) {
    if (!p->pair_ok) {
      set_error("lr_verify_attention: the CTA-pair tensor-core path does not support this shape");
      return LR_EUNSUPPORTED;
    }
    return launch_attn_pair(p, q, k, v, out, lse, scale, s);
  }
  bool use_tc = p->attention_path == 2 || (p->attention_path == 0 && p->tc_ok);
  if (use_tc) {
    if (!p->tc_ok) {
      set_error("lr_verify_attention: the tensor-core path does not support this shape");
      return LR_EUNSUPPORTED;
    }
    return launch_attn_tc(p, q, k, v, out, lse, scale, s);
  }
  return launch_attn_generic(p, q, k, v, out, lse, scale, s);
}

extern "C" int lr_accept_scratch_bytes(int32_t n_rows, size_t *bytes_out) {
  if (!bytes_out || n_rows < 0) {
    set_error("lr_accept_scratch_bytes: bad argument");
    return LR_EINVAL;
  }
  *bytes_out = 8 * ((size_t)n_rows + 1);
  return LR_OK;
}

extern "C" int lr_accept_greedy(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts,
                                const int32_t *cu_draft, int32_t n_branch, int32_t n_rows, int32_t *n_accept,
                                int32_t *bonus, int32_t *row_argmax, void *scratch, void *stream) {
  if (!ctx || !logits || !cu_draft || !n_accept || !bonus || !scratch || (!drafts && n_rows > n_branch)) {
    set_error("lr_accept_greedy: null argument");
    return LR_EINVAL;
  }
  if (n_branch < 0 || n_rows < n_branch) {
    set_error("lr_accept_greedy: n_rows %d < n_branch %d", n_rows, n_branch);
    return LR_EINVAL;
  }
  if (((uintptr_t)logits & 15) != 0 || (stride & 7) != 0 || stride < ctx->model.vocab || ((uintptr_t)scratch & 7) != 0) {
    set_error("lr_accept_greedy: logits must be 16-byte aligned with a row stride that is a multiple of 8 and >= vocab");
    return LR_EINVAL;
  }
  if (n_branch == 0) return LR_OK;
  return launch_accept(ctx, logits, stride, drafts, cu_draft, n_branch, n_rows, n_accept, bonus, row_argmax, scratch,
                       reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int lr_accept_greedy_static(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts,
                                       const int32_t *cu_draft, int32_t n_branch, int32_t n_rows, int32_t *n_accept,
                                       int32_t *bonus, int32_t *row_argmax, void *stream) {
  if (!ctx || !logits || !cu_draft || !n_accept || !bonus || (!drafts && n_rows > n_branch)) {
    set_error("lr_accept_greedy_static: null argument");
    return LR_EINVAL;
  }
  if (n_branch < 0 || n_rows < n_branch) {
    set_error("lr_accept_greedy_static: n_rows %d < n_branch %d", n_rows, n_branch);
    return LR_EINVAL;
  }
  if (((uintptr_t)logits & 15) != 0 || (stride & 7) != 0 || stride < ctx->model.vocab) {
    set_error("lr_accept_greedy_static: logits must be 16-byte aligned with a row stride that is a multiple of 8 and >= vocab");
    return LR_EINVAL;
  }
  if (n_branch == 0) return LR_OK;
  return launch_accept_static(ctx, logits, stride, drafts, cu_draft, n_branch, n_rows, n_accept, bonus, row_argmax,
                              reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int lr_accept_sample_scratch_bytes(const lr_ctx *ctx, int32_t n_rows, size_t *bytes_out) {
  if (!ctx || !bytes_out || n_rows < 0) {
    set_error("lr_accept_sample_scratch_bytes: bad argument");
    return LR_EINVAL;
  }
  *bytes_out = accept_sample_scratch_bytes(ctx->model.vocab, n_rows);
  return LR_OK;
}

extern "C" int lr_accept_sample(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts, const int32_t *cu_draft,
                                int32_t n_branch, int32_t n_rows, float temperature, const float *u_accept,
                                const float *u_final, int32_t *n_accept, int32_t *final_id, float *p_draft, void *scratch,
                                void *stream) {
  if (!ctx || !logits || !cu_draft || !u_final || !n_accept || !final_id || !scratch ||
      ((!drafts || !u_accept) && n_rows > n_branch)) {
    set_error("lr_accept_sample: null argument");
    return LR_EINVAL;
  }
  if (n_branch < 0 || n_rows < n_branch) {
    set_error("lr_accept_sample: n_rows %d < n_branch %d", n_rows, n_branch);
    return LR_EINVAL;
  }
  if (!(temperature > 0.f)) {
    set_error("lr_accept_sample: temperature must be positive (use lr_accept_greedy for the greedy rule)");
    return LR_EINVAL;
  }
  if (((uintptr_t)logits & 15) != 0 || (stride & 7) != 0 || stride < ctx->model.vocab || ((uintptr_t)scratch & 7) != 0) {
    set_error("lr_accept_sample: logits must be 16-byte aligned with a row stride that is a multiple of 8 and >= vocab");
    return LR_EINVAL;
  }
  if (n_branch == 0) return LR_OK;
  return launch_accept_sample(ctx, logits, stride, drafts, cu_draft, n_branch, n_rows, temperature, u_accept, u_final, n_accept,
                              final_id, p_draft, scratch, reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int lr_accept_sample_filtered_scratch_bytes(const lr_ctx *ctx, int32_t n_rows, size_t *bytes_out) {
  if (!ctx || !bytes_out || n_rows < 0) {
    set_error("lr_accept_sample_filtered_scratch_bytes: bad argument");
    return LR_EINVAL;
  }
  *bytes_out = accept_filtered_scratch_bytes(n_rows);
  return LR_OK;
}

extern "C" int lr_accept_sample_filtered(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts,
                                         const int32_t *cu_draft, int32_t n_branch, int32_t n_rows, float temperature,
                                         int32_t top_k, float top_p, const float *u_accept, const float *u_final,
                                         int32_t *n_accept, int32_t *final_id, float *p_draft, int32_t *n_kept, void *scratch,
                                         void *stream) {
  if (!ctx || !logits || !cu_draft || !u_final || !n_accept || !final_id || !scratch ||
      ((!drafts || !u_accept) && n_rows > n_branch)) {
    set_error("lr_accept_sample_filtered: null argument");
    return LR_EINVAL;
  }
  if (n_branch < 0 || n_rows < n_branch) {
    set_error("lr_accept_sample_filtered: n_rows %d < n_branch %d", n_rows, n_branch);
    return LR_EINVAL;
  }
  if (!(temperature > 0.f) || top_k < 0 || !(top_p > 0.f) || top_p > 1.f) {
    set_error("lr_accept_sample_filtered: temperature must be positive, top_k >= 0 (0 = off), top_p in (0, 1] (1 = off)");
    return LR_EINVAL;
  }
  if (((uintptr_t)logits & 15) != 0 || (stride & 7) != 0 || stride < ctx->model.vocab || ((uintptr_t)scratch & 7) != 0) {
    set_error("lr_accept_sample_filtered: logits must be 16-byte aligned with a row stride that is a multiple of 8 and >= vocab");
    return LR_EINVAL;
  }
  if (n_branch == 0) return LR_OK;
  return launch_accept_filtered(ctx, logits, stride, drafts, cu_draft, n_branch, n_rows, temperature, top_k, top_p, u_accept,
                                u_final, n_accept, final_id, p_draft, n_kept, scratch, reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int lr_commit(lr_plan *p, const uint8_t *verdict, const int32_t *n_accept, int32_t *n_steps, int32_t *survivor,
                         int32_t *committed, int32_t *keep_off, int32_t *keep_pages, int32_t *keep_valid,
                         int32_t *free_off, int32_t *free_pages, void *stream) {
  if (!p || !n_accept || !n_steps || !survivor || !committed || !keep_off || !keep_pages || !keep_valid || !free_off ||
      !free_pages || (!verdict && p->n_verdicts > 0)) {
    set_error("lr_commit: null argument");
    return LR_EINVAL;
  }
  return launch_commit(p, verdict, n_accept, n_steps, survivor, committed, keep_off, keep_pages, keep_valid, free_off,
                       free_pages, reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int lr_compact_scratch_bytes(const lr_plan *p, size_t *bytes_out) {
  if (!p || !bytes_out) {
    set_error("lr_compact_scratch_bytes: null argument");
    return LR_EINVAL;
  }
  *bytes_out = p->compact.bytes;
  return LR_OK;
}

extern "C" int lr_compact(lr_plan *p, const int32_t *keep_off, const int32_t *keep_pages, const int32_t *keep_valid, void *k_pool,
                          void *v_pool, int32_t *new_len, int32_t *n_pages_kept, void *scratch, void *stream) {
  if (!p || !keep_off || !keep_pages || !keep_valid || !k_pool || !v_pool || !new_len || !n_pages_kept || !scratch) {
    set_error("lr_compact: null argument");
    return LR_EINVAL;
  }
  if ((((uintptr_t)k_pool | (uintptr_t)v_pool) & 15) != 0 || ((uintptr_t)scratch & 255) != 0) {
    set_error("lr_compact: pools must be 16-byte aligned and the scratch 256-byte aligned");
    return LR_EINVAL;
  }
  return launch_compact(p, keep_off, keep_pages, keep_valid, k_pool, v_pool, new_len, n_pages_kept, scratch,
                        reinterpret_cast<cudaStream_t>(stream));
}

// ---- status --------------------------------------------------------------------
extern "C" int lr_poll_status(lr_plan *p, void *stream, int32_t *detail) {
  if (!p) {
    set_error("lr_poll_status: null plan");
    return LR_EINVAL;
  }
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int32_t st[2] = {0, 0};
  cudaError_t e = cudaMemcpyAsync(st, p->dev.status, sizeof(st), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(e, "lr_poll_status");
  if (detail) *detail = st[1];
  if (st[0] == kDevOk) return LR_OK;
  e = cudaMemsetAsync(p->dev.status, 0, sizeof(st), s);
  if (e != cudaSuccess) return cuda_fail(e, "lr_poll_status clear");
  if (st[0] == kDevTimeout) {
    set_error("device wait expired (detail %d)", st[1]);
    return LR_ETIMEOUT;
  }
  set_error("device bounds check failed (detail %d)", st[1]);
  return LR_EBOUNDS;
}

// ---- whole pass from host buffers --------------------------------------------------
namespace {
struct Staging {
  size_t q, logits, drafts, verdict, out, n_accept, bonus, n_steps, survivor, committed, keep_off, free_off, keep_pages,
      keep_valid, free_pages, scratch, total;
};
Staging staging_layout(const lr_plan *p) {
  Staging s;
  size_t off = 0;
  auto take = [&](size_t n) {
    size_t o = off;
    off = align_up(off + n, 256);
    return o;
  };
  const DevBatch &d = p->dev;
  const size_t qo = (size_t)d.n_q_rows * d.n_q_heads * d.head_dim * 2;
  s.q = take(qo);
  s.logits = take((size_t)p->n_rows_logits * p->ctx->model.vocab * 2 + 16);
  s.drafts = take((size_t)p->n_drafts * 4 + 4);
  s.verdict = take((size_t)p->n_verdicts + 4);
  s.out = take(qo);
  s.n_accept = take((size_t)d.n_branch * 4);
  s.bonus = take((size_t)d.n_branch * 4);
  s.n_steps = take((size_t)d.n_req * 4);
  s.survivor = take((size_t)d.n_req * 4);
  s.committed = take((size_t)d.n_req * 4);
  s.keep_off = take((size_t)(d.n_req + 1) * 4);
  s.free_off = take((size_t)(d.n_req + 1) * 4);
  s.keep_pages = take((size_t)d.n_page_slots * 4);
  s.keep_valid = take((size_t)d.n_page_slots * 4);
  s.free_pages = take((size_t)d.n_page_slots * 4);
  s.scratch = take(8 * ((size_t)p->n_rows_logits + 1));
  s.total = off;
  return s;
}
}  // namespace

extern "C" int lr_pass_staging_bytes(const lr_plan *p, size_t *bytes_out) {
  if (!p || !bytes_out) {
    set_error("lr_pass_staging_bytes: null argument");
    return LR_EINVAL;
  }
  *bytes_out = staging_layout(p).total;
  return LR_OK;
}

extern "C" int lr_verify_pass_host(lr_plan *p, const lr_pass_host_io *io, const void *k_pool, const void *v_pool,
                                   void *staging, size_t staging_bytes, float scale, void *stream) {
  if (!p || !io || !k_pool || !v_pool || !staging) {
    set_error("lr_verify_pass_host: null argument");
    return LR_EINVAL;
  }
  if (!io->q_h || !io->logits_h || !io->out_h || !io->n_accept_h || !io->bonus_id_h || !io->n_steps_accepted_h ||
      !io->survivor_h || !io->committed_len_h || !io->keep_off_h || !io->free_off_h || !io->keep_pages_h ||
      !io->keep_valid_h || !io->free_pages_h || (!io->draft_ids_h && p->n_drafts) || (!io->verdict_h && p->n_verdicts)) {
    set_error("lr_verify_pass_host: null host buffer");
    return LR_EINVAL;
  }
  const Staging L = staging_layout(p);
  if (staging_bytes < L.total || ((uintptr_t)staging & 255) != 0) {
    set_error("lr_verify_pass_host: staging of %zu bytes (256-byte aligned) needed", L.total);
    return LR_ENOMEM;
  }
  if (p->ctx->model.vocab % 8 != 0) {
    set_error("lr_verify_pass_host: dense logits rows need vocab to be a multiple of 8");
    return LR_EUNSUPPORTED;
  }
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  unsigned char *b = reinterpret_cast<unsigned char *>(staging);
  const DevBatch &d = p->dev;
  const size_t qo = (size_t)d.n_q_rows * d.n_q_heads * d.head_dim * 2;
  const int vocab = p->ctx->model.vocab;
  cudaError_t e = cudaMemcpyAsync(b + L.q, io->q_h, qo, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(b + L.logits, io->logits_h, (size_t)p->n_rows_logits * vocab * 2, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess && p->n_drafts) e = cudaMemcpyAsync(b + L.drafts, io->draft_ids_h, (size_t)p->n_drafts * 4, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess && p->n_verdicts) e = cudaMemcpyAsync(b + L.verdict, io->verdict_h, (size_t)p->n_verdicts, cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return cuda_fail(e, "lr_verify_pass_host: host-to-device copies");
  auto I = [&](size_t off) { return reinterpret_cast<int32_t *>(b + off); };
  if (int rc = lr_verify_attention(p, b + L.q, k_pool, v_pool, b + L.out, nullptr, scale, stream)) return rc;
  if (int rc = lr_accept_greedy(p->ctx, b + L.logits, vocab, I(L.drafts), d.cu_draft, d.n_branch, p->n_rows_logits,
                                I(L.n_accept), I(L.bonus), nullptr, b + L.scratch, stream))
    return rc;
  if (int rc = lr_commit(p, b + L.verdict, I(L.n_accept), I(L.n_steps), I(L.survivor), I(L.committed), I(L.keep_off),
                         I(L.keep_pages), I(L.keep_valid), I(L.free_off), I(L.free_pages), stream))
    return rc;
  // Results: the attention output goes straight to its host buffer; the ten integer arrays lie next to one another in
  // the staging buffer and leave in one copy, through a pinned buffer the plan keeps, then to the caller's arrays.
  e = cudaMemcpyAsync(io->out_h, b + L.out, qo, cudaMemcpyDeviceToHost, s);
  if (e != cudaSuccess) return cuda_fail(e, "lr_verify_pass_host: device-to-host copy of the output");
  const size_t small_bytes = L.scratch - L.n_accept;
  if (p->results_pinned_cap < small_bytes) {
    if (p->results_pinned) cudaFreeHost(p->results_pinned);
    p->results_pinned = nullptr;
    p->results_pinned_cap = 0;
    if (int rc = cuda_fail(cudaMallocHost(&p->results_pinned, small_bytes), "cudaMallocHost(pass results)")) return rc;
    p->results_pinned_cap = small_bytes;
  }
  e = cudaMemcpyAsync(p->results_pinned, b + L.n_accept, small_bytes, cudaMemcpyDeviceToHost, s);
  if (e != cudaSuccess) return cuda_fail(e, "lr_verify_pass_host: device-to-host copy of the integer results");
  const int rc = lr_poll_status(p, stream, nullptr);  // waits for the stream
  if (rc != LR_OK && rc != LR_ETIMEOUT && rc != LR_EBOUNDS) return rc;
  struct Back { void *dst; size_t off, n; } back[] = {
      {io->n_accept_h, L.n_accept, (size_t)d.n_branch * 4},
      {io->bonus_id_h, L.bonus, (size_t)d.n_branch * 4},
      {io->n_steps_accepted_h, L.n_steps, (size_t)d.n_req * 4},
      {io->survivor_h, L.survivor, (size_t)d.n_req * 4},
      {io->committed_len_h, L.committed, (size_t)d.n_req * 4},
      {io->keep_off_h, L.keep_off, (size_t)(d.n_req + 1) * 4},
      {io->free_off_h, L.free_off, (size_t)(d.n_req + 1) * 4},
      {io->keep_pages_h, L.keep_pages, (size_t)d.n_page_slots * 4},
      {io->keep_valid_h, L.keep_valid, (size_t)d.n_page_slots * 4},
      {io->free_pages_h, L.free_pages, (size_t)d.n_page_slots * 4},
  };
  for (const Back &k : back) memcpy(k.dst, reinterpret_cast<unsigned char *>(p->results_pinned) + (k.off - L.n_accept), k.n);
  return rc;
}

extern "C" const char *lr_strerror(int st) {
  switch (st) {
    case LR_OK: return "ok";
    case LR_EINVAL: return "invalid argument";
    case LR_EUNSUPPORTED: return "unsupported shape or device";
    case LR_ECUDA: return "CUDA error";
    case LR_ETIMEOUT: return "device-side wait expired";
    case LR_EBOUNDS: return "device-side bounds check failed";
    case LR_ENOMEM: return "buffer too small or out of host memory";
    default: return "unknown status";
  }
}

extern "C" const char *lr_last_error(void) { return lr::g_err; }
