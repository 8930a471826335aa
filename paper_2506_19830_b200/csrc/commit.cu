// Step-level commit on the paged KV cache (Algorithm 1, last two lines).
//
// Integer work on a few KB of tables: latency-bound, so it is one launch with no
// inter-CTA communication.  Every CTA recomputes the per-request decisions
// (j*, decisive branch, kept tail, list sizes) and their exclusive scans in
// shared memory -- O(requests x gamma) work -- and then the warps of all CTAs
// share the page-list writes, one warp per span or branch tail.
#include "lr_common.cuh"

namespace lr {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxReq = 4096;

__device__ __forceinline__ int pages_of(int n_tok) { return (n_tok + kPage - 1) / kPage; }

// exclusive scan of a[0..n) in shared memory, in place, by one CTA; returns nothing, total in *total
__device__ void block_exclusive_scan(int32_t *a, int n, int32_t *carry_slot) {
  __shared__ int32_t warp_sum[kThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (tid == 0) *carry_slot = 0;
  __syncthreads();
  for (int base = 0; base < n; base += kThreads) {
    int i = base + tid;
    int32_t x = (i < n) ? a[i] : 0;
    int32_t inc = x;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      int32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, off);
      if (lane >= off) inc += y;
    }
    if (lane == 31) warp_sum[wid] = inc;
    __syncthreads();
    int32_t wbase = 0;
    for (int w = 0; w < wid; ++w) wbase += warp_sum[w];
    int32_t carry = *carry_slot;
    if (i < n) a[i] = carry + wbase + inc - x;
    __syncthreads();
    if (tid == kThreads - 1) *carry_slot = carry + wbase + inc;
    __syncthreads();
  }
}

__global__ void __launch_bounds__(kThreads)
commit_kernel(DevBatch d, const uint8_t *__restrict__ verdict,
              const int32_t *__restrict__ n_accept, int32_t *__restrict__ n_steps_out, int32_t *__restrict__ survivor_out,
              int32_t *__restrict__ committed_out, int32_t *__restrict__ keep_off_out, int32_t *__restrict__ keep_pages,
              int32_t *__restrict__ keep_valid, int32_t *__restrict__ free_off_out, int32_t *__restrict__ free_pages) {
  extern __shared__ int32_t sm[];
  const int R = d.n_req;
  int32_t *s_keep = sm;            // keep count -> keep offset
  int32_t *s_free = sm + R;        // free count -> free offset
  int32_t *s_a = sm + 2 * R;       // j*
  int32_t *s_surv = sm + 3 * R;    // decisive branch or -1
  __shared__ int32_t s_total[2];
  const int tid = threadIdx.x;

  // ---- per-request decisions --------------------------------------------------
  for (int r = tid; r < R; r += kThreads) {
    const int s0 = d.req_span_off[r], s1 = d.req_span_off[r + 1];
    const int gamma = s1 - s0 - 1;
    const uint8_t *v = verdict + (s0 - r);
    int a = 0;
    while (a < gamma && v[a] != 0) ++a;  // j* = first rejected step, gamma if none
    int surv = -1;
    for (int b = d.req_br_off[r]; b < d.req_br_off[r + 1]; ++b)
      if (d.br_depth[b] == a) { surv = b; break; }
    int kept_tail = 0;
    if (surv >= 0) {
      int L = d.br_n_draft[surv];
      int na = n_accept[surv];
      if (na < 0 || na > L) {  // not a value the acceptance step can produce
        na = na < 0 ? 0 : L;
        d.status[0] = kDevBounds;
        d.status[1] = 300 + 0;
      }
      kept_tail = d.br_own_len[surv] - L + na;
    }
    int keep = pages_of(kept_tail), total = 0, len = kept_tail;
    for (int c = 0; c <= gamma; ++c) {
      int pg = pages_of(d.span_len[s0 + c]);
      total += pg;
      if (c <= a) { keep += pg; len += d.span_len[s0 + c]; }
    }
    for (int b = d.req_br_off[r]; b < d.req_br_off[r + 1]; ++b) total += pages_of(d.br_own_len[b]);
    s_keep[r] = keep;
    s_free[r] = total - keep;
    s_a[r] = a;
    s_surv[r] = surv;
    if (blockIdx.x == 0) {
      n_steps_out[r] = a;
      survivor_out[r] = surv;
      committed_out[r] = len;
    }
  }
  __syncthreads();
  block_exclusive_scan(s_keep, R, &s_total[0]);
  block_exclusive_scan(s_free, R, &s_total[1]);
  if (blockIdx.x == 0) {
    for (int r = tid; r < R; r += kThreads) {
      keep_off_out[r] = s_keep[r];
      free_off_out[r] = s_free[r];
    }
    if (tid == 0) {
      keep_off_out[R] = s_total[0];
      free_off_out[R] = s_total[1];
    }
  }

  // ---- page lists: one warp per span / branch tail ---------------------------------
  const int lane = tid & 31;
  const int warps_total = gridDim.x * (kThreads / 32);
  const int n_items = d.n_span + d.n_branch;
  for (int item = blockIdx.x * (kThreads / 32) + (tid >> 5); item < n_items; item += warps_total) {
    if (item < d.n_span) {
      const int s = item, r = d.span_req[s];
      const int s0 = d.req_span_off[r], c = s - s0, a = s_a[r];
      const int len = d.span_len[s], npg = pages_of(len);
      const int32_t *src = d.page_ids + d.span_slot[s];
      if (c <= a) {
        int off = s_keep[r];
        for (int cc = 0; cc < c; ++cc) off += pages_of(d.span_len[s0 + cc]);
        for (int p = lane; p < npg; p += 32) {
          keep_pages[off + p] = src[p];
          keep_valid[off + p] = min(kPage, len - p * kPage);
        }
      } else {
        int off = s_free[r];
        for (int cc = a + 1; cc < c; ++cc) off += pages_of(d.span_len[s0 + cc]);
        for (int p = lane; p < npg; p += 32) free_pages[off + p] = src[p];
      }
    } else {
      const int b = item - d.n_span, r = d.br_req[b];
      const int s0 = d.req_span_off[r], s1 = d.req_span_off[r + 1], a = s_a[r], surv = s_surv[r];
      int kept_tail = 0, kp = 0;
      if (surv >= 0) {
        int L = d.br_n_draft[surv], na = min(max(n_accept[surv], 0), L);
        kept_tail = d.br_own_len[surv] - L + na;
        kp = pages_of(kept_tail);
      }
      const int npg = pages_of(d.br_own_len[b]);
      const int32_t *src = d.page_ids + d.br_own_slot[b];
      if (b == surv) {
        int off = s_keep[r];
        for (int c = 0; c <= a; ++c) off += pages_of(d.span_len[s0 + c]);
        for (int p = lane; p < kp; p += 32) {
          keep_pages[off + p] = src[p];
          keep_valid[off + p] = min(kPage, kept_tail - p * kPage);
        }
      }
      int off = s_free[r];
      for (int c = a + 1; c < s1 - s0; ++c) off += pages_of(d.span_len[s0 + c]);
      for (int bb = d.req_br_off[r]; bb < b; ++bb) off += pages_of(d.br_own_len[bb]) - (bb == surv ? kp : 0);
      const int skip = (b == surv) ? kp : 0;
      for (int p = skip + lane; p < npg; p += 32) free_pages[off + p - skip] = src[p];
    }
  }
}

}  // namespace

int init_commit_kernel() {
  return cuda_fail(cudaFuncSetAttribute(commit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxReq * 16),
                   "commit_kernel shared-memory attribute");
}

int launch_commit(lr_plan *p, const uint8_t *verdict, const int32_t *n_accept, int32_t *n_steps, int32_t *survivor,
                  int32_t *committed, int32_t *keep_off, int32_t *keep_pages, int32_t *keep_valid, int32_t *free_off,
                  int32_t *free_pages, cudaStream_t s) {
  const DevBatch &d = p->dev;
  if (d.n_req > kMaxReq) {
    set_error("lr_commit: more than %d requests in one pass", kMaxReq);
    return LR_EUNSUPPORTED;
  }
  int grid = (d.n_page_slots + 511) / 512;
  grid = grid < 1 ? 1 : (grid > 64 ? 64 : grid);
  size_t smem = (size_t)d.n_req * 16;
  commit_kernel<<<grid, kThreads, smem, s>>>(d, verdict, n_accept, n_steps, survivor, committed,
                                              keep_off, keep_pages, keep_valid, free_off, free_pages);
  p->ctx->launches++;
  return cuda_fail(cudaGetLastError(), "commit_kernel launch");
}

}  // namespace lr
