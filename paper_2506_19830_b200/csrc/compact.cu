// Compaction of the committed KV after lr_commit: token k of a request's committed sequence goes to slot
// k % 16 of its kept page number k / 16.
//
// The moves are in place in the caller's pools and overlap (a page is both a source and a destination), so
// they go through a staging area in two stream-ordered phases: every displaced token is first copied out
// (gather), then copied to its place (scatter).  Tokens in front of the first partly filled page of a request
// stay where they are.  Three small kernels:
//   compact_scan_kernel     one CTA per request: exclusive scan of the valid counts of its kept pages
//                           (token offset of every page), the new length, the first displaced page;
//   compact_move_kernel<0>  a fixed grid over the displaced pages: tokens -> staging[token index]      (gather);
//   compact_move_kernel<1>  the same walk: staging -> destination page and slot                      (scatter).
// Bytes moved: 2 (K, V) x H_kv x D x 2 B per displaced token, read and written twice; the work is bound by
// the latency of three dependent launches, not by bandwidth.
#include <algorithm>

#include "lr_common.cuh"

namespace lr {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxReq = LR_COMPACT_MAX_REQUESTS;  // the move kernels keep one prefix sum per request in shared memory

__global__ void __launch_bounds__(kThreads)
compact_scan_kernel(const int32_t *__restrict__ keep_off, const int32_t *__restrict__ keep_valid, int32_t *__restrict__ tok_off,
                    int32_t *__restrict__ first_moved, int32_t *__restrict__ new_len, int32_t *__restrict__ n_pages_kept) {
  __shared__ int32_t warp_sum[kThreads / 32];
  __shared__ int32_t s_carry, s_first;
  const int r = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the keep list comes from the kernel launched just before
  const int i0 = keep_off[r], i1 = keep_off[r + 1];
  if (tid == 0) {
    s_carry = 0;
    s_first = i1;  // "no page is displaced"
  }
  __syncthreads();
  for (int base = i0; base < i1; base += kThreads) {
    const int i = base + tid;
    const int32_t x = i < i1 ? keep_valid[i] : 0;
    int32_t inc = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
      if (lane >= o) inc += y;
    }
    if (lane == 31) warp_sum[wid] = inc;
    __syncthreads();
    int32_t wbase = 0;
    for (int w = 0; w < wid; ++w) wbase += warp_sum[w];
    const int32_t carry = s_carry;
    const int32_t off = carry + wbase + inc - x;  // tokens of the request in front of page i
    if (i < i1) {
      tok_off[i] = off;
      if (off != (i - i0) * kPage) atomicMin(&s_first, i);  // displaced: an earlier page was not full
    }
    __syncthreads();
    if (tid == kThreads - 1) s_carry = carry + wbase + inc;
    __syncthreads();
  }
  if (tid == 0) {
    first_moved[r] = s_first;
    new_len[r] = s_carry;
    n_pages_kept[r] = (s_carry + kPage - 1) / kPage;
  }
}

// kScatter = false: pools -> staging; true: staging -> pools.  A fixed grid walks the displaced entries of the keep
// lists only: request r has keep_off[r+1] - first_moved[r] of them (none when nothing of it moves); every CTA builds
// the prefix sums of those counts in shared memory and takes the work items blockIdx.x, blockIdx.x + gridDim.x, ...
template <bool kScatter>
__global__ void __launch_bounds__(kThreads)
compact_move_kernel(DevBatch d, const int32_t *__restrict__ keep_off, const int32_t *__restrict__ keep_pages,
                    const int32_t *__restrict__ keep_valid, const int32_t *__restrict__ tok_off,
                    const int32_t *__restrict__ first_moved, const int32_t *__restrict__ stage_off, uint4 *__restrict__ k_pool,
                    uint4 *__restrict__ v_pool, uint4 *__restrict__ staging) {
  extern __shared__ int32_t s_off[];  // [n_req + 1] displaced entries in front of request r
  __shared__ int32_t warp_sum[kThreads / 32];
  __shared__ int32_t s_carry;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tid == 0) s_carry = 0;
  __syncthreads();
  for (int base = 0; base < d.n_req; base += kThreads) {
    const int r = base + tid;
    const int32_t x = r < d.n_req ? min(d.n_page_slots, max(0, keep_off[r + 1] - first_moved[r])) : 0;
    int32_t inc = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
      if (lane >= o) inc += y;
    }
    if (lane == 31) warp_sum[wid] = inc;
    __syncthreads();
    int32_t wbase = 0;
    for (int w = 0; w < wid; ++w) wbase += warp_sum[w];
    const int32_t carry = s_carry;
    if (r < d.n_req) s_off[r] = carry + wbase + inc - x;
    __syncthreads();
    if (tid == kThreads - 1) s_carry = carry + wbase + inc;
    __syncthreads();
  }
  const int32_t total = s_carry;
  if (tid == 0) s_off[d.n_req] = total;
  __syncthreads();
  const int vec_per_row = d.head_dim / 8;          // 16-byte vectors per (token, head)
  const int per_tok = d.n_kv_heads * vec_per_row;  // per pool
  // a work item is one KV head of one displaced page (8 KB of K and V): enough items to spread a few hundred pages
  for (int64_t item = blockIdx.x; item < (int64_t)total * d.n_kv_heads; item += gridDim.x) {
    const int32_t w = (int32_t)(item / d.n_kv_heads);
    const int h = (int)(item - (int64_t)w * d.n_kv_heads);
    int lo = 0, hi = d.n_req - 1;  // request of page w: largest r with s_off[r] <= w (requests without items are skipped)
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (s_off[mid] <= w) lo = mid; else hi = mid - 1;
    }
    const int r = lo;
    const int f = first_moved[r], i = f + (w - s_off[r]);
    if (f < 0 || i < 0 || i >= d.n_page_slots) {  // keep lists that do not come from lr_commit
      if (tid == 0) {
        d.status[0] = kDevBounds;
        d.status[1] = 402;
      }
      continue;
    }
    const int valid = keep_valid[i];
    const int64_t src_page = keep_pages[i];
    const int m0 = tok_off[i] - tok_off[f];  // index among the request's displaced tokens
    if (src_page < 0 || src_page >= d.n_pool_pages || valid < 0 || valid > kPage ||
        m0 + valid > stage_off[r + 1] - stage_off[r]) {  // never touch memory outside the pools or the staging area
      if (tid == 0) {
        d.status[0] = kDevBounds;
        d.status[1] = 400;
      }
      continue;
    }
    const int i0 = keep_off[r];
    const int k0 = tok_off[i];  // committed-sequence index of the page's first token
    for (int idx = tid; idx < valid * vec_per_row; idx += kThreads) {
      const int t = idx / vec_per_row, c = idx - t * vec_per_row, rem = h * vec_per_row + c;
      const int64_t s_idx = ((int64_t)(stage_off[r] + m0 + t) * 2) * per_tok + rem;  // [token][K, V][head][vector]
      if (!kScatter) {
        const int64_t src = ((src_page * d.n_kv_heads + h) * kPage + t) * vec_per_row + c;
        staging[s_idx] = k_pool[src];
        staging[s_idx + per_tok] = v_pool[src];
      } else {
        const int k = k0 + t;
        const int64_t dst_page = keep_pages[i0 + k / kPage];
        if (dst_page < 0 || dst_page >= d.n_pool_pages) {
          d.status[0] = kDevBounds;
          d.status[1] = 401;
          continue;
        }
        const int64_t dst = ((dst_page * d.n_kv_heads + h) * kPage + (k % kPage)) * vec_per_row + c;
        k_pool[dst] = staging[s_idx];
        v_pool[dst] = staging[s_idx + per_tok];
      }
    }
  }
}

}  // namespace

int launch_compact(lr_plan *p, const int32_t *keep_off, const int32_t *keep_pages, const int32_t *keep_valid, void *k_pool,
                   void *v_pool, int32_t *new_len, int32_t *n_pages_kept, void *scratch, cudaStream_t s) {
  const DevBatch &d = p->dev;
  unsigned char *base = reinterpret_cast<unsigned char *>(scratch);
  int32_t *tok_off = reinterpret_cast<int32_t *>(base + p->compact.o_tok_off);
  int32_t *first_moved = reinterpret_cast<int32_t *>(base + p->compact.o_first_moved);
  const int32_t *stage_off = d.compact_stage_off;  // per-request offsets into the staging area, fixed by the batch
  uint4 *staging = reinterpret_cast<uint4 *>(base + p->compact.o_staging);
  if (d.n_req > kMaxReq) {
    set_error("lr_compact: more than %d requests in one pass", kMaxReq);
    return LR_EUNSUPPORTED;
  }
  compact_scan_kernel<<<d.n_req, kThreads, 0, s>>>(keep_off, keep_valid, tok_off, first_moved, new_len, n_pages_kept);
  p->ctx->launches++;
  if (int rc = cuda_fail(cudaGetLastError(), "compact_scan_kernel launch")) return rc;
  const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((int64_t)d.n_page_slots * d.n_kv_heads, p->ctx->sm_count * 4));
  const size_t smem = sizeof(int32_t) * ((size_t)d.n_req + 1);
  compact_move_kernel<false><<<grid, kThreads, smem, s>>>(d, keep_off, keep_pages, keep_valid, tok_off, first_moved, stage_off,
                                                      reinterpret_cast<uint4 *>(k_pool), reinterpret_cast<uint4 *>(v_pool), staging);
  p->ctx->launches++;
  if (int rc = cuda_fail(cudaGetLastError(), "compact gather launch")) return rc;
  compact_move_kernel<true><<<grid, kThreads, smem, s>>>(d, keep_off, keep_pages, keep_valid, tok_off, first_moved, stage_off,
                                                     reinterpret_cast<uint4 *>(k_pool), reinterpret_cast<uint4 *>(v_pool), staging);
  p->ctx->launches++;
  return cuda_fail(cudaGetLastError(), "compact scatter launch");
}

}  // namespace lr
