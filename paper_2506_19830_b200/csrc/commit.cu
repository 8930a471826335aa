// Step-level commit on the paged KV cache (Algorithm 1, last two lines).
//
// Integer work on a few KB of tables: latency-bound, so it is one launch with no
// inter-CTA communication and as few dependent loads as possible.  Every CTA
// recomputes the per-request decisions (j*, decisive branch, kept tail, list
// sizes) -- one thread per request, with the verdict and depth scans unrolled in
// groups of 8 so that their loads are in flight together -- and the exclusive
// scans of the list sizes in shared memory.  The page lists are then written
// one thread per page slot: the plan holds, for every slot, the span or tail
// that owns it and prefix sums of pages per request, so a slot's place in the
// keep or free list is a handful of independent loads and adds.
#include "lr_common.cuh"

namespace lr {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxReq = LR_COMMIT_MAX_REQUESTS;
constexpr int kSmemPerReq = 7 * 4;  // bytes of shared memory per request

__device__ __forceinline__ int pages_of(int n_tok) { return (n_tok + kPage - 1) / kPage; }

// exclusive scan of a[0..n) in shared memory, in place, by one CTA; the total goes to *carry_slot
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
  int32_t *s_kp = sm + 4 * R;      // kept tail pages of the decisive branch
  int32_t *s_kt = sm + 5 * R;      // kept tail tokens
  int32_t *s_kchain = sm + 6 * R;  // pages of the kept chain spans (prefix and segments 1..j*)
  __shared__ int32_t s_total[2];
  const int tid = threadIdx.x;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // n_accept comes from the kernel launched just before
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // ---- per-request decisions --------------------------------------------------
  for (int r = tid; r < R; r += kThreads) {
    const int s0 = d.req_span_off[r], s1 = d.req_span_off[r + 1];
    const int b0 = d.req_br_off[r], b1 = d.req_br_off[r + 1];
    const int gamma = s1 - s0 - 1, base = s0 + r;
    const uint8_t *v = verdict + (s0 - r);
    int a = gamma;  // j* = first rejected step, gamma if none
    for (int c0 = 0; c0 < gamma && a == gamma; c0 += 8) {
      uint8_t w[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) w[k] = (c0 + k < gamma) ? v[c0 + k] : (uint8_t)1;
#pragma unroll
      for (int k = 7; k >= 0; --k)
        if (w[k] == 0) a = c0 + k;
    }
    int surv = -1;  // lowest-numbered branch of depth j*
    for (int i0 = b0; i0 < b1 && surv < 0; i0 += 8) {
      int dep[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) dep[k] = (i0 + k < b1) ? d.br_depth[i0 + k] : -1;
#pragma unroll
      for (int k = 7; k >= 0; --k)
        if (dep[k] == a) surv = i0 + k;
    }
    int kept_tail = 0;
    if (surv >= 0) {
      const int L = d.br_n_draft[surv], own = d.br_own_len[surv];
      int na = n_accept[surv];
      if (na < 0 || na > L) {  // not a value the acceptance step can produce
        na = na < 0 ? 0 : L;
        d.status[0] = kDevBounds;
        d.status[1] = 300;
      }
      kept_tail = own - L + na;
    }
    const int kchain = d.chain_pg[base + a + 1], chain_all = d.chain_pg[base + gamma + 1];
    const int tails_all = d.tail_pg[b0 + r + (b1 - b0)];
    const int len = d.chain_tok[base + a + 1] + kept_tail;
    const int kp = pages_of(kept_tail);
    s_keep[r] = kchain + kp;
    s_free[r] = chain_all + tails_all - kchain - kp;
    s_a[r] = a;
    s_surv[r] = surv;
    s_kp[r] = kp;
    s_kt[r] = kept_tail;
    s_kchain[r] = kchain;
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

  // ---- page lists: one thread per page slot --------------------------------------
  for (int i = blockIdx.x * kThreads + tid; i < d.n_page_slots; i += gridDim.x * kThreads) {
    const int item = d.slot_item[i];
    if (item < 0) continue;  // a slot no span refers to
    const int32_t pid = d.page_ids[i];
    if (item < d.n_span) {
      const int s = item, r = d.span_req[s];
      const int s0 = d.req_span_off[r], c = s - s0, a = s_a[r];
      const int idx = i - d.span_slot[s], before = d.chain_pg[s0 + r + c];
      if (c <= a) {
        const int dst = s_keep[r] + before + idx;
        keep_pages[dst] = pid;
        keep_valid[dst] = min(kPage, d.span_len[s] - idx * kPage);
      } else {
        free_pages[s_free[r] + before - s_kchain[r] + idx] = pid;
      }
    } else {
      const int b = item - d.n_span, r = d.br_req[b];
      const int s0 = d.req_span_off[r], s1 = d.req_span_off[r + 1], b0 = d.req_br_off[r];
      const int surv = s_surv[r], kp = s_kp[r], kchain = s_kchain[r];
      const int idx = i - d.br_own_slot[b];
      if (b == surv && idx < kp) {
        const int dst = s_keep[r] + kchain + idx;
        keep_pages[dst] = pid;
        keep_valid[dst] = min(kPage, s_kt[r] - idx * kPage);
      } else {
        const int chain_free = d.chain_pg[s0 + r + (s1 - s0)] - kchain;
        const int tails_before = d.tail_pg[b0 + r + (b - b0)];
        const int kept_before = (surv >= 0 && b >= surv) ? kp : 0;  // kept pages precede this one in tail order
        free_pages[s_free[r] + chain_free + tails_before - kept_before + idx] = pid;
      }
    }
  }
}

// Multi-branch drafting (Section 3, "Multi-Branch Drafting"): the draft steps form a tree and the kept steps are
// those of a walk from the prefix that moves, at every node, to the lowest-numbered child whose verdict is set.
// Same structure as commit_kernel; the walked nodes (at most kMaxTreeDepth, local indices below 256) are kept
// as bytes in shared memory, and a page slot finds its place from the walk of its request.
constexpr int kSmemPerReqTree = kSmemPerReq + kMaxTreeDepth;

__global__ void __launch_bounds__(kThreads)
commit_tree_kernel(DevBatch d, const uint8_t *__restrict__ verdict,
                   const int32_t *__restrict__ n_accept, int32_t *__restrict__ n_steps_out, int32_t *__restrict__ survivor_out,
                   int32_t *__restrict__ committed_out, int32_t *__restrict__ keep_off_out, int32_t *__restrict__ keep_pages,
                   int32_t *__restrict__ keep_valid, int32_t *__restrict__ free_off_out, int32_t *__restrict__ free_pages) {
  extern __shared__ int32_t sm[];
  const int R = d.n_req;
  int32_t *s_keep = sm, *s_free = sm + R, *s_a = sm + 2 * R, *s_surv = sm + 3 * R, *s_kp = sm + 4 * R, *s_kt = sm + 5 * R,
          *s_kchain = sm + 6 * R;
  uint8_t *s_walk = reinterpret_cast<uint8_t *>(sm + 7 * R);  // [R][kMaxTreeDepth]
  __shared__ int32_t s_total[2];
  const int tid = threadIdx.x;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  for (int r = tid; r < R; r += kThreads) {
    const int s0 = d.req_span_off[r], s1 = d.req_span_off[r + 1];
    const int b0 = d.req_br_off[r], b1 = d.req_br_off[r + 1];
    const int n_seg = s1 - s0 - 1, base = s0 + r;
    const uint8_t *v = verdict + (s0 - r);  // v[c - 1]: verdict of segment c
    int node = 0, a = 0, kchain = d.chain_pg[base + 1], tokens = d.chain_tok[base + 1];
    while (a < kMaxTreeDepth) {
      int next = -1;
      for (int k = d.child_off[s0 + node], k1 = d.child_off[s0 + node + 1]; k < k1 && next < 0; ++k) {
        const int c = d.child_list[k];
        if (v[c - 1] != 0) next = c;
      }
      if (next < 0) break;
      s_walk[r * kMaxTreeDepth + a++] = (uint8_t)next;
      node = next;
      kchain += d.chain_pg[base + node + 1] - d.chain_pg[base + node];
      tokens += d.chain_tok[base + node + 1] - d.chain_tok[base + node];
    }
    int surv = -1;  // lowest-numbered branch that continues the node where the walk stopped
    for (int i = b0; i < b1 && surv < 0; ++i)
      if (d.br_depth[i] == node) surv = i;
    int kept_tail = 0;
    if (surv >= 0) {
      const int L = d.br_n_draft[surv], own = d.br_own_len[surv];
      int na = n_accept[surv];
      if (na < 0 || na > L) {
        na = na < 0 ? 0 : L;
        d.status[0] = kDevBounds;
        d.status[1] = 301;
      }
      kept_tail = own - L + na;
    }
    const int chain_all = d.chain_pg[base + n_seg + 1], tails_all = d.tail_pg[b0 + r + (b1 - b0)];
    const int kp = pages_of(kept_tail);
    s_keep[r] = kchain + kp;
    s_free[r] = chain_all + tails_all - kchain - kp;
    s_a[r] = a;
    s_surv[r] = surv;
    s_kp[r] = kp;
    s_kt[r] = kept_tail;
    s_kchain[r] = kchain;
    if (blockIdx.x == 0) {
      n_steps_out[r] = a;
      survivor_out[r] = surv;
      committed_out[r] = tokens + kept_tail;
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

  for (int i = blockIdx.x * kThreads + tid; i < d.n_page_slots; i += gridDim.x * kThreads) {
    const int item = d.slot_item[i];
    if (item < 0) continue;
    const int32_t pid = d.page_ids[i];
    if (item < d.n_span) {
      const int s = item, r = d.span_req[s];
      const int s0 = d.req_span_off[r], c = s - s0, a = s_a[r], base = s0 + r;
      const int idx = i - d.span_slot[s];
      // pages of walked segments numbered below c (walked indices increase), and whether c itself was walked
      int walked_before = 0;
      bool on_walk = c == 0;
      for (int k = 0; k < a; ++k) {
        const int w = s_walk[r * kMaxTreeDepth + k];
        if (w < c) walked_before += d.chain_pg[base + w + 1] - d.chain_pg[base + w];
        on_walk |= w == c;
      }
      if (on_walk) {
        const int dst = s_keep[r] + (c == 0 ? 0 : d.chain_pg[base + 1] + walked_before) + idx;
        keep_pages[dst] = pid;
        keep_valid[dst] = min(kPage, d.span_len[s] - idx * kPage);
      } else {
        free_pages[s_free[r] + d.chain_pg[base + c] - d.chain_pg[base + 1] - walked_before + idx] = pid;
      }
    } else {
      const int b = item - d.n_span, r = d.br_req[b];
      const int s0 = d.req_span_off[r], s1 = d.req_span_off[r + 1], b0 = d.req_br_off[r];
      const int surv = s_surv[r], kp = s_kp[r], kchain = s_kchain[r];
      const int idx = i - d.br_own_slot[b];
      if (b == surv && idx < kp) {
        const int dst = s_keep[r] + kchain + idx;
        keep_pages[dst] = pid;
        keep_valid[dst] = min(kPage, s_kt[r] - idx * kPage);
      } else {
        const int chain_free = d.chain_pg[s0 + r + (s1 - s0)] - kchain;
        const int tails_before = d.tail_pg[b0 + r + (b - b0)];
        const int kept_before = (surv >= 0 && b >= surv) ? kp : 0;
        free_pages[s_free[r] + chain_free + tails_before - kept_before + idx] = pid;
      }
    }
  }
}

}  // namespace

int init_commit_kernel() {
  if (int rc = cuda_fail(cudaFuncSetAttribute(commit_tree_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              kMaxReq * kSmemPerReqTree), "commit_tree_kernel shared-memory attribute"))
    return rc;
  return cuda_fail(cudaFuncSetAttribute(commit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxReq * kSmemPerReq),
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
  // every CTA repeats the per-request phase, so few CTAs when there are many requests
  int grid = (d.n_page_slots + kThreads - 1) / kThreads;
  const int cap = d.n_req <= 64 ? 148 : (d.n_req <= 512 ? 32 : 8);
  grid = grid < 1 ? 1 : (grid > cap ? cap : grid);
  p->ctx->launches++;
  if (d.tree) {
    return cuda_fail(launch_dependent(commit_tree_kernel, dim3(grid), dim3(kThreads), (size_t)d.n_req * kSmemPerReqTree, s, d, verdict,
                                      n_accept, n_steps, survivor, committed, keep_off, keep_pages, keep_valid, free_off, free_pages),
                     "commit_tree_kernel launch");
  }
  size_t smem = (size_t)d.n_req * kSmemPerReq;
  return cuda_fail(launch_dependent(commit_kernel, dim3(grid), dim3(kThreads), smem, s, d, verdict, n_accept, n_steps, survivor, committed,
                                    keep_off, keep_pages, keep_valid, free_off, free_pages),
                   "commit_kernel launch");
}

}  // namespace lr
