// Stochastic token-level acceptance (rejection sampling) for point-mass draft distributions.
//
// Two kernels.  accept_stats_kernel streams the bf16 logits once -- the HBM-bound part: grid (chunks of 8192
// logits, rows); a CTA reduces its chunk to (raw maximum M_c, S_c = sum exp((x - M_c) / T)) and stores the pair.
// accept_sample_kernel, one CTA per branch, combines the pairs of a row in chunk order into (m, Z), gets
// P_i(d_i) = exp((x_d - m) / T) / Z for the drafts, walks the acceptance chain u_i < P_i(d_i), and draws the
// final token by inverse CDF over the stop row with the rejected token removed: first over the chunk
// weights S_c exp((M_c - m) / T) (no second pass over the row), then inside the one chunk that holds the
// target, which is read again and prefix-summed.  Every reduction has a fixed order: same inputs, same output.
#include <algorithm>

#include "lr_common.cuh"

namespace lr {

namespace {

constexpr int kThreads = 256;
constexpr int kVec = 4;                       // 16-byte vectors per thread
constexpr int kChunk = kThreads * kVec * 8;   // logits per chunk
constexpr int kRowBatch = 32;                 // rows of a branch handled at a time in the chain

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
__device__ __forceinline__ float ex2_approx(float x) {  // one MUFU operation; -inf gives 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float denan(float x) { return fmaxf(x, -INFINITY); }  // NaN counts as -inf (max drops a NaN operand)

// the 32 logits of thread `tid` in chunk `c` of a row: element e = c*kChunk + (k*kThreads + tid)*8 + j for the
// striped layout (coalesced), or e = c*kChunk + tid*32 + k*8 + j for the blocked layout (contiguous per thread)
template <bool kBlocked>
__device__ __forceinline__ void load_chunk(const uint16_t *rp, int32_t vocab, int c, int tid, float (&x)[kVec * 8]) {
  const int32_t n_vec = vocab >> 3;
#pragma unroll
  for (int k = 0; k < kVec; ++k) {
    const int32_t vi = c * (kChunk / 8) + (kBlocked ? tid * kVec + k : k * kThreads + tid);
    if (vi < n_vec) {
      const uint4 v = ld_stream(reinterpret_cast<const uint4 *>(rp) + vi);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        x[k * 8 + 2 * j] = denan(bf_lo(w[j]));
        x[k * 8 + 2 * j + 1] = denan(bf_hi(w[j]));
      }
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) {  // ragged end of the row (vocab not a multiple of 8), or beyond it
        const int32_t e = vi * 8 + j;
        x[k * 8 + j] = e < vocab ? denan(bf_lo((uint32_t)rp[e])) : -INFINITY;
      }
    }
  }
}

__device__ __forceinline__ float block_reduce_max(float v, float *s_red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = s_red[0];
#pragma unroll
  for (int w = 1; w < kThreads / 32; ++w) r = fmaxf(r, s_red[w]);
  __syncthreads();
  return r;
}
__device__ __forceinline__ float block_reduce_sum(float v, float *s_red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = s_red[0];
#pragma unroll
  for (int w = 1; w < kThreads / 32; ++w) r += s_red[w];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(kThreads)
accept_stats_kernel(const uint16_t *__restrict__ logits, int64_t row_stride, int32_t vocab, float k_log2,
                    float2 *__restrict__ stats) {
  __shared__ float s_red[kThreads / 32];
  const int c = blockIdx.x, row = blockIdx.y, n_chunks = gridDim.x;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the logits may come from the kernel launched just before
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  float x[kVec * 8];
  load_chunk<false>(logits + (int64_t)row * row_stride, vocab, c, threadIdx.x, x);
  float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;  // independent chains
#pragma unroll
  for (int i = 0; i < kVec * 8; i += 4) {
    m0 = fmaxf(m0, x[i]);
    m1 = fmaxf(m1, x[i + 1]);
    m2 = fmaxf(m2, x[i + 2]);
    m3 = fmaxf(m3, x[i + 3]);
  }
  const float M = block_reduce_max(fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)), s_red);
  float sum = 0.f;
  if (M > -INFINITY) {
    const float off = -M * k_log2;
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int i = 0; i < kVec * 8; i += 4) {
      a0 += ex2_approx(fmaf(x[i], k_log2, off));
      a1 += ex2_approx(fmaf(x[i + 1], k_log2, off));
      a2 += ex2_approx(fmaf(x[i + 2], k_log2, off));
      a3 += ex2_approx(fmaf(x[i + 3], k_log2, off));
    }
    sum = (a0 + a1) + (a2 + a3);
  }
  const float S = block_reduce_sum(sum, s_red);
  if (threadIdx.x == 0) stats[(int64_t)row * n_chunks + c] = make_float2(M, S);
}

__global__ void __launch_bounds__(kThreads)
accept_sample_kernel(const uint16_t *__restrict__ logits, int64_t row_stride, int32_t vocab, float k_log2,
                     const float2 *__restrict__ stats, int n_chunks, const int32_t *__restrict__ draft_ids,
                     const int32_t *__restrict__ cu_draft, const float *__restrict__ u_accept,
                     const float *__restrict__ u_final, int32_t *__restrict__ n_accept, int32_t *__restrict__ final_id,
                     float *__restrict__ p_draft) {
  extern __shared__ float2 s_st[];  // [kRowBatch][n_chunks]: the chunk pairs of a batch of rows
  __shared__ float s_red[kThreads / 32];
  __shared__ float s_m[kRowBatch], s_p[kRowBatch], s_u[kRowBatch], s_xd[kRowBatch];
  __shared__ int32_t s_tok[kRowBatch];
  __shared__ int s_n, s_stop;
  __shared__ int s_pick_chunk, s_pick_thread;
  __shared__ float s_pick_before;
  const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the statistics come from the kernel launched just before
  const int32_t d0 = cu_draft[b], L = cu_draft[b + 1] - d0, r0 = d0 + b;
  const float u_fin = u_final[b];  // fetched early: needed only after the chain
  static_assert(kRowBatch == 32, "the chain uses one lane per row of a batch");

  // ---- acceptance chain, kRowBatch rows at a time.  Everything a batch needs from global memory (the chunk
  //      pairs of its rows, the drafts, their logits, their uniforms) is fetched at once into shared memory.
  if (tid == 0) {
    s_n = L;
    s_stop = 0;
  }
  int i0 = 0;
  for (;; i0 += kRowBatch) {
    const int rows = min(kRowBatch, L + 1 - i0);
    __syncthreads();
    const float2 *src = stats + (int64_t)(r0 + i0) * n_chunks;  // consecutive rows are contiguous
    for (int idx = tid; idx < rows * n_chunks; idx += kThreads) s_st[idx] = src[idx];
    if (tid < rows) {
      const int i = i0 + tid;
      int32_t dtok = -1;
      float xd = -INFINITY, u = 2.f;  // row L has no draft: u = 2 never passes
      if (i < L) {
        dtok = draft_ids[d0 + i];
        u = u_accept[d0 + i];
        if (dtok >= 0 && dtok < vocab) xd = denan(bf_lo((uint32_t)logits[(int64_t)(r0 + i) * row_stride + dtok]));
        else dtok = -1;
      }
      s_tok[tid] = dtok;
      s_xd[tid] = xd;
      s_u[tid] = u;
    }
    __syncthreads();
    for (int k = warp; k < rows; k += kThreads / 32) {  // one warp per row combines the row's chunk pairs in order
      const float2 *st = s_st + k * n_chunks;
      float m = -INFINITY;
      for (int c = lane; c < n_chunks; c += 32) m = fmaxf(m, st[c].x);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
      float z = 0.f;
      for (int c0 = 0; c0 < n_chunks; c0 += 32) {  // chunk order: 32 at a time, butterfly inside
        const int c = c0 + lane;
        float t = 0.f;
        if (c < n_chunks) {
          const float2 v = st[c];
          if (v.y > 0.f) t = v.y * exp2f((v.x - m) * k_log2);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
        z += t;
      }
      if (lane == 0) {
        const float p = (s_tok[k] >= 0 && z > 0.f) ? exp2f((s_xd[k] - m) * k_log2) / z : 0.f;
        if (p_draft != nullptr && i0 + k < L) p_draft[d0 + i0 + k] = p;
        s_m[k] = m;
        s_p[k] = p;
      }
    }
    __syncthreads();
    if (warp == 0) {  // first rejected draft of the batch (kRowBatch == 32 rows = one per lane)
      const bool rej = lane < rows && !(s_u[lane] < s_p[lane]);  // row L has no draft: always "rejected"
      const unsigned mask = __ballot_sync(0xFFFFFFFFu, rej);
      if (lane == 0 && mask != 0u) {
        s_n = i0 + __ffs(mask) - 1;
        s_stop = 1;
      }
    }
    __syncthreads();
    if (s_stop) break;
  }
  const int n = s_n, kn = n - i0;  // the stop row is row kn of the batch in shared memory
  const float m = s_m[kn];
  const int64_t stop_row = r0 + n;
  const uint16_t *rp = logits + stop_row * row_stride;
  const int32_t dead = n < L ? s_tok[kn] : -1;  // the rejected token has weight 0 in the residual
  const float w_dead = dead >= 0 ? exp2f((s_xd[kn] - m) * k_log2) : 0.f;

  // ---- which chunk holds the target: warp 0 scans the chunk weights, 32 chunks at a time (inclusive prefix
  //      sums by shuffles, fixed order)
  if (warp == 0) {
    const float2 *st = s_st + kn * n_chunks;
    const int dead_chunk = dead >= 0 ? dead / kChunk : -1;
    auto weight = [&](int c) -> float {
      if (c >= n_chunks) return 0.f;
      const float2 v = st[c];
      float w = v.y > 0.f ? v.y * exp2f((v.x - m) * k_log2) : 0.f;
      if (c == dead_chunk) w = fmaxf(w - w_dead, 0.f);
      return w;
    };
    float total = 0.f;
    for (int c0 = 0; c0 < n_chunks; c0 += 32) {
      float t = weight(c0 + lane);
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const float y = __shfl_up_sync(0xFFFFFFFFu, t, o);
        if (lane >= o) t += y;
      }
      total += __shfl_sync(0xFFFFFFFFu, t, 31);
    }
    const float target = u_fin * total;
    float base = 0.f;
    int pick = -1, last_nonzero = 0;
    float before = 0.f;
    for (int c0 = 0; c0 < n_chunks && pick < 0; c0 += 32) {
      const float w = weight(c0 + lane);
      float t = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const float y = __shfl_up_sync(0xFFFFFFFFu, t, o);
        if (lane >= o) t += y;
      }
      const unsigned nz = __ballot_sync(0xFFFFFFFFu, w > 0.f);
      if (nz != 0u) last_nonzero = c0 + 31 - __clz(nz);
      const unsigned hit = __ballot_sync(0xFFFFFFFFu, w > 0.f && base + t > target);
      if (hit != 0u) {
        const int l = __ffs(hit) - 1;
        pick = c0 + l;
        before = base + __shfl_sync(0xFFFFFFFFu, t - w, l);
      }
      base += __shfl_sync(0xFFFFFFFFu, t, 31);
    }
    if (pick < 0) {  // rounding pushed the target past the last chunk: take the last chunk with any weight
      pick = last_nonzero;
      before = target;
    }
    if (lane == 0) {
      s_pick_chunk = pick;
      s_pick_before = target - before;  // what is still to be covered inside the chunk
    }
  }
  __syncthreads();

  // ---- inside the chunk: thread t owns 32 consecutive logits; exclusive scan of the thread sums, then a
  //      sequential walk in the one thread whose range holds the target
  const int pc = s_pick_chunk;
  const float remain = s_pick_before;
  float x[kVec * 8];
  load_chunk<true>(rp, vocab, pc, tid, x);
  float w[kVec * 8], mine = 0.f;
#pragma unroll
  for (int i = 0; i < kVec * 8; ++i) {
    const int32_t e = pc * kChunk + tid * 32 + i;
    w[i] = (e == dead || x[i] == -INFINITY) ? 0.f : exp2f((x[i] - m) * k_log2);
    mine += w[i];
  }
  float incl = mine;  // inclusive scan over the block, in thread order
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const float y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) s_red[warp] = incl;
  if (tid == 0) s_pick_thread = -1;
  __syncthreads();
  float base = 0.f;
  for (int k = 0; k < warp; ++k) base += s_red[k];
  const float before = base + incl - mine;
  const bool holds = before <= remain && before + mine > remain && mine > 0.f;
  if (holds) atomicMax(&s_pick_thread, tid);  // rounding can make two neighbours claim it: the later one decides
  __syncthreads();
  int pt = s_pick_thread;
  if (pt < 0) {  // rounding pushed the target past the end of the chunk: the last thread with any weight
    if (mine > 0.f) atomicMax(&s_pick_thread, tid);
    __syncthreads();
    pt = s_pick_thread;
  }
  if (tid == max(pt, 0)) {
    float cum = before;
    int pick = -1, last = 0;
#pragma unroll
    for (int i = 0; i < kVec * 8; ++i) {
      if (w[i] > 0.f) {
        last = i;
        if (pick < 0 && cum + w[i] > remain) pick = i;
        cum += w[i];
      }
    }
    if (pick < 0) pick = last;
    n_accept[b] = n;
    final_id[b] = pc * kChunk + tid * 32 + pick;
  }
}

}  // namespace

size_t accept_sample_scratch_bytes(int32_t vocab, int32_t n_rows) {
  const size_t n_chunks = ((size_t)vocab + kChunk - 1) / kChunk;
  return std::max<size_t>(8, (size_t)n_rows * n_chunks * sizeof(float2));
}

int launch_accept_sample(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts, const int32_t *cu_draft,
                         int32_t n_branch, int32_t n_rows, float temperature, const float *u_accept, const float *u_final,
                         int32_t *n_accept, int32_t *final_id, float *p_draft, void *scratch, cudaStream_t s) {
  const int32_t vocab = ctx->model.vocab;
  const int n_chunks = (vocab + kChunk - 1) / kChunk;
  if (n_rows > 65535) {
    set_error("lr_accept_sample: more than 65535 logits rows in one call");
    return LR_EUNSUPPORTED;
  }
  const float k_log2 = 1.4426950408889634f / temperature;
  auto *lg = reinterpret_cast<const uint16_t *>(logits);
  auto *st = reinterpret_cast<float2 *>(scratch);
  accept_stats_kernel<<<dim3((unsigned)n_chunks, (unsigned)n_rows), kThreads, 0, s>>>(lg, stride, vocab, k_log2, st);
  ctx->launches++;
  if (int rc = cuda_fail(cudaGetLastError(), "accept_stats_kernel launch")) return rc;
  const size_t smem = (size_t)kRowBatch * n_chunks * sizeof(float2);
  if (smem > 40 * 1024) {
    set_error("lr_accept_sample: vocabulary of %d entries needs %zu bytes of shared memory per branch (limit 40 KB)", vocab, smem);
    return LR_EUNSUPPORTED;
  }
  // programmatic dependent launch: the per-branch grid is set up while the streaming grid drains
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)n_branch, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, accept_sample_kernel, lg, stride, vocab, k_log2, (const float2 *)st, n_chunks, drafts,
                                     cu_draft, u_accept, u_final, n_accept, final_id, p_draft);
  ctx->launches++;
  return cuda_fail(e, "accept_sample_kernel launch");
}

}  // namespace lr
