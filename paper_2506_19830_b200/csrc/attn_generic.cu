// CUDA-core nested-prefix attention: the path for shapes whose packed query
// count is too small to be a dense contraction (and an on-device cross-check of
// the tensor-core path).  One warp per (query row, query head); the warp walks
// the spans the row may see -- prefix, segments 1..depth, its own tail up to and
// including itself -- 32 keys at a time: each lane scores one key, the warp
// combines them with shuffle reductions into a running (max, sum) in fp32, and
// the lanes then share the value rows, each owning head_dim/32 output channels.
#include "lr_common.cuh"

namespace lr {

namespace {

constexpr int kWarps = 4;

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xFFFFFFFFu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
  return x;
}
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

template <int D>
__global__ void __launch_bounds__(kWarps * 32)
attn_generic_kernel(DevBatch d, const uint16_t *__restrict__ q, const uint16_t *__restrict__ kpool,
                    const uint16_t *__restrict__ vpool, uint16_t *__restrict__ out, float *__restrict__ lse,
                    float scale_log2) {
  constexpr int EPL = D / 32;  // output channels per lane
  __shared__ float sq[kWarps][D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t wg = (int64_t)blockIdx.x * kWarps + warp;
  if (wg >= (int64_t)d.n_q_rows * d.n_q_heads) return;
  const int row = (int)(wg / d.n_q_heads), h = (int)(wg % d.n_q_heads), kv = h / d.group;

  // branch of this row: largest b with cu_q[b] <= row
  int lo = 0, hi = d.n_branch - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (d.cu_q[mid] <= row) lo = mid; else hi = mid - 1;
  }
  const int b = lo;
  const int i = row - d.cu_q[b], q_len = d.cu_q[b + 1] - d.cu_q[b];
  const int s0 = d.req_span_off[d.br_req[b]], n_seg = d.req_span_off[d.br_req[b] + 1] - s0 - 1;
  const int node = d.span_tin[s0 + d.br_depth[b]];  // depth-first number of the node the branch continues
  const int tail_vis = d.br_own_len[b] - q_len + i + 1;  // the query sees itself

  const uint16_t *qp = q + ((int64_t)row * d.n_q_heads + h) * D;
  for (int e = lane; e < D; e += 32) sq[warp][e] = bf_lo((uint32_t)qp[e]) * scale_log2;
  __syncwarp();

  float m = -INFINITY, l = 0.f, acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;

  for (int sp = 0; sp <= n_seg + 1; ++sp) {  // prefix, the segments the node descends from (index order), tail
    if (sp <= n_seg && (node < d.span_tin[s0 + sp] || node > d.span_last[s0 + sp])) continue;
    const int slot0 = (sp <= n_seg) ? d.span_slot[s0 + sp] : d.br_own_slot[b];
    const int len = (sp <= n_seg) ? d.span_len[s0 + sp] : tail_vis;
    for (int t0 = 0; t0 < len; t0 += 32) {
      const int t = t0 + lane;
      bool valid = t < len;
      int64_t page = 0;
      if (valid) {
        page = d.page_ids[slot0 + t / kPage];
        if (page < 0 || page >= d.n_pool_pages) {  // never dereference a page outside the pool
          d.status[0] = kDevBounds;
          d.status[1] = 100;
          valid = false;
          page = 0;
        }
      }
      float s = -INFINITY;
      if (valid) {
        const uint4 *kp = reinterpret_cast<const uint4 *>(kpool + ((page * d.n_kv_heads + kv) * kPage + (t % kPage)) * D);
        float a0 = 0.f, a1 = 0.f;
#pragma unroll
        for (int c = 0; c < D / 8; ++c) {
          uint4 kk = __ldg(kp + c);
          const float *qq = &sq[warp][c * 8];
          a0 = fmaf(qq[0], bf_lo(kk.x), a0); a1 = fmaf(qq[1], bf_hi(kk.x), a1);
          a0 = fmaf(qq[2], bf_lo(kk.y), a0); a1 = fmaf(qq[3], bf_hi(kk.y), a1);
          a0 = fmaf(qq[4], bf_lo(kk.z), a0); a1 = fmaf(qq[5], bf_hi(kk.z), a1);
          a0 = fmaf(qq[6], bf_lo(kk.w), a0); a1 = fmaf(qq[7], bf_hi(kk.w), a1);
        }
        s = a0 + a1;
      }
      const float bm = warp_max(s);
      if (bm == -INFINITY) continue;  // only after a bounds failure
      const float m_new = fmaxf(m, bm);
      const float p = valid ? exp2f(s - m_new) : 0.f;
      const float corr = exp2f(m - m_new);
      l = l * corr + warp_sum(p);
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] *= corr;
      const int n = min(32, len - t0);
      for (int j = 0; j < n; ++j) {
        const float pj = __shfl_sync(0xFFFFFFFFu, p, j);
        const int64_t pg = __shfl_sync(0xFFFFFFFFu, (long long)page, j);
        const uint16_t *vp = vpool + ((pg * d.n_kv_heads + kv) * kPage + ((t0 + j) % kPage)) * D + lane * EPL;
        if (EPL == 2) {
          uint32_t vv = __ldg(reinterpret_cast<const uint32_t *>(vp));
          acc[0] = fmaf(pj, bf_lo(vv), acc[0]);
          acc[1] = fmaf(pj, bf_hi(vv), acc[1]);
        } else {
          uint2 vv = __ldg(reinterpret_cast<const uint2 *>(vp));
          acc[0] = fmaf(pj, bf_lo(vv.x), acc[0]);
          acc[1] = fmaf(pj, bf_hi(vv.x), acc[1]);
          acc[2 % EPL] = fmaf(pj, bf_lo(vv.y), acc[2 % EPL]);
          acc[3 % EPL] = fmaf(pj, bf_hi(vv.y), acc[3 % EPL]);
        }
      }
      m = m_new;
    }
  }
  const float inv = 1.f / l;
  uint16_t *op = out + ((int64_t)row * d.n_q_heads + h) * D + lane * EPL;
#pragma unroll
  for (int e = 0; e < EPL; e += 2) {
    __nv_bfloat162 o2 = __floats2bfloat162_rn(acc[e] * inv, acc[e + 1] * inv);
    *reinterpret_cast<uint32_t *>(op + e) = *reinterpret_cast<uint32_t *>(&o2);
  }
  if (lse != nullptr && lane == 0) lse[(int64_t)row * d.n_q_heads + h] = (m + log2f(l)) * 0.6931471805599453f;
}

}  // namespace

int launch_attn_generic(lr_plan *p, const void *q, const void *k, const void *v, void *out, float *lse, float scale,
                        cudaStream_t s) {
  const DevBatch &d = p->dev;
  const int64_t warps = (int64_t)d.n_q_rows * d.n_q_heads;
  const unsigned grid = (unsigned)((warps + kWarps - 1) / kWarps);
  const float scale_log2 = scale * 1.4426950408889634f;
  auto *qq = reinterpret_cast<const uint16_t *>(q);
  auto *kk = reinterpret_cast<const uint16_t *>(k);
  auto *vv = reinterpret_cast<const uint16_t *>(v);
  auto *oo = reinterpret_cast<uint16_t *>(out);
  if (d.head_dim == 64)
    attn_generic_kernel<64><<<grid, kWarps * 32, 0, s>>>(d, qq, kk, vv, oo, lse, scale_log2);
  else if (d.head_dim == 128)
    attn_generic_kernel<128><<<grid, kWarps * 32, 0, s>>>(d, qq, kk, vv, oo, lse, scale_log2);
  else {
    set_error("lr_verify_attention: head_dim %d not supported", d.head_dim);
    return LR_EUNSUPPORTED;
  }
  p->ctx->launches++;
  return cuda_fail(cudaGetLastError(), "attn_generic_kernel launch");
}

}  // namespace lr
