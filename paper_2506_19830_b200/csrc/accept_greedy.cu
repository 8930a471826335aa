// Greedy token-level acceptance: one streaming pass over the bf16 logits.
//
// The logits are cut into equal contiguous ranges of 16-byte vectors, one per CTA
// of a fixed grid (a few CTAs per SM), whatever the row boundaries; a range that
// spans several rows is handled row segment by row segment.  Each segment is
// reduced to (max value, lowest index) and published with one 64-bit atomicMax
// on the row's key; a CTA then takes a ticket, and the one holding the last
// ticket turns the row keys into n_accept / bonus per branch and zeroes the
// scratch again.
//
// The work is bound by HBM reads: 2 bytes per logit, read once, 16-byte loads,
// eight independent loads in flight per thread.  The maximum is taken with
// packed bf16x2 max instructions on whole 16-byte vectors (about one
// instruction per logit); the index is resolved only inside the winning vector.
#include <algorithm>

#include "lr_common.cuh"

namespace lr {

namespace {

constexpr int kThreads = 256;
constexpr int kVecPerThread = 8;                          // 16-byte vectors in flight per thread
constexpr int kCtasPerSm = 4;

// Monotone map of a float (already NaN-free, -0 folded to +0) to an unsigned key.
__device__ __forceinline__ uint32_t order_key(float x) {
  uint32_t u = __float_as_uint(x == 0.0f ? 0.0f : x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ __nv_bfloat162 as_bf2(uint32_t u) {
  __nv_bfloat162 r;
  *reinterpret_cast<uint32_t *>(&r) = u;
  return r;
}

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// NaN counts as -inf.
__device__ __forceinline__ float denan(float x) { return (x != x) ? -INFINITY : x; }

// max over the 8 bf16 of a vector; NaNs are ignored by the packed max (an all-NaN
// vector gives NaN, which then fails every "greater than" test).
__device__ __forceinline__ float vec_max(const uint4 &v) {
  __nv_bfloat162 a = __hmax2(as_bf2(v.x), as_bf2(v.y));
  __nv_bfloat162 b = __hmax2(as_bf2(v.z), as_bf2(v.w));
  a = __hmax2(a, b);
  uint32_t u = *reinterpret_cast<uint32_t *>(&a);
  return fmaxf(bf_lo(u), bf_hi(u));
}

// index (0..7) of the first element of v equal to x (x is the vector's max, not NaN)
__device__ __forceinline__ int first_equal(const uint4 &v, float x) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  int idx = 7;
#pragma unroll
  for (int i = 3; i >= 0; --i) {
    if (bf_hi(w[i]) == x) idx = 2 * i + 1;
    if (bf_lo(w[i]) == x) idx = 2 * i;
  }
  return idx;
}

struct Best {
  float v;
  int32_t i;
};

__device__ __forceinline__ Best better(Best a, Best b) {
  // higher value wins; equal values: lower index wins
  if (b.v > a.v || (b.v == a.v && b.i < a.i)) return b;
  return a;
}

__global__ void __launch_bounds__(kThreads)
accept_greedy_kernel(const uint16_t *__restrict__ logits, int64_t row_stride, int32_t vocab,
                     const int32_t *__restrict__ draft_ids, const int32_t *__restrict__ cu_draft, int32_t n_branch,
                     int32_t n_rows, int32_t *__restrict__ n_accept, int32_t *__restrict__ bonus_id,
                     int32_t *__restrict__ row_argmax, unsigned long long *scratch) {
  unsigned int *counter = reinterpret_cast<unsigned int *>(scratch);
  unsigned long long *row_key = scratch + 1;
  const int tid = threadIdx.x;
  const int32_t n_vec = vocab >> 3;  // whole 16-byte vectors in a row
  // A row is n_vec vector units plus one unit for its ragged end (vocab not a multiple of 8).
  const int64_t upr = (int64_t)n_vec + 1, total = upr * n_rows;
  const int64_t per = (total + gridDim.x - 1) / gridDim.x;
  int64_t pos = (int64_t)blockIdx.x * per;
  const int64_t end = min(total, pos + per);
  __shared__ float s_v[kThreads / 32];
  __shared__ int32_t s_i[kThreads / 32];
  __shared__ int s_last;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the logits may come from the kernel launched just before
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // lr_commit's grid may be set up meanwhile

  while (pos < end) {
    const int row = (int)(pos / upr);
    const int32_t u0 = (int32_t)(pos - (int64_t)row * upr);
    const int32_t u1 = (int32_t)min(upr, (int64_t)u0 + (end - pos));
    const int32_t v_end = min(u1, n_vec);
    const uint16_t *rp = logits + (int64_t)row * row_stride;
    const uint4 *vp = reinterpret_cast<const uint4 *>(rp);
    // Per thread: vectors are visited in increasing index order and only a strictly
    // greater maximum replaces the current one, so the earliest maximum is kept.
    Best best;
    best.v = -INFINITY;
    best.i = 0x7FFFFFFF;  // "owns no element": loses every tie
    uint4 bv = make_uint4(0, 0, 0, 0);
    int32_t bvi = -1;
    for (int32_t base = u0; base < v_end; base += kThreads * kVecPerThread) {
      uint4 v[kVecPerThread];
#pragma unroll
      for (int k = 0; k < kVecPerThread; ++k) {
        const int32_t vi = base + k * kThreads + tid;
        if (vi < v_end) v[k] = ld_stream(vp + vi);
      }
#pragma unroll
      for (int k = 0; k < kVecPerThread; ++k) {
        const int32_t vi = base + k * kThreads + tid;
        if (vi < v_end) {
          const float m = denan(vec_max(v[k]));
          if (m > best.v || bvi < 0) {
            best.v = m;
            bv = v[k];
            bvi = vi;
          }
        }
      }
    }
    // a maximum of -inf means every element is -inf or NaN: the first one wins
    if (bvi >= 0) best.i = bvi * 8 + (best.v == -INFINITY ? 0 : first_equal(bv, best.v));
    // ragged end of the row: up to 7 single elements
    if (u1 == (int32_t)upr) {
      const int32_t e = n_vec * 8 + tid;
      if (e < vocab) {
        Best t;
        t.v = denan(bf_lo((uint32_t)rp[e]));
        t.i = e;
        best = better(best, t);
      }
    }
    // warp, then block reduction
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      Best o;
      o.v = __shfl_down_sync(0xFFFFFFFFu, best.v, off);
      o.i = __shfl_down_sync(0xFFFFFFFFu, best.i, off);
      best = better(best, o);
    }
    if ((tid & 31) == 0) {
      s_v[tid >> 5] = best.v;
      s_i[tid >> 5] = best.i;
    }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < kThreads / 32; ++w) {
        Best o;
        o.v = s_v[w];
        o.i = s_i[w];
        best = better(best, o);
      }
      if (best.i != 0x7FFFFFFF) {
        unsigned long long key =
            ((unsigned long long)order_key(best.v) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)best.i);
        atomicMax(row_key + row, key);
      }
    }
    __syncthreads();
    pos += u1 - u0;
  }
  if (tid == 0) {
    __threadfence();
    unsigned int t = atomicAdd(counter, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;

  // ---- last CTA: per-branch longest matching prefix + bonus ------------------
  __threadfence();
  volatile unsigned long long *vk = row_key;
  // One thread per branch, so that hundreds of branches cost one pass: the bounds of its draft range with two loads in
  // flight, then its rows eight at a time -- keys and drafts of a chunk are loaded together, so a chunk costs one
  // round trip to L2 whatever the branch count -- and the scan stops at the first mismatch.
  for (int b = tid; b < n_branch; b += kThreads) {
    const int32_t d0 = cu_draft[b], L = cu_draft[b + 1] - d0;
    const int32_t r0 = d0 + b;
    int32_t n = L, bonus = 0;
    bool found = false;
    for (int32_t i0 = 0; i0 <= L && !found; i0 += 8) {
      int32_t t[8], dr[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int32_t i = i0 + k;
        t[k] = 0;
        dr[k] = -1;
        if (i <= L) t[k] = (int32_t)(0xFFFFFFFFu - (uint32_t)(vk[r0 + i] & 0xFFFFFFFFull));
        if (i < L) dr[k] = draft_ids[d0 + i];
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int32_t i = i0 + k;
        // row L has no draft: the scan always stops there
        if (!found && i <= L && (i == L || dr[k] != t[k])) {
          found = true;
          n = i;
          bonus = t[k];
        }
      }
    }
    n_accept[b] = n;
    bonus_id[b] = bonus;
  }
  if (row_argmax != nullptr)
    for (int r = tid; r < n_rows; r += kThreads)
      row_argmax[r] = (int32_t)(0xFFFFFFFFu - (uint32_t)(vk[r] & 0xFFFFFFFFull));
  __syncthreads();
  for (int r = tid; r < n_rows; r += kThreads) row_key[r] = 0ull;
  if (tid == 0) *counter = 0u;
}

// Scratch of lr_accept_greedy_static: row keys + ticket counter for up to LR_ACCEPT_STATIC_MAX_ROWS rows.
// Lives in every context that loads the library, for the life of the process.
static __device__ __align__(256) unsigned long long g_static_scratch[LR_ACCEPT_STATIC_MAX_ROWS + 1];

}  // namespace

// Device address of g_static_scratch per device ordinal, resolved on the first call for that device.
static void *g_static_scratch_addr[64] = {nullptr};

int launch_accept_static(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts, const int32_t *cu_draft,
                         int32_t n_branch, int32_t n_rows, int32_t *n_accept, int32_t *bonus, int32_t *row_argmax,
                         cudaStream_t s) {
  if (n_rows > LR_ACCEPT_STATIC_MAX_ROWS) {
    set_error("lr_accept_greedy_static: %d logits rows, the built-in scratch holds at most %d; use lr_accept_greedy",
              n_rows, LR_ACCEPT_STATIC_MAX_ROWS);
    return LR_EINVAL;
  }
  if (ctx->device < 0 || ctx->device >= 64) {
    set_error("lr_accept_greedy_static: device ordinal %d not supported", ctx->device);
    return LR_EUNSUPPORTED;
  }
  // ctx's device is made current for the symbol look-up and the launch; the caller's own choice is put back afterwards
  int prev_device = -1;
  if (int rc = cuda_fail(cudaGetDevice(&prev_device), "cudaGetDevice")) return rc;
  if (prev_device != ctx->device)
    if (int rc = cuda_fail(cudaSetDevice(ctx->device), "cudaSetDevice")) return rc;
  int rc = LR_OK;
  void *ptr = g_static_scratch_addr[ctx->device];
  if (ptr == nullptr) {
    // In host code the array's name is only a handle; the kernel needs the address the symbol has
    // on *this* device.  Done once per device, with that device current.  The cache is written without a
    // lock (every writer stores the same value); the first call per device should still come from one thread.
    rc = cuda_fail(cudaGetSymbolAddress(&ptr, g_static_scratch), "cudaGetSymbolAddress(static scratch)");
    if (rc == LR_OK) g_static_scratch_addr[ctx->device] = ptr;
  }
  // Every call shares the array and it keeps what the last call left: start from zero regardless.
  if (rc == LR_OK) rc = cuda_fail(cudaMemsetAsync(ptr, 0, 8 * ((size_t)n_rows + 1), s), "cudaMemsetAsync(static scratch)");
  if (rc == LR_OK) rc = launch_accept(ctx, logits, stride, drafts, cu_draft, n_branch, n_rows, n_accept, bonus, row_argmax, ptr, s);
  if (prev_device != ctx->device) {
    const cudaError_t e = cudaSetDevice(prev_device);
    if (rc == LR_OK) rc = cuda_fail(e, "cudaSetDevice(restore)");
  }
  return rc;
}

int launch_accept(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts, const int32_t *cu_draft,
                  int32_t n_branch, int32_t n_rows, int32_t *n_accept, int32_t *bonus, int32_t *row_argmax,
                  void *scratch, cudaStream_t s) {
  const int32_t vocab = ctx->model.vocab;
  // equal ranges of at least one full round of loads per CTA, at most kCtasPerSm CTAs per SM
  const int64_t total = ((int64_t)(vocab >> 3) + 1) * n_rows;
  int64_t grid = (total + kThreads * kVecPerThread - 1) / (kThreads * kVecPerThread);
  grid = std::max<int64_t>(1, std::min<int64_t>(grid, (int64_t)ctx->sm_count * kCtasPerSm));
  accept_greedy_kernel<<<(unsigned)grid, kThreads, 0, s>>>(reinterpret_cast<const uint16_t *>(logits), stride, vocab, drafts,
                                                            cu_draft, n_branch, n_rows, n_accept, bonus, row_argmax,
                                                            reinterpret_cast<unsigned long long *>(scratch));
  ctx->launches++;
  return cuda_fail(cudaGetLastError(), "accept_greedy_kernel launch");
}

}  // namespace lr
