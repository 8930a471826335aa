// Tensor-core nested-prefix attention for sm_100a (head_dim 128).
//
// Work decomposition.  For one request the *extended chain* is the list of its
// KV pages in the order prefix, segments 1..gamma, branch tails; 8 consecutive
// pages form a 128-key tile.  All query rows of the request that share one KV
// head -- (query token, head-in-group) pairs, floor(128/G) tokens per 128-row
// M-tile -- are processed against a tile at once, so a KV page is fetched from
// HBM once for every branch and every GQA head that can see it.  A *group* is
// (request, KV head, pair of M-tiles); the tiles of all groups, weighted, are
// cut into equal contiguous ranges, one per CTA (one CTA per SM).  A range may
// cover parts of several groups (*pieces*).  A piece that is a whole group
// writes bf16 output directly; otherwise it writes an fp32 partial (running
// max, sum, unnormalised O) and a small second kernel merges the partials of a
// group in a fixed order.
//
// One CTA = 10 warps:
//   warp 0      TMA producer: per tile 16 + 16 bulk tensor copies (one per page
//               and 64-channel half, K then V) into a 4-stage ring of 32 KB
//               buffers in the 128-byte-swizzled layout the MMA descriptors read.
//   warp 1      MMA issuer: tcgen05.mma (M=128, N=128, K=16, bf16 -> fp32) for
//               S = Q K^T (both operands in shared memory) and O += P V (P read
//               from tensor memory, V from shared memory as the N-major operand).
//   warps 2-5   softmax of M-tile 0, one thread per query row (tcgen05.ld gives
//   warps 6-9   softmax of M-tile 1  a thread its whole row, so row max and row
//               sum need no cross-lane traffic): visibility masks, running max
//               with lazy rescaling of O in tensor memory, exp2, bf16 P written
//               back over S.
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each; P_m
// occupies the first 64 columns of S_m.
//
// Visibility.  Tiles made only of full prefix pages need no mask.  In every other
// tile each page carries (valid tokens, minimum depth, owning branch, tail
// offset) and every row carries (depth, branch, causal limit): a row sees the
// first n_ok tokens of a page, with n_ok from those six numbers.  V rows of
// invalid token slots are zeroed in shared memory before the PV product so that
// whatever the slack holds (NaN included) cannot reach the output.
//
// Every wait on an mbarrier is bounded; when one expires the CTA raises its abort
// flag, records LR_ETIMEOUT in the status word, drains what it has in flight,
// frees its tensor memory and returns.
#include <cuda.h>

#include "lr_common.cuh"

namespace lr {

namespace {

constexpr int kD = 128;
constexpr int kStages = 4;
constexpr int kTileBytes = 32768;  // [2 halves of 64 channels][128 keys or rows][128 B]
constexpr int kHalfBytes = 16384;
constexpr int kThreads = 320;
constexpr int kPagesPerTile = 8;
constexpr uint64_t kWaitLimitNs = 1000ull * 1000ull * 1000ull;  // one second per wait, measured on the global timer
constexpr uint64_t kDrainLimitNs = 50ull * 1000ull * 1000ull;
constexpr float kRescaleThreshold = 8.0f;  // log2 units: P stays below 2^8

struct __align__(8) Ctrl {
  uint64_t kv_full[kStages], kv_empty[kStages];
  uint64_t s_full[2], p_full[2], o_done[2];
  uint64_t q_full[2], piece_done[2], drain;
  uint32_t tmem_base;
  int abort_flag;
};
constexpr int kSmemBytes = 1024 + 2 * kTileBytes + kStages * kTileBytes + 1024;

// ---- PTX wrappers ----------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(20000u)  // suspend for at most 20 us per try
      : "memory");
  return ok;
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 2-D tiled bulk tensor copy global -> shared, completion on an mbarrier (no multicast).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: D fp32, A and B bf16, M = 128, N = 128; bit 16 selects an N-major B operand.
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | (16u << 17) | (8u << 24);
constexpr uint32_t kIdescPV = kIdescQK | (1u << 16);

__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  tc_wait_ld();
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
      "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
      "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
      "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
      "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
      "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
      "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
      "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&t);
}

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait: gives up after kWaitLimitNs of wall time.  Returns false when the wait expired or
// another role of the CTA gave up.
__device__ __forceinline__ bool wait_bar(uint64_t *bar, uint32_t parity, Ctrl *ctrl, int32_t *status, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  for (uint32_t i = 1;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 31u) == 0u) {
      if (*reinterpret_cast<volatile int *>(&ctrl->abort_flag)) return false;
      if (global_ns() - t0 > kWaitLimitNs) break;
    }
  }
  *reinterpret_cast<volatile int *>(&ctrl->abort_flag) = 1;
  status[0] = kDevTimeout;
  status[1] = code;
  return false;
}

struct RowInfo {
  int depth;       // segments the row sees; -1 for padding rows
  int branch;      // local branch index within the request; -1 for padding rows
  int limit;       // last tail token the row sees
  int64_t q_index; // (query row * n_q_heads + head), -1 for padding rows
};

// Row r (0..127) of M-tile mt of a group: token mt*T + r/G, head kv*G + r%G.
__device__ __forceinline__ RowInfo row_info(const DevBatch &d, const TcReq &rq, int T, int mt, int r, int kv) {
  RowInfo ri;
  ri.depth = -1;
  ri.branch = -1;
  ri.limit = -1;
  ri.q_index = -1;
  const int G = d.group;
  const int tok = mt * T + r / G;
  if (r < T * G && tok < rq.n_q) {
    const int row = rq.q_row0 + tok;
    int b = rq.br0;
    while (b + 1 < rq.br0 + rq.n_br && d.cu_q[b + 1] <= row) ++b;
    const int i = row - d.cu_q[b], q_len = d.cu_q[b + 1] - d.cu_q[b];
    ri.depth = d.br_depth[b];
    ri.branch = b - rq.br0;
    ri.limit = d.br_own_len[b] - q_len + i;
    ri.q_index = (int64_t)row * d.n_q_heads + kv * G + r % G;
  }
  return ri;
}

__device__ __forceinline__ int page_n_ok(uint32_t meta, const RowInfo &ri) {
  const int valid = meta & 31, need = (meta >> 5) & 255, owner = (meta >> 13) & 255, tb = meta >> 21;
  int n;
  if (owner == 0) n = (ri.depth >= need) ? valid : 0;
  else n = (owner - 1 == ri.branch) ? min(valid, ri.limit - tb * kPage + 1) : 0;
  return max(n, 0);
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map, DevBatch d, DevTcPlan tc,
               const uint16_t *__restrict__ q, uint16_t *__restrict__ out, float *__restrict__ lse, float scale_log2) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char *q_smem = smem;                         // 2 x 32 KB
  unsigned char *kv_smem = smem + 2 * kTileBytes;       // kStages x 32 KB
  Ctrl *ctrl = reinterpret_cast<Ctrl *>(kv_smem + kStages * kTileBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&ctrl->kv_full[s], 1);
      mbar_init(&ctrl->kv_empty[s], 1);
    }
    for (int m = 0; m < 2; ++m) {
      mbar_init(&ctrl->s_full[m], 1);
      mbar_init(&ctrl->p_full[m], 128);
      mbar_init(&ctrl->o_done[m], 1);
      mbar_init(&ctrl->q_full[m], 128);
      mbar_init(&ctrl->piece_done[m], 128);
    }
    mbar_init(&ctrl->drain, 1);
    ctrl->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctrl->tmem_base)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&ctrl->tmem_base);

  const int piece0 = tc.cta_piece_off[blockIdx.x], piece1 = tc.cta_piece_off[blockIdx.x + 1];
  const int T = tc.tokens_per_mtile;

  if (warp == 0) {
    // ======================= TMA producer ==========================================
    uint32_t it = 0;
    bool ok = true;
    for (int pc = piece0; pc < piece1 && ok; ++pc) {
      const TcPiece pi = tc.pieces[pc];
      const TcReq rq = tc.reqs[pi.req];
      for (int t = pi.tile_begin; t < pi.tile_end && ok; ++t) {
        const int npages = min(kPagesPerTile, rq.n_pages - t * kPagesPerTile);
        int64_t page = 0;
        if (lane < 16 && (lane >> 1) < npages) {
          page = tc.pages[rq.page_off + t * kPagesPerTile + (lane >> 1)].page;
          if (page < 0 || page >= d.n_pool_pages) {  // never fetch outside the pool
            d.status[0] = kDevBounds;
            d.status[1] = 200;
            page = 0;
          }
        }
        for (int op = 0; op < 2 && ok; ++op, ++it) {
          const uint32_t stage = it % kStages;
          ok = wait_bar(&ctrl->kv_empty[stage], ((it / kStages) & 1u) ^ 1u, ctrl, d.status, 210);
          if (!ok) break;
          if (lane == 0) mbar_arrive_expect_tx(&ctrl->kv_full[stage], (uint32_t)npages * 4096u);
          __syncwarp();
          if (lane < 16 && (lane >> 1) < npages) {
            const uint32_t dst = smem_u32(kv_smem + stage * kTileBytes) + (lane & 1) * kHalfBytes + (lane >> 1) * 2048;
            tma_load_2d(dst, op == 0 ? &k_map : &v_map, (lane & 1) * 64, (int32_t)((page * d.n_kv_heads + pi.kv_head) * kPage),
                        &ctrl->kv_full[stage]);
          }
        }
      }
    }
    if (!ok) {
      // give the copies already in flight a bounded time to land before the CTA exits
      for (uint32_t back = 1; back <= (uint32_t)kStages && back <= it; ++back) {
        const uint32_t j = it - back;
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(&ctrl->kv_full[j % kStages], (j / kStages) & 1u))
          if (global_ns() - t0 > kDrainLimitNs) break;
      }
    }
  } else if (warp == 1) {
    // ======================= MMA issuer =============================================
    uint32_t it = 0, q_phase[2] = {0, 0}, done_phase[2] = {0, 0}, p_phase[2] = {0, 0};
    bool ok = true;
    const uint32_t q_addr = smem_u32(q_smem), kv_addr = smem_u32(kv_smem);
    auto issue_qk = [&](int m, uint32_t stage) {
      const uint32_t a = q_addr + m * kTileBytes, b = kv_addr + stage * kTileBytes;
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_ss(tmem + m * 128, make_desc(a + h * kHalfBytes + kk * 32, 16, 1024),
                 make_desc(b + h * kHalfBytes + kk * 32, 16, 1024), kIdescQK, (h | kk) != 0);
    };
    auto issue_pv = [&](int m, uint32_t stage, bool acc) {
      const uint32_t b = kv_addr + stage * kTileBytes;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
        mma_ts(tmem + 256 + m * 128, tmem + m * 128 + ks * 8, make_desc(b + ks * 2048, kHalfBytes, 1024), kIdescPV,
               acc || ks != 0);
    };
    for (int pc = piece0; pc < piece1 && ok; ++pc) {
      const TcPiece pi = tc.pieces[pc];
      const TcReq rq = tc.reqs[pi.req];
      const int n_mt = min(2, (rq.n_q + T - 1) / T - 2 * pi.mgroup);
      for (int m = 0; m < n_mt && ok; ++m) {
        ok = wait_bar(&ctrl->q_full[m], q_phase[m], ctrl, d.status, 220);
        q_phase[m] ^= 1;
      }
      if (!ok) break;
      tc_fence_after();
      uint32_t sK = it % kStages;
      ok = wait_bar(&ctrl->kv_full[sK], (it / kStages) & 1u, ctrl, d.status, 221);
      ++it;
      if (!ok) break;
      tc_fence_after();
      if (lane == 0) {
        for (int m = 0; m < n_mt; ++m) {
          issue_qk(m, sK);
          tc_commit(&ctrl->s_full[m]);
        }
        tc_commit(&ctrl->kv_empty[sK]);
      }
      __syncwarp();
      for (int t = pi.tile_begin; t < pi.tile_end && ok; ++t) {
        const uint32_t sV = it % kStages;
        ok = wait_bar(&ctrl->kv_full[sV], (it / kStages) & 1u, ctrl, d.status, 222);
        ++it;
        if (!ok) break;
        if (t >= rq.n_dense_tiles) {
          // zero the V rows of token slots that hold no valid token (slack of a last page, absent pages)
          unsigned char *vs = kv_smem + sV * kTileBytes;
          for (int p = 0; p < kPagesPerTile; ++p) {
            const int valid = tc.pages[rq.page_off + t * kPagesPerTile + p].meta & 31;
            for (int idx = lane; idx < (kPage - valid) * 16; idx += 32) {
              const int key = p * kPage + valid + (idx >> 4), h = (idx >> 3) & 1, ch = idx & 7;
              *reinterpret_cast<uint4 *>(vs + h * kHalfBytes + key * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
            }
          }
          fence_proxy_async();
          __syncwarp();
        }
        const bool has_next = t + 1 < pi.tile_end;
        if (has_next) {
          sK = it % kStages;
          ok = wait_bar(&ctrl->kv_full[sK], (it / kStages) & 1u, ctrl, d.status, 223);
          ++it;
          if (!ok) break;
        }
        tc_fence_after();
        for (int m = 0; m < n_mt && ok; ++m) {
          ok = wait_bar(&ctrl->p_full[m], p_phase[m], ctrl, d.status, 224 + m);
          p_phase[m] ^= 1;
          if (!ok) break;
          tc_fence_after();
          if (lane == 0) {
            issue_pv(m, sV, t > pi.tile_begin);
            tc_commit(&ctrl->o_done[m]);
            if (has_next) {
              issue_qk(m, sK);
              tc_commit(&ctrl->s_full[m]);
            }
          }
          __syncwarp();
        }
        if (!ok) break;
        if (lane == 0) {
          tc_commit(&ctrl->kv_empty[sV]);
          if (has_next) tc_commit(&ctrl->kv_empty[sK]);
        }
        __syncwarp();
      }
      if (!ok) break;
      for (int m = 0; m < n_mt && ok; ++m) {
        ok = wait_bar(&ctrl->piece_done[m], done_phase[m], ctrl, d.status, 228);
        done_phase[m] ^= 1;
      }
      tc_fence_after();
    }
    if (!ok && lane == 0) {
      // let every MMA already issued retire before tensor memory is released
      tc_commit(&ctrl->drain);
      const uint64_t t0 = global_ns();
      while (!mbar_try_wait(&ctrl->drain, 0))
        if (global_ns() - t0 > kDrainLimitNs) break;
    }
    __syncwarp();
  } else {
    // ======================= softmax warpgroups ======================================
    const int m = (warp - 2) >> 2;                 // M-tile within the pair
    const int quarter = warp & 3;                  // tensor-memory lane quarter this warp may access
    const int r = quarter * 32 + lane;             // row within the M-tile
    const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
    const uint32_t s_addr = lane_base + m * 128, o_addr = lane_base + 256 + m * 128;
    uint32_t s_phase = 0, o_count = 0;
    bool ok = true;
    for (int pc = piece0; pc < piece1 && ok; ++pc) {
      const TcPiece pi = tc.pieces[pc];
      const TcReq rq = tc.reqs[pi.req];
      const int n_mt = min(2, (rq.n_q + T - 1) / T - 2 * pi.mgroup);
      if (m >= n_mt) continue;  // this M-tile does not exist in the piece
      RowInfo ri = row_info(d, rq, T, 2 * pi.mgroup + m, r, pi.kv_head);
      {
        // stage this row of Q: 16 chunks of 16 B into the swizzled K-major layout
        unsigned char *qs = q_smem + m * kTileBytes;
        const uint4 *src = reinterpret_cast<const uint4 *>(q + ri.q_index * kD);
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          uint4 v = make_uint4(0, 0, 0, 0);
          if (ri.q_index >= 0) v = __ldg(src + c);
          *reinterpret_cast<uint4 *>(qs + (c >> 3) * kHalfBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = v;
        }
        fence_proxy_async();
      }
      mbar_arrive(&ctrl->q_full[m]);
      float m_used = -INFINITY, l = 0.f;
      {
        for (int t = pi.tile_begin; t < pi.tile_end; ++t) {
          ok = wait_bar(&ctrl->s_full[m], s_phase, ctrl, d.status, 230 + m);
          s_phase ^= 1;
          if (!ok) break;
          tc_fence_after();
          const bool masked = t >= rq.n_dense_tiles;
          int n_ok[kPagesPerTile];
          if (masked) {
            const uint4 *mp = reinterpret_cast<const uint4 *>(tc.pages + rq.page_off + t * kPagesPerTile);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint4 w = __ldg(mp + j);
              n_ok[2 * j] = page_n_ok(w.y, ri);
              n_ok[2 * j + 1] = page_n_ok(w.w, ri);
            }
          }
          // pass 1: row maximum
          float mx = -INFINITY;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            float v[32];
            tmem_ld32(s_addr + ch * 32, v);
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              float x = v[c];
              if (masked && (c & 15) >= n_ok[2 * ch + (c >> 4)]) x = -INFINITY;
              mx = fmaxf(mx, x);
            }
          }
          mx *= scale_log2;
          // lazy rescale: only when the maximum grew by more than the threshold
          const bool grow = mx > m_used + kRescaleThreshold;
          if (__any_sync(0xFFFFFFFFu, grow)) {
            const float alpha = grow ? ex2(m_used - mx) : 1.0f;
            if (grow) {
              l *= alpha;
              m_used = mx;
            }
            if (t > pi.tile_begin) {
#pragma unroll
              for (int ch = 0; ch < 4; ++ch) {
                float v[32];
                tmem_ld32(o_addr + ch * 32, v);
#pragma unroll
                for (int c = 0; c < 32; ++c) v[c] *= alpha;
                tmem_st32(o_addr + ch * 32, v);
              }
              tc_wait_st();
            }
          }
          const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
          // pass 2: P = exp2(scale * s - m), row sum, bf16 P over the first half of S
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            float v[32];
            tmem_ld32(s_addr + ch * 32, v);
            uint32_t pk[16];
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
              float x0 = v[c], x1 = v[c + 1];
              if (masked && (c & 15) >= n_ok[2 * ch + (c >> 4)]) x0 = -INFINITY;
              if (masked && ((c + 1) & 15) >= n_ok[2 * ch + ((c + 1) >> 4)]) x1 = -INFINITY;
              const float p0 = ex2(fmaf(x0, scale_log2, neg_m)), p1 = ex2(fmaf(x1, scale_log2, neg_m));
              l += p0 + p1;
              pk[c >> 1] = pack_bf16(p0, p1);
            }
            tmem_st16(s_addr + ch * 16, pk);
          }
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(&ctrl->p_full[m]);
        }
        if (ok) {
          // epilogue: wait for the last PV of this piece, then normalise and store
          o_count += (uint32_t)(pi.tile_end - pi.tile_begin);
          ok = wait_bar(&ctrl->o_done[m], (o_count - 1) & 1u, ctrl, d.status, 240 + m);
        }
        if (ok) {
          tc_fence_after();
          if (pi.partial_slot < 0) {
            const float inv = 1.0f / l;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              float v[32];
              tmem_ld32(o_addr + ch * 32, v);
              if (ri.q_index >= 0) {
                uint4 *dst = reinterpret_cast<uint4 *>(out + ri.q_index * kD + ch * 32);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  dst[j] = make_uint4(pack_bf16(v[8 * j] * inv, v[8 * j + 1] * inv), pack_bf16(v[8 * j + 2] * inv, v[8 * j + 3] * inv),
                                      pack_bf16(v[8 * j + 4] * inv, v[8 * j + 5] * inv), pack_bf16(v[8 * j + 6] * inv, v[8 * j + 7] * inv));
              }
            }
            if (lse != nullptr && ri.q_index >= 0) lse[ri.q_index] = (m_used + log2f(l)) * 0.6931471805599453f;
          } else {
            const int64_t prow = (int64_t)pi.partial_slot * 256 + m * 128 + r;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              float v[32];
              tmem_ld32(o_addr + ch * 32, v);
              if (ri.q_index >= 0) {
                float4 *dst = reinterpret_cast<float4 *>(tc.partial_o + prow * kD + ch * 32);
#pragma unroll
                for (int j = 0; j < 8; ++j) dst[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
              }
            }
            if (ri.q_index >= 0) *reinterpret_cast<float2 *>(tc.partial_ml + prow * 2) = make_float2(m_used, l);
          }
          tc_fence_before();
        }
      }
      mbar_arrive(&ctrl->piece_done[m]);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// Merge of the split-KV partials of one group: O = sum_j 2^(m_j - M) O_j / sum_j 2^(m_j - M) l_j.
// One warp per query row (grid: groups x 32 CTAs of 8 warps); the slots are read in a fixed order.
__global__ void __launch_bounds__(256)
attn_tc_merge_kernel(DevBatch d, DevTcPlan tc, uint16_t *__restrict__ out, float *__restrict__ lse) {
  const TcGroup g = tc.groups[blockIdx.x];
  const TcReq rq = tc.reqs[g.req];
  const int T = tc.tokens_per_mtile, G = d.group;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.y * 8 + warp;
  const int mt = 2 * g.mgroup + (row >> 7), r = row & 127;
  const int tok = mt * T + r / G;
  if (r >= T * G || tok >= rq.n_q) return;
  const int64_t qi = (int64_t)(rq.q_row0 + tok) * d.n_q_heads + g.kv_head * G + r % G;
  const int64_t prow0 = (int64_t)g.partial_begin * 256 + row;
  // lane j holds (m, l) of slot j, 32 slots at a time
  float M = -INFINITY;
  for (int j0 = 0; j0 < g.n_partial; j0 += 32) {
    const int j = j0 + lane;
    float mj = -INFINITY;
    if (j < g.n_partial) {
      const float2 ml = *reinterpret_cast<const float2 *>(tc.partial_ml + (prow0 + (int64_t)j * 256) * 2);
      mj = ml.y > 0.f ? ml.x : -INFINITY;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mj = fmaxf(mj, __shfl_xor_sync(0xFFFFFFFFu, mj, o));
    M = fmaxf(M, mj);
  }
  float L = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int j0 = 0; j0 < g.n_partial; j0 += 32) {
    const int j = j0 + lane;
    float wl = 0.f, w = 0.f;
    if (j < g.n_partial) {
      const float2 ml = *reinterpret_cast<const float2 *>(tc.partial_ml + (prow0 + (int64_t)j * 256) * 2);
      if (ml.y > 0.f) {  // a piece that saw no key of the row contributes nothing
        w = exp2f(ml.x - M);
        wl = w * ml.y;
      }
    }
    const int n = min(32, g.n_partial - j0);
#pragma unroll 4
    for (int jj = 0; jj < n; ++jj) {
      const float wj = __shfl_sync(0xFFFFFFFFu, w, jj);
      L += __shfl_sync(0xFFFFFFFFu, wl, jj);
      const float4 o = *reinterpret_cast<const float4 *>(tc.partial_o + (prow0 + (int64_t)(j0 + jj) * 256) * kD + lane * 4);
      if (wj != 0.f) {
        acc.x = fmaf(wj, o.x, acc.x);
        acc.y = fmaf(wj, o.y, acc.y);
        acc.z = fmaf(wj, o.z, acc.z);
        acc.w = fmaf(wj, o.w, acc.w);
      }
    }
  }
  const float inv = 1.0f / L;
  uint2 pk = make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
  *reinterpret_cast<uint2 *>(out + qi * kD + lane * 4) = pk;
  if (lse != nullptr && lane == 0) lse[qi] = (M + log2f(L)) * 0.6931471805599453f;
}

// ---- tensor maps -------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int get_pool_map(lr_ctx *ctx, const void *pool, int64_t n_pages, const CUtensorMap **out) {
  for (auto &e : ctx->tmaps)
    if (e.ptr == pool && e.n_pages == n_pages) {
      *out = reinterpret_cast<const CUtensorMap *>(e.map);
      return LR_OK;
    }
  if (!ctx->tmap_encode) {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
      set_error("cuTensorMapEncodeTiled is not available from the driver");
      return LR_ECUDA;
    }
    ctx->tmap_encode = fn;
  }
  if (ctx->tmaps.size() >= 256) ctx->tmaps.erase(ctx->tmaps.begin());
  ctx->tmaps.emplace_back();
  lr_ctx::TmapEntry &ent = ctx->tmaps.back();
  ent.ptr = pool;
  ent.n_pages = n_pages;
  // the pool as a 2-D tensor [rows = pages * kv heads * 16][128 channels]; a box is one page half: 16 rows x 64 channels
  cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)n_pages * ctx->model.n_kv_heads * kPage};
  cuuint64_t strides[1] = {(cuuint64_t)kD * 2};
  cuuint32_t box[2] = {64, kPage};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->tmap_encode)(
      reinterpret_cast<CUtensorMap *>(ent.map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    ctx->tmaps.pop_back();
    set_error("cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return LR_ECUDA;
  }
  *out = reinterpret_cast<const CUtensorMap *>(ent.map);
  return LR_OK;
}

}  // namespace

int init_attn_tc_kernel() {
  return cuda_fail(cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes),
                   "attn_tc_kernel shared-memory attribute");
}

// ---- host planning -----------------------------------------------------------------
int tc_build_host_plan(const lr_ctx *ctx, const lr_batch *b, const int32_t *req_br_off, TcHostPlan &out, Image &img) {
  out = TcHostPlan();
  const lr_model &m = ctx->model;
  const int G = m.n_q_heads / m.n_kv_heads;
  if (m.head_dim != kD) return LR_OK;  // other head sizes take the CUDA-core path
  const int T = 128 / G;
  std::vector<TcPage> pages;
  std::vector<TcReq> reqs((size_t)b->n_req);
  struct Grp { int req, kv, mg, n_tiles, weight; };
  std::vector<Grp> grps;
  for (int r = 0; r < b->n_req; ++r) {
    const int s0 = b->req_span_off[r], s1 = b->req_span_off[r + 1];
    const int br0 = req_br_off[r], br1 = req_br_off[r + 1];
    TcReq &rq = reqs[r];
    memset(&rq, 0, sizeof(rq));
    rq.page_off = (int)pages.size();
    rq.br0 = br0;
    rq.n_br = br1 - br0;
    if (rq.n_br == 0) continue;  // a request without branches has no query rows
    if (rq.n_br > 254) return LR_OK;
    rq.q_row0 = b->cu_q[br0];
    rq.n_q = b->cu_q[br1] - b->cu_q[br0];
    int max_depth = 0;
    for (int i = br0; i < br1; ++i) max_depth = std::max(max_depth, b->br_depth[i]);
    auto add_span = [&](int slot, int len, int need, int owner) {
      const int n = (len + kPage - 1) / kPage;
      for (int p = 0; p < n; ++p) {
        TcPage e;
        e.page = b->page_ids[slot + p];
        const uint32_t valid = (uint32_t)std::min(kPage, len - p * kPage);
        e.meta = valid | ((uint32_t)need << 5) | ((uint32_t)owner << 13) | ((uint32_t)(owner ? p : 0) << 21);
        pages.push_back(e);
      }
      return n;
    };
    for (int i = br0; i < br1; ++i)
      if ((b->br_own_len[i] + kPage - 1) / kPage > 2047) return LR_OK;
    add_span(b->span_slot[s0], b->span_len[s0], 0, 0);
    rq.n_dense_tiles = (b->span_len[s0] / kPage) / kPagesPerTile;
    for (int c = 1; c <= max_depth && s0 + c < s1; ++c) add_span(b->span_slot[s0 + c], b->span_len[s0 + c], c, 0);
    for (int i = br0; i < br1; ++i) add_span(b->br_own_slot[i], b->br_own_len[i], 0, i - br0 + 1);
    rq.n_pages = (int)pages.size() - rq.page_off;
    while (pages.size() % kPagesPerTile) pages.push_back(TcPage{0, 0});  // absent pages of the last tile: nothing valid
    const int n_tiles = (rq.n_pages + kPagesPerTile - 1) / kPagesPerTile;
    const int n_mt = (rq.n_q + T - 1) / T;
    for (int kv = 0; kv < m.n_kv_heads; ++kv)
      for (int mg = 0; mg < (n_mt + 1) / 2; ++mg) {
        const int mts = std::min(2, n_mt - 2 * mg);
        grps.push_back(Grp{r, kv, mg, n_tiles, 1 + mts});
      }
  }
  if (grps.empty()) return LR_OK;
  // Cut the weighted tile sequence into n_cta contiguous ranges of equal weight: a tile belongs to the
  // CTA whose weight interval [total*c/n, total*(c+1)/n) holds the tile's start position.
  int64_t total_w = 0, total_tiles = 0;
  for (const Grp &g : grps) {
    total_w += (int64_t)g.n_tiles * g.weight;
    total_tiles += g.n_tiles;
  }
  const int n_cta = (int)std::min<int64_t>(ctx->sm_count, std::max<int64_t>(1, total_tiles / 2));
  std::vector<TcPiece> pieces;
  std::vector<int32_t> cta_off((size_t)n_cta + 1, 0);
  std::vector<TcGroup> groups(grps.size());
  int64_t w_pos = 0;
  int cta = 0, last_cta = -1;
  for (size_t gi = 0; gi < grps.size(); ++gi) {
    const Grp &g = grps[gi];
    const int first_piece = (int)pieces.size();
    for (int t = 0; t < g.n_tiles; ++t, w_pos += g.weight) {
      while (cta + 1 < n_cta && w_pos >= total_w * (cta + 1) / n_cta) {
        ++cta;
        cta_off[cta] = (int32_t)pieces.size();
      }
      if (!pieces.empty() && pieces.back().group_id == (int)gi && last_cta == cta) {
        pieces.back().tile_end = t + 1;  // same group, same CTA: extend the piece
      } else {
        TcPiece p;
        p.req = g.req; p.kv_head = g.kv; p.mgroup = g.mg; p.tile_begin = t; p.tile_end = t + 1;
        p.partial_slot = -1; p.group_id = (int)gi; p.pad = 0;
        pieces.push_back(p);
        last_cta = cta;
      }
    }
    TcGroup &tg = groups[gi];
    memset(&tg, 0, sizeof(tg));
    tg.req = g.req; tg.kv_head = g.kv; tg.mgroup = g.mg;
    tg.n_partial = (int)pieces.size() - first_piece;
    tg.partial_begin = first_piece;  // provisional: index of the group's first piece
  }
  for (int c = cta + 1; c <= n_cta; ++c) cta_off[c] = (int32_t)pieces.size();
  // partial slots for groups cut into several pieces
  int n_slots = 0;
  std::vector<TcGroup> merge_groups;
  for (size_t gi = 0; gi < grps.size(); ++gi) {
    TcGroup &tg = groups[gi];
    if (tg.n_partial >= 2) {
      const int first_piece = tg.partial_begin;
      tg.partial_begin = n_slots;
      for (int k = 0; k < tg.n_partial; ++k) pieces[first_piece + k].partial_slot = n_slots++;
      merge_groups.push_back(tg);
    }
  }
  out.ok = true;
  out.n_cta = n_cta;
  out.n_pieces = (int)pieces.size();
  out.n_groups = n_slots ? (int)merge_groups.size() : 0;
  out.n_partial_slots = n_slots;
  out.tokens_per_mtile = T;
  out.o_pages = img.add(pages.data(), pages.size() * sizeof(TcPage));
  out.o_pieces = img.add(pieces.data(), pieces.size() * sizeof(TcPiece));
  out.o_cta_piece_off = img.add(cta_off.data(), cta_off.size() * sizeof(int32_t));
  out.o_reqs = img.add(reqs.data(), reqs.size() * sizeof(TcReq));
  if (merge_groups.empty()) merge_groups.push_back(TcGroup{});  // keep the section non-empty
  out.o_groups = img.add(merge_groups.data(), merge_groups.size() * sizeof(TcGroup));
  out.s_ml = 0;
  out.s_o = ((size_t)n_slots * 256 * 2 * sizeof(float) + 255) / 256 * 256;
  out.scratch_bytes = out.s_o + (size_t)n_slots * 256 * kD * sizeof(float);
  out.scratch_zero_bytes = 0;
  return LR_OK;
}

void tc_bind_device_plan(const TcHostPlan &h, unsigned char *image_base, unsigned char *scratch_base, lr_plan *p) {
  p->tc_ok = h.ok;
  memset(&p->tc, 0, sizeof(p->tc));
  if (!h.ok) return;
  DevTcPlan &t = p->tc;
  t.pages = reinterpret_cast<const TcPage *>(image_base + h.o_pages);
  t.pieces = reinterpret_cast<const TcPiece *>(image_base + h.o_pieces);
  t.cta_piece_off = reinterpret_cast<const int32_t *>(image_base + h.o_cta_piece_off);
  t.reqs = reinterpret_cast<const TcReq *>(image_base + h.o_reqs);
  t.groups = reinterpret_cast<const TcGroup *>(image_base + h.o_groups);
  t.n_cta = h.n_cta;
  t.n_groups = h.n_groups;
  t.n_merge_groups = h.n_groups;
  t.tokens_per_mtile = h.tokens_per_mtile;
  t.partial_ml = reinterpret_cast<float *>(scratch_base + h.s_ml);
  t.partial_o = reinterpret_cast<float *>(scratch_base + h.s_o);
  t.tickets = nullptr;
}

int launch_attn_tc(lr_plan *p, const void *q, const void *k, const void *v, void *out, float *lse, float scale,
                   cudaStream_t s) {
  const CUtensorMap *km = nullptr, *vm = nullptr;
  if (int rc = get_pool_map(p->ctx, k, p->dev.n_pool_pages, &km)) return rc;
  CUtensorMap kmap = *km;  // the cache may reallocate when the second map is added
  if (int rc = get_pool_map(p->ctx, v, p->dev.n_pool_pages, &vm)) return rc;
  CUtensorMap vmap = *vm;
  const float scale_log2 = scale * 1.4426950408889634f;
  attn_tc_kernel<<<p->tc.n_cta, kThreads, kSmemBytes, s>>>(kmap, vmap, p->dev, p->tc, reinterpret_cast<const uint16_t *>(q),
                                                            reinterpret_cast<uint16_t *>(out), lse, scale_log2);
  p->ctx->launches++;
  if (int rc = cuda_fail(cudaGetLastError(), "attn_tc_kernel launch")) return rc;
  if (p->tc.n_merge_groups > 0) {
    dim3 grid((unsigned)p->tc.n_merge_groups, 32);
    attn_tc_merge_kernel<<<grid, 256, 0, s>>>(p->dev, p->tc, reinterpret_cast<uint16_t *>(out), lse);
    p->ctx->launches++;
    if (int rc = cuda_fail(cudaGetLastError(), "attn_tc_merge_kernel launch")) return rc;
  }
  return LR_OK;
}

}  // namespace lr
