// Tensor-core nested-prefix attention for sm_100a (head_dim 128) on CTA pairs.
//
// Work decomposition.  For one request the *extended chain* is the list of its KV pages in the order prefix,
// segments, branch tails; 8 consecutive pages form a 128-key tile.  All query rows of the request that share one KV
// head -- (query token, head-in-group) pairs, floor(128/G) tokens per 128-row M-tile -- are processed against a tile
// at once, so a KV page is fetched from HBM once for every branch and every GQA head that can see it.  A *group* is
// (request, KV head, one or two M-tiles); the tiles of all groups, in order, are cut into contiguous ranges, one per
// CTA pair; a range may cover parts of several groups (*pieces*).
//
// A pair is a cluster of two CTAs on the two SMs of one TPC.  CTA c owns M-tile c of the piece: its Q tile in its
// shared memory, its score buffers and output accumulator in its tensor memory, its softmax warps.  Every KV tile is
// split between the two: CTA c fetches the K rows of keys 64c..64c+63 and, of the V rows of all 128 keys, channels
// 64c..64c+63 -- half of the bytes each, every byte of the tile crossing L2 -> shared memory once per pair.  One
// thread of CTA 0 issues tcgen05.mma with cta_group::2 (M = 256): S = Q K^T (N = 128 keys, the B operand half from
// either CTA) and O += P V (N = 128 channels), which write each CTA's 128 rows into that CTA's tensor memory.
//
// One CTA = 7 warps:
//   warps 0-3  softmax, one thread per query row (tcgen05.ld 32x32b gives a thread its row): scores of a whole
//              128-key tile per step, exponentials against the row's running reference exponent with the maximum
//              computed beside them, lazy rescale of O (only when the maximum grew by more than 2^8), exact redo
//              when it would have overflowed; bf16 P written over the first half of the score buffer.
//   warp 4     TMA producer of this CTA's halves: per tile 4 boxes of 4 KB (K pages) and 8 boxes of 2 KB (V page
//              halves) into a ring of 16 KB stages; the Q tile of each piece (double-buffered).  Every copy is for
//              this CTA alone and completes on this CTA's own barrier.
//   warp 5     gate: waits for each stage to land, zeroes the V rows of token slots that hold no valid token (so
//              that whatever the slack holds, NaN included, cannot reach the output) and then tells CTA 0 that this
//              CTA's half is ready (a remote mbarrier arrive).
//   warp 6     (CTA 0 only) MMA issuer for the pair.  Three score buffers: the QK product runs two tiles ahead of
//              the PV product, so the softmax of one tile overlaps the products around it.
// Completion of the products is signalled to both CTAs with tcgen05.commit multicast to the same barrier in each.
// Tensor memory (512 columns per CTA): S0 | S1 | S2 | O, 128 fp32 columns each; P_b occupies the first 64 columns
// of S_b.
//
// Split KV.  A piece that is the only contributor to its M-tile writes bf16 output.  Otherwise it writes an fp32
// partial (reference exponent, sum, unnormalised O) and takes a ticket on the M-tile's counter; the contributor that
// draws the last ticket merges all partials in slot order (bit-reproducible) and writes the output.  No second
// kernel and no waiting on other CTAs.
//
// Every wait on an mbarrier is bounded by the global timer; when one expires the CTA raises the abort flag of both
// CTAs of the pair, records LR_ETIMEOUT in the status word, drains what it has in flight and goes to the common
// exit, where both CTAs meet before tensor memory is released.
#include <cuda.h>

#include <algorithm>

#include "lr_common.cuh"

namespace lr {

namespace {

constexpr int kD = 128;
constexpr int kStages = 5;
constexpr int kPartBytes = 16384;   // one CTA's half of a K tile (64 keys x 128 channels) or of a V tile (128 keys x 64 channels)
constexpr int kStageBytes = 2 * kPartBytes;  // ring position p of a piece: [K half of tile p | V half of tile p - 2]
constexpr int kQBytes = 32768;      // one M-tile of Q: [2 halves of 64 channels][128 rows][128 B]
constexpr int kHalfBytes = 16384;
constexpr int kAtomBytes = 1024;    // 8 rows x 128 bytes, one 128-byte-swizzle atom
constexpr int kThreads = 384;  // 8 softmax warps, producer, gate, two issuers
constexpr int kPagesPerTile = 8;
constexpr int kSBufs = 2;          // score buffers; P has buffers of its own, so a score buffer is free as soon as it has been read
constexpr uint64_t kDrainLimitNs = 50ull * 1000ull * 1000ull;
constexpr long long kStaggerCycles = 700;
constexpr float kRescaleThreshold = 8.0f;  // log2 units: the reference exponent follows the row maximum within 2^8

struct __align__(8) Ctrl {
  uint64_t kv_full[kStages], kv_empty[kStages], kv_ready[kStages];
  uint64_t q_full[2], q_empty[2], q_ready[2];
  uint64_t s_full[kSBufs], p_full[kSBufs];
  uint64_t o_done[2], epi_done, drain, drain_qk;  // o_done[u & 1]: the PV product of tile u has retired
  uint32_t tmem_base;
  int abort_flag;
  uint32_t ticket;
  float l_xch[2][128];  // row sums of the two column halves, exchanged once per piece
};
constexpr int kCtrlBytes = 2048;
static_assert(sizeof(Ctrl) <= kCtrlBytes, "Ctrl must fit behind the tiles");
constexpr int kSmemBytes = 2 * kQBytes + kStages * kStageBytes + kCtrlBytes;  // the base must be 1024-aligned
static_assert(kSmemBytes <= 227 * 1024, "shared memory per CTA");

// ---- PTX wrappers ----------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// arrive on a barrier of any CTA of the cluster (address from map_to_cta)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ uint32_t mbar_test_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void bar_sync_softmax() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Arrives on the barrier at this shared-memory offset in BOTH CTAs of the pair once every tcgen05.mma issued so far
// by this thread has completed.
__device__ __forceinline__ void tc_commit_pair(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(smem_u32(bar)),
               "h"((uint16_t)3)
               : "memory");
}

// Tiled bulk tensor copies global -> shared for this CTA alone, completion on this CTA's own mbarrier.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, int32_t z, int32_t w, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
      "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "r"(w)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, int32_t z, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
      "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptors: D fp32, A and B bf16, M = 256 over the pair (bits 24-28 = M/16), N = 128 (bits 17-22 = N/8).
// QK: both operands K-major.  PV: bit 16 selects the N-major B operand (V rows are keys, channels contiguous).
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | (16u << 24) | ((128u >> 3) << 17);
constexpr uint32_t kIdescQK = kIdescBase;
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16);

__device__ __forceinline__ void mma2_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void mma2_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}

// tcgen05.ld / tcgen05.st, shape 32x32b: thread i of the warp owns lane (base + i), consecutive columns.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr)
               : "memory");
}
// 64 columns of a row and the wait for them in one statement, so that nothing can be scheduled between the load and
// the point where its registers are valid.
__device__ __forceinline__ void tmem_ld64_wait(uint32_t taddr, uint32_t (&r)[64]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];\n\ttcgen05.wait::ld.sync.aligned;"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
               : "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// packed fp32 pairs: d = a * b + c and d = a + b on both halves with one instruction each
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
  float2 d;
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d.x), "=f"(d.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
  return d;
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
  float2 d;
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d.x), "=f"(d.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&t);
}
__device__ __forceinline__ float bits_f(uint32_t u) { return __uint_as_float(u); }

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// What every role of a CTA needs for a bounded wait.
struct WaitCtx {
  Ctrl *ctrl;
  int32_t *status;
  uint32_t peer_abort_addr;  // the other CTA's abort flag
  uint64_t limit_ns;
};

__device__ __forceinline__ void raise_abort(const WaitCtx &w, int code) {
  *reinterpret_cast<volatile int *>(&w.ctrl->abort_flag) = 1;
  asm volatile("st.relaxed.cluster.shared::cluster.u32 [%0], %1;" ::"r"(w.peer_abort_addr), "r"(1u) : "memory");
  w.status[0] = kDevTimeout;
  w.status[1] = code;
}

// Bounded wait: gives up after the limit of wall time.  Returns false when the wait expired or another role of
// the pair gave up.
__device__ __forceinline__ bool wait_bar(uint64_t *bar, uint32_t parity, const WaitCtx &w, int code) {
  if (mbar_test_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  for (uint32_t i = 1;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 7u) == 0u) {
      if (*reinterpret_cast<volatile int *>(&w.ctrl->abort_flag)) return false;
      if (global_ns() - t0 > w.limit_ns) break;
    }
  }
  raise_abort(w, code);
  return false;
}

// The same for a whole warp: every lane waits, and the warp goes on only if every lane's wait succeeded (so that a
// warp never executes its warp-wide instructions half in and half out of an abort).
__device__ __forceinline__ bool wait_bar_warp(uint64_t *bar, uint32_t parity, const WaitCtx &w, int code) {
  return __all_sync(0xFFFFFFFFu, wait_bar(bar, parity, w, code)) != 0;
}

// ---- ring order ----------------------------------------------------------------------
// The QK product runs two tiles ahead of the PV product, so ring position p (0 .. n + 1) of a piece of n tiles holds
// the K half of tile p (p < n) beside the V half of tile p - 2 (p >= 2): what the issuer consumes together.

struct RowInfo {
  int depth;       // depth-first number of the node the row's branch continues (on a chain: segments it sees); -1 for padding rows
  int branch;      // local branch index within the request; -1 for padding rows
  int limit;       // last tail token the row sees
  int64_t q_index; // (query row * n_q_heads + head), -1 for padding rows
};

// Row r (0..127) of M-tile mt of (request, KV head): token mt*T + r/G, head kv*G + r%G.
__device__ __forceinline__ RowInfo row_info(const DevBatch &d, const TcRow *rows, const TcReq &rq, int T, int mt, int r, int kv) {
  RowInfo ri;
  ri.depth = -1;
  ri.branch = -1;
  ri.limit = -1;
  ri.q_index = -1;
  const int G = d.group;
  const int tok = mt * T + r / G;
  if (r < T * G && tok < rq.n_q) {
    const int row = rq.q_row0 + tok;
    const int2 w = __ldg(reinterpret_cast<const int2 *>(rows + row));
    ri.depth = w.x & 0xFFFF;
    ri.branch = w.x >> 16;
    ri.limit = w.y;
    ri.q_index = (int64_t)row * d.n_q_heads + kv * G + r % G;
  }
  return ri;
}

__device__ __forceinline__ int page_n_ok(uint32_t meta, const RowInfo &ri) {
  const int valid = meta & 31, need = (meta >> 5) & 255, owner = (meta >> 13) & 255, tb = meta >> 21;
  int n;
  if (owner == 0) n = (ri.depth >= need && ri.depth <= tb) ? valid : 0;  // the row's node lies in the span's subtree
  else n = (owner - 1 == ri.branch) ? min(valid, ri.limit - tb * kPage + 1) : 0;
  return max(n, 0);
}

// -inf on the score columns of one 64-key half that the row does not see (n_ok[p] = visible tokens of page p)
__device__ __forceinline__ void mask_half(uint32_t (&v)[64], const int *n_ok) {
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    const int n = n_ok[p];
    if (n < kPage) {
#pragma unroll
      for (int c = 0; c < kPage; ++c)
        if (c >= n) v[p * kPage + c] = 0xFF800000u;
    }
  }
}
__device__ __forceinline__ float max_half(const uint32_t (&v)[64]) {
  float a = -INFINITY, b = -INFINITY, c = -INFINITY, e = -INFINITY;
#pragma unroll
  for (int i = 0; i < 64; i += 8) {
    a = max3(a, bits_f(v[i]), bits_f(v[i + 1]));
    b = max3(b, bits_f(v[i + 2]), bits_f(v[i + 3]));
    c = max3(c, bits_f(v[i + 4]), bits_f(v[i + 5]));
    e = max3(e, bits_f(v[i + 6]), bits_f(v[i + 7]));
  }
  return fmaxf(fmaxf(a, b), fmaxf(c, e));
}
// 2^x for a pair of arguments without the special-function unit: x = n + f with n = round(x) (adding 1.5 * 2^23 leaves
// n in the low mantissa bits), 2^f on [-0.5, 0.5] by a cubic (minimax fit, relative error 7.5e-5 -- a thirtieth of the
// rounding of the bf16 weight it becomes), and n added to the exponent field.  Arguments below -125 give 2^-125.
__device__ __forceinline__ float2 exp2_fma(float2 x) {
  x.x = fmaxf(x.x, -125.0f);
  x.y = fmaxf(x.y, -125.0f);
  const float2 y = fadd2(x, make_float2(12582912.0f, 12582912.0f));
  const float2 t = fadd2(y, make_float2(-12582912.0f, -12582912.0f));
  const float2 f = ffma2(t, make_float2(-1.0f, -1.0f), x);
  float2 p = ffma2(make_float2(0.0551716685f, 0.0551716685f), f, make_float2(0.2426111251f, 0.2426111251f));
  p = ffma2(p, f, make_float2(0.6932609677f, 0.6932609677f));
  p = ffma2(p, f, make_float2(0.9999280572f, 0.9999280572f));
  float2 r;
  r.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(y.x) << 23));
  r.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(y.y) << 23));
  return r;
}

// P = exp2(scale * s - m) for 64 scores -> 32 packed bf16 pairs; returns their fp32 sum.  The special-function unit
// delivers one exponential per lane every 8.5 cycles and is what bounds the sweep; with POLY, kPolyOf8 of every 8 pairs
// are computed on the FMA pipe instead (only where every score is finite: tiles that need no mask).
#ifndef LR_POLY_OF_8
#define LR_POLY_OF_8 3
#endif
constexpr int kPolyOf8 = LR_POLY_OF_8;
template <bool POLY>
__device__ __forceinline__ float exp_half(const uint32_t (&v)[64], uint32_t (&pk)[32], float scale_log2, float neg_m) {
  const float2 sc = make_float2(scale_log2, scale_log2), nm = make_float2(neg_m, neg_m);
  float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
  for (int i = 0; i < 64; i += 4) {
    float2 y0 = ffma2(make_float2(bits_f(v[i]), bits_f(v[i + 1])), sc, nm);
    float2 y1 = ffma2(make_float2(bits_f(v[i + 2]), bits_f(v[i + 3])), sc, nm);
    const int pair0 = ((i >> 1) & 7), pair1 = pair0 + 1;  // position of the two pairs in their block of 8 pairs
    if (POLY && (pair0 * kPolyOf8) / 8 != ((pair0 + 1) * kPolyOf8) / 8) {
      y0 = exp2_fma(y0);
    } else {
      y0.x = ex2(y0.x);
      y0.y = ex2(y0.y);
    }
    if (POLY && (pair1 * kPolyOf8) / 8 != ((pair1 + 1) * kPolyOf8) / 8) {
      y1 = exp2_fma(y1);
    } else {
      y1.x = ex2(y1.x);
      y1.y = ex2(y1.y);
    }
    acc0 = fadd2(acc0, y0);
    acc1 = fadd2(acc1, y1);
    pk[i >> 1] = pack_bf16(y0.x, y0.y);
    pk[(i >> 1) + 1] = pack_bf16(y1.x, y1.y);
  }
  acc0 = fadd2(acc0, acc1);
  return acc0.x + acc0.y;
}

// One softmax thread's state and per-piece constants, passed to the non-inlined epilogue.  Two threads share a row:
// thread g of the row owns output channels 64 g .. 64 g + 63.
struct EpiArgs {
  uint32_t o_addr;     // this thread's lane quarter of the output accumulator, at its channel half
  int slot, target;    // as in PrPiece
  int r, g;            // row of the M-tile, channel half
  int64_t q_index;     // -1 for padding rows
  float m, l;          // reference exponent (log2 units) and sum of the row over this piece's keys
};

// Output of half a row: bf16 (slot < 0) or an fp32 partial.  Not inlined: its buffers must not weigh on the
// register allocation of the sweep.
__device__ __noinline__ void store_row(const EpiArgs a, uint16_t *__restrict__ out, float *__restrict__ lse,
                                       float *__restrict__ partial_o, float *__restrict__ partial_ml) {
  if (a.slot < 0) {
    const float inv = 1.0f / a.l;
#pragma unroll 1
    for (int ch = 0; ch < 2; ++ch) {
      uint32_t o[32];
      tmem_ld32(a.o_addr + ch * 32, o);
      tc_wait_ld();
      if (a.q_index >= 0) {
        uint4 *dst = reinterpret_cast<uint4 *>(out + a.q_index * kD + a.g * 64 + ch * 32);
#pragma unroll
        for (int jj = 0; jj < 4; ++jj)
          dst[jj] = make_uint4(pack_bf16(bits_f(o[8 * jj]) * inv, bits_f(o[8 * jj + 1]) * inv),
                               pack_bf16(bits_f(o[8 * jj + 2]) * inv, bits_f(o[8 * jj + 3]) * inv),
                               pack_bf16(bits_f(o[8 * jj + 4]) * inv, bits_f(o[8 * jj + 5]) * inv),
                               pack_bf16(bits_f(o[8 * jj + 6]) * inv, bits_f(o[8 * jj + 7]) * inv));
      }
    }
    if (lse != nullptr && a.q_index >= 0 && a.g == 0) lse[a.q_index] = (a.m + log2f(a.l)) * 0.6931471805599453f;
  } else {
#pragma unroll 1
    for (int ch = 0; ch < 2; ++ch) {
      uint32_t o[32];
      tmem_ld32(a.o_addr + ch * 32, o);
      tc_wait_ld();
      if (a.q_index >= 0) {
        // chunk-major: 16-byte chunk k of row r at [slot][k][r], so a warp's store is 512 contiguous bytes
        uint4 *dst = reinterpret_cast<uint4 *>(partial_o) + ((int64_t)a.slot * 32 + (a.g * 2 + ch) * 8) * 128 + a.r;
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) dst[jj * 128] = make_uint4(o[4 * jj], o[4 * jj + 1], o[4 * jj + 2], o[4 * jj + 3]);
      }
    }
    if (a.q_index >= 0 && a.g == 0) *reinterpret_cast<float2 *>(partial_ml + ((int64_t)a.slot * 128 + a.r) * 2) = make_float2(a.m, a.l);
  }
}

// Merge of the partials of one M-tile by the contributor that arrived last: O = sum_j 2^(m_j - M) O_j / sum_j
// 2^(m_j - M) l_j, slots in increasing order whoever merges.  One thread per (row, channel half), 32 channels at a time.
__device__ __noinline__ void merge_row(int slot_begin, int n_slots, int r, int g, int64_t q_index, uint16_t *__restrict__ out,
                                       float *__restrict__ lse, const float *partial_o, const float *partial_ml) {
  if (q_index < 0) return;
  const float2 *ml = reinterpret_cast<const float2 *>(partial_ml) + (int64_t)slot_begin * 128 + r;
  float M = -INFINITY;
  for (int j = 0; j < n_slots; ++j) {
    const float2 v = __ldcg(ml + (int64_t)j * 128);
    if (v.y > 0.f) M = fmaxf(M, v.x);  // a contributor that saw no key of the row adds nothing
  }
  float L = 0.f;
  for (int j = 0; j < n_slots; ++j) {
    const float2 v = __ldcg(ml + (int64_t)j * 128);
    if (v.y > 0.f) L = fmaf(exp2f(v.x - M), v.y, L);
  }
  const float inv = 1.0f / L;
#pragma unroll 1
  for (int ch = 0; ch < 2; ++ch) {
    float acc[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) acc[c] = 0.f;
    const float4 *po = reinterpret_cast<const float4 *>(partial_o) + ((int64_t)slot_begin * 32 + (g * 2 + ch) * 8) * 128 + r;
    for (int j = 0; j < n_slots; ++j) {
      const float2 v = __ldcg(ml + (int64_t)j * 128);
      if (v.y > 0.f) {
        const float w = exp2f(v.x - M);
        float4 o[8];
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) o[jj] = __ldcg(po + ((int64_t)j * 32 + jj) * 128);
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
          acc[4 * jj] = fmaf(w, o[jj].x, acc[4 * jj]);
          acc[4 * jj + 1] = fmaf(w, o[jj].y, acc[4 * jj + 1]);
          acc[4 * jj + 2] = fmaf(w, o[jj].z, acc[4 * jj + 2]);
          acc[4 * jj + 3] = fmaf(w, o[jj].w, acc[4 * jj + 3]);
        }
      }
    }
    uint4 *dst = reinterpret_cast<uint4 *>(out + q_index * kD + g * 64 + ch * 32);
#pragma unroll
    for (int jj = 0; jj < 4; ++jj)
      dst[jj] = make_uint4(pack_bf16(acc[8 * jj] * inv, acc[8 * jj + 1] * inv), pack_bf16(acc[8 * jj + 2] * inv, acc[8 * jj + 3] * inv),
                           pack_bf16(acc[8 * jj + 4] * inv, acc[8 * jj + 5] * inv), pack_bf16(acc[8 * jj + 6] * inv, acc[8 * jj + 7] * inv));
  }
  if (lse != nullptr && g == 0) lse[q_index] = (M + log2f(L)) * 0.6931471805599453f;
}

__global__ void __launch_bounds__(kThreads, 1)
attn_pair_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
                 const __grid_constant__ CUtensorMap q_map, DevBatch d, DevPairPlan pp, uint16_t *__restrict__ out,
                 float *__restrict__ lse, float scale_log2) {
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char *q_smem = smem;                       // 2 x 32 KB
  unsigned char *kv_smem = smem + 2 * kQBytes;        // kStages x 16 KB
  Ctrl *ctrl = reinterpret_cast<Ctrl *>(kv_smem + kStages * kStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t cta = cluster_ctarank();             // 0: issues the products of the pair
  const int pair = blockIdx.x >> 1;
  // the swizzled tiles need a 1024-byte aligned base; both CTAs of a pair see the same offset, so both skip the work
  const bool aligned = (smem_u32(smem) & 1023u) == 0u;
  if (!aligned && threadIdx.x == 0) {
    d.status[0] = kDevBounds;
    d.status[1] = 250;
  }

  // rows of a Q tile that no copy writes must hold finite values
  for (int i = threadIdx.x; i < 2 * kQBytes / 16; i += kThreads) reinterpret_cast<uint4 *>(q_smem)[i] = make_uint4(0, 0, 0, 0);
  fence_proxy_async();
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&ctrl->kv_full[s], 1);
      mbar_init(&ctrl->kv_empty[s], 2);  // one arrival per issuer warp
      mbar_init(&ctrl->kv_ready[s], 2);  // one arrival per gate warp of the pair (used in CTA 0 only)
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&ctrl->q_full[b], 1);
      mbar_init(&ctrl->q_empty[b], 1);
      mbar_init(&ctrl->q_ready[b], 2);
    }
    for (int b = 0; b < kSBufs; ++b) {
      mbar_init(&ctrl->s_full[b], 1);
      mbar_init(&ctrl->p_full[b], 16);   // one arrival per softmax warp of the pair (used in CTA 0 only)
    }
    mbar_init(&ctrl->o_done[0], 1);
    mbar_init(&ctrl->o_done[1], 1);
    mbar_init(&ctrl->epi_done, 16);
    mbar_init(&ctrl->drain, 1);
    mbar_init(&ctrl->drain_qk, 1);
    ctrl->abort_flag = 0;
    ctrl->ticket = 0;
    fence_barrier_init();
  }
  if (warp == 8) {  // the same warp of both CTAs allocates (and later frees) the pair's tensor memory
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctrl->tmem_base)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the other CTA's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&ctrl->tmem_base);
  // inputs may come from the kernel launched just before this one
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  WaitCtx wc;
  wc.ctrl = ctrl;
  wc.status = d.status;
  wc.peer_abort_addr = map_to_cta(smem_u32(&ctrl->abort_flag), cta ^ 1u);
  wc.limit_ns = (uint64_t)pp.wait_limit_us * 1000ull;

  const PrHead *head = pp.heads + pair;
  const int piece0 = aligned ? head->piece0 : 0, piece1 = aligned ? head->piece1 : 0;
  const int T = pp.tokens_per_mtile;
  const int G = d.group;

  if (warp == 8) {
    // ======================= TMA producer of this CTA's halves ==========================
    uint32_t ring = 0, pc_idx = 0;
    bool ok = true;
    const uint32_t q_box_bytes = (uint32_t)(64 * G * T * 2);
    for (int pc = piece0; pc < piece1 && ok; ++pc, ++pc_idx) {
      const PrPiece pi = pc == piece0 ? head->first : pp.pieces[pc];
      const TcReq rq = pc == piece0 ? head->first_req : pp.reqs[pi.req];
      const int n = pi.tile_end - pi.tile_begin;
      const uint32_t qb = pc_idx & 1u;
      // the Q tile of the piece, once the products of the piece two before no longer read the buffer
      ok = wait_bar_warp(&ctrl->q_empty[qb], ((pc_idx >> 1) & 1u) ^ 1u, wc, 205);
      if (!ok) break;
      const bool has_q = (int)cta < pi.n_mt;
      if (lane == 0) {
        if (has_q) mbar_arrive_expect_tx(&ctrl->q_full[qb], 2u * q_box_bytes);
        else mbar_arrive(&ctrl->q_full[qb]);
      }
      __syncwarp();
      if (has_q && lane < 2)
        tma_load_3d(smem_u32(q_smem) + qb * kQBytes + lane * kHalfBytes, &q_map, lane * 64, pi.kv_head * G,
                    rq.q_row0 + (pi.mtile0 + (int)cta) * T, &ctrl->q_full[qb]);
      // Page ids arrive 32 at a time (one per lane = 4 tiles) and one chunk ahead of their first use, so no step of
      // the loop waits for a load it has just issued.  Pages past the end of the request are absent (no copy).
      auto load_chunk = [&](int c) -> int32_t {
        const int idx = c * 32 + lane;
        int32_t pg = 0;
        if (idx < rq.n_pages) {
          pg = pp.pages[rq.page_off + idx].page;
          if (pg < 0 || pg >= d.n_pool_pages) {  // never fetch outside the pool
            d.status[0] = kDevBounds;
            d.status[1] = 200;
            pg = 0;
          }
        }
        return pg;
      };
      int c_cur = pi.tile_begin >> 2;
      int32_t pg_nxt = load_chunk(c_cur + 1), pg_cur;
      if (pc == piece0) {  // the first chunk of the first piece comes with the pair's head record
        pg_cur = head->first_pages[lane];
        if (c_cur * 32 + lane < rq.n_pages && (pg_cur < 0 || pg_cur >= d.n_pool_pages)) {
          d.status[0] = kDevBounds;
          d.status[1] = 201;
          pg_cur = 0;
        }
      } else {
        pg_cur = load_chunk(c_cur);
      }
      for (int pos = 0; pos < n + 2 && ok; ++pos, ++ring) {
        const int tk = pi.tile_begin + pos, tv = pi.tile_begin + pos - 2;  // K tile and V tile of the position
        const bool has_k = pos < n, has_v = pos >= 2;
        if (has_v && (tv >> 2) > c_cur) {  // the V index is the oldest tile still needed
          ++c_cur;
          pg_cur = pg_nxt;
          pg_nxt = load_chunk(c_cur + 1);
        }
        // lanes 0-3 copy this CTA's K pages (4 cta .. 4 cta + 3 of the tile), lanes 8-15 its half of the 8 V pages
        const bool v_lane = lane >= 8;
        const int t = v_lane ? tv : tk;
        const int pidx = v_lane ? (lane & 7) : (int)(4u * cta) + (lane & 3);
        const int src = ((t & 3) * 8 + pidx) & 31;  // the lane that holds the page's id, in this chunk or the next
        const int32_t from_cur = __shfl_sync(0xFFFFFFFFu, pg_cur, src), from_nxt = __shfl_sync(0xFFFFFFFFu, pg_nxt, src);
        const int32_t page = (t >> 2) == c_cur ? from_cur : from_nxt;
        const int k_in_tile = has_k ? min(kPagesPerTile, rq.n_pages - tk * kPagesPerTile) : 0;  // pages of the tile that exist
        const int v_in_tile = has_v ? min(kPagesPerTile, rq.n_pages - tv * kPagesPerTile) : 0;
        const int mine_k = max(0, min(4, k_in_tile - (int)(4u * cta)));
        const uint32_t stage = ring % kStages;
        ok = wait_bar_warp(&ctrl->kv_empty[stage], ((ring / kStages) & 1u) ^ 1u, wc, 210);
        if (!ok) break;
        if (lane == 0) {
          const uint32_t bytes = (uint32_t)mine_k * 4096u + (uint32_t)v_in_tile * 2048u +
                                 ((pair == 0 && cta == 0 && ring == 0) ? pp.phantom_tx_bytes : 0u);
          if (bytes > 0) mbar_arrive_expect_tx(&ctrl->kv_full[stage], bytes);
          else mbar_arrive(&ctrl->kv_full[stage]);
        }
        __syncwarp();
        const uint32_t dst = smem_u32(kv_smem + stage * kStageBytes);
        const int32_t w4 = (int32_t)(((int64_t)page * d.n_kv_heads + pi.kv_head) * 2);  // first 8-key group of the page
        if (lane < mine_k) tma_load_4d(dst + lane * 4096, &k_map, 0, 0, 0, w4, &ctrl->kv_full[stage]);
        if (v_lane && lane - 8 < v_in_tile) tma_load_4d(dst + kPartBytes + (lane - 8) * 2048, &v_map, 0, 0, (int32_t)cta, w4, &ctrl->kv_full[stage]);
      }
    }
    if (!ok) {
      // give the copies already in flight a bounded time to land before the CTA exits
      for (uint32_t back = 1; back <= (uint32_t)kStages && back <= ring; ++back) {
        const uint32_t j = ring - back;
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(&ctrl->kv_full[j % kStages], (j / kStages) & 1u))
          if (global_ns() - t0 > kDrainLimitNs) break;
      }
    }
  } else if (warp == 9) {
    // ======================= gate: this CTA's half of a stage is ready ===================
    uint32_t ring = 0, pc_idx = 0;
    bool ok = true;
    const uint32_t ready0 = map_to_cta(smem_u32(&ctrl->kv_ready[0]), 0), qready0 = map_to_cta(smem_u32(&ctrl->q_ready[0]), 0);
    for (int pc = piece0; pc < piece1 && ok; ++pc, ++pc_idx) {
      const PrPiece pi = pc == piece0 ? head->first : pp.pieces[pc];
      const TcReq rq = pc == piece0 ? head->first_req : pp.reqs[pi.req];
      const int n = pi.tile_end - pi.tile_begin;
      const uint32_t qb = pc_idx & 1u;
      ok = wait_bar_warp(&ctrl->q_full[qb], (pc_idx >> 1) & 1u, wc, 215);
      if (!ok) break;
      if (lane == 0) mbar_arrive_cluster(qready0 + qb * 8u);
      for (int pos = 0; pos < n + 2 && ok; ++pos, ++ring) {
        const int tv = pi.tile_begin + pos - 2;
        const uint32_t stage = ring % kStages;
        ok = wait_bar_warp(&ctrl->kv_full[stage], (ring / kStages) & 1u, wc, 216);
        if (!ok) break;
        if (pos >= 2 && tv >= rq.n_dense_tiles) {
          // zero the V rows (this CTA's 64 channels = one 128-byte row each) of token slots that hold no valid
          // token: the slack of a span's last page, and pages past the end of the request
          unsigned char *vs = kv_smem + stage * kStageBytes + kPartBytes;
          const TcPage *pg = pp.pages + rq.page_off + tv * kPagesPerTile;
          for (int p = 0; p < kPagesPerTile; ++p) {
            const int valid = __ldg(&pg[p].meta) & 31;
            for (int idx = lane; idx < (kPage - valid) * 8; idx += 32) {
              const int key = p * kPage + valid + (idx >> 3);
              *reinterpret_cast<uint4 *>(vs + (key >> 3) * kAtomBytes + (key & 7) * 128 + (idx & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
          }
          fence_proxy_async();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(ready0 + stage * 8u);
      }
    }
  } else if (warp == 10 || warp == 11) {
    if (cta == 0) {
      // ======================= MMA issuers of the pair ===================================
      // Issuing a tcgen05.mma holds its thread for about as long as the tensor pipe needs for it, so one thread that
      // also does the waiting and committing cannot keep the pipe busy.  Warp 10 issues every PV product (one thread,
      // so O accumulates in a fixed order), warp 11 every QK product; the pipe takes them as they come.  Both walk
      // the ring positions of every piece and both observe every phase of the barriers they share.
      const bool is_pv = warp == 10;
      uint32_t ring = 0, pc_idx = 0, unit = 0;  // ring position, piece count, tiles of the pieces before this one
      bool ok = true;
      const uint32_t q_addr = smem_u32(q_smem), kv_addr = smem_u32(kv_smem);
      const uint32_t p_tmem = tmem + kSBufs * 128, o_tmem = tmem + 384;  // S0 | S1 | P0 P1 | O
      // Descriptors differ from a base only in the start-address field (units of 16 bytes).
      // Q: K-major, 8-row groups 1024 bytes apart.  K half: K-major, 8-key groups 2048 bytes apart (two 64-channel
      // atoms per group).  V half: N-major, one 64-channel atom per 8-key group, groups 1024 bytes apart.
      const uint64_t qdesc0 = make_desc(q_addr, 16, 1024), kdesc0 = make_desc(kv_addr, 16, 2 * kAtomBytes),
                     vdesc0 = make_desc(kv_addr, kAtomBytes, kAtomBytes);
      auto issue_qk = [&](uint32_t qb, uint32_t stage, uint32_t buf) {  // S_buf = Q K^T over the 128 keys of the tile
        const uint64_t a = qdesc0 + (uint64_t)(qb * (kQBytes >> 4)), b = kdesc0 + (uint64_t)(stage * (kStageBytes >> 4));
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            mma2_ss(tmem + buf * 128, a + (uint64_t)(h * (kHalfBytes >> 4) + kk * 2), b + (uint64_t)(h * (kAtomBytes >> 4) + kk * 2),
                    kIdescQK, (h | kk) != 0);
      };
      auto issue_pv = [&](uint32_t stage, uint32_t buf, bool acc) {  // O (+)= P_buf V over the 128 keys of the tile
        const uint64_t b = vdesc0 + (uint64_t)(stage * (kStageBytes >> 4) + (kPartBytes >> 4));
#pragma unroll
        for (int k = 0; k < 8; ++k)
          mma2_ts(o_tmem, p_tmem + buf * 64 + k * 8, b + (uint64_t)(k * (2 * kAtomBytes >> 4)), kIdescPV, acc || k != 0);
      };
      for (int pc = piece0; pc < piece1 && ok; ++pc, ++pc_idx) {
        const PrPiece pi = pc == piece0 ? head->first : pp.pieces[pc];
        const int n = pi.tile_end - pi.tile_begin;
        const uint32_t qb = pc_idx & 1u;
        if (!is_pv) {
          ok = wait_bar_warp(&ctrl->q_ready[qb], (pc_idx >> 1) & 1u, wc, 220);
          if (!ok) break;
        }
        // position pos: O += P V for tile pos - 2 (warp 10) and S = Q K^T for tile pos (warp 11)
        for (int pos = 0; pos < n + 2 && ok; ++pos, ++ring) {
          const uint32_t stage = ring % kStages;
          ok = wait_bar_warp(&ctrl->kv_ready[stage], (ring / kStages) & 1u, wc, 221);
          if (!ok) break;
          const bool has_pv = pos >= 2, has_qk = pos < n;
          const uint32_t u_pv = unit + (uint32_t)(pos - 2), u_qk = unit + (uint32_t)pos;
          if (has_pv) {
            if (is_pv && pos == 2 && pc_idx > 0) {  // the epilogue of the previous piece has read O
              ok = wait_bar_warp(&ctrl->epi_done, (pc_idx - 1) & 1u, wc, 223);
              if (!ok) break;
            }
            // Both CTAs have read the scores of tile pos - 2 and put their P in place: the PV product may run, and
            // the score buffer may take tile pos.
            ok = wait_bar_warp(&ctrl->p_full[u_pv % kSBufs], (u_pv / kSBufs) & 1u, wc, 224);
            if (!ok) break;
          }
          tc_fence_after();
          if (lane == 0) {
            if (is_pv) {
              if (has_pv) {
                issue_pv(stage, u_pv % kSBufs, pos != 2);
                tc_commit_pair(&ctrl->o_done[u_pv & 1u]);
              }
            } else if (has_qk) {
              issue_qk(qb, stage, u_qk % kSBufs);
              tc_commit_pair(&ctrl->s_full[u_qk % kSBufs]);
              if (pos + 1 == n) tc_commit_pair(&ctrl->q_empty[qb]);  // last QK of the piece
            }
            // one of the two arrivals that release the stage (at once when this warp had nothing to issue from it)
            tc_commit_pair(&ctrl->kv_empty[stage]);
          }
          __syncwarp();
        }
        unit += (uint32_t)n;
      }
      if (!ok && lane == 0) {
        // let every MMA already issued by this thread retire before tensor memory is released
        uint64_t *drain = is_pv ? &ctrl->drain : &ctrl->drain_qk;
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(drain)) : "memory");
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(drain, 0))
          if (global_ns() - t0 > kDrainLimitNs) break;
      }
      __syncwarp();
    }
  } else {
    // ======================= softmax warps ============================================
    // Two threads per query row: thread g of a row turns the scores of keys 64 g .. 64 g + 63 of every tile into
    // weights and owns output channels 64 g .. 64 g + 63.  Both read the whole row for its maximum, so both hold the
    // same reference exponent and take the same decisions without talking to each other; the sums of the two halves
    // meet once per piece.
    const int quarter = warp & 3;                  // tensor-memory lane quarter this warp may access
    const int g = warp >> 2;                       // column half
    const int r = quarter * 32 + lane;             // row within the M-tile
    const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
    const uint32_t o_addr = lane_base + 384 + g * 64;
    const uint32_t p_full0 = map_to_cta(smem_u32(&ctrl->p_full[0]), 0), epi_done0 = map_to_cta(smem_u32(&ctrl->epi_done), 0);
    uint32_t unit = 0;  // tiles of all pieces so far
    bool ok = true;
    for (int pc = piece0; pc < piece1; ++pc) {
      const PrPiece pi = pc == piece0 ? head->first : pp.pieces[pc];
      const TcReq rq = pc == piece0 ? head->first_req : pp.reqs[pi.req];
      const int n = pi.tile_end - pi.tile_begin;
      const bool has_rows = (int)cta < pi.n_mt;
      RowInfo ri;
      ri.depth = ri.branch = ri.limit = -1;
      ri.q_index = -1;
      if (has_rows) ri = row_info(d, pp.rows, rq, T, pi.mtile0 + (int)cta, r, pi.kv_head);
      // a warp none of whose rows is a query row only keeps the barrier protocol going
      const bool warp_live = __any_sync(0xFFFFFFFFu, ri.q_index >= 0);
      // Rows that are no query row (padding of the M-tile) run along with a fixed reference exponent and take no part
      // in the decisions below; nothing of them is ever stored.
      const bool live_row = ri.q_index >= 0;
      float m_used = live_row ? -INFINITY : 0.f, l = 0.f;
      // O *= alpha on this thread's 64 channels.  Every PV product issued so far (tiles before this one) must have
      // retired first.
      auto rescale_o = [&](float alpha, uint32_t units_done) -> bool {
        if (!wait_bar_warp(&ctrl->o_done[(units_done - 1) & 1u], ((units_done - 1) >> 1) & 1u, wc, 235)) return false;
        tc_fence_after();
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t o[32];
          tmem_ld32(o_addr + ch * 32, o);
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(bits_f(o[c]) * alpha);
          tmem_st32(o_addr + ch * 32, o);
        }
        tc_wait_st();
        return true;
      };
      for (int j = 0; j < n && ok; ++j) {
        const uint32_t u = unit + (uint32_t)j;
        const uint32_t buf = u % kSBufs;
        const uint32_t s_addr = lane_base + buf * 128;
        const int t = pi.tile_begin + j;
        const bool masked = t >= rq.n_dense_tiles;
        ok = wait_bar_warp(&ctrl->s_full[buf], (u / kSBufs) & 1u, wc, 230);
        if (!ok) break;
        if (j == 0 && g == 1) {
          // The two halves of a row share the special-function unit of their scheduler.  In step, both load scores
          // and take maxima at the same time and then both queue for exponentials; half a tile out of step, the
          // exponentials of one run under the loads of the other.  Nothing brings them back into step afterwards
          // (they only meet in p_full), so the second half starts each piece late once.
          const long long c0 = clock64();
          while (clock64() - c0 < kStaggerCycles) {}
        }
        tc_fence_after();
        if (warp_live) {
          int n_ok[kPagesPerTile];
          if (masked) {
            const uint4 *mp = reinterpret_cast<const uint4 *>(pp.pages + rq.page_off + t * kPagesPerTile);
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
              const uint4 w = __ldg(mp + jj);
              n_ok[2 * jj] = page_n_ok(w.y, ri);
              n_ok[2 * jj + 1] = page_n_ok(w.w, ri);
            }
          }
          // The maximum of the whole row first (the other half only for that), so that the reference exponent is
          // settled before any weight of the tile exists: it follows the row maximum lazily, only when that has
          // grown by more than 2^8 -- O is rescaled then, after the PV products issued so far have retired -- and
          // otherwise every weight stays below 2^8.
          float mx;
          {
            uint32_t w[64];
            tmem_ld64_wait(s_addr + (1 - g) * 64, w);
            if (masked) mask_half(w, n_ok + 4 * (1 - g));
            mx = max_half(w);
          }
          uint32_t v[64];
          tmem_ld64_wait(s_addr + g * 64, v);
          if (masked) mask_half(v, n_ok + 4 * g);
          mx = fmaxf(mx, max_half(v)) * scale_log2;
          const bool grow = live_row && mx > m_used + kRescaleThreshold;  // also the first visible key of a row (m = -inf)
          if (__any_sync(0xFFFFFFFFu, grow)) {
            const float alpha = grow ? ex2(m_used - mx) : 1.0f;
            if (grow) {
              l *= alpha;
              m_used = mx;
            }
            if (j != 0) {
              ok = rescale_o(alpha, u);
              if (!ok) break;
            }
          }
          const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;  // a row that sees nothing yet: every score is -inf, P = 0
          uint32_t pk[32];
          l += masked ? exp_half<false>(v, pk, scale_log2, neg_m) : exp_half<true>(v, pk, scale_log2, neg_m);
          // The P buffer of this tile is the one the PV product of tile u - 2 read: that product has long retired, but
          // nothing else orders the two.  o_done[b] completes once per two tiles, and between this thread's waits for
          // tiles u - 4 and u - 2 on it at most the product of tile u - 2 can have completed (that of tile u needs
          // this warp's arrival below): a parity wait tells the two states apart.
          if (u >= 2) {
            ok = wait_bar_warp(&ctrl->o_done[u & 1u], ((u - 2) >> 1) & 1u, wc, 236);
            if (!ok) break;
          }
          tmem_st32(lane_base + kSBufs * 128 + buf * 64 + g * 32, pk);
          tc_wait_st();
        } else if (u >= 2) {  // keep the phases of o_done observed in order
          ok = wait_bar_warp(&ctrl->o_done[u & 1u], ((u - 2) >> 1) & 1u, wc, 236);
          if (!ok) break;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(p_full0 + buf * 8u);
      }
      unit += (uint32_t)n;
      if (ok && n > 0) {
        // epilogue: wait for the last PV product of the piece, then store
        ok = wait_bar_warp(&ctrl->o_done[(unit - 1) & 1u], ((unit - 1) >> 1) & 1u, wc, 240);
      }
      const int slot = pi.slot[cta], target = pi.target[cta];
      // the row sum is the sum of its two halves (same reference exponent in both)
      ctrl->l_xch[g][r] = l;
      bar_sync_softmax();
      const float l_row = l + ctrl->l_xch[1 - g][r];
      if (ok && n > 0 && warp_live && slot != -2) {
        tc_fence_after();
        EpiArgs a;
        a.o_addr = o_addr;
        a.slot = slot;
        a.target = target;
        a.r = r;
        a.g = g;
        a.q_index = ri.q_index;
        a.m = m_used;
        a.l = l_row;
        store_row(a, out, lse, pp.partial_o, pp.partial_ml);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(epi_done0);  // one arrival per warp and piece, whatever happened above
      // Every softmax thread of the CTA takes part in the barriers below (a warp without query rows included).  The
      // first also closes the exchange of the row sums: nobody writes l_xch for the next piece before all have read.
      bar_sync_softmax();
      if (slot >= 0) {
        // The contributor that draws the last ticket of the M-tile merges; the decision is uniform over the CTA.
        // The partial stores of all threads are ordered before the barrier above, and the fence of the ticket taker
        // after it orders them (cumulatively) before the ticket; the merging CTA mirrors this on its side.
        if (threadIdx.x == 0) {
          __threadfence();
          ctrl->ticket = atomicAdd(pp.counters + target, 1u);
          __threadfence();
        }
        const TcTarget tg = pp.targets[target];
        bar_sync_softmax();
        const bool last = *reinterpret_cast<volatile uint32_t *>(&ctrl->ticket) == (uint32_t)tg.n_slots - 1u;
        bar_sync_softmax();  // everybody has read the ticket before the next piece may overwrite it
        if (last) {
          if (ok) merge_row(tg.slot_begin, tg.n_slots, r, g, ri.q_index, out, lse, pp.partial_o, pp.partial_ml);
          if (threadIdx.x == 0) pp.counters[target] = 0u;  // ready for the next launch, also after an aborted pass
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // no product of the pair is in flight and nobody reads tensor memory any more
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// ---- tensor maps -------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// A KV pool of n pages is viewed as [8-key groups][2 channel halves][8 keys][64 channels].
// kind 10: box = one page of one KV head (4 KB): two 8-key groups of two 1024-byte swizzle atoms each (K)
// kind 11: box = one channel half of one page of one KV head (2 KB): two 8-key groups of one atom each (V)
// kind 12: Q of n rows as [rows][q heads][128], box = 64 channels x G heads x T tokens
int get_pair_map(lr_ctx *ctx, int kind, const void *ptr, int64_t n, const CUtensorMap **out) {
  for (auto &e : ctx->tmaps)
    if (e.ptr == ptr && e.n == n && e.kind == kind) {
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
  ent.ptr = ptr;
  ent.n = n;
  ent.kind = kind;
  const lr_model &m = ctx->model;
  CUresult r;
  if (kind == 10 || kind == 11) {
    cuuint64_t dims[4] = {64, 8, 2, (cuuint64_t)n * m.n_kv_heads * (kPage / 8)};
    cuuint64_t strides[3] = {(cuuint64_t)kD * 2, 128, (cuuint64_t)kD * 2 * 8};
    cuuint32_t box[4] = {64, 8, kind == 10 ? 2u : 1u, kPage / 8};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    r = reinterpret_cast<EncodeTiledFn>(ctx->tmap_encode)(
        reinterpret_cast<CUtensorMap *>(ent.map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(ptr), dims, strides, box,
        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    const int G = m.n_q_heads / m.n_kv_heads, T = 128 / G;
    cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)m.n_q_heads, (cuuint64_t)n};
    cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)m.n_q_heads * kD * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)T};
    cuuint32_t estr[3] = {1, 1, 1};
    r = reinterpret_cast<EncodeTiledFn>(ctx->tmap_encode)(
        reinterpret_cast<CUtensorMap *>(ent.map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box,
        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) {
    ctx->tmaps.pop_back();
    set_error("cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return LR_ECUDA;
  }
  *out = reinterpret_cast<const CUtensorMap *>(ent.map);
  return LR_OK;
}

}  // namespace

int init_attn_pair_kernel() {
  return cuda_fail(cudaFuncSetAttribute(attn_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes),
                   "attn_pair_kernel shared-memory attribute");
}

// ---- host planning -----------------------------------------------------------------
int pair_build_host_plan(const lr_ctx *ctx, const lr_batch *b, const int32_t *req_br_off, const int32_t *span_tin,
                         const int32_t *span_last, PairHostPlan &out, Image &img) {
  out = PairHostPlan();
  const lr_model &m = ctx->model;
  const int G = m.n_q_heads / m.n_kv_heads;
  if (m.head_dim != kD) return LR_OK;  // other head sizes take the CUDA-core path
  if ((int64_t)b->n_pool_pages * m.n_kv_heads * kPage >= ((int64_t)1 << 31)) return LR_OK;  // tensor-map coordinates are 32-bit
  const int T = 128 / G;
  const int n_q_rows = b->cu_q[b->n_branch];
  std::vector<TcPage> pages;
  std::vector<TcRow> rows((size_t)std::max(1, n_q_rows));
  std::vector<TcReq> reqs;  // one per page list (request x pair of M-tiles); PrPiece.req indexes it
  struct Grp { int req, kv, mtile0, n_mt, n_tiles, first_piece, n_pieces; };
  std::vector<Grp> grps;
  // One page list per (request, pair of M-tiles): the prefix, the segments some branch of the group descends from and
  // the tails of its own branches up to the last token one of its rows sees.  Pages no row of the group can see are
  // left out, so no tile of the sweep is fully masked for everybody.
  reqs.clear();
  for (int r = 0; r < b->n_req; ++r) {
    const int s0 = b->req_span_off[r], s1 = b->req_span_off[r + 1];
    const int br0 = req_br_off[r], br1 = req_br_off[r + 1];
    if (br1 == br0) continue;  // a request without branches has no query rows
    if (br1 - br0 > 254) return LR_OK;
    const int q_row0 = b->cu_q[br0], n_q = b->cu_q[br1] - b->cu_q[br0];
    for (int i = br0; i < br1; ++i) {
      const int tin = span_tin[s0 + b->br_depth[i]];
      if ((b->br_own_len[i] + kPage - 1) / kPage > 2047) return LR_OK;
      const int q_len = b->cu_q[i + 1] - b->cu_q[i];
      for (int k = 0; k < q_len; ++k) {
        TcRow &w = rows[(size_t)b->cu_q[i] + k];
        w.depth_branch = tin | ((i - br0) << 16);
        w.limit = b->br_own_len[i] - q_len + k;
      }
    }
    const int n_mtiles = (n_q + T - 1) / T;
    for (int m0 = 0; m0 < n_mtiles; m0 += 2) {
      const int mts = std::min(2, n_mtiles - m0);
      const int row_lo = q_row0 + m0 * T, row_hi = q_row0 + std::min(n_q, (m0 + mts) * T);  // query rows of the group
      TcReq rq;
      memset(&rq, 0, sizeof(rq));
      rq.page_off = (int)pages.size();
      rq.q_row0 = q_row0;
      rq.n_q = n_q;
      std::vector<unsigned char> node_used((size_t)(s1 - s0), 0);  // by depth-first number: a branch of the group continues it
      std::vector<int> tail_limit((size_t)(br1 - br0), -1);        // last tail token a row of the group sees, per branch
      for (int i = br0; i < br1; ++i) {
        const int lo = std::max(row_lo, b->cu_q[i]), hi = std::min(row_hi, b->cu_q[i + 1]);
        if (lo >= hi) continue;
        node_used[span_tin[s0 + b->br_depth[i]]] = 1;
        tail_limit[i - br0] = rows[(size_t)hi - 1].limit;
      }
      auto add_span = [&](int slot, int len, int n_pg, int need, int last, int owner) {
        for (int p = 0; p < n_pg; ++p) {
          TcPage e;
          e.page = b->page_ids[slot + p];
          const uint32_t valid = (uint32_t)std::min(kPage, len - p * kPage);
          e.meta = valid | ((uint32_t)need << 5) | ((uint32_t)owner << 13) | ((uint32_t)(owner ? p : last) << 21);
          pages.push_back(e);
        }
      };
      add_span(b->span_slot[s0], b->span_len[s0], (b->span_len[s0] + kPage - 1) / kPage, 0, 255, 0);
      rq.n_dense_tiles = (b->span_len[s0] / kPage) / kPagesPerTile;
      for (int c = 1; s0 + c < s1; ++c) {
        bool seen = false;
        for (int t = span_tin[s0 + c]; t <= span_last[s0 + c] && !seen; ++t) seen = node_used[t];
        if (seen) add_span(b->span_slot[s0 + c], b->span_len[s0 + c], (b->span_len[s0 + c] + kPage - 1) / kPage, span_tin[s0 + c], span_last[s0 + c], 0);
      }
      for (int i = br0; i < br1; ++i)
        if (tail_limit[i - br0] >= 0) add_span(b->br_own_slot[i], b->br_own_len[i], tail_limit[i - br0] / kPage + 1, 0, 0, i - br0 + 1);
      rq.n_pages = (int)pages.size() - rq.page_off;
      while (pages.size() % kPagesPerTile) pages.push_back(TcPage{0, 0});  // absent pages of the last tile: nothing valid
      const int n_tiles = (rq.n_pages + kPagesPerTile - 1) / kPagesPerTile;
      const int list = (int)reqs.size();
      reqs.push_back(rq);
      for (int kv = 0; kv < m.n_kv_heads; ++kv) grps.push_back(Grp{list, kv, m0, mts, n_tiles, 0, 0});
    }
  }
  if (grps.empty()) return LR_OK;
  // Contiguous partition of the tile sequence (groups in order, tiles in order) over at most max_pairs pairs that
  // minimises the largest load.  A tile costs the same whatever the group holds (the pair applies it to both
  // M-tiles at once); a tile that needs masks (anything past the full prefix pages) costs 7/5 of a dense one; every
  // piece -- a pair's share of one group -- kPieceStartTiles tiles more (Q load, pipeline ramp, epilogue, a partial
  // to merge).  For a load limit L the greedy fill needs the fewest pairs possible; the smallest feasible L is found
  // by bisection.
  constexpr int kPieceStartTiles = 3, kDense = 5, kMasked = 7;  // costs in fifths of a dense tile
  auto tile_cost = [&](const Grp &g, int t) -> int64_t { return t >= reqs[g.req].n_dense_tiles ? kMasked : kDense; };
  int64_t total_w = 0, total_tiles = 0, lo = 0;
  for (const Grp &g : grps) {
    total_w += (int64_t)kPieceStartTiles * kDense;
    for (int t = 0; t < g.n_tiles; ++t) total_w += tile_cost(g, t);
    total_tiles += g.n_tiles;
    lo = std::max<int64_t>(lo, (int64_t)(kPieceStartTiles * kDense + kMasked));
  }
  const int64_t max_pairs = std::min<int64_t>(std::max(1, ctx->sm_count / 2), std::max<int64_t>(1, total_tiles / 2));
  std::vector<PrPiece> pieces;
  std::vector<int32_t> pair_off;
  auto walk = [&](int64_t L, bool emit) -> int64_t {
    int64_t n = 0, load = 0;
    for (size_t gi = 0; gi < grps.size(); ++gi) {
      Grp &g = grps[gi];
      if (emit) g.first_piece = (int)pieces.size();
      const int64_t start = (int64_t)kPieceStartTiles * kDense;
      const int n_dense = std::min(g.n_tiles, reqs[g.req].n_dense_tiles);
      bool new_piece = true;
      int t = 0;
      while (t < g.n_tiles) {
        const int run_end = t < n_dense ? n_dense : g.n_tiles;
        const int64_t cost = tile_cost(g, t);
        if (n == 0 || load + cost + (new_piece ? start : 0) > L) {  // open the next pair: its share of this group is a new piece
          ++n;
          load = 0;
          new_piece = true;
          if (emit) pair_off.push_back((int32_t)pieces.size());
        }
        if (new_piece) load += start;
        const int k = (int)std::max<int64_t>(1, std::min<int64_t>(run_end - t, (L - load) / cost));
        load += (int64_t)k * cost;
        if (emit) {
          if (new_piece) {
            PrPiece p;
            memset(&p, 0, sizeof(p));
            p.req = g.req; p.kv_head = g.kv; p.mtile0 = g.mtile0; p.n_mt = g.n_mt; p.tile_begin = t; p.tile_end = t + k;
            p.slot[0] = p.slot[1] = -2;
            p.target[0] = p.target[1] = -1;
            pieces.push_back(p);
          } else {
            pieces.back().tile_end = t + k;
          }
        }
        new_piece = false;
        t += k;
      }
      if (emit) g.n_pieces = (int)pieces.size() - g.first_piece;
    }
    return n;
  };
  int64_t hi = total_w;  // one pair takes everything
  while (lo < hi) {
    const int64_t mid = lo + (hi - lo) / 2;
    if (walk(mid, false) <= max_pairs) hi = mid; else lo = mid + 1;
  }
  const int n_pairs = (int)walk(lo, true);
  pair_off.push_back((int32_t)pieces.size());
  // Targets (one M-tile of one group) and the pieces that contribute to them, in piece order.
  int n_slots = 0;
  std::vector<TcTarget> targets;
  for (const Grp &g : grps)
    for (int mt = 0; mt < g.n_mt; ++mt) {
      if (g.n_pieces == 1) {
        pieces[g.first_piece].slot[mt] = -1;
        continue;
      }
      TcTarget tg;
      memset(&tg, 0, sizeof(tg));
      tg.req = g.req; tg.kv_head = g.kv; tg.mtile = g.mtile0 + mt;
      tg.slot_begin = n_slots; tg.n_slots = g.n_pieces;
      tg.q_row0 = reqs[g.req].q_row0; tg.n_q = reqs[g.req].n_q;
      for (int k = 0; k < g.n_pieces; ++k) {
        pieces[g.first_piece + k].slot[mt] = n_slots++;
        pieces[g.first_piece + k].target[mt] = (int32_t)targets.size();
      }
      targets.push_back(tg);
    }
  out.ok = true;
  out.n_pairs = n_pairs;
  out.n_pieces = (int)pieces.size();
  out.n_targets = (int)targets.size();
  out.n_partial_slots = n_slots;
  out.tokens_per_mtile = T;
  out.n_pages = (int)pages.size();
  static_assert(sizeof(PrHead) == 256, "one pair head = 256 bytes");
  std::vector<PrHead> heads((size_t)n_pairs);
  for (int c = 0; c < n_pairs; ++c) {
    PrHead &h = heads[c];
    memset(&h, 0, sizeof(h));
    h.piece0 = pair_off[c];
    h.piece1 = pair_off[c + 1];
    if (h.piece1 > h.piece0) {
      h.first = pieces[h.piece0];
      h.first_req = reqs[h.first.req];
      const int c0 = h.first.tile_begin >> 2;
      for (int k = 0; k < 32; ++k) {
        const int idx = c0 * 32 + k;
        h.first_pages[k] = idx < h.first_req.n_pages ? pages[(size_t)h.first_req.page_off + idx].page : -1;
      }
    }
  }
  out.o_heads = img.add(heads.data(), heads.size() * sizeof(PrHead));
  out.o_pages = img.add(pages.data(), pages.size() * sizeof(TcPage));
  out.o_rows = img.add(rows.data(), rows.size() * sizeof(TcRow));
  out.o_pieces = img.add(pieces.data(), pieces.size() * sizeof(PrPiece));
  if (reqs.empty()) reqs.push_back(TcReq{});
  out.o_reqs = img.add(reqs.data(), reqs.size() * sizeof(TcReq));
  if (targets.empty()) targets.push_back(TcTarget{});  // keep the section non-empty
  out.o_targets = img.add(targets.data(), targets.size() * sizeof(TcTarget));
  // scratch behind the image: ticket counters (zeroed at upload, left zero by every launch), (exponent, sum) pairs,
  // fp32 partial outputs
  out.s_counters = 0;
  out.scratch_zero_bytes = ((size_t)std::max(1, out.n_targets) * sizeof(uint32_t) + 255) / 256 * 256;
  out.s_ml = out.scratch_zero_bytes;
  out.s_o = out.s_ml + ((size_t)n_slots * 128 * 2 * sizeof(float) + 255) / 256 * 256;
  out.scratch_bytes = out.s_o + (size_t)n_slots * 128 * kD * sizeof(float);
  return LR_OK;
}

void pair_bind_device_plan(const PairHostPlan &h, unsigned char *image_base, unsigned char *scratch_base, lr_plan *p) {
  p->pair_ok = h.ok;
  p->pr_pieces = h.n_pieces;
  p->pr_partial_slots = h.n_partial_slots;
  p->o_pr_pages = h.o_pages;
  p->o_pr_heads = h.o_heads;
  p->n_pr_pages = h.ok ? h.n_pages : 0;
  p->n_pr_heads = h.ok ? h.n_pairs : 0;
  memset(&p->pr, 0, sizeof(p->pr));
  if (!h.ok) return;
  DevPairPlan &t = p->pr;
  t.heads = reinterpret_cast<const PrHead *>(image_base + h.o_heads);
  t.pages = reinterpret_cast<const TcPage *>(image_base + h.o_pages);
  t.rows = reinterpret_cast<const TcRow *>(image_base + h.o_rows);
  t.pieces = reinterpret_cast<const PrPiece *>(image_base + h.o_pieces);
  t.reqs = reinterpret_cast<const TcReq *>(image_base + h.o_reqs);
  t.targets = reinterpret_cast<const TcTarget *>(image_base + h.o_targets);
  t.n_pairs = h.n_pairs;
  t.n_targets = h.n_targets;
  t.tokens_per_mtile = h.tokens_per_mtile;
  t.wait_limit_us = 1000000u;  // one second per wait, measured on the global timer
  t.phantom_tx_bytes = 0;
  t.counters = reinterpret_cast<uint32_t *>(scratch_base + h.s_counters);
  t.partial_ml = reinterpret_cast<float *>(scratch_base + h.s_ml);
  t.partial_o = reinterpret_cast<float *>(scratch_base + h.s_o);
}

int launch_attn_pair(lr_plan *p, const void *q, const void *k, const void *v, void *out, float *lse, float scale,
                     cudaStream_t s) {
  const CUtensorMap *mp = nullptr;
  if (int rc = get_pair_map(p->ctx, 10, k, p->dev.n_pool_pages, &mp)) return rc;
  const CUtensorMap kmap = *mp;  // the cache may reallocate when the next map is added
  if (int rc = get_pair_map(p->ctx, 11, v, p->dev.n_pool_pages, &mp)) return rc;
  const CUtensorMap vmap = *mp;
  if (int rc = get_pair_map(p->ctx, 12, q, p->dev.n_q_rows, &mp)) return rc;
  const CUtensorMap qmap = *mp;
  const float scale_log2 = scale * 1.4426950408889634f;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(2u * (unsigned)p->pr.n_pairs, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, attn_pair_kernel, kmap, vmap, qmap, p->dev, p->pr, reinterpret_cast<uint16_t *>(out), lse,
                                     scale_log2);
  p->ctx->launches++;
  return cuda_fail(e, "attn_pair_kernel launch");
}

}  // namespace lr
