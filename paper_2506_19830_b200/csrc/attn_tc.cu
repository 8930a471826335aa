// Tensor-core nested-prefix attention for sm_100a (head_dim 128).
//
// Work decomposition.  For one request the *extended chain* is the list of its
// KV pages in the order prefix, segments 1..gamma, branch tails; 8 consecutive
// pages form a 128-key tile.  All query rows of the request that share one KV
// head -- (query token, head-in-group) pairs, floor(128/G) tokens per 128-row
// M-tile -- are processed against a tile at once, so a KV page is fetched from
// HBM once for every branch and every GQA head that can see it.  A *group* is
// (request, KV head, one or two M-tiles); the tiles of all groups, weighted, are
// cut into equal contiguous ranges, one per CTA (one CTA per SM); a range may
// cover parts of several groups (*pieces*).
//
// A CTA runs two independent *streams*, each with its own score tile S, output
// accumulator O (both in tensor memory), MMA issuer warp and softmax warpgroup:
// for a piece with two M-tiles stream s is M-tile s over every tile; for a piece
// with one M-tile stream s takes every other tile (a split of the keys inside
// the CTA).  While one stream is in its softmax the tensor pipe works for the
// other.  A stream whose result is the only contribution to its M-tile writes
// bf16 output; otherwise it writes an fp32 partial (reference exponent, sum,
// unnormalised O) and a small second kernel merges the partials of an M-tile in
// a fixed order.  The two streams of a one-M-tile piece hold partial results of the
// same rows; they are combined inside the CTA (stream 0 reads stream 1's accumulator
// from tensor memory) and leave as one result.
//
// One CTA = 12 warps in three warpgroups (registers are moved from the service warps to the
// softmax warpgroups with setmaxnreg):
//   warp 8      TMA producer: the Q tiles of a piece (3-D boxes: 64 channels x G
//               heads x T tokens, so that the rows land packed) and, per tile,
//               8 + 8 bulk tensor copies (one 4 KB box per page, K and V) into a
//               5-stage ring of 32 KB buffers.  A box is a 4-D view of the page,
//               [8-key group][channel half][8 keys][64 channels], so a tile lies in
//               shared memory as 1024-byte swizzle atoms, the two channel halves of
//               an 8-key group side by side (groups 2048 bytes apart): the layout
//               the MMA descriptors read with SBO = 2048.  One box per page rather
//               than one per page half matters: the producer spends about 100
//               cycles per box, and 32 boxes per tile made it a bottleneck.
//               Every copy is for this CTA alone.
//   warps 9, 10 MMA issuers of stream 0 and 1 (warp 11 idles): tcgen05.mma (M=128, N=128, K=16,
//               bf16 -> fp32) for S = Q K^T (both operands in shared memory) and
//               O += P V (P read from tensor memory, V from shared memory as the
//               N-major operand).  Issue blocks while the tensor pipe is full, so
//               one issuer per stream lets the waits of one overlap the MMAs of
//               the other.
//   warps 0-3   softmax of stream 0, one thread per query row: tcgen05.ld gives a
//   warps 4-7   softmax of stream 1  thread its whole row of S in registers, so
//               row max and row sum need no cross-lane traffic.  One sweep:
//               max (3-input max), lazy rescale of O in tensor memory only when
//               the maximum grew by more than 2^8, exp2 with packed fp32 FMA/ADD,
//               bf16 P written back over S.
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each; P_s
// occupies the first 64 columns of S_s.
//
// Visibility.  Tiles made only of full prefix pages need no mask.  In every other
// tile each page carries (valid tokens, first and last node number that sees it,
// owning branch, tail offset) and every row carries (node number, branch, causal
// limit): a row sees the first n_ok tokens of a page, with n_ok from those
// numbers.  Node numbers are depth-first, so "the row's node descends from the
// page's segment" is an interval test; on the nested chain the number is the
// depth and the interval is [segment index, gamma].  V rows of
// invalid token slots are zeroed in shared memory before the PV product so that
// whatever the slack holds (NaN included) cannot reach the output.
//
// Every wait on an mbarrier is bounded by the global timer; when one expires the
// CTA raises its abort flag, records LR_ETIMEOUT in the status word, drains what
// it has in flight, frees its tensor memory and returns.
#include <cuda.h>

#include <algorithm>

#include "lr_common.cuh"

namespace lr {

namespace {

constexpr int kD = 128;
constexpr int kStages = 5;
constexpr int kTileBytes = 32768;  // [2 halves of 64 channels][128 keys or rows][128 B]
constexpr int kHalfBytes = 16384;
constexpr int kAtomBytes = 1024;   // K/V tiles: 8 keys x 64 channels, one 128-byte-swizzle atom
constexpr int kGroupBytes = 2048;  // ... two atoms (the two channel halves) per 8-key group
constexpr int kThreads = 384;
constexpr int kPagesPerTile = 8;
constexpr uint64_t kDrainLimitNs = 50ull * 1000ull * 1000ull;
constexpr float kRescaleThreshold = 8.0f;  // log2 units: the reference exponent follows the row maximum within 2^8
constexpr float kRedoThreshold = 64.0f;    // log2 units: beyond this a tile is redone with its own maximum as reference

struct __align__(8) Ctrl {
  uint64_t kv_full[kStages], kv_empty[kStages];
  uint64_t q_full, q_empty;
  uint64_t s_full[2][2], p_full[2][2], o_done[2];  // [stream][half]
  uint64_t epi_done, drain[2];
  uint64_t xch;           // stream 1 -> stream 0: its (m, l) are published and its accumulator is final
  uint32_t tmem_base;
  int abort_flag;
  uint64_t wait_limit_ns;  // bound of every wait, measured on the global timer
  float2 ml_xch[128];     // (reference exponent, row sum) of stream 1's rows, for the in-CTA combination
};
constexpr int kCtrlBytes = 2048;
static_assert(sizeof(Ctrl) <= kCtrlBytes, "Ctrl must fit behind the tiles");
constexpr int kSmemBytes = 2 * kTileBytes + kStages * kTileBytes + kCtrlBytes;  // tiles, then Ctrl; the base must be 1024-aligned
static_assert(kSmemBytes <= 227 * 1024, "shared memory per CTA");

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
// both tests in flight together: bit 0 = first barrier's phase complete, bit 1 = second's
__device__ __forceinline__ uint32_t mbar_test_wait2(uint64_t *bar_a, uint32_t parity_a, uint64_t *bar_b, uint32_t parity_b) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .b32 a, b;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 q, [%3], %4;\n\t"
      "selp.b32 a, 1, 0, p;\n\tselp.b32 b, 2, 0, q;\n\tor.b32 %0, a, b;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar_a)), "r"(parity_a), "r"(smem_u32(bar_b)), "r"(parity_b)
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

// Tiled bulk tensor copies global -> shared for this CTA alone, completion on an mbarrier.
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
// Instruction descriptors: D fp32, A and B bf16, M = 128 (bits 24-28 = M/16), N in bits 17-22 (= N/8).
// QK: N = 64 keys of a half-tile, both operands K-major.  PV: N = 128 channels, bit 16 selects the N-major B operand.
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | (8u << 24);
constexpr uint32_t kIdescQK = kIdescBase | ((64u >> 3) << 17);
constexpr uint32_t kIdescPV = kIdescBase | ((128u >> 3) << 17) | (1u << 16);

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

// tcgen05.ld / tcgen05.st, shape 32x32b: thread i of the warp owns lane (base + i), consecutive columns.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, uint32_t (&r)[64]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
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

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait: gives up after kWaitLimitNs of wall time.  Returns false when the wait expired or
// another role of the CTA gave up.
__device__ __forceinline__ bool wait_bar_lane(uint64_t *bar, uint32_t parity, Ctrl *ctrl, int32_t *status, int code) {
  if (mbar_test_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  for (uint32_t i = 1;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 31u) == 0u) {
      if (*reinterpret_cast<volatile int *>(&ctrl->abort_flag)) return false;
      if (global_ns() - t0 > ctrl->wait_limit_ns) break;
    }
  }
  *reinterpret_cast<volatile int *>(&ctrl->abort_flag) = 1;
  status[0] = kDevTimeout;
  status[1] = code;
  return false;
}

// Every wait of the kernel is made by a whole warp: the warp goes on only if every lane's wait succeeded, so that it
// never executes its warp-wide instructions half in and half out of an abort.
__device__ __forceinline__ bool wait_bar(uint64_t *bar, uint32_t parity, Ctrl *ctrl, int32_t *status, int code) {
  return __all_sync(0xFFFFFFFFu, wait_bar_lane(bar, parity, ctrl, status, code)) != 0;
}

// ---- ring order ----------------------------------------------------------------------
// Within a piece of n tiles the producer emits K and V tiles in the order the MMA issuers first
// touch them.  With la = K tiles issued ahead of the first PV (1 for two M-tiles, 2 for the
// even/odd split): K(0..min(la,n)-1), then for u = 0..n-1: V(u), and K(u+la) while u+la < n.
struct RingOrder {
  int n, la, la_c, np;  // np = number of (V, K) pairs
  __device__ __forceinline__ RingOrder(int n_, int mode) : n(n_), la(mode == 2 ? 1 : 2) {
    la_c = min(la, n);
    np = max(0, n - la);
  }
  __device__ __forceinline__ int pos_k(int t) const { return t < la ? t : la_c + 2 * (t - la) + 1; }
  __device__ __forceinline__ int pos_v(int u) const { return u < np ? la_c + 2 * u : la_c + 2 * np + (u - np); }
  // step i (= ring position within the piece) of the 2n steps -> tile, and whether it is a V tile
  __device__ __forceinline__ int step(int i, bool &is_v) const {
    if (i < la_c) { is_v = false; return i; }
    const int j = i - la_c;
    if (j < 2 * np) { is_v = !(j & 1); return (j >> 1) + ((j & 1) ? la : 0); }
    is_v = true;
    return np + (j - 2 * np);
  }
};

struct RowInfo {
  int depth;       // depth-first number of the node the row's branch continues (on a chain: segments it sees); -1 for padding rows
  int branch;      // local branch index within the request; -1 for padding rows
  int limit;       // last tail token the row sees
  int64_t q_index; // (query row * n_q_heads + head), -1 for padding rows
};

// Row r (0..127) of M-tile mt of (request, KV head): token mt*T + r/G, head kv*G + r%G.
__device__ __forceinline__ RowInfo row_info(const DevBatch &d, const DevTcPlan &tc, const TcReq &rq, int T, int mt, int r, int kv) {
  RowInfo ri;
  ri.depth = -1;
  ri.branch = -1;
  ri.limit = -1;
  ri.q_index = -1;
  const int G = d.group;
  const int tok = mt * T + r / G;
  if (r < T * G && tok < rq.n_q) {
    const int row = rq.q_row0 + tok;
    const int2 w = __ldg(reinterpret_cast<const int2 *>(tc.rows + row));
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

__device__ __forceinline__ float bits_f(uint32_t u) { return __uint_as_float(u); }

// -inf on the score columns of one 64-key half that the row does not see
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
// P = exp2(scale * s - m) for 64 scores -> 32 packed bf16 pairs; returns the fp32 sum
__device__ __forceinline__ float exp_half(const uint32_t (&v)[64], uint32_t (&pk)[32], float scale_log2, float neg_m) {
  const float2 sc = make_float2(scale_log2, scale_log2), nm = make_float2(neg_m, neg_m);
  float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
  for (int i = 0; i < 64; i += 4) {
    float2 y0 = ffma2(make_float2(bits_f(v[i]), bits_f(v[i + 1])), sc, nm);
    float2 y1 = ffma2(make_float2(bits_f(v[i + 2]), bits_f(v[i + 3])), sc, nm);
    y0.x = ex2(y0.x);
    y0.y = ex2(y0.y);
    y1.x = ex2(y1.x);
    y1.y = ex2(y1.y);
    acc0 = fadd2(acc0, y0);
    acc1 = fadd2(acc1, y1);
    pk[i >> 1] = pack_bf16(y0.x, y0.y);
    pk[(i >> 1) + 1] = pack_bf16(y1.x, y1.y);
  }
  acc0 = fadd2(acc0, acc1);
  return acc0.x + acc0.y;
}

// exp_half on v, and beside it (in the shadow of the MUFU) the maximum of the raw scores
__device__ __forceinline__ float exp_half_max(const uint32_t (&v)[64], uint32_t (&pk)[32], float scale_log2, float neg_m,
                                              float &raw_max) {
  const float2 sc = make_float2(scale_log2, scale_log2), nm = make_float2(neg_m, neg_m);
  float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
  float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
  for (int i = 0; i < 64; i += 4) {
    float2 y0 = ffma2(make_float2(bits_f(v[i]), bits_f(v[i + 1])), sc, nm);
    float2 y1 = ffma2(make_float2(bits_f(v[i + 2]), bits_f(v[i + 3])), sc, nm);
    m0 = max3(m0, bits_f(v[i]), bits_f(v[i + 1]));
    y0.x = ex2(y0.x);
    y0.y = ex2(y0.y);
    m1 = max3(m1, bits_f(v[i + 2]), bits_f(v[i + 3]));
    y1.x = ex2(y1.x);
    y1.y = ex2(y1.y);
    acc0 = fadd2(acc0, y0);
    acc1 = fadd2(acc1, y1);
    pk[i >> 1] = pack_bf16(y0.x, y0.y);
    pk[(i >> 1) + 1] = pack_bf16(y1.x, y1.y);
  }
  raw_max = fmaxf(m0, m1);
  acc0 = fadd2(acc0, acc1);
  return acc0.x + acc0.y;
}

// The store epilogue of a softmax thread: row r of the accumulator at o_addr (and, when the CTA's two streams worked on
// the same rows, of the other stream's at o_other, weighted) goes out as bf16 (slot < 0) or as an fp32 partial.
// Not inlined: its two 64-register row buffers must not weigh on the register allocation of the sweep.
__device__ __noinline__ void store_rows(uint32_t o_addr, uint32_t o_other, int slot, bool pair, float w_self, float w_other, float m_out,
                                        float l_out, int r, int64_t q_index, uint16_t *__restrict__ out, float *__restrict__ lse,
                                        float *__restrict__ partial_o, float *__restrict__ partial_ml) {
          const bool any_other = pair && __any_sync(0xFFFFFFFFu, w_other > 0.f);
          if (slot < 0) {
            const float inv = 1.0f / l_out, a = w_self * inv, b = w_other * inv;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
              uint32_t o[64];
              tmem_ld64(o_addr + hf * 64, o);
              tc_wait_ld();
#pragma unroll
              for (int c = 0; c < 64; ++c) o[c] = __float_as_uint(bits_f(o[c]) * a);
              if (any_other) {  // the loads are warp-wide; a row whose other stream saw nothing keeps its own values
                uint32_t p[64];
                tmem_ld64(o_other + hf * 64, p);
                tc_wait_ld();
                if (w_other > 0.f) {
#pragma unroll
                  for (int c = 0; c < 64; ++c) o[c] = __float_as_uint(fmaf(bits_f(p[c]), b, bits_f(o[c])));
                }
              }
              if (q_index >= 0) {
                uint4 *dst = reinterpret_cast<uint4 *>(out + q_index * kD + hf * 64);
#pragma unroll
                for (int jj = 0; jj < 8; ++jj)
                  dst[jj] = make_uint4(pack_bf16(bits_f(o[8 * jj]), bits_f(o[8 * jj + 1])), pack_bf16(bits_f(o[8 * jj + 2]), bits_f(o[8 * jj + 3])),
                                       pack_bf16(bits_f(o[8 * jj + 4]), bits_f(o[8 * jj + 5])), pack_bf16(bits_f(o[8 * jj + 6]), bits_f(o[8 * jj + 7])));
              }
            }
            if (lse != nullptr && q_index >= 0) lse[q_index] = (m_out + log2f(l_out)) * 0.6931471805599453f;
          } else {
            const int64_t prow = (int64_t)slot * 128 + r;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
              uint32_t o[64];
              tmem_ld64(o_addr + hf * 64, o);
              tc_wait_ld();
              if (pair) {
#pragma unroll
                for (int c = 0; c < 64; ++c) o[c] = __float_as_uint(bits_f(o[c]) * w_self);
                if (any_other) {
                  uint32_t p[64];
                  tmem_ld64(o_other + hf * 64, p);
                  tc_wait_ld();
                  if (w_other > 0.f) {
#pragma unroll
                    for (int c = 0; c < 64; ++c) o[c] = __float_as_uint(fmaf(bits_f(p[c]), w_other, bits_f(o[c])));
                  }
                }
              }
              if (q_index >= 0) {
                // chunk-major: 16-byte chunk k of row r at [slot][k][r], so a warp's store is 512 contiguous bytes
                uint4 *dst = reinterpret_cast<uint4 *>(partial_o) + ((int64_t)slot * 32 + hf * 16) * 128 + r;
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) dst[jj * 128] = make_uint4(o[4 * jj], o[4 * jj + 1], o[4 * jj + 2], o[4 * jj + 3]);
              }
            }
            if (q_index >= 0) *reinterpret_cast<float2 *>(partial_ml + prow * 2) = make_float2(m_out, l_out);
          }
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
               const __grid_constant__ CUtensorMap q_map, DevBatch d, DevTcPlan tc, uint16_t *__restrict__ out,
               float *__restrict__ lse, float scale_log2) {
  extern __shared__ __align__(1024) unsigned char smem[];
  if ((smem_u32(smem) & 1023u) != 0u) {  // the swizzled tiles need a 1024-byte aligned base
    if (threadIdx.x == 0) {
      d.status[0] = kDevBounds;
      d.status[1] = 250;
    }
    return;
  }
  unsigned char *q_smem = smem;                         // 2 x 32 KB
  unsigned char *kv_smem = smem + 2 * kTileBytes;       // kStages x 32 KB
  Ctrl *ctrl = reinterpret_cast<Ctrl *>(kv_smem + kStages * kTileBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // rows of a Q tile that no copy writes must hold finite values
  for (int i = threadIdx.x; i < 2 * kTileBytes / 16; i += kThreads) reinterpret_cast<uint4 *>(q_smem)[i] = make_uint4(0, 0, 0, 0);
  fence_proxy_async();
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&ctrl->kv_full[s], 1);
      mbar_init(&ctrl->kv_empty[s], 2);  // one arrival per MMA issuer
    }
    mbar_init(&ctrl->q_full, 1);
    mbar_init(&ctrl->q_empty, 2);
    for (int s = 0; s < 2; ++s) {
      for (int h = 0; h < 2; ++h) {
        mbar_init(&ctrl->s_full[s][h], 1);
        mbar_init(&ctrl->p_full[s][h], 128);
      }
      mbar_init(&ctrl->o_done[s], 1);
      mbar_init(&ctrl->drain[s], 1);
    }
    mbar_init(&ctrl->epi_done, 256);
    mbar_init(&ctrl->xch, 128);
    ctrl->abort_flag = 0;
    ctrl->wait_limit_ns = (uint64_t)tc.wait_limit_us * 1000ull;
    fence_barrier_init();
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctrl->tmem_base)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&ctrl->tmem_base);
  // inputs may come from the kernel launched just before this one
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const TcCtaHead *head = tc.heads + blockIdx.x;
  const int piece0 = head->piece0, piece1 = head->piece1;
  const int T = tc.tokens_per_mtile;
  const int G = d.group;

  if (warp >= 8) {
   // service warpgroup: needs few registers; the softmax threads hold a whole row of scores in theirs
   // setmaxnreg.inc blocks until its request fits into what the CTA was launched with (168 registers x 384
   // threads), so the totals after the moves must not exceed that: 72 x 128 + 216 x 256 = 168 x 384.
   asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
   if (warp == 8) {
    // ======================= TMA producer ==========================================
    uint32_t ring = 0, q_count = 0;
    bool ok = true;
    const uint32_t q_box_bytes = (uint32_t)(64 * G * T * 2);
    for (int pc = piece0; pc < piece1 && ok; ++pc) {
      const TcPiece pi = pc == piece0 ? head->first : tc.pieces[pc];
      const TcReq rq = pc == piece0 ? head->first_req : tc.reqs[pi.req];
      const int n = pi.tile_end - pi.tile_begin;
      // Q tiles of the piece, once the MMAs of the previous piece no longer read the buffers
      ok = wait_bar(&ctrl->q_empty, (q_count & 1u) ^ 1u, ctrl, d.status, 205);
      if (!ok) break;
      if (lane == 0) mbar_arrive_expect_tx(&ctrl->q_full, (uint32_t)pi.n_mt * 2u * q_box_bytes);
      __syncwarp();
      if (lane < 2 * pi.n_mt)
        tma_load_3d(smem_u32(q_smem) + (lane >> 1) * kTileBytes + (lane & 1) * kHalfBytes, &q_map, (lane & 1) * 64, pi.kv_head * G,
                    rq.q_row0 + (pi.mtile0 + (lane >> 1)) * T, &ctrl->q_full);
      ++q_count;
      const RingOrder ord(n, pi.n_mt);
      // Page ids arrive 32 at a time (one per lane = 4 tiles) and one chunk ahead of their first use,
      // so no step of the loop waits for a load it has just issued.
      auto load_chunk = [&](int c) -> int32_t {
        const int idx = c * 32 + lane;
        int32_t pg = -1;  // absent page
        if (idx < rq.n_pages) {
          pg = tc.pages[rq.page_off + idx].page;
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
      if (pc == piece0) {  // the first chunk of the first piece comes with the CTA head
        pg_cur = head->first_pages[lane];
        if (c_cur * 32 + lane < rq.n_pages && (pg_cur < 0 || pg_cur >= d.n_pool_pages)) {
          d.status[0] = kDevBounds;
          d.status[1] = 201;
          pg_cur = 0;
        }
      } else {
        pg_cur = load_chunk(c_cur);
      }
      for (int i = 0; i < 2 * n && ok; ++i, ++ring) {
        bool is_v;
        const int t = pi.tile_begin + ord.step(i, is_v);
        if (is_v && (t >> 2) > c_cur) {  // the V index is the oldest tile still needed
          ++c_cur;
          pg_cur = pg_nxt;
          pg_nxt = load_chunk(c_cur + 1);
        }
        const int32_t page = __shfl_sync(0xFFFFFFFFu, (t >> 2) == c_cur ? pg_cur : pg_nxt, (t & 3) * 8 + (lane & 7));
        const int npages = min(kPagesPerTile, rq.n_pages - t * kPagesPerTile);
        const uint32_t stage = ring % kStages;
        ok = wait_bar(&ctrl->kv_empty[stage], ((ring / kStages) & 1u) ^ 1u, ctrl, d.status, 210);
        if (!ok) break;
        if (lane == 0)
          mbar_arrive_expect_tx(&ctrl->kv_full[stage], (uint32_t)npages * 4096u + ((blockIdx.x == 0 && ring == 0) ? tc.phantom_tx_bytes : 0u));
        __syncwarp();
        if (lane < 8 && page >= 0) {  // one 4 KB box per page: two 8-key groups x two d halves
          const uint32_t dst = smem_u32(kv_smem + stage * kTileBytes) + lane * 4096;
          tma_load_4d(dst, is_v ? &v_map : &k_map, 0, 0, 0, (int32_t)(((int64_t)page * d.n_kv_heads + pi.kv_head) * 2),
                      &ctrl->kv_full[stage]);
        }
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
   } else if (warp == 9 || warp == 10) {
    // ======================= MMA issuer of stream s ====================================
    // Both issuers walk every ring position of a piece in order: a position this stream uses is
    // consumed by its MMAs (released by a tcgen05.commit), one it does not use (the other
    // stream's tiles in the even/odd split) is released with a plain arrive once it has landed.
    // So neither issuer nor the producer can get a whole ring ahead of the other.
    const int s = warp - 9;
    uint32_t ring_base = 0, waited = 0, p_cnt = 0, pc_idx = 0;
    bool ok = true;
    const uint32_t q_addr = smem_u32(q_smem), kv_addr = smem_u32(kv_smem);
    const uint32_t s_tmem = tmem + s * 128, o_tmem = tmem + 256 + s * 128;
    // Descriptors differ from a base only in the start-address field (units of 16 bytes).
    const uint64_t qdesc0 = make_desc(q_addr, 16, 1024), kdesc0 = make_desc(kv_addr, 16, kGroupBytes),
                   vdesc0 = make_desc(kv_addr, kAtomBytes, kGroupBytes);
    auto issue_qk = [&](int m, uint32_t stage, int half) {  // S_s[half] = Q_m K^T over 64 of the 128 keys
      const uint64_t a = qdesc0 + (uint64_t)(m * (kTileBytes >> 4)),
                     b = kdesc0 + (uint64_t)(stage * (kTileBytes >> 4) + half * (8 * kGroupBytes >> 4));
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_ss(s_tmem + half * 64, a + (uint64_t)(h * (kHalfBytes >> 4) + kk * 2), b + (uint64_t)(h * (kAtomBytes >> 4) + kk * 2),
                 kIdescQK, (h | kk) != 0);
    };
    auto issue_pv = [&](uint32_t stage, int half, bool acc) {  // O_s (+)= P_s[half] V over 64 of the 128 keys
      const uint64_t b = vdesc0 + (uint64_t)(stage * (kTileBytes >> 4) + half * (8 * kGroupBytes >> 4));
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4)
        mma_ts(o_tmem, s_tmem + half * 64 + k4 * 8, b + (uint64_t)(k4 * (2 * kGroupBytes >> 4)), kIdescPV, acc || k4 != 0);
    };
    for (int pc = piece0; pc < piece1 && ok; ++pc, ++pc_idx) {
      const TcPiece pi = pc == piece0 ? head->first : tc.pieces[pc];
      const TcReq rq = pc == piece0 ? head->first_req : tc.reqs[pi.req];
      const int n = pi.tile_end - pi.tile_begin, mode = pi.n_mt;
      const RingOrder ord(n, mode);
      const int my_units = mode == 2 ? n : (n - s + 1) / 2;
      const int m_tile = mode == 2 ? s : 0;
      // waits, in ring order, until absolute ring position `pos` has landed; positions on the way
      // belong to the other stream and are released here
      auto need = [&](uint32_t pos, int code) -> bool {
        while (waited <= pos) {
          if (!wait_bar(&ctrl->kv_full[waited % kStages], (waited / kStages) & 1u, ctrl, d.status, code)) return false;
          if (waited < pos && lane == 0) mbar_arrive(&ctrl->kv_empty[waited % kStages]);
          ++waited;
        }
        return true;
      };
      // after the MMAs that read the stage: arrives when they retire (the other issuer arrives for itself)
      auto release = [&](uint32_t pos) { tc_commit(&ctrl->kv_empty[pos % kStages]); };
      ok = wait_bar(&ctrl->q_full, pc_idx & 1u, ctrl, d.status, 220);
      if (!ok) break;
      if (my_units > 0) {
        const uint32_t pos = ring_base + ord.pos_k(mode == 2 ? 0 : s);
        ok = need(pos, 221);
        if (!ok) break;
        tc_fence_after();
        if (lane == 0) {
          issue_qk(m_tile, pos % kStages, 0);
          tc_commit(&ctrl->s_full[s][0]);
          issue_qk(m_tile, pos % kStages, 1);
          tc_commit(&ctrl->s_full[s][1]);
          release(pos);
          if (my_units == 1) tc_commit(&ctrl->q_empty);  // last QK of the piece: this stream is done with the Q buffers
        }
        __syncwarp();
      } else {
        if (lane == 0) mbar_arrive(&ctrl->q_empty);
        // nothing to issue in this piece: still observe the previous piece's epilogue phase, so that the parity
        // wait of a later piece never finds this issuer two phases behind
        if (pc_idx > 0) {
          ok = wait_bar(&ctrl->epi_done, (pc_idx - 1) & 1u, ctrl, d.status, 228);
          if (!ok) break;
        }
      }
      for (int j = 0; j < my_units && ok; ++j) {
        const int t = mode == 2 ? j : 2 * j + s;
        const uint32_t pos_v = ring_base + ord.pos_v(t), sV = pos_v % kStages;
        if (mode == 2 && j + 1 < my_units && waited == pos_v &&
            mbar_test_wait2(&ctrl->kv_full[pos_v % kStages], (pos_v / kStages) & 1u, &ctrl->kv_full[(pos_v + 1) % kStages],
                            ((pos_v + 1) / kStages) & 1u) == 3u)
          waited = pos_v + 2;  // V of this tile and K of the next (the position right behind it) have both landed
        ok = need(pos_v, 222);
        if (!ok) break;
        if (pi.tile_begin + t >= rq.n_dense_tiles) {
          // zero the V rows of token slots that hold no valid token (slack of a last page, absent pages);
          // with two M-tiles both issuers write the same zeros
          unsigned char *vs = kv_smem + sV * kTileBytes;
          const TcPage *pg = tc.pages + rq.page_off + (pi.tile_begin + t) * kPagesPerTile;
          for (int p = 0; p < kPagesPerTile; ++p) {
            const int valid = pg[p].meta & 31;
            for (int idx = lane; idx < (kPage - valid) * 16; idx += 32) {
              const int key = p * kPage + valid + (idx >> 4), h = (idx >> 3) & 1, ch = idx & 7;
              *reinterpret_cast<uint4 *>(vs + (key >> 3) * kGroupBytes + h * kAtomBytes + (key & 7) * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
            }
          }
          fence_proxy_async();
          __syncwarp();
        }
        const bool has_next = j + 1 < my_units;
        uint32_t pos_k = 0;
        if (has_next) {
          pos_k = ring_base + ord.pos_k(mode == 2 ? j + 1 : 2 * (j + 1) + s);
          ok = need(pos_k, 226);
          if (!ok) break;
        }
        if (j == 0 && pc_idx > 0) {  // the epilogue of the previous piece has read O_0 and O_1
          ok = wait_bar(&ctrl->epi_done, (pc_idx - 1) & 1u, ctrl, d.status, 223);
          if (!ok) break;
        }
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          // P of this half is in place: O += P V, then the buffer takes the scores of the next tile's half
          ok = wait_bar(&ctrl->p_full[s][half], p_cnt & 1u, ctrl, d.status, 224 + s);
          if (!ok) break;
          tc_fence_after();
          if (lane == 0) {
            issue_pv(sV, half, (j | half) != 0);
            tc_commit(&ctrl->o_done[s]);
            if (half == 1) release(pos_v);
            if (has_next) {
              issue_qk(m_tile, pos_k % kStages, half);
              tc_commit(&ctrl->s_full[s][half]);
              if (half == 1) {
                release(pos_k);
                if (j + 2 == my_units) tc_commit(&ctrl->q_empty);  // last QK of the piece
              }
            }
          }
          __syncwarp();
        }
        ++p_cnt;
      }
      if (!ok) break;
      // positions of the piece this stream never touched (the tail of the other stream's tiles)
      ring_base += 2u * (uint32_t)n;
      if (waited < ring_base) {
        ok = need(ring_base - 1, 227);
        if (!ok) break;
        if (lane == 0) mbar_arrive(&ctrl->kv_empty[(ring_base - 1) % kStages]);
      }
    }
    if (!ok && lane == 0) {
      // let every MMA already issued retire before tensor memory is released
      tc_commit(&ctrl->drain[s]);
      const uint64_t t0 = global_ns();
      while (!mbar_try_wait(&ctrl->drain[s], 0))
        if (global_ns() - t0 > kDrainLimitNs) break;
    }
    __syncwarp();
   }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    // ======================= softmax warpgroups ======================================
    const int s = warp >> 2;                       // stream
    const int quarter = warp & 3;                  // tensor-memory lane quarter this warp may access
    const int r = quarter * 32 + lane;             // row within the M-tile
    const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
    const uint32_t s_addr = lane_base + s * 128, o_addr = lane_base + 256 + s * 128;
    uint32_t s_cnt = 0, o_cnt = 0;  // tiles / half-units of this stream so far
    uint32_t x_cnt = 0;             // pieces so far in which the two streams were combined
    bool ok = true;
    for (int pc = piece0; pc < piece1; ++pc) {
      const TcPiece pi = pc == piece0 ? head->first : tc.pieces[pc];
      const TcReq rq = pc == piece0 ? head->first_req : tc.reqs[pi.req];
      const int n = pi.tile_end - pi.tile_begin, mode = pi.n_mt;
      const int my_units = mode == 2 ? n : (n - s + 1) / 2;
      if (ok && my_units > 0) {
        const RowInfo ri = row_info(d, tc, rq, T, mode == 2 ? pi.mtile0 + s : pi.mtile0, r, pi.kv_head);
        float m_used = -INFINITY, l = 0.f, m_new = 0.f;
        bool pend = false;
        // O *= alpha.  The PV product of the previous half-unit must have retired first; the one before
        // it has (its commit precedes the s_full this thread has just seen).
        auto rescale_o = [&](float alpha, uint32_t done_needed) -> bool {
          if (!wait_bar(&ctrl->o_done[s], (done_needed - 1) & 1u, ctrl, d.status, 235 + s)) return false;
          tc_fence_after();
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
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
        for (int j = 0; j < my_units && ok; ++j) {
          const int t = pi.tile_begin + (mode == 2 ? j : 2 * j + s);
          const bool masked = t >= rq.n_dense_tiles;
          int n_ok[kPagesPerTile];
          if (masked) {
            const uint4 *mp = reinterpret_cast<const uint4 *>(tc.pages + rq.page_off + t * kPagesPerTile);
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
              const uint4 w = __ldg(mp + jj);
              n_ok[2 * jj] = page_n_ok(w.y, ri);
              n_ok[2 * jj + 1] = page_n_ok(w.w, ri);
            }
          }
#pragma unroll 1  // one copy of the sweep: the unrolled pair was slower (instruction fetch)
          for (int half = 0; half < 2; ++half) {
            const uint32_t sh_addr = s_addr + half * 64;
            const uint32_t g = o_cnt + (uint32_t)(2 * j + half);  // half-units of this stream before this one
            const bool first = (j | half) == 0;
            ok = wait_bar(&ctrl->s_full[s][half], s_cnt & 1u, ctrl, d.status, 230 + s);
            if (!ok) break;
            tc_fence_after();
            uint32_t v[64];
            tmem_ld64(sh_addr, v);
            tc_wait_ld();
            if (masked) mask_half(v, n_ok + 4 * half);
            // A growth of the maximum noticed in an earlier half-unit is applied now.
            if (__any_sync(0xFFFFFFFFu, pend)) {
              const float alpha = pend ? ex2(m_used - m_new) : 1.0f;
              if (pend) {
                l *= alpha;
                m_used = m_new;
                pend = false;
              }
              ok = rescale_o(alpha, g);
              if (!ok) break;
            }
            uint32_t pk[32];
            float sum = 0.f, mx;
            // Fast path: exponentials against the running reference exponent; the maximum of the 64 scores is
            // computed beside them and only checked afterwards.
            bool fast = __all_sync(0xFFFFFFFFu, m_used > -INFINITY);
            if (fast) {
              float raw;
              sum = exp_half_max(v, pk, scale_log2, -m_used, raw);
              mx = raw * scale_log2;
              if (__any_sync(0xFFFFFFFFu, mx > m_used + kRedoThreshold)) fast = false;  // could overflow: redo exactly
            } else {
              mx = max_half(v) * scale_log2;
            }
            if (!fast) {
              // Exact path (first half-unit of a stream, rows that have seen no key yet, a jump of the
              // scores): adopt the maximum before the exponentials.
              const bool grow = mx > m_used + kRescaleThreshold;
              if (__any_sync(0xFFFFFFFFu, grow)) {
                const float alpha = grow ? ex2(m_used - mx) : 1.0f;
                if (grow) {
                  l *= alpha;
                  m_used = mx;
                }
                if (!first) {
                  ok = rescale_o(alpha, g);
                  if (!ok) break;
                }
              }
              sum = exp_half(v, pk, scale_log2, (m_used == -INFINITY) ? 0.f : -m_used);
            } else if (mx > m_used + kRescaleThreshold) {
              pend = true;
              m_new = mx;
            }
            l += sum;
            tmem_st32(sh_addr, pk);
            tc_wait_st();
            tc_fence_before();
            // Observe every completion of o_done in order (a parity wait must never fall two phases behind):
            // the PV product of the previous half-unit has long retired by now.  Before the arrive below,
            // because the PV product of this half-unit can only be issued after it.
            if (g > 0) {
              ok = wait_bar(&ctrl->o_done[s], (g - 1) & 1u, ctrl, d.status, 237 + s);
              if (!ok) break;
            }
            mbar_arrive(&ctrl->p_full[s][half]);
          }
          ++s_cnt;
        }
        if (ok) {
          // epilogue: wait for the last PV of this stream, then normalise and store
          o_cnt += 2u * (uint32_t)my_units;
          ok = wait_bar(&ctrl->o_done[s], (o_cnt - 1) & 1u, ctrl, d.status, 240 + s);
        }
        // The two streams of a one-M-tile piece hold partial results of the same rows (even and odd tiles).
        // Stream 1 publishes its (m, l); stream 0 reads them and stream 1's accumulator -- the same tensor-memory
        // lanes, so the thread of row r can load both -- and writes one combined result.
        const bool pair = mode == 1 && n >= 2;
        float m_out = m_used, l_out = l, w_self = 1.0f, w_other = 0.0f;
        bool writer = true;
        if (ok && pair) {
          if (s == 1) {
            ctrl->ml_xch[r] = make_float2(m_used, l);
            tc_fence_before();
            mbar_arrive(&ctrl->xch);
            writer = false;
          } else {
            ok = wait_bar(&ctrl->xch, x_cnt & 1u, ctrl, d.status, 242);
            if (ok) {
              tc_fence_after();
              const float2 other = ctrl->ml_xch[r];
              m_out = fmaxf(m_used, other.x);
              w_self = l > 0.f ? ex2(m_used - m_out) : 0.f;       // a stream that saw no key of the row has l = 0
              w_other = other.y > 0.f ? ex2(other.x - m_out) : 0.f;
              l_out = w_self * l + w_other * other.y;
            }
          }
        }
        if (pair) ++x_cnt;
        if (ok && writer) {
          tc_fence_after();
          store_rows(o_addr, lane_base + 256 + (1 - s) * 128, pi.slot[pair ? 0 : s], pair, w_self, w_other, m_out, l_out, r, ri.q_index, out,
                     lse, tc.partial_o, tc.partial_ml);
          tc_fence_before();
        }
      }
      // One arrival per thread and piece.  A stream with units in this piece cannot get here before the previous
      // piece's phase is complete (its PV products were issued behind a wait for it); a stream with none must look
      // itself, or its arrival would be counted into the previous phase while the other stream is still storing.
      if (my_units == 0 && pc > piece0 && ok) ok = wait_bar(&ctrl->epi_done, (uint32_t)(pc - piece0 - 1) & 1u, ctrl, d.status, 243);
      mbar_arrive(&ctrl->epi_done);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// Merge of the partials of one M-tile: O = sum_j 2^(m_j - M) O_j / sum_j 2^(m_j - M) l_j.
// One thread per (query row, 16-byte chunk of channels); a warp holds 32 consecutive rows of one chunk, which
// is how the partials are laid out ([slot][chunk][row]).  Grid: targets x 16 CTAs of 256 threads.  The slots
// are combined in a fixed order.
__global__ void __launch_bounds__(256)
attn_tc_merge_kernel(DevBatch d, DevTcPlan tc, uint16_t *__restrict__ out, float *__restrict__ lse) {
  const TcTarget g = tc.targets[blockIdx.x];
  const int T = tc.tokens_per_mtile, G = d.group;
  const int item = blockIdx.y * 256 + threadIdx.x;  // 0 .. 4095
  const int k = item >> 7, r = item & 127;           // chunk of 4 channels, row
  const int tok = g.mtile * T + r / G;
  const bool live = r < T * G && tok < g.n_q;
  // the partials come from the kernel launched just before this one
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (!live) return;
  const int64_t qi = (int64_t)(g.q_row0 + tok) * d.n_q_heads + g.kv_head * G + r % G;
  const float2 *ml = reinterpret_cast<const float2 *>(tc.partial_ml) + (int64_t)g.slot_begin * 128 + r;
  const float4 *po = reinterpret_cast<const float4 *>(tc.partial_o) + ((int64_t)g.slot_begin * 32 + k) * 128 + r;
  // Eight slots at a time, the (exponent, sum) pairs and the partial outputs of a batch requested together: one
  // round trip to memory per batch.  The running maximum moves between batches (never within one), in slot order,
  // so the result depends on nothing but the partials.
  float M = -INFINITY, L = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int j0 = 0; j0 < g.n_slots; j0 += 8) {
    float4 o[8];
    float2 v[8];
#pragma unroll
    for (int jj = 0; jj < 8; ++jj)
      if (j0 + jj < g.n_slots) {
        v[jj] = ml[(int64_t)(j0 + jj) * 128];
        o[jj] = po[(int64_t)(j0 + jj) * 32 * 128];
      }
    float mb = M;
#pragma unroll
    for (int jj = 0; jj < 8; ++jj)
      if (j0 + jj < g.n_slots && v[jj].y > 0.f) mb = fmaxf(mb, v[jj].x);  // a stream that saw no key of the row contributes nothing
    if (mb > M) {
      const float a = exp2f(M - mb);  // 0 while nothing has been accumulated (M = -inf)
      L *= a;
      acc.x *= a;
      acc.y *= a;
      acc.z *= a;
      acc.w *= a;
      M = mb;
    }
#pragma unroll
    for (int jj = 0; jj < 8; ++jj)
      if (j0 + jj < g.n_slots && v[jj].y > 0.f) {
        const float w = exp2f(v[jj].x - M);
        L = fmaf(w, v[jj].y, L);
        acc.x = fmaf(w, o[jj].x, acc.x);
        acc.y = fmaf(w, o[jj].y, acc.y);
        acc.z = fmaf(w, o[jj].z, acc.z);
        acc.w = fmaf(w, o[jj].w, acc.w);
      }
  }
  const float inv = 1.0f / L;
  uint2 pk = make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
  *reinterpret_cast<uint2 *>(out + qi * kD + k * 4) = pk;
  if (lse != nullptr && k == 0) lse[qi] = (M + log2f(L)) * 0.6931471805599453f;
}

// ---- tensor maps -------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// kind 0: a KV pool of n pages viewed as [8-key groups][2 channel halves][8 keys][64 channels]; box = one page of one
//         KV head (4 KB), which lands in shared memory as two 8-key groups of two 1024-byte swizzle atoms each
// kind 1: Q of n rows as [rows][q heads][128], box = 64 channels x G heads x T tokens
int get_map(lr_ctx *ctx, int kind, const void *ptr, int64_t n, const CUtensorMap **out) {
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
  if (kind == 0) {
    // [8-key group][channel half][key in group][64 channels]: one box = one page of one KV head (4 KB)
    cuuint64_t dims[4] = {64, 8, 2, (cuuint64_t)n * m.n_kv_heads * (kPage / 8)};
    cuuint64_t strides[3] = {(cuuint64_t)kD * 2, 128, (cuuint64_t)kD * 2 * 8};
    cuuint32_t box[4] = {64, 8, 2, kPage / 8};
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

int init_attn_tc_kernel() {
  return cuda_fail(cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes),
                   "attn_tc_kernel shared-memory attribute");
}

// ---- host planning -----------------------------------------------------------------
// most CTAs worth using for a number of tiles (tiny problems: not one CTA per tile, their partial results cost more than they save)
static int64_t max_ctas_for_tiles(int64_t tiles) { return tiles >= 64 ? tiles : tiles / 2; }

int tc_build_host_plan(const lr_ctx *ctx, const lr_batch *b, const int32_t *req_br_off, const int32_t *span_tin,
                       const int32_t *span_last, TcHostPlan &out, Image &img) {
  out = TcHostPlan();
  const lr_model &m = ctx->model;
  const int G = m.n_q_heads / m.n_kv_heads;
  if (m.head_dim != kD) return LR_OK;  // other head sizes take the CUDA-core path
  if ((int64_t)b->n_pool_pages * m.n_kv_heads * kPage >= ((int64_t)1 << 31)) return LR_OK;  // tensor-map coordinates are 32-bit
  const int T = 128 / G;
  const int n_q_rows = b->cu_q[b->n_branch];
  std::vector<TcPage> pages;
  std::vector<TcRow> rows((size_t)std::max(1, n_q_rows));
  std::vector<TcReq> reqs;  // one per page list (request x group of M-tiles); TcPiece.req indexes it
  struct Grp { int req, kv, mtile0, n_mt, n_tiles, weight, first_piece, n_pieces; };
  std::vector<Grp> grps;
  // Two M-tiles per group read every KV tile once for both, which is what a large pass needs.  A small pass --
  // a few tiles per SM -- is dominated by the partial results of its key split instead; there every M-tile is a
  // group of its own: a CTA then spends its two streams on the even and odd tiles of one M-tile, combines them
  // on chip and writes one partial where the paired form writes two (the second reader of a KV tile finds it
  // in L2).  Measured crossover: about 6 paired tiles per SM.
  int m_step = 2;
  {
    int64_t paired = 0;
    for (int r = 0; r < b->n_req; ++r) {
      const int br0 = req_br_off[r], br1 = req_br_off[r + 1];
      if (br1 == br0) continue;
      int64_t n_pg = 0;
      for (int sp = b->req_span_off[r]; sp < b->req_span_off[r + 1]; ++sp) n_pg += (b->span_len[sp] + kPage - 1) / kPage;
      for (int i = br0; i < br1; ++i) n_pg += (b->br_own_len[i] + kPage - 1) / kPage;
      const int64_t n_mt = (b->cu_q[br1] - b->cu_q[br0] + T - 1) / T;
      paired += (n_pg + kPagesPerTile - 1) / kPagesPerTile * m.n_kv_heads * ((n_mt + 1) / 2);
    }
    if (paired <= 6 * (int64_t)ctx->sm_count) m_step = 1;
  }
  // One page list per (request, group of M-tiles): the prefix, the segments some branch of the group descends from and
  // the tails of its own branches up to the last token one of its rows sees.  Pages no row of the group can see --
  // other branches' tails, segments off its paths through the tree -- are left out, so no tile of the sweep is fully
  // masked for everybody.  (The prefix pages appear in every list of the request: 8 bytes per page and list.)
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
    for (int m0 = 0; m0 < n_mtiles; m0 += m_step) {
      const int mts = std::min(m_step, n_mtiles - m0);
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
      for (int kv = 0; kv < m.n_kv_heads; ++kv) grps.push_back(Grp{list, kv, m0, mts, n_tiles, mts == 2 ? 16 : 10, 0, 0});
    }
  }
  if (grps.empty()) return LR_OK;
  // Contiguous partition of the tile sequence (groups in order, tiles in order) over at most max_cta CTAs that
  // minimises the largest CTA load.  A tile costs its group's weight (10 with one M-tile, 16 with two: per-CTA cycle
  // counts on the ragged serving workload gave 2360 and 3790 cycles a tile); every piece -- a CTA's share of one
  // group -- costs kPieceStartTiles tiles more (Q load, pipeline ramp, epilogue: measured 1.7 to 1.8 tiles), so a CTA
  // that spans a group boundary gets fewer tiles; a tile that needs masks (anything past the full prefix pages) costs 8/5 of a dense one (measured: 1.3 to 2.3 times, depending on the workload; 9/5 was no better).  For a load limit L the greedy fill (a CTA takes tiles while it stays within L) needs the fewest
  // CTAs possible; the smallest feasible L is found by bisection.  At most one CTA per two tiles: smaller shares
  // only add partial results to merge.
  constexpr int kPieceStartTiles = 2, kDense = 5, kMasked = 8;  // costs in fifths of a dense tile
  auto tile_cost = [&](const Grp &g, int t) -> int64_t {
    return (int64_t)g.weight * (t >= reqs[g.req].n_dense_tiles ? kMasked : kDense);
  };
  int64_t total_w = 0, total_tiles = 0, lo = 0;
  for (const Grp &g : grps) {
    total_w += (int64_t)kPieceStartTiles * kDense * g.weight;
    for (int t = 0; t < g.n_tiles; ++t) total_w += tile_cost(g, t);
    total_tiles += g.n_tiles;
    lo = std::max<int64_t>(lo, (int64_t)(kPieceStartTiles * kDense + kMasked) * g.weight);
  }
  const int64_t max_cta = std::min<int64_t>(ctx->sm_count, std::max<int64_t>(1, max_ctas_for_tiles(total_tiles)));
  // walks the partition for limit L; with `emit` it also records the pieces.  A group is a run of dense tiles
  // followed by a run of masked ones, each of uniform cost, so a walk takes O(CTAs + groups) steps.
  std::vector<TcPiece> pieces;
  std::vector<int32_t> cta_off;
  auto walk = [&](int64_t L, bool emit) -> int64_t {
    int64_t n = 0, load = 0;
    for (size_t gi = 0; gi < grps.size(); ++gi) {
      Grp &g = grps[gi];
      if (emit) g.first_piece = (int)pieces.size();
      const int64_t start = (int64_t)kPieceStartTiles * kDense * g.weight;
      const int n_dense = std::min(g.n_tiles, reqs[g.req].n_dense_tiles);
      bool new_piece = true;
      int t = 0;
      while (t < g.n_tiles) {
        const int run_end = t < n_dense ? n_dense : g.n_tiles;
        const int64_t cost = tile_cost(g, t);
        if (n == 0 || load + cost + (new_piece ? start : 0) > L) {  // open the next CTA: its share of this group is a new piece
          ++n;
          load = 0;
          new_piece = true;
          if (emit) cta_off.push_back((int32_t)pieces.size());
        }
        if (new_piece) load += start;
        const int k = (int)std::max<int64_t>(1, std::min<int64_t>(run_end - t, (L - load) / cost));
        load += (int64_t)k * cost;
        if (emit) {
          if (new_piece) {
            TcPiece p;
            p.req = g.req; p.kv_head = g.kv; p.mtile0 = g.mtile0; p.n_mt = g.n_mt; p.tile_begin = t; p.tile_end = t + k;
            p.slot[0] = p.slot[1] = -2;
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
  int64_t hi = total_w;  // one CTA takes everything
  while (lo < hi) {
    const int64_t mid = lo + (hi - lo) / 2;
    if (walk(mid, false) <= max_cta) hi = mid; else lo = mid + 1;
  }
  const int n_cta = (int)walk(lo, true);
  cta_off.push_back((int32_t)pieces.size());
  // Targets (one M-tile of one group) and the streams that contribute to them, in piece order.
  int n_slots = 0;
  std::vector<TcTarget> targets;
  for (const Grp &g : grps)
    for (int mt = 0; mt < g.n_mt; ++mt) {
      std::vector<int32_t *> contrib;
      for (int k = 0; k < g.n_pieces; ++k) {
        TcPiece &p = pieces[g.first_piece + k];
        if (g.n_mt == 2) contrib.push_back(&p.slot[mt]);
        else contrib.push_back(&p.slot[0]);  // the two streams of a one-M-tile piece are combined inside the CTA
      }
      if (contrib.size() == 1) { *contrib[0] = -1; continue; }
      TcTarget tg;
      memset(&tg, 0, sizeof(tg));
      tg.req = g.req; tg.kv_head = g.kv; tg.mtile = g.mtile0 + mt;
      tg.slot_begin = n_slots; tg.n_slots = (int)contrib.size();
      tg.q_row0 = reqs[g.req].q_row0; tg.n_q = reqs[g.req].n_q;
      for (int32_t *c : contrib) *c = n_slots++;
      targets.push_back(tg);
    }
  out.ok = true;
  out.n_cta = n_cta;
  out.n_pieces = (int)pieces.size();
  out.n_targets = (int)targets.size();
  out.n_partial_slots = n_slots;
  out.tokens_per_mtile = T;
  static_assert(sizeof(TcCtaHead) == 256, "one CTA head = 256 bytes");
  std::vector<TcCtaHead> heads((size_t)n_cta);
  for (int c = 0; c < n_cta; ++c) {
    TcCtaHead &h = heads[c];
    memset(&h, 0, sizeof(h));
    h.piece0 = cta_off[c];
    h.piece1 = cta_off[c + 1];
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
  out.o_heads = img.add(heads.data(), heads.size() * sizeof(TcCtaHead));
  out.o_pages = img.add(pages.data(), pages.size() * sizeof(TcPage));
  out.n_pages = (int)pages.size();
  out.o_rows = img.add(rows.data(), rows.size() * sizeof(TcRow));
  out.o_pieces = img.add(pieces.data(), pieces.size() * sizeof(TcPiece));
  out.o_cta_piece_off = img.add(cta_off.data(), cta_off.size() * sizeof(int32_t));
  if (reqs.empty()) reqs.push_back(TcReq{});
  out.o_reqs = img.add(reqs.data(), reqs.size() * sizeof(TcReq));
  if (targets.empty()) targets.push_back(TcTarget{});  // keep the section non-empty
  out.o_targets = img.add(targets.data(), targets.size() * sizeof(TcTarget));
  out.s_ml = 0;
  out.s_o = ((size_t)n_slots * 128 * 2 * sizeof(float) + 255) / 256 * 256;
  out.scratch_bytes = out.s_o + (size_t)n_slots * 128 * kD * sizeof(float);
  out.scratch_zero_bytes = 0;
  return LR_OK;
}

void tc_bind_device_plan(const TcHostPlan &h, unsigned char *image_base, unsigned char *scratch_base, lr_plan *p) {
  p->tc_ok = h.ok;
  p->tc_pieces = h.n_pieces;
  p->o_tc_pages = h.o_pages;
  p->o_tc_heads = h.o_heads;
  p->n_tc_pages = h.ok ? h.n_pages : 0;
  p->n_tc_heads = h.ok ? h.n_cta : 0;
  p->tc_partial_slots = h.n_partial_slots;
  memset(&p->tc, 0, sizeof(p->tc));
  if (!h.ok) return;
  DevTcPlan &t = p->tc;
  t.heads = reinterpret_cast<const TcCtaHead *>(image_base + h.o_heads);
  t.pages = reinterpret_cast<const TcPage *>(image_base + h.o_pages);
  t.rows = reinterpret_cast<const TcRow *>(image_base + h.o_rows);
  t.pieces = reinterpret_cast<const TcPiece *>(image_base + h.o_pieces);
  t.cta_piece_off = reinterpret_cast<const int32_t *>(image_base + h.o_cta_piece_off);
  t.reqs = reinterpret_cast<const TcReq *>(image_base + h.o_reqs);
  t.targets = reinterpret_cast<const TcTarget *>(image_base + h.o_targets);
  t.n_cta = h.n_cta;
  t.n_targets = h.n_targets;
  t.tokens_per_mtile = h.tokens_per_mtile;
  t.wait_limit_us = 1000000u;  // one second per wait
  t.phantom_tx_bytes = 0;
  t.partial_ml = reinterpret_cast<float *>(scratch_base + h.s_ml);
  t.partial_o = reinterpret_cast<float *>(scratch_base + h.s_o);
}

int launch_attn_tc(lr_plan *p, const void *q, const void *k, const void *v, void *out, float *lse, float scale,
                   cudaStream_t s) {
  const CUtensorMap *mp = nullptr;
  if (int rc = get_map(p->ctx, 0, k, p->dev.n_pool_pages, &mp)) return rc;
  const CUtensorMap kmap = *mp;  // the cache may reallocate when the next map is added
  if (int rc = get_map(p->ctx, 0, v, p->dev.n_pool_pages, &mp)) return rc;
  const CUtensorMap vmap = *mp;
  if (int rc = get_map(p->ctx, 1, q, p->dev.n_q_rows, &mp)) return rc;
  const CUtensorMap qmap = *mp;
  const float scale_log2 = scale * 1.4426950408889634f;
  attn_tc_kernel<<<p->tc.n_cta, kThreads, kSmemBytes, s>>>(kmap, vmap, qmap, p->dev, p->tc, reinterpret_cast<uint16_t *>(out), lse,
                                                            scale_log2);
  p->ctx->launches++;
  if (int rc = cuda_fail(cudaGetLastError(), "attn_tc_kernel launch")) return rc;
  if (p->tc.n_targets > 0) {
    // programmatic dependent launch: the merge grid is set up while the attention grid drains
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)p->tc.n_targets, 16, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, attn_tc_merge_kernel, p->dev, p->tc, reinterpret_cast<uint16_t *>(out), lse);
    p->ctx->launches++;
    if (int rc = cuda_fail(e, "attn_tc_merge_kernel launch")) return rc;
  }
  return LR_OK;
}

}  // namespace lr
