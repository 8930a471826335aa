// Stochastic token-level acceptance with the sampling filters of Section 4 "Setup" (top-k, top-p) applied to
// the target distribution before the rejection-sampling rule of Background, "Speculative Decoding".
//
// The filters keep a leading part of the ranking of a row's tokens by probability (descending; equal
// probabilities in index order).  With bf16 logits the ranking is the ranking of a 16-bit ordered key (-0 and +0
// sharing one), so the
// kept set of a row is described by a cut: every token whose key is above cut_key, and of the tokens whose key
// equals cut_key those with an index up to cut_idx.  filter_rows_kernel (one CTA per row) finds the cut:
//   pass 0   row maximum m;
//   pass 1   token counts per key over the window of the 8192 largest keys from m down (64 octaves: every positive
//            logit when m > 0), one shared-memory atomic per token; the tokens below the window only add their
//            mass to a per-thread sum.  Masses are w = exp2((x - m) log2(e) / T) as integers in units of 2^-40:
//            all tokens of a key have the same mass, so a key's mass is count x w exactly, and integer sums do not
//            depend on the order of the additions -- the result is the same on every run;
//   scan     counts and masses of the window's keys from the top down: the key holding the last token top-k
//            keeps, then, with W_k = mass of the top k, the key at which the mass reaches top_p W_k;
//   more     if a cut lies below the window, the window moves down to the next key that occurs (one more pass
//            each time) until it holds the cut; if top-p's cut lies above the window top-k ended in, the search
//            starts again from the top;
//   last     only when the cut splits a group of equal keys: the index of the last token kept in the group.
// After pass 0 the row comes from L2.  accept_filtered_kernel (one CTA per branch) walks the acceptance chain
// with P'(d) = w_d / Z' for kept tokens and 0 for the others, and draws the final token by inverse CDF over the
// kept tokens of the stop row in index order, in the same integer masses (no rounding: the draw is exact given
// the masses).
#include <algorithm>

#include "lr_common.cuh"

namespace lr {

namespace {

constexpr int kFT = 1024;          // threads of filter_rows_kernel
constexpr int kWin = 8192;         // keys per window
constexpr int kPer = kWin / kFT;   // window positions per thread in the scan
constexpr int kST = 1024;          // threads of accept_filtered_kernel
typedef unsigned long long u64;
constexpr int32_t kNoKey = INT32_MIN;

struct RowCut {  // what the second kernel needs to know about a row (32 bytes)
  float m;          // row maximum (finite: a row without a finite logit gets -3e38)
  int32_t cut_key;  // key32 of the last kept group of equal logits; kNoKey: everything is kept
  int32_t cut_idx;  // largest index kept inside that group
  int32_t n_kept;
  u64 z_fix;        // mass of the kept set
  u64 reserved;
};

// Order-preserving key of a bf16 value given as fp32 bits (low 16 bits zero): sign-magnitude turned into two's
// complement, so that a larger value has a larger key and -0 and +0 share key 0.  A multiple of 65536; key32 >> 16
// ("key16") lies in [-32768, 32767].  A NaN lies beyond the infinities; its mass is 0 (below), so wherever it lands
// it changes no sum.
__device__ __forceinline__ int32_t key32(uint32_t f) {
  const uint32_t s = (uint32_t)((int32_t)f >> 31);
  return (int32_t)(((f & 0x7FFFFFFFu) ^ s) - s);
}
__device__ __forceinline__ uint32_t f_of_key16(int32_t key16) {
  return key16 >= 0 ? (uint32_t)key16 << 16 : (0x8000u | (uint32_t)(-key16)) << 16;
}
// mass of a token in units of 2^-40 relative to the row maximum (at most 2^40): a subtraction, a multiply-add, one
// exponential, one conversion.  The conversion turns NaN into 0.
__device__ __forceinline__ u64 wfix_of(uint32_t f, float m, float k_log2) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(fmaf(__uint_as_float(f) - m, k_log2, 40.f)));
  u64 r;
  asm("cvt.rni.u64.f32 %0, %1;" : "=l"(r) : "f"(y));
  return r;
}

// f(e, bits) for every token e of the row (bits = the logit as fp32 bits), threads striding over 16-byte vectors
template <int kT, class F>
__device__ __forceinline__ void row_strided(const uint16_t *rp, int32_t vocab, F &&f) {
  const int32_t n_vec = vocab >> 3;
  const uint4 *vp = reinterpret_cast<const uint4 *>(rp);
  for (int32_t v0 = 0; v0 < n_vec; v0 += 4 * kT) {
    uint4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int32_t vi = v0 + k * kT + (int32_t)threadIdx.x;
      if (vi < n_vec) v[k] = __ldg(vp + vi);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int32_t vi = v0 + k * kT + (int32_t)threadIdx.x;
      if (vi < n_vec) {
        const uint32_t w[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          f(vi * 8 + 2 * j, w[j] << 16);
          f(vi * 8 + 2 * j + 1, w[j] & 0xFFFF0000u);
        }
      }
    }
  }
  const int32_t e = n_vec * 8 + (int32_t)threadIdx.x;  // vocab not a multiple of 8
  if (e < vocab) f(e, (uint32_t)__ldg(rp + e) << 16);
}

// the same with every thread owning a contiguous range of the row, ranges in thread order: visiting threads in
// order and each thread's tokens in order is index order
template <int kT, class F>
__device__ __forceinline__ void row_blocked(const uint16_t *rp, int32_t vocab, F &&f) {
  const int32_t n_vec = vocab >> 3, per = (n_vec + kT - 1) / kT;
  const int32_t v_begin = min(n_vec, (int32_t)threadIdx.x * per), v_end = min(n_vec, v_begin + per);
  const uint4 *vp = reinterpret_cast<const uint4 *>(rp);
  for (int32_t v0 = v_begin; v0 < v_end; v0 += 4) {  // four loads in flight
    uint4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (v0 + k < v_end) v[k] = __ldg(vp + v0 + k);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (v0 + k < v_end) {
        const int32_t vi = v0 + k;
        const uint32_t w[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          f(vi * 8 + 2 * j, w[j] << 16);
          f(vi * 8 + 2 * j + 1, w[j] & 0xFFFF0000u);
        }
      }
    }
  }
  if (threadIdx.x == kT - 1)
    for (int32_t e = n_vec * 8; e < vocab; ++e) f(e, (uint32_t)__ldg(rp + e) << 16);
}

// maximum of a row, two bf16 at a time (max.bf16x2 returns the other operand when one is NaN); never below -3e38
template <int kT>
__device__ __forceinline__ float row_max(const uint16_t *rp, int32_t vocab, float *s_w, float &thread_max) {
  const int32_t n_vec = vocab >> 3;
  const uint4 *vp = reinterpret_cast<const uint4 *>(rp);
  constexpr uint32_t kNegInf2 = 0xFF80FF80u;
  uint32_t a = kNegInf2, b = kNegInf2;
  auto mx = [](uint32_t x, uint32_t y) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(y));
    return r;
  };
  for (int32_t v0 = 0; v0 < n_vec; v0 += 4 * kT) {
    uint4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int32_t vi = v0 + k * kT + (int32_t)threadIdx.x;
      v[k] = vi < n_vec ? __ldg(vp + vi) : make_uint4(kNegInf2, kNegInf2, kNegInf2, kNegInf2);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      a = mx(a, mx(v[k].x, v[k].y));
      b = mx(b, mx(v[k].z, v[k].w));
    }
  }
  a = mx(a, b);
  float m = fmaxf(__uint_as_float(a << 16), __uint_as_float(a & 0xFFFF0000u));
  const int32_t e = n_vec * 8 + (int32_t)threadIdx.x;
  if (e < vocab) m = fmaxf(m, __uint_as_float((uint32_t)__ldg(rp + e) << 16));
  thread_max = m;  // the largest logit among the tokens this thread looked at
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = m;
  __syncthreads();
  float r = s_w[0];
#pragma unroll
  for (int k = 1; k < kT / 32; ++k) r = fmaxf(r, s_w[k]);
  __syncthreads();
  return fmaxf(r, -3.0e38f);
}

// inclusive scan over the block in thread order; `total` receives the sum over the block
template <int kT, class T>
__device__ __forceinline__ T block_scan(T v, T *s_w, T &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const T y = __shfl_up_sync(0xFFFFFFFFu, v, o);
    if (lane >= o) v += y;
  }
  if (lane == 31) s_w[warp] = v;
  __syncthreads();
  T base = 0, all = 0;
#pragma unroll
  for (int k = 0; k < kT / 32; ++k) {
    const T t = s_w[k];
    if (k < warp) base += t;
    all += t;
  }
  __syncthreads();
  total = all;
  return v + base;
}

struct KeyCut {  // the last token kept: a key, and how many of the tokens with that key
  int32_t key;         // key16
  uint32_t j;          // tokens of the key that are kept (>= 1 when found)
  uint32_t cnt_key;    // tokens of the key
  uint32_t cnt_above;  // tokens with a larger key
  u64 mass_above;      // their mass
  u64 w_key;           // mass of one token of the key
};

// A window of kWin consecutive keys, hi down to hi - kWin + 1: per-key token counts in shared memory (position d
// is key hi - d; keys here are key16), and what lies above the window.
struct Window {
  int32_t hi;
  int32_t next_hi;     // the largest key below the window that occurs in the row; kNoKey if none
  uint32_t cnt_above;
  u64 mass_above;
  uint32_t cnt;        // tokens inside
  u64 mass;            // their mass
};

struct FilterShared {
  uint32_t cnt[kWin];
  u64 w64[kFT / 32];
  uint32_t w32[kFT / 32];
  float wf[kFT / 32];
  int32_t wi[kFT / 32];
  KeyCut cut;
  int32_t cut_idx;
};

template <int kT>
__device__ __forceinline__ int32_t block_max_i32(int32_t v, int32_t *s_w) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = v;
  __syncthreads();
  int32_t r = s_w[0];
#pragma unroll
  for (int k = 1; k < kT / 32; ++k) r = max(r, s_w[k]);
  __syncthreads();
  return r;
}

// One pass over the row: counts of the keys inside the window starting at `hi`.  On the first window (kFirst) the
// mass of everything below the window is summed too, so that the mass of the whole row is known.  Tokens whose
// logit is below `floor_x` are left out altogether (-inf: none is; a NaN always is).
template <bool kFirst>
__device__ __forceinline__ void build_window(FilterShared &sh, const uint16_t *rp, int32_t vocab, float m, float k_log2,
                                             float floor_x, int32_t hi, Window &win, u64 &mass_below) {
  for (int i = threadIdx.x; i < kWin; i += kFT) sh.cnt[i] = 0;
  __syncthreads();
  int32_t nh = kNoKey;
  u64 rest = 0;
  const int32_t hi32 = hi * 65536;
  row_strided<kFT>(rp, vocab, [&](int32_t, uint32_t f) {
    if (!(__uint_as_float(f) >= floor_x)) return;
    const int32_t k32 = key32(f);
    if (k32 <= hi32) {  // keys above the window were counted by an earlier pass (a NaN beyond +inf: never)
      const uint32_t d = ((uint32_t)hi32 - (uint32_t)k32) >> 16;
      if (d < (uint32_t)kWin) {
        atomicAdd(&sh.cnt[d], 1u);
      } else {
        nh = max(nh, k32);
        if (kFirst) rest += wfix_of(f, m, k_log2);
      }
    }
  });
  __syncthreads();
  win.hi = hi;
  nh = block_max_i32<kFT>(nh, sh.wi);
  win.next_hi = nh == kNoKey ? kNoKey : nh >> 16;
  if (kFirst) {
    u64 all;
    block_scan<kFT, u64>(rest, sh.w64, all);
    mass_below = all;
  }
}

// Per-thread view of the window: thread t owns positions t kPer .. t kPer + kPer - 1 (keys descending)
struct Mine {
  uint32_t c_excl;  // tokens of the window before this thread's positions
  u64 m_excl;       // their mass
  uint32_t c_sum;
  u64 m_sum;
};

__device__ __forceinline__ u64 w_of_pos(const Window &win, int pos, float m, float k_log2) {
  return wfix_of(f_of_key16(win.hi - pos), m, k_log2);
}

__device__ __forceinline__ void scan_window(FilterShared &sh, Window &win, Mine &me, float m, float k_log2) {
  me.c_sum = 0;
  me.m_sum = 0;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const uint32_t c = sh.cnt[threadIdx.x * kPer + i];
    if (c != 0) {
      me.c_sum += c;
      me.m_sum += (u64)c * w_of_pos(win, threadIdx.x * kPer + i, m, k_log2);  // all tokens of a key weigh the same
    }
  }
  me.c_excl = block_scan<kFT, uint32_t>(me.c_sum, sh.w32, win.cnt) - me.c_sum;
  me.m_excl = block_scan<kFT, u64>(me.m_sum, sh.w64, win.mass) - me.m_sum;
}

// The key of the window at which the token count (from the top of the ranking) reaches k, or at which the mass
// reaches t; the caller has made sure that it lies inside the window.  Every thread returns the same value.
template <bool kByMass>
__device__ __forceinline__ KeyCut locate(FilterShared &sh, const Window &win, const Mine &me, uint32_t k, u64 t, float m,
                                         float k_log2) {
  const uint32_t k_rel = k - win.cnt_above;
  const u64 t_rel = t - win.mass_above;
  const bool mine = kByMass ? (me.m_sum > 0 && me.m_excl < t_rel && t_rel <= me.m_excl + me.m_sum)
                            : (me.c_excl < k_rel && k_rel <= me.c_excl + me.c_sum);
  if (mine) {
    uint32_t cnt = me.c_excl;
    u64 mass = me.m_excl;
    bool done = false;
    for (int i = 0; i < kPer; ++i) {
      const uint32_t c = sh.cnt[threadIdx.x * kPer + i];
      if (c != 0 && !done) {
        const int pos = threadIdx.x * kPer + i;
        const u64 w = w_of_pos(win, pos, m, k_log2);
        const bool here = kByMass ? (w > 0 && mass + (u64)c * w >= t_rel) : (cnt + c >= k_rel);
        if (here) {
          KeyCut r;
          r.key = win.hi - pos;
          r.cnt_key = c;
          r.cnt_above = win.cnt_above + cnt;
          r.mass_above = win.mass_above + mass;
          r.w_key = w;
          r.j = kByMass ? (uint32_t)((t_rel - mass + w - 1) / w) : (k_rel - cnt);
          sh.cut = r;
          done = true;
        }
        cnt += c;
        mass += (u64)c * w;
      }
    }
  }
  __syncthreads();
  const KeyCut r = sh.cut;
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(kFT, 1)
filter_rows_kernel(const uint16_t *__restrict__ logits, int64_t row_stride, int32_t vocab, float k_log2, int32_t top_k,
                   float top_p, RowCut *__restrict__ cuts, int32_t *__restrict__ n_kept_out) {
  __shared__ FilterShared sh;
  const int tid = threadIdx.x;
  const int64_t row = blockIdx.x;
  const uint16_t *rp = logits + row * row_stride;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the logits may come from the kernel launched just before
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // ---- pass 0: the row maximum
  if (tid == 0) {
    sh.cut_idx = INT32_MAX;
    sh.cut.j = 0;
  }
  float thread_max;
  const float m = row_max<kFT>(rp, vocab, sh.wf, thread_max);
  const int32_t key_top = key32(__float_as_uint(m)) >> 16;

  // ---- pass 1: the window that starts at the largest key, and the mass of the whole row
  Window win;
  Mine me;
  u64 mass_below = 0;
  win.cnt_above = 0;
  win.mass_above = 0;
  const uint32_t cnt_total = (uint32_t)vocab;
  const bool by_k = top_k > 0 && (uint32_t)top_k < cnt_total;
  const bool by_p = top_p < 1.f;
  // With top-k on and k no larger than the number of threads, the k-th largest of the threads' own maxima (each is
  // the logit of a different token) is a lower bound of the k-th largest logit of the row: tokens below it cannot be
  // kept, and the passes that follow skip them after one comparison.
  float floor_x = -INFINITY;
  if (by_k && top_k <= kFT) {
    for (int i = tid; i < kWin; i += kFT) sh.cnt[i] = 0;
    __syncthreads();
    const int32_t k32 = key32(__float_as_uint(thread_max));
    const uint32_t d = ((uint32_t)(key_top * 65536) - (uint32_t)k32) >> 16;  // thread_max <= m
    if (thread_max > -INFINITY && d < (uint32_t)kWin) atomicAdd(&sh.cnt[d], 1u);
    __syncthreads();
    win.hi = key_top;
    scan_window(sh, win, me, m, k_log2);
    if ((uint32_t)top_k <= win.cnt) {
      const KeyCut kc = locate<false>(sh, win, me, (uint32_t)top_k, 0, m, k_log2);
      floor_x = __uint_as_float(f_of_key16(kc.key));
    }
    __syncthreads();
  }
  // the mass of the whole row is needed only when top-k does not cut: else the mass of the top k takes its place
  if (by_k) build_window<false>(sh, rp, vocab, m, k_log2, floor_x, key_top, win, mass_below);
  else build_window<true>(sh, rp, vocab, m, k_log2, floor_x, key_top, win, mass_below);
  scan_window(sh, win, me, m, k_log2);
  const u64 mass_total = win.mass + mass_below;

  auto advance = [&]() -> bool {  // the next window down; false when nothing is left below
    if (win.next_hi == kNoKey) return false;
    win.cnt_above += win.cnt;
    win.mass_above += win.mass;
    u64 unused;
    build_window<false>(sh, rp, vocab, m, k_log2, floor_x, win.next_hi, win, unused);
    scan_window(sh, win, me, m, k_log2);
    return true;
  };

  KeyCut cut;
  bool have_cut = false;
  u64 w_k = mass_total;  // mass of what top-k keeps
  uint32_t n_all = cnt_total;

  if (by_k) {
    const uint32_t k = (uint32_t)top_k;
    bool ok = true;
    while (ok && k > win.cnt_above + win.cnt) ok = advance();
    if (ok) {
      cut = locate<false>(sh, win, me, k, 0, m, k_log2);
      have_cut = true;
      w_k = cut.mass_above + (u64)cut.j * cut.w_key;
    } else {  // fewer than k tokens that are numbers: every window was visited, nothing is cut
      w_k = win.mass_above + win.mass;
      n_all = win.cnt_above + win.cnt;
    }
  }
  if (by_p && w_k > 0) {
    // rank r stays iff the mass ranked before it is below top_p W_k: the last one kept is the first rank at which
    // the mass, itself included, reaches t
    const double t_d = ceil((double)top_p * (double)w_k);
    u64 t = t_d < 1.0 ? 1ull : (u64)t_d;
    if (t > w_k) t = w_k;
    bool ok = true;
    if (t <= win.mass_above) {  // the top-k search went past it: start again from the top
      win.cnt_above = 0;
      win.mass_above = 0;
      u64 unused;
      build_window<false>(sh, rp, vocab, m, k_log2, floor_x, key_top, win, unused);
      scan_window(sh, win, me, m, k_log2);
    }
    while (ok && t > win.mass_above + win.mass) ok = advance();
    if (ok) {
      KeyCut cp = locate<true>(sh, win, me, 0, t, m, k_log2);
      if (have_cut && cp.key == cut.key) cp.j = min(cp.j, cut.j);  // (already implied by t <= W_k)
      cut = cp;
      have_cut = true;
    }
  }

  // ---- last pass, only when the cut splits a group of equal keys: the index of the last one kept
  if (have_cut && cut.j < cut.cnt_key) {
    uint32_t mine = 0;
    const int32_t cut32 = cut.key * 65536;
    row_blocked<kFT>(rp, vocab, [&](int32_t, uint32_t f) { mine += key32(f) == cut32 ? 1u : 0u; });
    uint32_t all;
    const uint32_t before = block_scan<kFT, uint32_t>(mine, sh.w32, all) - mine;
    if (before < cut.j && cut.j <= before + mine) {
      uint32_t seen = before;
      row_blocked<kFT>(rp, vocab, [&](int32_t e, uint32_t f) {
        if (key32(f) == cut32 && ++seen == cut.j) sh.cut_idx = e;
      });
    }
    __syncthreads();
  }
  if (tid == 0) {
    RowCut rc;
    rc.m = m;
    rc.cut_key = have_cut ? cut.key * 65536 : kNoKey;
    rc.cut_idx = sh.cut_idx;
    rc.n_kept = have_cut ? (int32_t)(cut.cnt_above + cut.j) : (int32_t)n_all;
    rc.z_fix = have_cut ? cut.mass_above + (u64)cut.j * cut.w_key : w_k;
    rc.reserved = 0;
    cuts[row] = rc;
    if (n_kept_out != nullptr) n_kept_out[row] = rc.n_kept;
  }
}

__device__ __forceinline__ bool is_kept(int32_t key, int32_t e, const RowCut &rc) {
  return key > rc.cut_key || (key == rc.cut_key && e <= rc.cut_idx);
}

__global__ void __launch_bounds__(kST)
accept_filtered_kernel(const uint16_t *__restrict__ logits, int64_t row_stride, int32_t vocab, float k_log2,
                       const RowCut *__restrict__ cuts, const int32_t *__restrict__ draft_ids,
                       const int32_t *__restrict__ cu_draft, const float *__restrict__ u_accept,
                       const float *__restrict__ u_final, int32_t *__restrict__ n_accept, int32_t *__restrict__ final_id,
                       float *__restrict__ p_draft) {
  __shared__ u64 s_w64[kST / 32];
  __shared__ int s_n;
  __shared__ int32_t s_final;
  const int b = blockIdx.x, tid = threadIdx.x;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the cuts come from the kernel launched just before
  const int32_t d0 = cu_draft[b], L = cu_draft[b + 1] - d0, r0 = d0 + b;
  if (tid == 0) {
    s_n = L;
    s_final = 0;
  }
  __syncthreads();

  // ---- acceptance chain: draft i passes iff u_i < P'_i(d_i); the first one that does not ends it
  for (int i = tid; i < L; i += kST) {
    const RowCut rc = cuts[r0 + i];
    const int32_t d = draft_ids[d0 + i];
    float p = 0.f;
    if (d >= 0 && d < vocab && rc.z_fix > 0) {
      const uint32_t f = (uint32_t)logits[(int64_t)(r0 + i) * row_stride + d] << 16;
      if (is_kept(key32(f), d, rc)) p = (float)wfix_of(f, rc.m, k_log2) / (float)rc.z_fix;
    }
    if (p_draft != nullptr) p_draft[d0 + i] = p;
    if (!(u_accept[d0 + i] < p)) atomicMin(&s_n, i);
  }
  __syncthreads();
  const int n = s_n;

  // ---- the final token: inverse CDF over the kept tokens of the stop row, the rejected one removed
  const RowCut rc = cuts[r0 + n];
  const uint16_t *rp = logits + (int64_t)(r0 + n) * row_stride;
  int32_t dead = -1;
  u64 w_dead = 0;
  if (n < L) {
    const int32_t d = draft_ids[d0 + n];
    if (d >= 0 && d < vocab) {
      const uint32_t f = (uint32_t)rp[d] << 16;
      if (is_kept(key32(f), d, rc)) {
        dead = d;
        w_dead = wfix_of(f, rc.m, k_log2);
      }
    }
  }
  const u64 total = rc.z_fix - w_dead;
  // smallest v whose cumulative mass exceeds u * total; the masses are integers, so "exceeds floor(u * total)"
  u64 target = (u64)((double)u_final[b] * (double)total);
  if (total > 0 && target >= total) target = total - 1;
  u64 mine = 0;
  row_blocked<kST>(rp, vocab, [&](int32_t e, uint32_t bts) {
    if (e != dead && is_kept(key32(bts), e, rc)) mine += wfix_of(bts, rc.m, k_log2);
  });
  u64 all;
  const u64 before = block_scan<kST, u64>(mine, s_w64, all) - mine;
  if (mine > 0 && before <= target && target < before + mine) {
    u64 cum = before;
    bool done = false;
    row_blocked<kST>(rp, vocab, [&](int32_t e, uint32_t bts) {
      if (!done && e != dead && is_kept(key32(bts), e, rc)) {
        cum += wfix_of(bts, rc.m, k_log2);
        if (cum > target) {
          s_final = e;
          done = true;
        }
      }
    });
  }
  __syncthreads();
  if (tid == 0) {
    n_accept[b] = n;
    final_id[b] = s_final;
  }
}

}  // namespace

size_t accept_filtered_scratch_bytes(int32_t n_rows) { return std::max<size_t>(32, (size_t)n_rows * sizeof(RowCut)); }

int launch_accept_filtered(lr_ctx *ctx, const void *logits, int64_t stride, const int32_t *drafts, const int32_t *cu_draft,
                           int32_t n_branch, int32_t n_rows, float temperature, int32_t top_k, float top_p,
                           const float *u_accept, const float *u_final, int32_t *n_accept, int32_t *final_id, float *p_draft,
                           int32_t *n_kept, void *scratch, cudaStream_t s) {
  const int32_t vocab = ctx->model.vocab;
  const float k_log2 = 1.4426950408889634f / temperature;
  auto *lg = reinterpret_cast<const uint16_t *>(logits);
  auto *cuts = reinterpret_cast<RowCut *>(scratch);
  filter_rows_kernel<<<(unsigned)n_rows, kFT, 0, s>>>(lg, stride, vocab, k_log2, top_k, top_p, cuts, n_kept);
  ctx->launches++;
  if (int rc = cuda_fail(cudaGetLastError(), "filter_rows_kernel launch")) return rc;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)n_branch, 1, 1);
  cfg.blockDim = dim3(kST, 1, 1);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, accept_filtered_kernel, lg, stride, vocab, k_log2, (const RowCut *)cuts, drafts, cu_draft,
                                     u_accept, u_final, n_accept, final_id, p_draft);
  ctx->launches++;
  return cuda_fail(e, "accept_filtered_kernel launch");
}

}  // namespace lr
