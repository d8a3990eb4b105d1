// Gather attention of the token-level path (Main Results: Token Position-Decay on a selector that keeps the top
// 2048 tokens per query), for sm_100a: O[t, h] = softmax_s(Q[t, h] . K[s, kv(h)] * scale) V[s, kv(h)] over the tokens
// s of list (kv(h), t).  Every (query token, kv head) gathers its own K / V rows, so the kernel is bound by how fast
// rows come out of the L2; everything is arranged so that nothing else is in the way:
//
//   * the rows are gathered by four producer warps with 16-byte cp.async copies - a warp instruction fetches two
//     whole 256-byte rows, each chunk written straight to its place in the 128-byte-swizzled operand layout of the
//     tensor cores - 128 keys per tile through a ring of stages, completion counted on mbarriers (TMA row gathers,
//     tile::gather4, were measured first: 2.1 TB/s, the copy engine takes about 16 cycles per 128-byte row);
//   * both contractions run on the tcgen05 tensor cores in the TRANSPOSED orientation, keys (then head-dimension
//     columns) on the 128 TMEM lanes and the group's query heads, padded to 16, on the columns:
//         S^T [128 keys x 16] = K_tile [128 x 128] . Q_g^T          (A = the gathered K rows, K-major)
//         O^T [128 cols x 16] += V_tile^T [128 x 128 keys] . P^T    (A = the gathered V rows, MN-major; B = P^T from
//                                                                    shared memory)
//     so the CUDA cores only see 16 numbers per key: one thread per key, online softmax with one reference per head
//     shared by the CTA (raised lazily, by more than 2^8), the row sums kept per thread and added up once per item;
//   * persistent CTAs (one per SM) walk the (token, kv head) items, longest lists first; Q K^T of tile i+1 is issued
//     before P V of tile i (S^T is double-buffered), copies run up to two tiles ahead, across items.
//
// P is rounded to bf16 before P V, as in the block-sparse kernel.  Every wait is bounded; a wait that gives up
// records {4, CTA, role, barrier} in the status words below, the CTA drains its copies, frees its tensor memory and
// returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>

#include "stem_internal.h"
#include "stem_ptx.cuh"

namespace stem {

namespace {

using namespace ptx;

constexpr int kThreads = 288;             // warps 0-3 softmax / epilogue, warps 4-7 copies, warp 8 MMAs
constexpr int kMmaWarp = 8;
constexpr int kKeys = 128;                // keys per tile
constexpr int kNPad = 16;                 // query heads of a group, padded to the smallest N of a 128-row MMA
constexpr int kStages = 3;
constexpr int kHalf = kKeys * 128;        // one 64-column half of a K or V tile: 128 rows x 128 bytes
constexpr int kKvTile = 2 * kHalf;        // 32 KB
constexpr int kSmallHalf = kNPad * 128;   // one 64-column half of a [16 x 128] bf16 operand (Q_g, P^T)
constexpr int kSmall = 2 * kSmallHalf;    // 4 KB
constexpr int kOffK = 0, kOffV = kKvTile, kOffQ = 2 * kKvTile, kOffP = 2 * kKvTile + kSmall;
constexpr int kStageBytes = 2 * kKvTile + 2 * kSmall;  // 72 KB
constexpr int kSBuf = 3;                                // S^T buffers in tensor memory: Q K^T runs up to two tiles ahead of P V
constexpr int kOffRed = kStages * kStageBytes;          // float [kSBuf][4][16] tile maxima, float [2][4][16] row sums
constexpr int kOffBars = kOffRed + (kSBuf + 2) * 4 * kNPad * 4;
// barriers: k_full[3] v_full[3] empty[3] s_full[kSBuf] p_ready[kSBuf] red[kSBuf] sum[2] pv_done[kPvBars] o_free
constexpr int kPvBars = 4;
constexpr int kNumBars = 3 * kStages + 3 * kSBuf + 2 + kPvBars + 1;
constexpr int kOffTmem = kOffBars + kNumBars * 8;
constexpr int kOffAbort = kOffTmem + 8;
constexpr int kSmemBytes = kOffAbort + 8 + 1024;  // slack for manual 1024-byte alignment
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
static_assert(kPvBars > kStages, "a P V completion barrier must never be a phase behind its waiter");
constexpr uint64_t kWaitLimitNs = 400ull * 1000 * 1000;
constexpr float kRescale = 8.f;           // log2 units
constexpr int kTmemCols = 64;             // S^T of kSBuf tiles (16 columns each) and O^T (16 columns)
constexpr uint32_t kColS = 0, kColO = kSBuf * kNPad;

constexpr int kRoleSoftmax = 0, kRoleCopy = 1, kRoleMma = 2;
enum : int { kBarKFull = 0, kBarVFull, kBarEmpty, kBarSFull, kBarPReady, kBarRed, kBarSum, kBarPvDone, kBarOFree, kBarDrain /* the issuing warp's poll */ };

__device__ int32_t g_token_status[4];

struct TokArgs {
  const __nv_bfloat16 *Q, *K, *V;
  __nv_bfloat16* O;
  float* lse;
  const int32_t* sel_idx;
  const int32_t* sel_cnt;
  int64_t q_st, q_sh, kv_st, kv_sh;
  int N, Hq, Hkv, G, k_max, n_items;
  float scale_log2;
};

struct Ctx {
  volatile int* abort;
  int role;
};

// Raises the CTA-wide abort flag; the first give-up of the launch is recorded in the status words.
__device__ __forceinline__ void give_up(const Ctx& c, int which) {
  if (!*c.abort) {
    *c.abort = 1;
    if (atomicCAS(&g_token_status[0], 0, 4) == 0) {
      g_token_status[1] = (int32_t)blockIdx.x;
      g_token_status[2] = c.role;
      g_token_status[3] = which;
    }
  }
}
// Bounded wait; false on expiry, or when another role of the CTA has given up.
__device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity, const Ctx& c, int which) {
  if (mbar_wait_bounded(bar, parity, kWaitLimitNs, c.abort)) return true;
  give_up(c, which);
  return false;
}

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ float lds_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void sts_f32(uint32_t addr, float v) { asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory"); }
__device__ __forceinline__ void sts_bf16(uint32_t addr, float v) {
  const __nv_bfloat16 b = __float2bfloat16_rn(v);
  asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(*(const unsigned short*)&b) : "memory");
}
__device__ __forceinline__ float warp_max(float v) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
  return r;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// One arrival on `bar` once every cp.async this thread has issued so far has landed (the barrier's count
// includes these arrivals).
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

// Byte offset of element (row, 16-byte chunk) inside a K-major operand of 64-column halves with 128-byte swizzle:
// 8-row groups of 1024 bytes, the chunk index XORed with the row inside its group.
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((chunk ^ (row & 7)) << 4));
}

constexpr uint32_t kIdescS = make_idesc_ex(kKeys, kNPad, 0, 0);     // K rows (K-major) x Q_g (K-major)
constexpr uint32_t kIdescPV = make_idesc_ex(kKeys, kNPad, 1, 0);    // V rows as V^T (MN-major) x P^T (K-major)

template <int GP>
__global__ void __launch_bounds__(kThreads, 1)
token_attn_tc_kernel(const TokArgs a) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = ((uint32_t)__cvta_generic_to_shared(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem_gen = smem_raw + (smem_base - (uint32_t)__cvta_generic_to_shared(smem_raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bars = smem_base + kOffBars;
  auto k_full = [&](int s) { return bars + 8 * s; };
  auto v_full = [&](int s) { return bars + 8 * (kStages + s); };
  auto empty = [&](int s) { return bars + 8 * (2 * kStages + s); };
  auto s_full = [&](int b) { return bars + 8 * (3 * kStages + b); };
  auto p_ready = [&](int b) { return bars + 8 * (3 * kStages + kSBuf + b); };
  auto red_bar = [&](int b) { return bars + 8 * (3 * kStages + 2 * kSBuf + b); };
  auto sum_bar = [&](int b) { return bars + 8 * (3 * kStages + 3 * kSBuf + b); };
  // P V of tile g completes phase g / kPvBars of pv_done(g % kPvBars).  A parity wait tells only phases one apart,
  // and a softmax thread that asks for tile g knows no more than that P V of tile g - kStages is complete (its stage
  // was refilled): with more barriers than stages the barrier it waits on is never a phase behind.
  auto pv_done = [&](uint32_t g) { return bars + 8 * (3 * kStages + 3 * kSBuf + 2 + (g % kPvBars)); };
  const uint32_t o_free = bars + 8 * (3 * kStages + 3 * kSBuf + 2 + kPvBars);
  volatile int* abort_flag = (volatile int*)(smem_gen + kOffAbort);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(k_full(s), 128); mbar_init(v_full(s), 128); mbar_init(empty(s), 1); }  // full: an arrival per copying thread
    for (int b = 0; b < kSBuf; ++b) { mbar_init(s_full(b), 1); mbar_init(p_ready(b), 4); mbar_init(red_bar(b), 4); }
    for (int b = 0; b < 2; ++b) mbar_init(sum_bar(b), 4);
    for (uint32_t b = 0; b < kPvBars; ++b) mbar_init(pv_done(b), 1);
    mbar_init(o_free, 4);
    *abort_flag = 0;
    mbar_init_fence();
  }
  // the rows of the Q_g and P^T operands beyond the group's heads stay zero for the whole kernel
  for (int s = 0; s < kStages; ++s)
    for (int e = threadIdx.x; e < 2 * kSmall / 16; e += kThreads)
      *(uint4*)(smem_gen + s * kStageBytes + kOffQ + e * 16) = make_uint4(0, 0, 0, 0);
  fence_async_smem();
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_base + kOffTmem), "n"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *(volatile uint32_t*)(smem_gen + kOffTmem);

  // item i of this CTA: (query token, kv head), long lists first; n = its list length
  auto item_of = [&](int i, int& t, int& kvh, int& n) {
    t = a.N - 1 - i / a.Hkv;
    kvh = i - (i / a.Hkv) * a.Hkv;
    n = min(max(a.sel_cnt[(int64_t)kvh * a.N + t], 0), min(a.k_max, t + 1));
  };

  if (warp < 4) {
    // ============================== softmax and epilogue: thread = key of the tile, then output column ==========
    // GP = the group's heads rounded up to 4, 8 or 16: the columns of S^T / O^T this role looks at (the columns
    // beyond the group's heads come from zero rows of Q_g: finite, never stored)
    const Ctx ctx{abort_flag, kRoleSoftmax};
    const int m = warp * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    const uint32_t red_s = smem_base + kOffRed, sums_s = red_s + kSBuf * 4 * kNPad * 4;
    uint32_t gs = 0;   // tiles so far
    uint32_t ord = 0;  // non-empty items so far
    bool ok = true;
    for (int i = blockIdx.x; i < a.n_items && ok; i += gridDim.x) {
      int t, kvh, n;
      item_of(i, t, kvh, n);
      if (n == 0) {
        for (int h = 0; h < a.G; ++h) a.O[((int64_t)t * a.Hq + kvh * a.G + h) * kHeadDim + m] = __float2bfloat16_rn(0.f);
        if (a.lse && m < a.G) a.lse[(int64_t)(kvh * a.G + m) * a.N + t] = -INFINITY;
        continue;
      }
      float m_ref[GP], l_thr[GP];
#pragma unroll
      for (int h = 0; h < GP; ++h) { m_ref[h] = -INFINITY; l_thr[h] = 0.f; }
      const int ntiles = (n + kKeys - 1) / kKeys;
      for (int ti = 0; ti < ntiles; ++ti, ++gs) {
        const int sb = gs % kSBuf, st = gs % kStages;
        const uint32_t sb_par = (gs / kSBuf) & 1;
        ok = __all_sync(0xffffffffu, wait(s_full(sb), sb_par, ctx, kBarSFull));
        if (!ok) break;
        tc_fence_after();
        uint32_t sr[kNPad];
        tmem_ld16_sync(lane_addr + kColS + sb * kNPad, sr);
        const bool valid = ti * kKeys + m < n;
        float sv[GP];
        // maxima of the tile per head: one warp-wide reduction each, the four warps through shared memory
        const uint32_t red_w = red_s + (uint32_t)((sb * 4 + warp) * kNPad * 4);
#pragma unroll
        for (int h = 0; h < GP; ++h) {
          sv[h] = valid ? __uint_as_float(sr[h]) * a.scale_log2 : -INFINITY;
          const float wm = warp_max(sv[h]);
          if (lane == 0) sts_f32(red_w + h * 4, wm);
        }
        if (lane == 0) mbar_arrive(red_bar(sb));
        ok = __all_sync(0xffffffffu, wait(red_bar(sb), sb_par, ctx, kBarRed));
        if (!ok) break;
        bool rescale = false;
        float alpha[GP];
#pragma unroll
        for (int h = 0; h < GP; ++h) {
          const uint32_t r4 = red_s + (uint32_t)((sb * 4 * kNPad + h) * 4);
          const float mt = fmaxf(fmaxf(lds_f32(r4), lds_f32(r4 + kNPad * 4)), fmaxf(lds_f32(r4 + 2 * kNPad * 4), lds_f32(r4 + 3 * kNPad * 4)));
          alpha[h] = 1.f;
          if (ti == 0) {
            m_ref[h] = mt;
          } else if (mt > m_ref[h] + kRescale) {
            alpha[h] = exp2f(m_ref[h] - mt);
            m_ref[h] = mt;
            rescale = true;  // the same decision in all 128 threads: it depends on shared values only
          }
        }
        if (rescale) {
          // O^T must be quiescent: P V of the previous tile complete (that of this tile waits for p_ready below)
          ok = __all_sync(0xffffffffu, wait(pv_done(gs - 1), ((gs - 1) / kPvBars) & 1, ctx, kBarPvDone));
          if (!ok) break;
          tc_fence_after();
          uint32_t orr[kNPad];
          tmem_ld16_sync(lane_addr + kColO, orr);
#pragma unroll
          for (int h = 0; h < GP; ++h) {
            orr[h] = __float_as_uint(__uint_as_float(orr[h]) * alpha[h]);
            l_thr[h] *= alpha[h];
          }
          tmem_st16(lane_addr + kColO, orr);
          tmem_st_wait();
        }
        // P^T of this key into the stage's operand buffer (row = head, column = key), bf16
        const uint32_t pbuf = smem_base + st * kStageBytes + kOffP + (m >> 6) * kSmallHalf + (m & 7) * 2;
        const int chunk = (m & 63) >> 3;
#pragma unroll
        for (int h = 0; h < GP; ++h) {
          const float p = fast_exp2(sv[h] - m_ref[h]);  // 0 for a key past the end of the list
          l_thr[h] += p;
          sts_bf16(pbuf + swz(h, chunk), p);
        }
        fence_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_ready(sb));
      }
      if (!ok) break;
      // ---- epilogue: P V of the item's last tile complete -> O^T / l -> bf16 -> global memory
      ok = __all_sync(0xffffffffu, wait(pv_done(gs - 1), ((gs - 1) / kPvBars) & 1, ctx, kBarPvDone));
      if (!ok) break;
      tc_fence_after();
      uint32_t orr[kNPad];
      tmem_ld16_sync(lane_addr + kColO, orr);
      tc_fence_before();
      // row sums: this thread's keys -> warp -> CTA
      const int ob = ord & 1;
      const uint32_t sum_w = sums_s + (uint32_t)((ob * 4 + warp) * kNPad * 4);
#pragma unroll
      for (int h = 0; h < GP; ++h) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) l_thr[h] += __shfl_xor_sync(0xffffffffu, l_thr[h], d);
        if (lane == 0) sts_f32(sum_w + h * 4, l_thr[h]);
      }
      if (lane == 0) {
        mbar_arrive(sum_bar(ob));
        mbar_arrive(o_free);  // O^T is in registers: the next item's P V may overwrite it
      }
      ok = __all_sync(0xffffffffu, wait(sum_bar(ob), (ord >> 1) & 1, ctx, kBarSum));
      if (!ok) break;
#pragma unroll
      for (int h = 0; h < GP; ++h) {
        if (h < a.G) {
          const uint32_t s4 = sums_s + (uint32_t)((ob * 4 * kNPad + h) * 4);
          const float l = (lds_f32(s4) + lds_f32(s4 + kNPad * 4)) + (lds_f32(s4 + 2 * kNPad * 4) + lds_f32(s4 + 3 * kNPad * 4));
          a.O[((int64_t)t * a.Hq + kvh * a.G + h) * kHeadDim + m] = __float2bfloat16_rn(__uint_as_float(orr[h]) / l);
          if (a.lse && m == 0) a.lse[(int64_t)(kvh * a.G + h) * a.N + t] = (m_ref[h] + log2f(l)) * 0.6931471805599453f;
        }
      }
      ++ord;
    }
  } else if (warp < kMmaWarp) {
    // ============================== copies: thread pw * 32 + lane owns row pw * 32 + lane of every tile ==========
    const Ctx ctx{abort_flag, kRoleCopy};
    const int pw = warp - 4;
    const int sub = lane >> 4, c16 = lane & 15;  // a warp instruction copies rows 2 i and 2 i + 1 whole: 16 chunks each
    uint32_t g = 0;
    bool ok = true;
    // the list entry of this thread's row in the next tile is fetched one tile ahead
    auto first_item = [&](int from, int& t, int& kvh, int& n) -> int {
      int i = from;
      for (; i < a.n_items; i += gridDim.x) {
        item_of(i, t, kvh, n);
        if (n > 0) break;
      }
      return i;
    };
    int t = 0, kvh = 0, n = 0;
    int i = first_item(blockIdx.x, t, kvh, n);
    int ti = 0;
    auto row_of = [&](int t_, int kvh_, int n_, int ti_) -> int {
      const int e = ti_ * kKeys + pw * 32 + lane;
      // past the end of the list: the query token itself (a valid row; its probability is masked to zero)
      return e < n_ ? min(max(a.sel_idx[((int64_t)kvh_ * a.N + t_) * a.k_max + e], 0), t_) : t_;
    };
    int row = i < a.n_items ? row_of(t, kvh, n, 0) : 0;
    while (i < a.n_items && ok) {
      const int ntiles = (n + kKeys - 1) / kKeys;
      // this tile's coordinates; then step to the next tile (possibly of the next item) and fetch its list entry
      const int c_t = t, c_kvh = kvh, c_row = row;
      int n_i = i, n_t = t, n_kvh = kvh, n_n = n, n_ti = ti + 1;
      if (n_ti == ntiles) {
        n_ti = 0;
        n_i = first_item(i + gridDim.x, n_t, n_kvh, n_n);
      }
      if (n_i < a.n_items) row = row_of(n_t, n_kvh, n_n, n_ti);

      const int st = g % kStages;
      if (g >= kStages) {
        ok = __all_sync(0xffffffffu, wait(empty(st), ((g / kStages) - 1) & 1, ctx, kBarEmpty));
        if (!ok) break;
      }
      const uint32_t stage_s = smem_base + st * kStageBytes;
      if (pw == 0) {
        // the group's query vectors: G rows of 16 chunks
        const __nv_bfloat16* qrow = a.Q + (int64_t)c_t * a.q_st + (int64_t)(c_kvh * a.G) * a.q_sh;
        for (int e = lane; e < a.G * 16; e += 32) {
          const int h = e >> 4, c = e & 15;
          cp_async16(stage_s + kOffQ + (c >> 3) * kSmallHalf + swz(h, c & 7), qrow + (int64_t)h * a.q_sh + c * 8);
        }
      }
      const __nv_bfloat16* kbase = a.K + (int64_t)c_kvh * a.kv_sh + c16 * 8;
      const __nv_bfloat16* vbase = a.V + (int64_t)c_kvh * a.kv_sh + c16 * 8;
      const uint32_t dst0 = stage_s + (c16 >> 3) * kHalf;
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        const int r = pw * 32 + 2 * q + sub;
        const int tok = __shfl_sync(0xffffffffu, c_row, 2 * q + sub);
        cp_async16(dst0 + kOffK + swz(r, c16 & 7), kbase + (int64_t)tok * a.kv_st);
      }
      cp_async_arrive(k_full(st));
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        const int r = pw * 32 + 2 * q + sub;
        const int tok = __shfl_sync(0xffffffffu, c_row, 2 * q + sub);
        cp_async16(dst0 + kOffV + swz(r, c16 & 7), vbase + (int64_t)tok * a.kv_st);
      }
      cp_async_arrive(v_full(st));
      ++g;
      i = n_i; t = n_t; kvh = n_kvh; n = n_n; ti = n_ti;
    }
    // no copy of this thread may be in flight when the CTA ends
    asm volatile("cp.async.wait_all;" ::: "memory");
  } else {
    // ============================== MMAs ==============================
    // Two cursors walk the CTA's tiles: cq (next Q K^T) and cp (next P V).  Whatever has its inputs is issued, P V
    // first because it frees a stage; Q K^T of tile g needs S^T buffer g % kSBuf, free once P V of tile g - kSBuf has
    // been issued (that waited for the softmax of that tile).  Lane 0 polls without suspending and broadcasts.
    const Ctx ctx{abort_flag, kRoleMma};
    const bool leader = elect_one();
    struct Cursor {
      int i, n, ti, ntiles;
      uint32_t g, ord;
    };
    auto seek = [&](Cursor& c) {  // to the first non-empty item at or behind c.i
      for (; c.i < a.n_items; c.i += gridDim.x) {
        int t, kvh;
        item_of(c.i, t, kvh, c.n);
        if (c.n > 0) break;
      }
      c.ti = 0;
      c.ntiles = (c.n + kKeys - 1) / kKeys;
    };
    auto step = [&](Cursor& c) {
      ++c.g;
      if (++c.ti == c.ntiles) {
        ++c.ord;
        c.i += gridDim.x;
        seek(c);
      }
    };
    Cursor cq{(int)blockIdx.x, 0, 0, 0, 0u, 0u};
    seek(cq);
    Cursor cp = cq;
    bool ok = true;
    uint64_t idle_since = 0;
    uint32_t idle = 0;
    while (cp.i < a.n_items && ok) {
      int what = 0;  // 1: P V of cp, 2: Q K^T of cq
      if (lane == 0) {
        if (cp.g < cq.g) {
          const bool first = cp.ti == 0;
          if (mbar_test(p_ready(cp.g % kSBuf), (cp.g / kSBuf) & 1) && mbar_test(v_full(cp.g % kStages), (cp.g / kStages) & 1) &&
              (!(first && cp.ord > 0) || mbar_test(o_free, (cp.ord - 1) & 1)))
            what = 1;
        }
        if (what == 0 && cq.i < a.n_items && cq.g < cp.g + kSBuf && mbar_test(k_full(cq.g % kStages), (cq.g / kStages) & 1)) what = 2;
      }
      what = __shfl_sync(0xffffffffu, what, 0);
      if (what == 0) {
        if (idle == 0) idle_since = globaltimer();
        __nanosleep(20);  // the issue slots belong to the softmax and copy warps that share this scheduler
        if ((++idle & 63u) == 0u && (*abort_flag || globaltimer() - idle_since > kWaitLimitNs)) {
          give_up(ctx, kBarDrain);
          ok = false;
          break;
        }
        continue;
      }
      idle = 0;
      fence_async_smem();  // operands written through the generic proxy (cp.async, the softmax threads' stores)
      tc_fence_after();
      if (what == 1) {
        const int st = cp.g % kStages;
        if (leader) {
          const uint32_t v_addr = smem_base + st * kStageBytes + kOffV, p_addr = smem_base + st * kStageBytes + kOffP;
#pragma unroll
          for (int k = 0; k < kKeys / 16; ++k)
            mma_ss(tmem + kColO, smem_desc(v_addr + k * 2048, kHalf, 1024), smem_desc(p_addr + (k >> 2) * kSmallHalf + (k & 3) * 32),
                   kIdescPV, (cp.ti == 0 && k == 0) ? 0u : 1u);
          tc_commit(empty(st));
          tc_commit(pv_done(cp.g));
        }
        __syncwarp();
        step(cp);
      } else {
        const int st = cq.g % kStages, sb = cq.g % kSBuf;
        if (leader) {
          const uint32_t k_addr = smem_base + st * kStageBytes + kOffK, q_addr = smem_base + st * kStageBytes + kOffQ;
#pragma unroll
          for (int k = 0; k < kHeadDim / 16; ++k)
            mma_ss(tmem + kColS + sb * kNPad, smem_desc(k_addr + (k >> 2) * kHalf + (k & 3) * 32),
                   smem_desc(q_addr + (k >> 2) * kSmallHalf + (k & 3) * 32), kIdescS, k ? 1u : 0u);
          tc_commit(s_full(sb));
        }
        __syncwarp();
        step(cq);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    if (*abort_flag) {
      const uint64_t t0 = globaltimer();
      while (globaltimer() - t0 < 2000000ull) {}  // 2 ms: far beyond any MMA still in flight
    }
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kTmemCols) : "memory");
  }
}

}  // namespace

int token_attn_max_group() { return kNPad; }

cudaError_t launch_token_attention(const void* Q, const void* K, const void* V, int64_t q_st, int64_t q_sh, int64_t kv_st,
                                   int64_t kv_sh, int N, int Hq, int Hkv, int k_max, const int32_t* sel_idx,
                                   const int32_t* sel_cnt, float softmax_scale, void* O, float* lse, cudaStream_t s) {
  static bool attr_set[64] = {};
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  if (!attr_set[dev & 63]) {
    e = cudaFuncSetAttribute(token_attn_tc_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(token_attn_tc_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(token_attn_tc_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set[dev & 63] = true;
  }
  TokArgs a{};
  a.Q = (const __nv_bfloat16*)Q;
  a.K = (const __nv_bfloat16*)K;
  a.V = (const __nv_bfloat16*)V;
  a.O = (__nv_bfloat16*)O;
  a.lse = lse;
  a.sel_idx = sel_idx;
  a.sel_cnt = sel_cnt;
  a.q_st = q_st; a.q_sh = q_sh; a.kv_st = kv_st; a.kv_sh = kv_sh;
  a.N = N; a.Hq = Hq; a.Hkv = Hkv; a.G = Hq / Hkv; a.k_max = k_max;
  a.n_items = N * Hkv;
  a.scale_log2 = softmax_scale * 1.4426950408889634f;
  const int grid = std::min(a.n_items, sms);
  if (a.G <= 4) token_attn_tc_kernel<4><<<grid, kThreads, kSmemBytes, s>>>(a);
  else if (a.G <= 8) token_attn_tc_kernel<8><<<grid, kThreads, kSmemBytes, s>>>(a);
  else token_attn_tc_kernel<16><<<grid, kThreads, kSmemBytes, s>>>(a);
  return cudaGetLastError();
}

// Reads (and clears) the status words of the gather-attention kernel after the caller synchronised the stream.
cudaError_t token_status_words(int32_t* out4) {
  cudaError_t e = cudaMemcpyFromSymbol(out4, g_token_status, sizeof(g_token_status));
  if (e != cudaSuccess) return e;
  if (out4[0] != 0) {
    const int32_t zero[4] = {0, 0, 0, 0};
    e = cudaMemcpyToSymbol(g_token_status, zero, sizeof(zero));
  }
  return e;
}

}  // namespace stem
