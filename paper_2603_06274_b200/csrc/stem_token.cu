// Token Position-Decay on a token-level top-k selector (Main Results: integration with a sparse-attention
// model whose indexer keeps the top 2048 tokens per query; there k_start = 2048 and mu = 0.7).  Selection
// granularity is one token: query token t keeps k(t) of its t+1 causal tokens, k(t) from Eq. 3 at token
// positions, ranked by an indexer score the caller supplies (one score matrix per kv head: the heads of a
// group share the selection), and attends over exactly those tokens.  This file holds the selection:
//
//   token_select_kernel   one CTA per (list head, query token): exact top-k of the row's candidates by
//                         (score descending, token id ascending) with a radix selection, a byte per pass, on
//                         order-preserving keys through shared-memory histograms (it stops as soon as the bin that
//                         holds the rank is taken whole); the forced tokens (the first
//                         `stem` and the last `local`, the token itself included) are kept outside the
//                         ranking; the list comes out ascending.  The row's keys are converted once into
//                         shared memory (rows of up to 51 200 tokens; longer rows are re-read from the L2).
//
// The attention over the lists is in stem_token_attn.cu.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "stem_internal.h"

namespace stem {

namespace {

// Monotone map float -> uint32 with -0 == +0 and NaN below everything (as -inf).
__device__ __forceinline__ uint32_t score_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) u = 0xff800000u;
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kSelThreads = 256;

// Number of keys equal to the threshold in the segments of the warps before warp w.
__device__ __forceinline__ int eq_before_all(const int* seg_eq, int w) {
  int n = 0;
  for (int q = 0; q < w; ++q) n += seg_eq[q];
  return n;
}

// kInSmem: the row's candidate keys are converted once and kept in (dynamic) shared memory, so the score row is
// read from memory a single time; rows too long for that are re-read from memory (they stay in the L2).
template <bool kInSmem>
__global__ void __launch_bounds__(kSelThreads) token_select_kernel(const float* __restrict__ scores, int N, int k_max,
                                                                   const int32_t* __restrict__ k_tok, int stem, int local,
                                                                   int32_t* __restrict__ sel_idx, int32_t* __restrict__ sel_cnt) {
  extern __shared__ uint32_t s_keys[];
  __shared__ int hist[kSelThreads / 32][256];  // one histogram per warp: fewer colliding atomics
  __shared__ uint32_t s_prefix;
  __shared__ int s_need, s_whole;
  const int t = N - 1 - (int)blockIdx.x;  // long rows first
  const int lh = blockIdx.y;
  const int warp = threadIdx.x >> 5;
  const int i = t + 1;                                                    // causal tokens 0 .. t
  const int n_stem = min(stem, i);
  const int c_lo = n_stem, c_hi = max(max(i - local, 0), n_stem);         // candidates [c_lo, c_hi)
  const int n_cand = c_hi - c_lo;
  const int n_forced = i - n_cand;
  const int need = max(min(k_tok[t] - n_forced, n_cand), 0);
  const float* row = scores + ((int64_t)lh * N + t) * N;
  int32_t* out = sel_idx + ((int64_t)lh * N + t) * k_max;
  auto key_at = [&](int c) -> uint32_t { return kInSmem ? s_keys[c - c_lo] : score_key(row[c]); };

  const bool ranked = need > 0 && need < n_cand;  // otherwise none or all of the candidates are taken
  if (kInSmem && ranked) {
    for (int c = c_lo + (int)threadIdx.x; c < c_hi; c += kSelThreads) s_keys[c - c_lo] = score_key(row[c]);
    __syncthreads();
  }
  // ---- the need-th largest key: most significant byte first, a histogram per byte
  uint32_t prefix = 0u;   // the bytes decided so far (in the high bits)
  uint32_t decided = 0u;  // their bit mask
  int k = need;           // rank wanted among the keys that match the prefix
  bool whole = false;     // the bin that holds the rank is taken whole: the remaining bytes need no pass
  if (ranked) {
    for (int pass = 0; pass < 4 && !whole; ++pass) {
      const int shift = 24 - 8 * pass;
      const uint32_t mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
#pragma unroll
      for (int w = 0; w < kSelThreads / 32; ++w) hist[w][threadIdx.x] = 0;
      __syncthreads();
      for (int c = c_lo + (int)threadIdx.x; c < c_hi; c += kSelThreads) {
        const uint32_t key = key_at(c);
        if ((key & mask) == prefix) atomicAdd(&hist[warp][(key >> shift) & 255u], 1);
      }
      __syncthreads();
      {
        int tot = 0;
#pragma unroll
        for (int w = 0; w < kSelThreads / 32; ++w) tot += hist[w][threadIdx.x];
        __syncthreads();
        hist[0][threadIdx.x] = tot;
      }
      __syncthreads();
      if (warp == 0) {
        // the largest byte value b with (number of keys whose byte is >= b) >= k: lane l owns the bins 8 l .. 8 l + 7
        const int lane = threadIdx.x & 31;
        int mine = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) mine += hist[0][8 * lane + q];
        int above = mine;  // keys in the bins of this lane and of the lanes above it
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int u = __shfl_down_sync(0xffffffffu, above, d);
          if (lane + d < 32) above += u;
        }
        const uint32_t reach = __ballot_sync(0xffffffffu, above >= k);  // lanes at or below the one that holds the rank
        const int owner = 31 - __clz((int)reach);                        // reach != 0: lane 0 counts every key
        if (lane == owner) {
          int acc = above - mine, b = 8 * lane + 7;
          for (; b > 8 * lane; --b) {
            if (acc + hist[0][b] >= k) break;
            acc += hist[0][b];
          }
          s_prefix = prefix | ((uint32_t)b << shift);
          s_need = k - acc;
          s_whole = hist[0][b] == k - acc;
        }
      }
      __syncthreads();
      prefix = s_prefix;
      k = s_need;
      whole = s_whole != 0;
      decided |= 0xffu << shift;
      __syncthreads();
    }
  }
  // keys whose decided bytes are above `prefix` are taken; of those equal to it all (whole) or the first k by token id
  const int k_eq = whole ? 0x7fffffff : k;

  // ---- emission in ascending token order: stem tokens, selected candidates, local tokens
  for (int j = threadIdx.x; j < n_stem; j += kSelThreads) out[j] = j;
  int written = n_stem;
  if (need > 0 && !ranked) {
    for (int c = c_lo + (int)threadIdx.x; c < c_hi; c += kSelThreads) out[n_stem + (c - c_lo)] = c;
    written += n_cand;
  } else if (ranked) {
    // every warp owns one contiguous segment of the candidates: it counts its keys above and equal to the
    // threshold, the counts of the warps before it give its first output position, and it then writes its
    // selected tokens in order (ballots and popcounts, no block-wide step inside the loops)
    const int lane = threadIdx.x & 31;
    const int seg = ((n_cand + kSelThreads / 32 - 1) / (kSelThreads / 32) + 31) & ~31;
    const int s_lo = c_lo + warp * seg, s_hi = min(s_lo + seg, c_hi);
    int n_gt = 0, n_eq = 0;
    for (int c0 = s_lo; c0 < s_hi; c0 += 32) {
      const int c = c0 + lane;
      const uint32_t key = c < s_hi ? key_at(c) : 0u;
      n_gt += __popc(__ballot_sync(0xffffffffu, c < s_hi && (key & decided) > prefix));
      n_eq += __popc(__ballot_sync(0xffffffffu, c < s_hi && (key & decided) == prefix));
    }
    __shared__ int seg_gt[kSelThreads / 32], seg_eq[kSelThreads / 32];
    if (lane == 0) { seg_gt[warp] = n_gt; seg_eq[warp] = n_eq; }
    __syncthreads();
    int eq_before = 0, pos = n_stem, all_sel = 0;
#pragma unroll
    for (int w = 0; w < kSelThreads / 32; ++w) {
      const int take = seg_gt[w] + min(max(k_eq - eq_before_all(seg_eq, w), 0), seg_eq[w]);
      if (w < warp) { pos += take; eq_before += seg_eq[w]; }
      all_sel += take;
    }
    const uint32_t below = (1u << lane) - 1u;
    for (int c0 = s_lo; c0 < s_hi; c0 += 32) {
      const int c = c0 + lane;
      const uint32_t key = c < s_hi ? key_at(c) : 0u;
      const bool gt = c < s_hi && (key & decided) > prefix;
      const bool eq = c < s_hi && (key & decided) == prefix;
      const uint32_t eq_mask = __ballot_sync(0xffffffffu, eq);
      const bool sel = gt || (eq && eq_before + __popc(eq_mask & below) < k_eq);
      const uint32_t sel_mask = __ballot_sync(0xffffffffu, sel);
      if (sel) out[pos + __popc(sel_mask & below)] = c;
      pos += __popc(sel_mask);
      eq_before += __popc(eq_mask);
    }
    written += all_sel;
  }
  for (int j = c_hi + (int)threadIdx.x; j < i; j += kSelThreads) out[written + (j - c_hi)] = j;
  const int total = written + (i - c_hi);
  for (int q = total + (int)threadIdx.x; q < k_max; q += kSelThreads) out[q] = -1;
  if (threadIdx.x == 0) sel_cnt[(int64_t)lh * N + t] = total;
}

}  // namespace

cudaError_t launch_token_select(const float* scores, int N, int H_list, int k_max, const int32_t* k_tok, int stem, int local,
                                int32_t* sel_idx, int32_t* sel_cnt, cudaStream_t s) {
  const dim3 grid((unsigned)N, (unsigned)H_list);
  const size_t row_bytes = (size_t)N * sizeof(uint32_t);
  constexpr size_t kSmemLimit = 200 * 1024;
  if (row_bytes <= kSmemLimit) {
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (!attr_set[dev & 63]) {
      e = cudaFuncSetAttribute(token_select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit);
      if (e != cudaSuccess) return e;
      attr_set[dev & 63] = true;
    }
    token_select_kernel<true><<<grid, kSelThreads, row_bytes, s>>>(scores, N, k_max, k_tok, stem, local, sel_idx, sel_cnt);
  } else {
    token_select_kernel<false><<<grid, kSelThreads, 0, s>>>(scores, N, k_max, k_tok, stem, local, sel_idx, sel_cnt);
  }
  return cudaGetLastError();
}

}  // namespace stem
