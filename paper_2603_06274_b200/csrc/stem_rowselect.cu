// Alg. 1 steps 3b-3c from a stored metric: Token Position-Decay budget and top-k block selection,
// one warp per (head, query-block row).
//
// A row's forced blocks are its first `stem` and last `local` causal blocks; the candidates are the
// causal blocks between them.  The row takes the need = k_eff(r) - #forced best candidates by
// (metric descending, block id ascending), metric compared as an order-preserving 32-bit key with
// -0 == +0 and NaN as -inf.  The warp holds the candidates' keys in registers (candidate c of the row
// in lane c % 32, register c / 32), finds the need-th largest key by a most-significant-bit-first
// radix descent, one warp-wide population count per varying key bit, and writes the selected block
// ids in ascending order.  For the descent each lane keeps its 32 keys bit-transposed (word b holds
// bit b of every key), so that one AND and one popc per lane count a bit over the whole row.
#include <cuda_runtime.h>

#include "stem_internal.h"

namespace stem {

namespace {

constexpr int kThreads = 256;

// Monotone map float -> uint32 with -0 == +0 and NaN below everything (as -inf).  Every key is >= 1.
__device__ __forceinline__ uint32_t metric_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) u = 0xff800000u;  // NaN -> -inf
  if (u == 0x80000000u) u = 0u;                          // -0 -> +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// In-register transpose of a 32 x 32 bit matrix: afterwards bit t of w[b] is bit b of the old w[t].
__device__ __forceinline__ void transpose32(uint32_t (&w)[32]) {
#pragma unroll
  for (int s = 0; s < 5; ++s) {
    const int j = 16 >> s;
    const uint32_t m = s == 0 ? 0xffff0000u : s == 1 ? 0xff00ff00u : s == 2 ? 0xf0f0f0f0u : s == 3 ? 0xccccccccu : 0xaaaaaaaau;
#pragma unroll
    for (int k = 0; k < 32; ++k) {
      if (k & j) continue;
      // swap the high-j-bit part of row k with the low-j-bit part of row k + j
      const uint32_t t = ((w[k] >> j) ^ w[k + j]) & (m >> j);
      w[k] ^= t << j;
      w[k + j] ^= t;
    }
  }
}

struct SelArgs {
  const float* M;
  int32_t* sel_idx;
  int32_t* sel_cnt;
  RowTables rows;
  int64_t m_tot;
  int Hq, R_tot, k_max, stem, local;
};

// SETS = 32-key register sets per lane: rows of up to SETS * 1024 candidates.
template <int SETS>
__global__ void __launch_bounds__(kThreads, SETS == 1 ? 4 : 2) select_rows_kernel(const SelArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t item = (int64_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
  if (item >= (int64_t)a.Hq * a.R_tot) return;
  // rows in descending order so that the long rows of a launch start first
  const int h = (int)(item % a.Hq);
  const int R = a.R_tot - 1 - (int)(item / a.Hq);
  const int seq = a.rows.row_seq[R];
  const int r = a.rows.row_r[R];
  const int nb = a.rows.seq_nblk[seq];
  const int i = r + 1;
  const int n_stem = min(a.stem, i);
  const int c_lo = n_stem, c_hi = max(max(i - a.local, 0), n_stem);  // candidates [c_lo, c_hi)
  const int n_cand = c_hi - c_lo;
  const int n_forced = i - n_cand;
  const int need = max(min(a.rows.row_keff[R] - n_forced, n_cand), 0);
  int32_t* out = a.sel_idx + ((int64_t)h * a.R_tot + R) * a.k_max;
  const float* mrow = a.M + (int64_t)h * a.m_tot + a.rows.seq_m_off[seq] + (int64_t)r * nb;
  const uint32_t lt_mask = (1u << lane) - 1u;

  // ---- keys of the candidates (0 = no candidate; every real key is >= 1), then bit-transposed in place
  uint32_t tw[SETS][32];
  uint32_t act[SETS], gt[SETS];  // per key of this lane (bit t <-> register t): still in the descent / known > T
  uint32_t vary = 0u;
  const uint32_t key0 = n_cand > 0 ? metric_key(mrow[c_lo]) : 0u;
#pragma unroll
  for (int s = 0; s < SETS; ++s) {
    act[s] = 0u;
    gt[s] = 0u;
#pragma unroll
    for (int t = 0; t < 32; ++t) {
      const int j = c_lo + (s * 32 + t) * 32 + lane;
      uint32_t kx = 0u;
      if ((s * 32 + t) * 32 < n_cand && j < c_hi) {
        kx = metric_key(mrow[j]);
        act[s] |= 1u << t;
        vary |= kx ^ key0;
      }
      tw[s][t] = kx;
    }
    transpose32(tw[s]);
  }

  // ---- threshold: the need-th largest key T; gt = keys above it, act = keys equal to it
  int rem = 0;  // how many of the keys equal to T are taken (the first ones by block id)
  if (need == 0) {
#pragma unroll
    for (int s = 0; s < SETS; ++s) act[s] = 0u;
  } else if (need == n_cand) {
#pragma unroll
    for (int s = 0; s < SETS; ++s) { gt[s] = act[s]; act[s] = 0u; }
  } else {
    vary = __reduce_or_sync(0xffffffffu, vary);
    int k = need;  // rank wanted among the keys still active
#pragma unroll
    for (int b = 31; b >= 0; --b) {
      if (!((vary >> b) & 1u)) continue;  // warp-uniform: all candidates agree on this bit
      int cnt = 0;
#pragma unroll
      for (int s = 0; s < SETS; ++s) cnt += __popc(tw[s][b] & act[s]);
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      if (cnt >= k) {
#pragma unroll
        for (int s = 0; s < SETS; ++s) act[s] &= tw[s][b];
      } else {
        k -= cnt;
#pragma unroll
        for (int s = 0; s < SETS; ++s) { gt[s] |= act[s] & tw[s][b]; act[s] &= ~tw[s][b]; }
      }
    }
    rem = k;
  }
  // Equal keys beyond the ones needed are the rare case; otherwise every key equal to T is taken.
  int n_eq = 0;
#pragma unroll
  for (int s = 0; s < SETS; ++s) n_eq += __popc(act[s]);
  n_eq = __reduce_add_sync(0xffffffffu, n_eq);
  const bool ties = n_eq > rem;

  // ---- emission in ascending block order: stem blocks, selected candidates, local blocks
  for (int j = lane; j < n_stem; j += 32) out[j] = j;
  int base = n_stem, eq_before = 0;
#pragma unroll
  for (int s = 0; s < SETS; ++s) {
    const uint32_t sel = ties ? gt[s] : (gt[s] | act[s]);
#pragma unroll
    for (int t = 0; t < 32; ++t) {
      if ((s * 32 + t) * 32 >= n_cand) break;  // warp-uniform
      bool take = (sel >> t) & 1u;
      if (ties) {
        const bool eq = (act[s] >> t) & 1u;
        const uint32_t eqb = __ballot_sync(0xffffffffu, eq);
        take = take || (eq && eq_before + __popc(eqb & lt_mask) < rem);
        eq_before += __popc(eqb);
      }
      const uint32_t selb = __ballot_sync(0xffffffffu, take);
      if (take) out[base + __popc(selb & lt_mask)] = c_lo + (s * 32 + t) * 32 + lane;
      base += __popc(selb);
    }
  }
  for (int j = c_hi + lane; j < i; j += 32) out[base + (j - c_hi)] = j;
  const int total = base + (i - c_hi);
  for (int q = total + lane; q < a.k_max; q += 32) out[q] = -1;
  if (lane == 0) a.sel_cnt[(int64_t)h * a.R_tot + R] = total;
}

}  // namespace

int row_select_max_blocks() { return 2 * 1024; }

cudaError_t launch_select_rows(const Plan& p, const float* M, int32_t* sel_idx, int32_t* sel_cnt, cudaStream_t s) {
  SelArgs a{};
  a.M = M; a.sel_idx = sel_idx; a.sel_cnt = sel_cnt; a.rows = p.rows; a.m_tot = p.m_tot;
  a.Hq = p.cfg.num_q_heads; a.R_tot = p.R_tot; a.k_max = p.k_max;
  a.stem = p.cfg.stem_blocks; a.local = p.cfg.local_blocks;
  const int64_t items = (int64_t)a.Hq * a.R_tot;
  const int grid = (int)((items + kThreads / 32 - 1) / (kThreads / 32));
  if (p.max_nblk <= 1024)
    select_rows_kernel<1><<<grid, kThreads, 0, s>>>(a);
  else
    select_rows_kernel<2><<<grid, kThreads, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace stem
