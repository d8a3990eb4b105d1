// Alg. 1 steps 3b-3c from a stored metric: Token Position-Decay budget and top-k block selection,
// one warp per (head, query-block row).
//
// A row's forced blocks are its first `stem` and last `local` causal blocks; the candidates are the
// causal blocks between them.  The row takes the need = k_eff(r) - #forced best candidates by
// (metric descending, block id ascending), metric compared as an order-preserving 32-bit key with
// -0 == +0 and NaN as -inf.
// Each lane holds a run of consecutive blocks of the row as bit planes (word b = bit b of every key
// of the lane), and the need-th largest key is found by a most-significant-bit-first radix descent
// that costs one AND + popc per lane and one warp reduction per key bit.  The selected ids come out
// in ascending order by a warp prefix sum over the lanes' counts.  Two kernels:
//   select_rows_kernel    from float metrics (the public M): coalesced loads, a turn through shared
//                         memory into lane-contiguous runs of candidates, key conversion and an
//                         in-register bit transpose per lane;
//   select_planes_kernel  from the bit planes the metric kernel writes for the fused path: one
//                         128-byte line per lane, nothing to convert or transpose.
// Both are bound by the integer pipe, so the stages are written for few logic instructions.
#include <cuda_runtime.h>

#include "stem_internal.h"
#include "stem_ptx.cuh"

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

using ptx::transpose32;

struct SelArgs {
  const float* M;
  const uint32_t* Mt;  // bit-plane form (select_planes_kernel)
  int32_t* sel_idx;
  int32_t* sel_cnt;
  RowTables rows;
  int64_t m_tot, mt_tot;
  int Hq, R_tot, k_max, stem, local;
};

// The mask of the n lowest set bits of m.
__device__ __forceinline__ uint32_t lowest_bits(uint32_t m, int n) {
  uint32_t r = 0u;
  while (n > 0 && m != 0u) {
    const uint32_t b = m & (0u - m);
    r |= b;
    m ^= b;
    --n;
  }
  return r;
}

// SETS = 32-key register sets per lane: rows of up to SETS * 1024 candidates.
template <int SETS>
__global__ void __launch_bounds__(kThreads, SETS == 1 ? 4 : 2) select_rows_kernel(const SelArgs a) {
  constexpr int kStride = 32 * SETS + 1;  // words of shared memory per lane (odd: conflict-free both ways)
  extern __shared__ uint32_t stage_all[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* stage = stage_all + warp * 32 * kStride;
  const int64_t item = (int64_t)blockIdx.x * (kThreads / 32) + warp;
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
  const float* mrow = a.M + (int64_t)h * a.m_tot + a.rows.seq_m_off[seq] + (int64_t)(r - a.rows.seq_r0[seq]) * nb + c_lo;
  const int per = (n_cand + 31) >> 5;  // candidates per lane

  uint32_t sel[SETS];  // per key of this lane (bit t <-> its t-th candidate): selected
#pragma unroll
  for (int s = 0; s < SETS; ++s) sel[s] = 0u;

  if (need > 0) {
    // ---- keys: coalesced loads, through shared memory into runs of `per` consecutive candidates per lane
    const uint32_t magic = ((1u << 20) + per - 1) / per;  // q / per == (q * magic) >> 20 for q < 2048
    for (int q = lane; q < n_cand; q += 32) {
      const uint32_t owner = ((uint32_t)q * magic) >> 20;
      stage[owner * kStride + (q - owner * per)] = metric_key(mrow[q]);
    }
    __syncwarp();
    uint32_t tw[SETS][32];
    uint32_t act[SETS], gt[SETS];  // still in the descent / known to be above the threshold
    const int mine = min(max(n_cand - lane * per, 0), per);  // candidates of this lane
#pragma unroll
    for (int s = 0; s < SETS; ++s) {
      gt[s] = 0u;
      const int cnt_s = min(max(mine - 32 * s, 0), 32);
      act[s] = cnt_s >= 32 ? 0xffffffffu : ((1u << cnt_s) - 1u);
#pragma unroll
      for (int t = 0; t < 32; ++t) {
        uint32_t kx = 0u;
        if (32 * s + t < per) {  // warp-uniform
          kx = stage[lane * kStride + 32 * s + t];
          if (32 * s + t >= mine) kx = 0u;
        }
        tw[s][t] = kx;
      }
      transpose32(tw[s]);
    }

    // ---- the need-th largest key by radix descent; gt = keys above it, act = keys still undecided.
    // Straight-line over all 32 bits (a bit all undecided keys agree on changes nothing: its count is
    // 0 or all of them); at the end the undecided keys are all equal.  The loop is kept free of
    // branches: with warp-uniform branches around the warp reduction in the unrolled loop this
    // compiler produced wrong lists.
    int k = need;  // rank wanted among the undecided keys
#pragma unroll
    for (int b = 31; b >= 0; --b) {
      int cnt = 0;
#pragma unroll
      for (int s = 0; s < SETS; ++s) cnt += __popc(tw[s][b] & act[s]);
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      const bool inside = cnt >= k;  // the k-th largest has this bit set
      k -= inside ? 0 : cnt;
#pragma unroll
      for (int s = 0; s < SETS; ++s) {
        const uint32_t ones = act[s] & tw[s][b];
        gt[s] |= inside ? 0u : ones;
        act[s] = inside ? ones : (act[s] ^ ones);
      }
    }
    const int rem = k;  // of the undecided keys the first `rem` by block id are taken
    // ---- the equal keys that are taken: the first `rem` in lane-major order
    int n_eq = 0;
#pragma unroll
    for (int s = 0; s < SETS; ++s) n_eq += __popc(act[s]);
    int before = n_eq;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, before, d);
      if (lane >= d) before += v;
    }
    before -= n_eq;  // equal keys in lower lanes
    int quota = min(max(rem - before, 0), n_eq);
#pragma unroll
    for (int s = 0; s < SETS; ++s) {
      const int take = min(quota, __popc(act[s]));
      sel[s] = gt[s] | (take == __popc(act[s]) ? act[s] : lowest_bits(act[s], take));
      quota -= take;
    }
  }

  // ---- emission in ascending block order: stem blocks, selected candidates, local blocks
  for (int j = lane; j < n_stem; j += 32) out[j] = j;
  int n_sel = 0;
#pragma unroll
  for (int s = 0; s < SETS; ++s) n_sel += __popc(sel[s]);
  int pos = n_sel;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, pos, d);
    if (lane >= d) pos += v;
  }
  const int n_taken = __shfl_sync(0xffffffffu, pos, 31);  // == need
  pos += n_stem - n_sel;
#pragma unroll
  for (int s = 0; s < SETS; ++s) {
    uint32_t m = sel[s];
    while (m != 0u) {
      const int t = __ffs((int)m) - 1;
      m &= m - 1u;
      out[pos++] = c_lo + lane * per + 32 * s + t;
    }
  }
  const int base = n_stem + n_taken;
  for (int j = c_hi + lane; j < i; j += 32) out[base + (j - c_hi)] = j;
  const int total = base + (i - c_hi);
  for (int q = total + lane; q < a.k_max; q += 32) out[q] = -1;
  if (lane == 0) a.sel_cnt[(int64_t)h * a.R_tot + R] = total;
}

// Inclusive prefix sum over the lanes of a warp.
__device__ __forceinline__ int warp_scan(int v, int lane) {
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int u = __shfl_up_sync(0xffffffffu, v, d);
    if (lane >= d) v += u;
  }
  return v;
}

// The same selection from the bit-plane metric the metric kernel writes for the fused path: row r of
// a sequence holds, for every group of 32 columns, 32 words, word k = bit k of the 32 keys.  Lane L
// owns group L (and group 32 + L for sequences of more than 1024 blocks): it loads its 32 planes
// as one 128-byte line and needs neither key conversion nor transposition.
template <int SETS>
__global__ void __launch_bounds__(kThreads, SETS == 1 ? 4 : 2) select_planes_kernel(const SelArgs a) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t item = (int64_t)blockIdx.x * (kThreads / 32) + warp;
  if (item >= (int64_t)a.Hq * a.R_tot) return;
  const int h = (int)(item % a.Hq);
  const int R = a.R_tot - 1 - (int)(item / a.Hq);  // long rows first
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
  const int stride = (nb + 31) & ~31;
  const uint32_t* prow = a.Mt + (int64_t)h * a.mt_tot + a.rows.seq_mt_off[seq] + (int64_t)(r - a.rows.seq_r0[seq]) * stride;

  uint32_t sel[SETS];
#pragma unroll
  for (int s = 0; s < SETS; ++s) sel[s] = 0u;

  // Launched as a programmatic dependent of the metric kernel, the set-up above overlaps its tail.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (need > 0) {
    uint32_t tw[SETS][32], act[SETS], gt[SETS];
#pragma unroll
    for (int s = 0; s < SETS; ++s) {
      const int j0 = 32 * (lane + 32 * s);  // first column of this lane's group
      gt[s] = 0u;
      // candidates among the columns j0 .. j0 + 31
      const int lo = min(max(c_lo - j0, 0), 32), hi = min(max(c_hi - j0, 0), 32);
      const uint32_t upto_hi = hi >= 32 ? 0xffffffffu : ((1u << hi) - 1u);
      act[s] = hi > lo ? (upto_hi & ~((1u << lo) - 1u)) : 0u;  // lo < 32 when hi > lo
      if (act[s] != 0u) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const uint4 v = *(const uint4*)(prow + j0 + q * 4);
          tw[s][q * 4] = v.x; tw[s][q * 4 + 1] = v.y; tw[s][q * 4 + 2] = v.z; tw[s][q * 4 + 3] = v.w;
        }
      } else {
#pragma unroll
        for (int k = 0; k < 32; ++k) tw[s][k] = 0u;
      }
    }
    // Radix descent as in select_rows_kernel, over all 32 bits: a bit all undecided keys agree on
    // changes nothing (its count is 0 or all of them), so the bits need not be screened first.
    int k = need;
#pragma unroll
    for (int b = 31; b >= 0; --b) {
      // straight-line step: keys with the bit set are either where the k-th largest lies (cnt >= k)
      // or all above it
      int cnt = 0;
#pragma unroll
      for (int s = 0; s < SETS; ++s) cnt += __popc(tw[s][b] & act[s]);
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      const bool inside = cnt >= k;
      k -= inside ? 0 : cnt;
#pragma unroll
      for (int s = 0; s < SETS; ++s) {
        const uint32_t ones = act[s] & tw[s][b];
        gt[s] |= inside ? 0u : ones;
        act[s] = inside ? ones : (act[s] ^ ones);
      }
    }
    // of the undecided keys the first k in column order (set-major, then lane, then bit) are taken
    int rem = k;
#pragma unroll
    for (int s = 0; s < SETS; ++s) {
      const int n_eq = __popc(act[s]);
      const int incl = warp_scan(n_eq, lane);
      const int take = min(max(rem - (incl - n_eq), 0), n_eq);
      sel[s] = gt[s] | (take == n_eq ? act[s] : lowest_bits(act[s], take));
      rem -= __shfl_sync(0xffffffffu, incl, 31);
    }
  }

  // ---- emission in ascending block order: stem blocks, selected candidates, local blocks
  for (int j = lane; j < n_stem; j += 32) out[j] = j;
  int base = n_stem;
#pragma unroll
  for (int s = 0; s < SETS; ++s) {
    const int n_sel = __popc(sel[s]);
    const int incl = warp_scan(n_sel, lane);
    int pos = base + incl - n_sel;
    uint32_t m = sel[s];
    while (m != 0u) {
      const int t = __ffs((int)m) - 1;
      m &= m - 1u;
      out[pos++] = 32 * (lane + 32 * s) + t;
    }
    base += __shfl_sync(0xffffffffu, incl, 31);
  }
  for (int j = c_hi + lane; j < i; j += 32) out[base + (j - c_hi)] = j;
  const int total = base + (i - c_hi);
  for (int q = total + lane; q < a.k_max; q += 32) out[q] = -1;
  if (lane == 0) a.sel_cnt[(int64_t)h * a.R_tot + R] = total;
}

}  // namespace

int row_select_max_blocks() { return 2 * 1024; }

static SelArgs make_args(const Plan& p, int32_t* sel_idx, int32_t* sel_cnt) {
  SelArgs a{};
  a.sel_idx = sel_idx; a.sel_cnt = sel_cnt; a.rows = p.rows; a.m_tot = p.m_tot; a.mt_tot = p.mt_tot;
  a.Hq = p.H_list; a.R_tot = p.R_tot; a.k_max = p.k_max;
  a.stem = p.cfg.stem_blocks; a.local = p.cfg.local_blocks;
  return a;
}

static cudaLaunchConfig_t make_config(const SelArgs& a, size_t smem, cudaStream_t s, cudaLaunchAttribute* attr, bool dependent) {
  const int64_t items = (int64_t)a.Hq * a.R_tot;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((items + kThreads / 32 - 1) / (kThreads / 32)));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
  return cfg;
}

cudaError_t launch_select_rows(const Plan& p, const float* M, bool dependent, int32_t* sel_idx, int32_t* sel_cnt,
                               cudaStream_t s) {
  SelArgs a = make_args(p, sel_idx, sel_cnt);
  a.M = M;
  constexpr int kSmem1 = (kThreads / 32) * 32 * 33 * 4, kSmem2 = (kThreads / 32) * 32 * 65 * 4;
  // the attribute belongs to the device's context: set it once per device of this process
  static bool attr_set[64] = {};
  const int dev_slot = p.device & 63;
  if (!attr_set[dev_slot]) {
    cudaError_t e = cudaFuncSetAttribute(select_rows_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem2);
    if (e != cudaSuccess) return e;
    attr_set[dev_slot] = true;
  }
  cudaLaunchAttribute attr[1];
  if (p.max_nblk <= 1024) {
    cudaLaunchConfig_t cfg = make_config(a, kSmem1, s, attr, dependent);
    return cudaLaunchKernelEx(&cfg, select_rows_kernel<1>, a);
  }
  cudaLaunchConfig_t cfg = make_config(a, kSmem2, s, attr, dependent);
  return cudaLaunchKernelEx(&cfg, select_rows_kernel<2>, a);
}

cudaError_t launch_select_planes(const Plan& p, const uint32_t* Mt, bool dependent, int32_t* sel_idx, int32_t* sel_cnt,
                                 cudaStream_t s) {
  SelArgs a = make_args(p, sel_idx, sel_cnt);
  a.Mt = Mt;
  cudaLaunchAttribute attr[1];
  cudaLaunchConfig_t cfg = make_config(a, 0, s, attr, dependent);
  if (p.max_nblk <= 1024) return cudaLaunchKernelEx(&cfg, select_planes_kernel<1>, a);
  return cudaLaunchKernelEx(&cfg, select_planes_kernel<2>, a);
}

}  // namespace stem
