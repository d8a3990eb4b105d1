// Alg. 1 steps 3a-3c on pooled blocks.
//   metric   M[h,r,j] = score_scale * Qbar[h,r].Kbar[kv(h),j] + beta * MV[kv(h),j],  j <= r   (Eq. 7)
//   select   forced stem/local blocks plus the top (k_eff(r) - |forced|) remaining causal blocks,
//            order (metric descending, block id ascending), emitted ascending            (Alg. 1 "TopK")
//
// One CTA owns a tile: the g query heads of one kv head times a run of consecutive rows of one
// sequence (at most 32 pooled query vectors).  The metric rows of the tile live in shared memory
// only; they are written to global memory only when the caller asked for M.  The contraction is
// fp32 FMA (a 10-bit tensor-core mantissa would move top-k boundaries).
#include "stem_internal.h"

namespace stem {

namespace {

constexpr int kThreads = 256;
constexpr int kNQ = 32;        // pooled query vector slots per tile
constexpr int kChunk = 64;     // key blocks scored per step
constexpr int kKPad = 132;     // padded row length of the Kbar chunk (floats): conflict-free float4 reads

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, bool pred) {
  const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
  const int bytes = pred ? 16 : 0;  // src-size 0 -> zero fill
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem), "r"(bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }

// Monotone map float -> uint32 with -0 == +0 and NaN below everything (as -inf).
__device__ __forceinline__ uint32_t order_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) u = 0xff800000u;  // NaN -> -inf
  if (u == 0x80000000u) u = 0u;                          // -0 -> +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct TileArgs {
  const float* qbar; const float* kbar; const float* mv;
  const float* M_in; float* M_out;
  int32_t* sel_idx; int32_t* sel_cnt;
  const int32_t* tiles;
  RowTables rows;
  int Hq, Hkv, g, R_tot, k_max, rows_per_tile, ncols_pad, nq_slots;
  int stem, local;
  int64_t m_tot;
  float beta, score_scale;
  int mode;
};

__global__ void __launch_bounds__(kThreads, 1) score_select_kernel(TileArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* qs = (float*)smem_raw;                              // [kNQ][128]
  float* ks = qs + kNQ * kHeadDim;                           // [2][kChunk][kKPad]
  float* mrow = ks + 2 * kChunk * kKPad;                     // [nq_slots][ncols_pad]
  uint32_t* hist = (uint32_t*)(mrow + (size_t)a.nq_slots * a.ncols_pad);  // [8][256]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x, kvh = blockIdx.y;
  const int b = a.tiles[2 * tile], r0 = a.tiles[2 * tile + 1];
  const int nblk = a.rows.seq_nblk[b];
  const int row_off = a.rows.seq_row_off[b];
  const int64_t m_off = a.rows.seq_m_off[b];
  const int n_rows = min(a.rows_per_tile, nblk - r0);
  const int nq = n_rows * a.g;            // valid vectors: v = rr * g + gh
  const int r_last = r0 + n_rows - 1;
  const int n_cols = r_last + 1;

  if (a.mode & kFromPooled) {
    // ---- stage the pooled query vectors of the tile (zero for unused slots)
    for (int e = tid; e < kNQ * (kHeadDim / 4); e += kThreads) {
      const int v = e / (kHeadDim / 4), c4 = e % (kHeadDim / 4);
      float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
      if (v < nq) {
        const int rr = v / a.g, gh = v % a.g;
        const int h = kvh * a.g + gh;
        val = *(const float4*)(a.qbar + ((int64_t)h * a.R_tot + row_off + r0 + rr) * kHeadDim + c4 * 4);
      }
      *(float4*)(qs + v * kHeadDim + c4 * 4) = val;
    }
    const float* kb = a.kbar + ((int64_t)kvh * a.R_tot + row_off) * kHeadDim;
    const float* mvb = a.mv + (int64_t)kvh * a.R_tot + row_off;
    const int n_chunks = (n_cols + kChunk - 1) / kChunk;

    auto load_chunk = [&](int ch, int buf) {
      float* dst = ks + buf * kChunk * kKPad;
      for (int e = tid; e < kChunk * (kHeadDim / 4); e += kThreads) {
        const int row = e / (kHeadDim / 4), c4 = e % (kHeadDim / 4);
        const int j = ch * kChunk + row;
        const bool ok = j < nblk;
        cp_async16(dst + row * kKPad + c4 * 4, kb + (int64_t)(ok ? j : 0) * kHeadDim + c4 * 4, ok);
      }
      cp_async_commit();
    };

    load_chunk(0, 0);
    const int col = tid & (kChunk - 1), qgrp = tid / kChunk;  // 4 groups x 8 vectors
    for (int ch = 0; ch < n_chunks; ++ch) {
      if (ch + 1 < n_chunks) { load_chunk(ch + 1, (ch + 1) & 1); cp_async_wait<1>(); }
      else cp_async_wait<0>();
      __syncthreads();
      const float* kp = ks + (ch & 1) * kChunk * kKPad + col * kKPad;
      const float* qp = qs + qgrp * 8 * kHeadDim;
      float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
      const bool active = qgrp * 8 < a.nq_slots;
#pragma unroll 4
      for (int c4 = 0; c4 < (active ? kHeadDim / 4 : 0); ++c4) {
        const float4 kv = *(const float4*)(kp + c4 * 4);
#pragma unroll
        for (int v = 0; v < 8; ++v) {
          const float4 qv = *(const float4*)(qp + v * kHeadDim + c4 * 4);
          acc[v] = fmaf(qv.x, kv.x, acc[v]);
          acc[v] = fmaf(qv.y, kv.y, acc[v]);
          acc[v] = fmaf(qv.z, kv.z, acc[v]);
          acc[v] = fmaf(qv.w, kv.w, acc[v]);
        }
      }
      const int j = ch * kChunk + col;
      const float bias = (j < nblk) ? a.beta * mvb[j] : 0.f;
      if (active) {
#pragma unroll
        for (int v = 0; v < 8; ++v) mrow[(size_t)(qgrp * 8 + v) * a.ncols_pad + j] = fmaf(a.score_scale, acc[v], bias);
      }
      __syncthreads();
    }
  } else {
    // ---- metric rows come from global memory
    for (int v = warp; v < nq; v += kThreads / 32) {
      const int rr = v / a.g, gh = v % a.g;
      const int h = kvh * a.g + gh, r = r0 + rr;
      const float* src = a.M_in + (int64_t)h * a.m_tot + m_off + (int64_t)r * nblk;
      for (int j = lane; j <= r; j += 32) mrow[(size_t)v * a.ncols_pad + j] = src[j];
    }
    __syncthreads();
  }

  if (a.mode & kWriteMetric) {
    for (int v = warp; v < nq; v += kThreads / 32) {
      const int rr = v / a.g, gh = v % a.g;
      const int h = kvh * a.g + gh, r = r0 + rr;
      float* dst = a.M_out + (int64_t)h * a.m_tot + m_off + (int64_t)r * nblk;
      for (int j = lane; j <= r; j += 32) dst[j] = mrow[(size_t)v * a.ncols_pad + j];
    }
  }
  if (!(a.mode & kSelect)) return;

  // ---- selection: one warp per pooled query vector
  uint32_t* hw = hist + warp * 256;
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int v = warp; v < nq; v += kThreads / 32) {
    const int rr = v / a.g, gh = v % a.g;
    const int h = kvh * a.g + gh, r = r0 + rr;
    const int R = row_off + r;
    const int i = r + 1;
    const int n_stem = min(a.stem, i);
    const int lo_local = max(0, i - a.local);
    const int k_eff = a.rows.row_keff[R];
    const int n_forced = n_stem + (i - lo_local) - max(0, n_stem - lo_local);
    const int n_free = max(0, lo_local - n_stem);
    int need = min(max(0, k_eff - n_forced), n_free);
    const float* mr = mrow + (size_t)v * a.ncols_pad;

    uint32_t thr = 0u;      // keys above thr are taken
    int need_eq = 0;        // plus this many keys equal to thr, smallest block ids first
    if (need >= n_free) {
      thr = 0u; need_eq = 0;
      if (n_free > 0) { thr = 0u; need_eq = n_free; }  // every free block: all keys are > 0 or counted as equal
    } else if (need > 0) {
      uint32_t prefix = 0u;
      int need_rem = need;
#pragma unroll 1
      for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
#pragma unroll
        for (int q = 0; q < 8; ++q) hw[lane * 8 + q] = 0u;
        __syncwarp();
        for (int j = n_stem + lane; j < lo_local; j += 32) {
          const uint32_t key = order_key(mr[j]);
          if (pass == 0 || (key >> (shift + 8)) == prefix) atomicAdd(&hw[(key >> shift) & 255u], 1u);
        }
        __syncwarp();
        uint32_t c[8];
        uint32_t lane_sum = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) { c[q] = hw[lane * 8 + q]; lane_sum += c[q]; }
        uint32_t incl = lane_sum;  // becomes the count in lanes >= this lane
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const uint32_t t = __shfl_down_sync(0xffffffffu, incl, off);
          if (lane + off < 32) incl += t;
        }
        const uint32_t above = incl - lane_sum;
        const bool found = (above < (uint32_t)need_rem) && ((uint32_t)need_rem <= incl);
        int bin = 0, new_need = 0;
        if (found) {
          uint32_t cum = above;
#pragma unroll
          for (int q = 7; q >= 0; --q) {
            if (cum + c[q] >= (uint32_t)need_rem) { bin = lane * 8 + q; new_need = need_rem - (int)cum; break; }
            cum += c[q];
          }
        }
        const uint32_t fb = __ballot_sync(0xffffffffu, found);
        const int src = __ffs(fb) - 1;
        bin = __shfl_sync(0xffffffffu, bin, src);
        new_need = __shfl_sync(0xffffffffu, new_need, src);
        prefix = (prefix << 8) | (uint32_t)bin;
        need_rem = new_need;
        __syncwarp();
      }
      thr = prefix;
      need_eq = need_rem;
    } else {
      thr = 0xffffffffu; need_eq = 0;  // forced blocks only
    }

    int32_t* out = a.sel_idx + ((int64_t)h * a.R_tot + R) * a.k_max;
    int base = 0, eq_taken = 0;
    const bool all_free = (need >= n_free);
    for (int j0 = 0; j0 < i; j0 += 32) {
      const int j = j0 + lane;
      const bool valid = j < i;
      const bool forced = valid && (j < n_stem || j >= lo_local);
      const bool is_free = valid && !forced;
      uint32_t key = 0u;
      if (is_free) key = order_key(mr[j]);
      const bool gt = is_free && !all_free && key > thr;
      const bool eq = is_free && (all_free || key == thr);
      const uint32_t eqb = __ballot_sync(0xffffffffu, eq);
      const int eq_rank = eq_taken + __popc(eqb & lt_mask);
      const bool take = forced || gt || (eq && eq_rank < need_eq);
      const uint32_t tb = __ballot_sync(0xffffffffu, take);
      if (take) {
        const int pos = base + __popc(tb & lt_mask);
        if (pos < a.k_max) out[pos] = j;
      }
      base += __popc(tb);
      eq_taken += __popc(eqb);
    }
    for (int q = base + lane; q < a.k_max; q += 32) out[q] = -1;
    if (lane == 0) a.sel_cnt[(int64_t)h * a.R_tot + R] = min(base, a.k_max);
  }
}

}  // namespace

cudaError_t launch_score_select(const Plan& p, int mode, const float* qbar, const float* kbar, const float* mv,
                                const float* M_in, float* M_out, int32_t* sel_idx, int32_t* sel_cnt, cudaStream_t s) {
  TileArgs a{};
  a.qbar = qbar; a.kbar = kbar; a.mv = mv; a.M_in = M_in; a.M_out = M_out;
  a.sel_idx = sel_idx; a.sel_cnt = sel_cnt;
  a.tiles = p.d_sel_tiles; a.rows = p.rows;
  a.Hq = p.cfg.num_q_heads; a.Hkv = p.cfg.num_kv_heads; a.g = a.Hq / a.Hkv;
  a.R_tot = p.R_tot; a.k_max = p.k_max; a.rows_per_tile = p.sel_rows_per_tile;
  a.ncols_pad = (p.max_nblk + kChunk - 1) / kChunk * kChunk;
  a.stem = p.cfg.stem_blocks; a.local = p.cfg.local_blocks;
  a.m_tot = p.m_tot; a.beta = p.cfg.beta; a.score_scale = p.score_scale; a.mode = mode;
  a.nq_slots = (p.sel_nq + 7) / 8 * 8;
  const size_t smem = (size_t)kNQ * kHeadDim * 4 + 2 * kChunk * kKPad * 4 + (size_t)a.nq_slots * a.ncols_pad * 4 + 8 * 256 * 4;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(score_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)p.n_sel_tiles, (unsigned)a.Hkv);
  score_select_kernel<<<grid, kThreads, smem, s>>>(a);
  return cudaGetLastError();
}

}  // namespace stem
