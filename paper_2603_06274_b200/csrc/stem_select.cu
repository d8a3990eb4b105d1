// Alg. 1 steps 3a-3c on pooled blocks.
//   metric   M[h,r,j] = score_scale * Qbar[h,r].Kbar[kv(h),j] + beta * MV[kv(h),j],  j <= r   (Eq. 7)
//   select   forced stem/local blocks plus the top (k_eff(r) - |forced|) remaining causal blocks,
//            order (metric descending, block id ascending), emitted ascending            (Alg. 1 "TopK")
//
// One CTA owns a tile: the g query heads of one kv head times a run of consecutive rows of one
// sequence (at most 32 pooled query vectors).  The metric rows of the tile live in shared memory
// only; they are written to global memory only when the caller asked for M.
//
// Scoring is a small fp32 GEMM on the FMA pipe (a 10-bit tensor-core mantissa would move top-k
// boundaries): Qbar^T of the tile stays in shared memory, Kbar^T (stored transposed by the pooling
// kernel, block index contiguous) streams through a double-buffered 64-column chunk, and each
// thread keeps an 8 x 2 register tile over a quarter of the head dimension; the four quarters sit
// in the four lane groups of a warp and are added by shuffles in a fixed order.  Both operands are
// laid out in shared memory so that a warp's loads of one step fall into whole 128-byte lines.
//
// Selection: one warp per row holds the row's order-preserving keys in registers and brackets the
// k-th largest key by counting passes (interpolated and midpoint thresholds in turn, leaving early
// as soon as a threshold has exactly the wanted number of keys at or above it); ties at the
// threshold are resolved towards smaller block ids with ballots while the ascending list is emitted.
#include "stem_internal.h"

namespace stem {

namespace {

constexpr int kThreads = 512;
constexpr int kNQ = 32;      // pooled query vector slots per tile
constexpr int kChunk = 64;   // key blocks scored per step

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }

// Monotone map float -> uint32 with -0 == +0 and NaN below everything (as -inf).  Every key is >= 1.
__device__ __forceinline__ uint32_t order_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7fffffffu) > 0x7f800000u) u = 0xff800000u;  // NaN -> -inf
  if (u == 0x80000000u) u = 0u;                          // -0 -> +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct TileArgs {
  const float* qbar; const float* kbar_t; const float* mv;
  const float* M_in; float* M_out;
  int32_t* sel_idx; int32_t* sel_cnt;
  const int32_t* tiles;
  RowTables rows;
  int Hq, Hkv, g, R_tot, k_max, rows_per_tile, ncols_pad, nq_slots, kt_width;
  int stem, local;
  int64_t m_tot;
  float beta, score_scale;
  int mode;
};

// KPL = keys per lane held in registers during selection (32 * KPL >= ncols_pad).
template <int KPL>
__global__ void __launch_bounds__(kThreads, 1) score_select_kernel(TileArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // Element (d, x) of an operand with d = ds * 32 + dd is stored at ((dd * G + x / W) * 4 + ds) * W + x % W,
  // G groups of W consecutive vectors / columns: the four d-quarters a warp reads together are adjacent.
  float* qt = (float*)smem_raw;                   // Qbar^T of the tile: 128 d x kNQ, W = 8
  float* kt = qt + kHeadDim * kNQ;                // Kbar^T chunk, double-buffered: 2 x (128 d x kChunk), W = 16
  float* mrow = kt + 2 * kHeadDim * kChunk;       // [nq_slots][ncols_pad] metric rows

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x / a.Hkv, kvh = blockIdx.x - tile * a.Hkv;
  const int b = a.tiles[2 * tile], r0 = a.tiles[2 * tile + 1];
  const int nblk = a.rows.seq_nblk[b];
  const int row_off = a.rows.seq_row_off[b];
  const int64_t m_off = a.rows.seq_m_off[b];
  const int n_rows = min(a.rows_per_tile, nblk - r0);
  const int nq = n_rows * a.g;            // valid vectors: v = rr * g + gh
  const int r_last = r0 + n_rows - 1;
  const int n_cols = r_last + 1;

  if (a.mode & kFromPooled) {
    // Kbar^T of this kv head and sequence: [128 d][kt_width], columns of the sequence start at a
    // multiple of kChunk and its region is padded to a multiple of kChunk, so whole chunks are in bounds.
    const float* kb = a.kbar_t + (int64_t)kvh * kHeadDim * a.kt_width + a.rows.seq_kt_off[b];
    const float* mvb = a.mv + (int64_t)kvh * a.R_tot + row_off;
    const int n_chunks = (n_cols + kChunk - 1) / kChunk;
    auto load_chunk = [&](int ch, int buf) {
      float* dst = kt + buf * kHeadDim * kChunk;
      for (int e = tid; e < kHeadDim * (kChunk / 4); e += kThreads) {
        const int d = e / (kChunk / 4), c4 = e - d * (kChunk / 4);
        const int ds = d >> 5, dd = d & 31;
        cp_async16(dst + ((dd * 4 + (c4 >> 2)) * 4 + ds) * 16 + (c4 & 3) * 4,
                   kb + (int64_t)d * a.kt_width + ch * kChunk + c4 * 4);
      }
      cp_async_commit();
    };
    load_chunk(0, 0);  // in flight while the query vectors are staged
    // ---- Qbar^T of the tile (lanes run over the vectors)
    for (int e = tid; e < kNQ * (kHeadDim / 4); e += kThreads) {
      const int v = e & (kNQ - 1), c4 = e / kNQ;
      float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
      if (v < nq) {
        const int rr = v / a.g, gh = v - rr * a.g;
        const int h = kvh * a.g + gh;
        val = *(const float4*)(a.qbar + ((int64_t)h * a.R_tot + row_off + r0 + rr) * kHeadDim + c4 * 4);
      }
      const int ds = c4 >> 3, dd = (c4 & 7) * 4;
      float* dst = qt + ((dd * 4 + (v >> 3)) * 4 + ds) * 8 + (v & 7);
      dst[0] = val.x; dst[128] = val.y; dst[256] = val.z; dst[384] = val.w;  // dd + 1 is 4 * 4 * 8 floats further
    }
    // thread tile: 8 vectors x 2 columns over one quarter of the head dimension
    const int vg = warp >> 2, cg = warp & 3;      // vectors vg * 8 .., columns cg * 16 .. of the chunk
    const int ds = lane >> 3, kp = lane & 7;
    const float* qp = qt + (vg * 4 + ds) * 8;
    for (int ch = 0; ch < n_chunks; ++ch) {
      cp_async_wait<0>();
      __syncthreads();  // chunk ch has landed and the other buffer is free again
      if (ch + 1 < n_chunks) load_chunk(ch + 1, (ch + 1) & 1);
      const float* kp_s = kt + (ch & 1) * kHeadDim * kChunk + (cg * 4 + ds) * 16 + kp * 2;
      float acc[8][2];
#pragma unroll
      for (int i = 0; i < 8; ++i) { acc[i][0] = 0.f; acc[i][1] = 0.f; }
#pragma unroll 8
      for (int dd = 0; dd < 32; ++dd) {
        const float4 qa = *(const float4*)(qp + dd * 128);
        const float4 qb = *(const float4*)(qp + dd * 128 + 4);
        const float2 kk = *(const float2*)(kp_s + dd * 256);
        const float qv[8] = {qa.x, qa.y, qa.z, qa.w, qb.x, qb.y, qb.z, qb.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          acc[i][0] = fmaf(qv[i], kk.x, acc[i][0]);
          acc[i][1] = fmaf(qv[i], kk.y, acc[i][1]);
        }
      }
      // quarters: (0 + 1) + (2 + 3)
#pragma unroll
      for (int i = 0; i < 8; ++i) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          acc[i][c] += __shfl_xor_sync(0xffffffffu, acc[i][c], 8);
          acc[i][c] += __shfl_xor_sync(0xffffffffu, acc[i][c], 16);
        }
      }
      if (ds == 0) {
        const int j = ch * kChunk + cg * 16 + kp * 2;
        const float bias0 = (j < nblk) ? a.beta * mvb[j] : 0.f;
        const float bias1 = (j + 1 < nblk) ? a.beta * mvb[j + 1] : 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (vg * 8 + i < a.nq_slots) {
            float2 out;
            out.x = fmaf(a.score_scale, acc[i][0], bias0);
            out.y = fmaf(a.score_scale, acc[i][1], bias1);
            *(float2*)(mrow + (size_t)(vg * 8 + i) * a.ncols_pad + j) = out;
          }
        }
      }
    }
    __syncthreads();
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
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int v = warp; v < nq; v += kThreads / 32) {
    const int rr = v / a.g, gh = v % a.g;
    const int h = kvh * a.g + gh, r = r0 + rr;
    const int R = row_off + r;
    const int i = r + 1;                          // causal blocks of the row
    const int n_stem = min(a.stem, i);
    const int lo_local = max(0, i - a.local);
    const int k_eff = a.rows.row_keff[R];
    const int n_forced = n_stem + (i - lo_local) - max(0, n_stem - lo_local);
    const int n_free = max(0, lo_local - n_stem);  // candidates: blocks n_stem .. lo_local-1
    const int need = min(max(0, k_eff - n_forced), n_free);
    const float* mr = mrow + (size_t)v * a.ncols_pad;

    // keys of the free candidates; lane l holds blocks q * 32 + l.  0 = not a candidate (below every key).
    // Only the first ng groups of eight key slots can hold candidates of this row (warp-uniform).
    const int ng = min(KPL / 8, (lo_local + 255) >> 8);
    uint32_t key[KPL];
#pragma unroll
    for (int q8 = 0; q8 < KPL / 8; ++q8) {
#pragma unroll
      for (int q = q8 * 8; q < q8 * 8 + 8; ++q) {
        const int j = q * 32 + lane;
        key[q] = (q8 < ng && j >= n_stem && j < lo_local) ? order_key(mr[j]) : 0u;
      }
    }
    // f(t) = number of candidates with key >= t (t >= 1)
    auto count_ge = [&](uint32_t t) -> int {
      int c4[4] = {0, 0, 0, 0};  // independent chains
#pragma unroll
      for (int q8 = 0; q8 < KPL / 8; ++q8) {
        if (q8 >= ng) break;
#pragma unroll
        for (int q = q8 * 8; q < q8 * 8 + 8; ++q) c4[q & 3] += key[q] >= t ? 1 : 0;
      }
      return __reduce_add_sync(0xffffffffu, (c4[0] + c4[1]) + (c4[2] + c4[3]));
    };

    // thr / need_eq: take every key > thr, plus the need_eq candidates with key == thr of smallest block id
    uint32_t thr = 0xffffffffu;
    int need_eq = 0;
    if (need >= n_free) {
      thr = 0u;            // every candidate (all keys are >= 1)
    } else if (need > 0) {
      // Bracket the need-th largest key: f(lo) >= need > f(hi).  Candidates alternate between the
      // point where a linear model of f between the bracket ends reaches `need` and the midpoint
      // (which bounds the number of steps by twice the key width); the search stops as soon as a
      // threshold has exactly `need` keys at or above it, or when the bracket is one key wide.
      uint32_t kmax = 0u, kmin = 0xffffffffu;
#pragma unroll
      for (int q8 = 0; q8 < KPL / 8; ++q8) {
        if (q8 >= ng) break;
#pragma unroll
        for (int q = q8 * 8; q < q8 * 8 + 8; ++q) {
          kmax = max(kmax, key[q]);
          kmin = min(kmin, key[q] != 0u ? key[q] : 0xffffffffu);
        }
      }
      uint32_t lo = __reduce_min_sync(0xffffffffu, kmin);       // f(lo) = n_free > need
      uint32_t hi = __reduce_max_sync(0xffffffffu, kmax) + 1u;  // f(hi) = 0 < need (keys stay below 0xff800001)
      int c_lo = n_free, c_hi = 0;
#pragma unroll 1
      for (int step = 0; c_lo != need && hi - lo > 1u; ++step) {
        uint32_t cand = lo + ((hi - lo) >> 1);
        if ((step & 1) == 0) {
          const float fr = (float)(c_lo - need) / (float)(c_lo - c_hi);
          cand = lo + (uint32_t)((float)(hi - lo) * fr);
        }
        cand = min(max(cand, lo + 1u), hi - 1u);
        const int c = count_ge(cand);
        if (c >= need) { lo = cand; c_lo = c; } else { hi = cand; c_hi = c; }
      }
      if (c_lo == need) {
        thr = lo - 1u;           // key >= lo  <=>  key > lo - 1 (lo >= 1)
      } else {
        thr = lo;                // lo is the need-th largest key and is tied across the boundary
        need_eq = need - c_hi;   // c_hi = f(lo + 1) = keys above it
      }
    }

    int32_t* out = a.sel_idx + ((int64_t)h * a.R_tot + R) * a.k_max;
    int base = 0, eq_taken = 0;
#pragma unroll
    for (int q = 0; q < KPL; ++q) {
      const int j = q * 32 + lane;
      if (q * 32 >= i) break;  // warp-uniform
      const bool forced = j < i && (j < n_stem || j >= lo_local);
      const bool gt = key[q] > thr;
      const bool eq = key[q] == thr && key[q] != 0u;
      const uint32_t eqb = __ballot_sync(0xffffffffu, eq);
      const bool take = forced || gt || (eq && eq_taken + __popc(eqb & lt_mask) < need_eq);
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

size_t score_select_fixed_smem() { return (size_t)(kHeadDim * kNQ + 2 * kHeadDim * kChunk) * sizeof(float); }

template <int KPL>
cudaError_t launch_kpl(const TileArgs& a, dim3 grid, size_t smem, cudaStream_t s) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(score_select_kernel<KPL>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  score_select_kernel<KPL><<<grid, kThreads, smem, s>>>(a);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score_select(const Plan& p, int mode, const float* qbar, const float* kbar_t, const float* mv,
                                const float* M_in, float* M_out, int32_t* sel_idx, int32_t* sel_cnt, cudaStream_t s) {
  TileArgs a{};
  a.qbar = qbar; a.kbar_t = kbar_t; a.mv = mv; a.M_in = M_in; a.M_out = M_out;
  a.sel_idx = sel_idx; a.sel_cnt = sel_cnt;
  a.tiles = p.d_sel_tiles; a.rows = p.rows;
  a.Hq = p.cfg.num_q_heads; a.Hkv = p.cfg.num_kv_heads; a.g = a.Hq / a.Hkv;
  a.R_tot = p.R_tot; a.k_max = p.k_max; a.rows_per_tile = p.sel_rows_per_tile;
  a.ncols_pad = (p.max_nblk + kChunk - 1) / kChunk * kChunk;
  a.kt_width = p.kt_width;
  a.stem = p.cfg.stem_blocks; a.local = p.cfg.local_blocks;
  a.m_tot = p.m_tot; a.beta = p.cfg.beta; a.score_scale = p.score_scale; a.mode = mode;
  a.nq_slots = (p.sel_nq + 7) / 8 * 8;
  const size_t smem = score_select_fixed_smem() + (size_t)a.nq_slots * a.ncols_pad * sizeof(float);
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)p.n_sel_tiles * (unsigned)a.Hkv);
  const int kpl = a.ncols_pad / 32;  // ncols_pad is a multiple of 64
  if (kpl <= 8) return launch_kpl<8>(a, grid, smem, s);
  if (kpl <= 16) return launch_kpl<16>(a, grid, smem, s);
  if (kpl <= 32) return launch_kpl<32>(a, grid, smem, s);
  if (kpl <= 64) return launch_kpl<64>(a, grid, smem, s);
  return cudaErrorInvalidValue;
}

}  // namespace stem
