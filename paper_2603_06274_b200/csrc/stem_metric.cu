// Alg. 1 step 2, Eq. 7: the block metric as a dense contraction on the tensor cores (sm_100a).
//
//   M[h, r, j] = score_scale * Qbar[h, r] . Kbar[kv(h), j] + beta * MV[kv(h), j],   j <= r
//
// Selection is decided on these values, so the contraction has to be as exact as an fp32 dot
// product.  The pooling kernel therefore hands over every pooled fp32 vector as three bf16 parts
// (x = hi + mid + lo, each the bf16 rounding of what the previous parts leave: 24 mantissa bits in
// all), and the kernel adds the six partial products that matter
//     mid.mid + hi.lo + lo.hi + hi.mid + mid.hi + hi.hi          (smallest terms first)
// as tcgen05.mma (bf16 x bf16, exact products, fp32 accumulation in tensor memory); the dropped
// terms are below 2^-24 of the leading one.  A pooled value that is not finite makes its row or
// column of M NaN (which ranks below every number).
//
// One CTA per (128 x 128 tile of one sequence's causal triangle, kv head): the Kbar parts stay in
// shared memory while the Qbar parts of the group's query heads stream through (TMA, K-major,
// 128-byte swizzle, one half of the head dimension per buffer); one warp issues the copies and the
// 2 x 24 MMAs per head into one of two accumulators, the other four warps
// read the accumulator (one row per thread), apply scale and bias, and either turn the tile through
// shared memory and write the causal part of it with coalesced stores (the public M), or write each
// row's selection keys as bit planes, one 128-byte line per 32 columns (the fused path's workspace
// form, read by the bit-plane selection kernel).  Waits are bounded.
#include <cuda.h>
#include <cuda_bf16.h>

#include "stem_internal.h"
#include "stem_ptx.cuh"

namespace stem {

namespace {

constexpr int kThreads = 288;                         // warps 0-7: epilogue (two warps per 32 accumulator rows, two 32-column
                                                      // pieces each); warp 8: copies + MMAs
constexpr int kTile = 128;
constexpr int kPartBytes = kTile * 128;               // one operand part, one 64-column half of d (bf16): 16 KB
constexpr int kSmemB = 0;                             // Kbar parts, both halves: [half][part], resident for the whole CTA
constexpr int kSmemA = kSmemB + 6 * kPartBytes;       // Qbar parts of one head: [half][part], refilled head by head
constexpr int kSmemStage = kSmemA + 6 * kPartBytes;   // 8 warps x 32 rows x 32 columns fp32 (float output only)
constexpr int kSmemBias = kSmemStage + 8 * 32 * 32 * 4;  // 128 floats
constexpr int kSmemBars = kSmemBias + kTile * 4;      // b_full, a_full[2], a_empty[2], acc_full[2], acc_empty[2]
constexpr int kSmemTmem = kSmemBars + 9 * 8;
constexpr int kSmemTotal = kSmemTmem + 16;
constexpr int kSmemBytes = kSmemTotal + 1024;         // slack for manual 1024-byte alignment
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
constexpr uint64_t kWaitLimitNs = 200ull * 1000 * 1000;

using namespace ptx;

// Bounded wait; false when the time limit ran out (the status words then say so).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t* status) {
  if (mbar_wait_bounded(bar, parity, kWaitLimitNs)) return true;
  if (atomicCAS(status + 4, 0, 2) == 0) { status[5] = (int32_t)blockIdx.x; status[6] = (int32_t)blockIdx.y; }
  return false;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = N = 128.
constexpr uint32_t kIdesc = make_idesc(kTile, kTile, 0);

struct GemmArgs {
  const int32_t* tiles;  // [n_tiles][3] (sequence, row tile, column tile), column tile <= row tile
  const float* mv;       // [H_kv, KB_tot]
  float* M;
  int32_t* status;
  RowTables rows;
  int64_t m_tot, mt_tot;
  int Hq, Hkv, g, R_tot, KB_tot;  // Hq = heads of the metric (the list heads), g = of them per kv head
  float beta, scale;
  int as_keys;  // write bit planes of the metric's selection keys (for launch_select_planes) instead of floats
};

__global__ void __launch_bounds__(kThreads, 1)
metric_gemm_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, const GemmArgs a) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = ((uint32_t)__cvta_generic_to_shared(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem_gen = smem_raw + (smem_base - (uint32_t)__cvta_generic_to_shared(smem_raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bars = smem_base + kSmemBars;
  const uint32_t b_full = bars, a_full = bars + 8, a_empty = bars + 24, acc_full = bars + 40, acc_empty = bars + 56;
  float* bias = (float*)(smem_gen + kSmemBias);

  // One CTA works on one tile of one sequence's causal triangle for the g query heads of a kv head:
  // the Kbar parts stay in shared memory, the Qbar parts of the heads stream through, and two
  // accumulators in tensor memory let the epilogue of one head overlap the MMAs of the next.
  const int seq = a.tiles[3 * blockIdx.x], ti = a.tiles[3 * blockIdx.x + 1], tj = a.tiles[3 * blockIdx.x + 2];
  const int kvh = blockIdx.y, g = a.g;
  const int nb = a.rows.seq_nblk[seq];   // key blocks of the sequence
  const int r0 = a.rows.seq_r0[seq];     // first row of its query chunk
  const int R0 = a.rows.seq_row_off[seq] + ti * kTile;  // first query row of A (Qbar numbering)
  const int C0 = a.rows.seq_kb_off[seq] + tj * kTile;   // first key block of B (Kbar numbering)

  if (threadIdx.x == 0) {
    mbar_init(b_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(a_full + 8 * i, 1);
      mbar_init(a_empty + 8 * i, 1);
      mbar_init(acc_full + 8 * i, 1);
      mbar_init(acc_empty + 8 * i, 8);  // one arrival per epilogue warp
    }
    mbar_init_fence();
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_base + kSmemTmem), "n"(256)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Launched as a programmatic dependent of the pooling kernel, everything above overlaps its tail;
  // its outputs are read only below this point.  (Without that launch attribute both are no-ops.)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (threadIdx.x < kTile) {
    const int c = threadIdx.x;  // bias of column c of the tile (the same for every head of the group)
    bias[c] = (tj * kTile + c < nb) ? a.beta * a.mv[(int64_t)kvh * a.KB_tot + C0 + c] : 0.f;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *(volatile uint32_t*)(smem_gen + kSmemTmem);

  if (warp == 8) {
    // ============================== copies and MMAs ==============================
    const bool leader = elect_one();
    bool ok = true;
    auto load_a = [&](const int hh, const int half) {  // the three Qbar parts of one head, one half of d
      if (leader) {
        mbar_expect_tx(a_full + 8 * half, 3 * kPartBytes);
#pragma unroll
        for (int s = 0; s < 3; ++s)
          tma_load_3d(smem_base + kSmemA + (half * 3 + s) * kPartBytes, &map_q, a_full + 8 * half, 64 * half, R0,
                      s * a.Hq + kvh * g + hh);
      }
      __syncwarp();
    };
    if (leader) {
      mbar_expect_tx(b_full, 6 * kPartBytes);
#pragma unroll
      for (int half = 0; half < 2; ++half)
#pragma unroll
        for (int s = 0; s < 3; ++s)
          tma_load_3d(smem_base + kSmemB + (half * 3 + s) * kPartBytes, &map_k, b_full, 64 * half, C0, s * a.Hkv + kvh);
    }
    __syncwarp();
    load_a(0, 0);
    load_a(0, 1);
    // parts of A x parts of B, smallest products first: (mid,mid) (hi,lo) (lo,hi) (hi,mid) (mid,hi) (hi,hi)
    constexpr int kPairs[6][2] = {{1, 1}, {0, 2}, {2, 0}, {0, 1}, {1, 0}, {0, 0}};
#pragma unroll 1
    for (int st = 0; st < 2 * g; ++st) {
      const int hh = st >> 1, half = st & 1;
      const uint32_t acc_tmem = tmem + (uint32_t)(hh & 1) * 128u;
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(a_full + 8 * half, hh & 1, a.status));
      if (ok && st == 0) ok = __all_sync(0xffffffffu, mbar_wait(b_full, 0, a.status));
      // the accumulator was last used by head hh - 2: its epilogue must have read it
      if (ok && half == 0 && hh >= 2) ok = __all_sync(0xffffffffu, mbar_wait(acc_empty + 8 * (hh & 1), ((hh >> 1) - 1) & 1, a.status));
      if (!ok) break;
      tc_fence_after();
      if (leader) {
        uint32_t accf = half;  // the first MMA of a head overwrites the accumulator
#pragma unroll
        for (int q = 0; q < 6; ++q) {
          const uint32_t a_addr = smem_base + kSmemA + (half * 3 + kPairs[q][0]) * kPartBytes;
          const uint32_t b_addr = smem_base + kSmemB + (half * 3 + kPairs[q][1]) * kPartBytes;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            mma_ss(acc_tmem, smem_desc(a_addr + k * 32), smem_desc(b_addr + k * 32), kIdesc, accf);
            accf = 1u;
          }
        }
        tc_commit(a_empty + 8 * half);
        if (half == 1) tc_commit(acc_full + 8 * (hh & 1));
      }
      __syncwarp();
      if (hh + 1 < g) {  // refill this half's buffer with the next head's parts once the MMAs have read it
        ok = __all_sync(0xffffffffu, mbar_wait(a_empty + 8 * half, hh & 1, a.status));
        if (!ok) break;
        load_a(hh + 1, half);
      }
    }
  } else {
    // ============================== epilogue ==============================
    // A single warp per scheduler cannot keep the integer pipe busy (dependent chains), so two warps
    // share each quarter of the accumulator rows: warps 0-3 take columns 0-63, warps 4-7 columns 64-127.
    const int quarter = warp & 3, gq0 = (warp >> 2) * 2;
    const int m = quarter * 32 + lane;  // row of the tile == TMEM lane
    const int rl = ti * kTile + m;      // row inside the chunk
    const int r = r0 + rl;              // row inside the sequence
    const int stride = (nb + 31) & ~31;
    float* stage = (float*)(smem_gen + kSmemStage) + warp * 32 * 32;
    bool ok = true;
#pragma unroll 1
    for (int hh = 0; hh < g && ok; ++hh) {
      const int h = kvh * g + hh;
      ok = __all_sync(0xffffffffu, mbar_wait(acc_full + 8 * (hh & 1), (hh >> 1) & 1, a.status));
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem + (uint32_t)(hh & 1) * 128u + ((uint32_t)(quarter * 32) << 16);
      uint32_t* dst_planes = (uint32_t*)a.M + (int64_t)h * a.mt_tot + a.rows.seq_mt_off[seq] + (int64_t)rl * stride + tj * kTile;
      float* mseq = a.M + (int64_t)h * a.m_tot + a.rows.seq_m_off[seq];
#pragma unroll 1
      for (int gq = gq0; gq < gq0 + 2; ++gq) {
        float v[32];
        tmem_ld32_sync(taddr + gq * 32, v);
        if (gq == gq0 + 1) {
          // the accumulator is in registers: the MMAs of head hh + 2 may overwrite it
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(acc_empty + 8 * (hh & 1));
        }
        if (a.as_keys) {
          // For the selection: the keys of the row, 32 columns at a time, as 32 bit planes (word k =
          // bit k of the 32 keys), one 128-byte line of the row.  key = bits ^ (negative ? all ones :
          // sign bit) of the value with -0 -> +0 and NaN -> -inf; the exclusive-or is applied to the
          // planes (32 operations for 32 keys) instead of to the keys.
          uint32_t w[32];
#pragma unroll
          for (int c = 0; c < 32; ++c)
            w[c] = __float_as_uint(fmaxf(fmaf(a.scale, v[c], bias[gq * 32 + c]) + 0.0f, __int_as_float(0xff800000)));
          transpose32(w);
          const uint32_t neg = w[31];  // bit t: value t is negative
#pragma unroll
          for (int k = 0; k < 31; ++k) w[k] ^= neg;
          w[31] = ~neg;
          if (r < nb && tj * kTile + gq * 32 < stride) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              *(uint4*)(dst_planes + gq * 32 + q * 4) = make_uint4(w[q * 4], w[q * 4 + 1], w[q * 4 + 2], w[q * 4 + 3]);
          }
        } else {
          // The public M: the warp's 32 x 32 piece through shared memory (rows swizzled by 16-byte
          // chunks), then one 128-byte store per row, causal part only.
#pragma unroll
          for (int c4 = 0; c4 < 8; ++c4) {
            float4 o;
            o.x = fmaf(a.scale, v[c4 * 4 + 0], bias[gq * 32 + c4 * 4 + 0]);
            o.y = fmaf(a.scale, v[c4 * 4 + 1], bias[gq * 32 + c4 * 4 + 1]);
            o.z = fmaf(a.scale, v[c4 * 4 + 2], bias[gq * 32 + c4 * 4 + 2]);
            o.w = fmaf(a.scale, v[c4 * 4 + 3], bias[gq * 32 + c4 * 4 + 3]);
            *(float4*)(stage + lane * 32 + ((c4 ^ (lane & 7)) << 2)) = o;
          }
          __syncwarp();
          const int cg = tj * kTile + gq * 32 + lane;  // this lane's column inside the sequence
          for (int mm = 0; mm < 32; ++mm) {
            const int rr = r0 + ti * kTile + quarter * 32 + mm;  // row inside the sequence
            if (rr >= nb) break;
            if (cg <= rr) mseq[(int64_t)(rr - r0) * nb + cg] = stage[mm * 32 + (((lane >> 2) ^ (mm & 7)) << 2) + (lane & 3)];
          }
          __syncwarp();
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(256) : "memory");
  }
}

// [planes, rows, 128] bf16, dense: TMA dims (innermost first) = (128, rows, planes);
// one box = 64 columns x 128 rows of one plane, 128-byte swizzled; rows past the end read as zero.
bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t planes) {
  return make_bf16_map_3d(map, base, {(uint64_t)kHeadDim, (uint64_t)rows, (uint64_t)planes},
                          {(uint64_t)kHeadDim * 2, (uint64_t)rows * kHeadDim * 2}, {64u, (uint32_t)kTile, 1u});
}

}  // namespace

cudaError_t launch_metric_gemm(const Plan& p, const void* qsplit, const void* ksplit, const float* mv, float* M,
                               bool as_keys, bool dependent, int32_t* status, cudaStream_t s) {
  CUtensorMap mq, mk;
  if (!make_map(&mq, qsplit, p.R_tot, 3 * (int64_t)p.H_list) ||
      !make_map(&mk, ksplit, p.KB_tot, 3 * (int64_t)p.cfg.num_kv_heads))
    return cudaErrorInvalidValue;
  GemmArgs a{};
  (void)status;
  a.tiles = p.d_gemm_tiles; a.mv = mv; a.M = M; a.status = status; a.rows = p.rows; a.m_tot = p.m_tot; a.mt_tot = p.mt_tot;
  a.Hq = p.H_list; a.Hkv = p.cfg.num_kv_heads; a.g = a.Hq / a.Hkv; a.R_tot = p.R_tot; a.KB_tot = p.KB_tot;
  a.beta = p.cfg.beta; a.scale = p.score_scale; a.as_keys = as_keys ? 1 : 0;
  // the attribute belongs to the device's context: set it once per device of this process
  static bool attr_set[64] = {};
  const int dev_slot = p.device & 63;
  if (!attr_set[dev_slot]) {
    cudaError_t e = cudaFuncSetAttribute(metric_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set[dev_slot] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)p.n_gemm_tiles, (unsigned)a.Hkv);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, metric_gemm_kernel, mq, mk, a);
}

}  // namespace stem
