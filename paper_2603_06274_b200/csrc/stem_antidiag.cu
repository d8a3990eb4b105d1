// Alg. 1 step 1 / step 3a in the anti-diagonal scoring mode (Overall Algorithm: "anti-diagonal scoring";
// Alg. 1 step 1 comment, stride = B): the routing term of block pair (r, j) is the mean of the token
// scores along the main anti-diagonal of the B x B score block,
//
//   M[h, r, j] = score_scale * (1/B) * sum_{s < B} q[rB + B-1-s] . k[jB + s]  +  beta * MV[kv(h), j],   j <= r.
//
// With the tokens of a query block taken in reverse order, a block is one row of B*d numbers, and the
// anti-diagonal sums of all block pairs are one dense contraction with inner dimension B*d:
// [N_blk x B*d] x [B*d x N_blk] per head, on the tcgen05 tensor cores.  A 4-D tensor map (d, head, token in
// block, block) lets one TMA box fetch "64 columns of token t of 128 consecutive blocks" as a 128-row
// K-major operand tile; the query map is walked with t = B-1-s, the key map with t = s.
//
// One CTA per (128 x 128 tile of one sequence's causal triangle, query head): warp 4 issues the copies
// through a ring of stages, warp 5 the MMAs into one TMEM accumulator, warps 0-3 write the tile as floats
// (the public M) or as bit planes of the selection keys (the fused path's workspace form).  Only FULL
// blocks go through the contraction (the maps end at the last full block, so nothing is read past a
// sequence); a sequence's partial last block, whose anti-diagonal is truncated (the mean is over the
// pairs whose two tokens exist), is one metric row that a small second kernel computes with plain FMAs.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>

#include "stem_internal.h"
#include "stem_ptx.cuh"

namespace stem {

namespace {

using namespace ptx;

constexpr int kThreads = 192;
constexpr int kTile = 128;
constexpr int kStages = 6;
constexpr int kPartBytes = kTile * 128;  // one operand tile of a step: 128 rows x 64 columns bf16
constexpr int kSmemA = 0;
constexpr int kSmemB = kSmemA + kStages * kPartBytes;
constexpr int kSmemBias = kSmemB + kStages * kPartBytes;
constexpr int kSmemBars = kSmemBias + kTile * 4;  // full[kStages], empty[kStages], acc_full
constexpr int kSmemTmem = kSmemBars + (2 * kStages + 1) * 8;
constexpr int kSmemBytes = kSmemTmem + 16 + 1024;  // slack for manual 1024-byte alignment
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
constexpr uint64_t kWaitLimitNs = 200ull * 1000 * 1000;
constexpr int kMaxSeqs = 8;

struct MapSet {
  CUtensorMap q[kMaxSeqs], k[kMaxSeqs];
};

struct AntiArgs {
  const int32_t* tiles;  // [n_tiles][3] (sequence, row tile, column tile)
  const float* mv;       // [H_kv, KB_tot]
  float* M;
  int32_t* status;
  RowTables rows;
  int64_t m_tot, mt_tot;
  int Hq, g, KB_tot, block;
  float beta, scale;     // scale = score_scale / B
  int as_keys;
  // the partial-row kernel
  const __nv_bfloat16 *Q, *K;
  int64_t q_st, q_sh, kv_st, kv_sh;
  int batch;
};

// Bounded wait; false when the time limit ran out (the status words then say so).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t* status) {
  if (mbar_wait_bounded(bar, parity, kWaitLimitNs)) return true;
  if (atomicCAS(status + 4, 0, 3) == 0) { status[5] = (int32_t)blockIdx.x; status[6] = (int32_t)blockIdx.y; }
  return false;
}

constexpr uint32_t kIdesc = make_idesc(kTile, kTile, 0);

// Selection key of a metric value: monotone map float -> uint32 with -0 == +0 and NaN below everything.
__device__ __forceinline__ uint32_t metric_key(float f) {
  uint32_t u = __float_as_uint(fmaxf(f + 0.0f, __int_as_float(0xff800000)));  // -0 -> +0, NaN -> -inf
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <int BLK>
__global__ void __launch_bounds__(kThreads, 1)
antidiag_metric_kernel(const __grid_constant__ MapSet maps, const AntiArgs a) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = ((uint32_t)__cvta_generic_to_shared(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem_gen = smem_raw + (smem_base - (uint32_t)__cvta_generic_to_shared(smem_raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bars = smem_base + kSmemBars;
  auto full = [&](int s) { return bars + 8 * s; };
  auto empty = [&](int s) { return bars + 8 * (kStages + s); };
  const uint32_t acc_full = bars + 8 * 2 * kStages;
  float* bias = (float*)(smem_gen + kSmemBias);

  const int seq = a.tiles[3 * blockIdx.x], ti = a.tiles[3 * blockIdx.x + 1], tj = a.tiles[3 * blockIdx.x + 2];
  const int h = blockIdx.y, kvh = h / a.g;
  const int nb = a.rows.seq_nblk[seq];
  const int r0 = a.rows.seq_r0[seq];
  // full blocks of the sequence: all of them, or all but the last when that one is partial
  const int last_ntok = a.rows.kb_ntok[a.rows.seq_kb_first[seq] + nb - 1];
  const int nfull = last_ntok == BLK ? nb : nb - 1;
  // nothing to do when the tile holds no full row or no full column
  if (r0 + ti * kTile >= nfull || tj * kTile >= nfull) return;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
    mbar_init(acc_full, 1);
    mbar_init_fence();
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_base + kSmemTmem), "n"(128)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Launched as a programmatic dependent of the pooling kernel (which writes MV), everything above overlaps
  // its tail.  (Without that launch attribute both are no-ops.)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (threadIdx.x < kTile) {
    const int c = threadIdx.x;
    bias[c] = (tj * kTile + c < nb) ? a.beta * a.mv[(int64_t)kvh * a.KB_tot + a.rows.seq_kb_off[seq] + tj * kTile + c] : 0.f;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *(volatile uint32_t*)(smem_gen + kSmemTmem);
  constexpr int kIters = 2 * BLK;  // (token of the block, half of the head dimension)

  if (warp == 4) {
    // ============================== copies ==============================
    const bool leader = elect_one();
    bool ok = true;
#pragma unroll 1
    for (int it = 0; it < kIters && ok; ++it) {
      const int st = it % kStages, s = it >> 1, half = it & 1;
      if (it >= kStages) ok = __all_sync(0xffffffffu, mbar_wait(empty(st), ((it / kStages) - 1) & 1, a.status));
      if (!ok) break;
      if (leader) {
        mbar_expect_tx(full(st), 2 * kPartBytes);
        // query tokens in reverse order, key tokens in order: step s pairs q[B-1-s] with k[s]
        tma_load_4d(smem_base + kSmemA + st * kPartBytes, &maps.q[seq], full(st), 64 * half, h, BLK - 1 - s, ti * kTile);
        tma_load_4d(smem_base + kSmemB + st * kPartBytes, &maps.k[seq], full(st), 64 * half, kvh, s, tj * kTile);
      }
      __syncwarp();
    }
  } else if (warp == 5) {
    // ============================== MMAs ==============================
    const bool leader = elect_one();
    bool ok = true;
#pragma unroll 1
    for (int it = 0; it < kIters && ok; ++it) {
      const int st = it % kStages;
      ok = __all_sync(0xffffffffu, mbar_wait(full(st), (it / kStages) & 1, a.status));
      if (!ok) break;
      tc_fence_after();
      if (leader) {
        const uint32_t a_addr = smem_base + kSmemA + st * kPartBytes, b_addr = smem_base + kSmemB + st * kPartBytes;
#pragma unroll
        for (int k = 0; k < 4; ++k) mma_ss(tmem, smem_desc(a_addr + k * 32), smem_desc(b_addr + k * 32), kIdesc, (it | k) ? 1u : 0u);
        tc_commit(empty(st));
        if (it == kIters - 1) tc_commit(acc_full);
      }
      __syncwarp();
    }
  } else {
    // ============================== epilogue ==============================
    const int m = warp * 32 + lane;       // row of the tile == TMEM lane
    const int rl = ti * kTile + m;        // row inside the chunk
    const int r = r0 + rl;                // row inside the sequence
    const int stride = (nb + 31) & ~31;
    if (__all_sync(0xffffffffu, mbar_wait(acc_full, 0, a.status))) {
      tc_fence_after();
      const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16);
      uint32_t* dst_planes = (uint32_t*)a.M + (int64_t)h * a.mt_tot + a.rows.seq_mt_off[seq] + (int64_t)rl * stride + tj * kTile;
      float* mrow = a.M + (int64_t)h * a.m_tot + a.rows.seq_m_off[seq] + (int64_t)rl * nb;
#pragma unroll 1
      for (int gq = 0; gq < 4; ++gq) {
        float v[32];
        tmem_ld32_sync(taddr + gq * 32, v);
        if (r >= nfull) continue;  // rows of the partial block (or past the end) belong to the other kernel
        if (a.as_keys) {
          uint32_t w[32];
#pragma unroll
          for (int c = 0; c < 32; ++c)
            w[c] = __float_as_uint(fmaxf(fmaf(a.scale, v[c], bias[gq * 32 + c]) + 0.0f, __int_as_float(0xff800000)));
          transpose32(w);
          const uint32_t neg = w[31];  // bit t: value t is negative
#pragma unroll
          for (int k = 0; k < 31; ++k) w[k] ^= neg;
          w[31] = ~neg;
          if (tj * kTile + gq * 32 < stride) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              *(uint4*)(dst_planes + gq * 32 + q * 4) = make_uint4(w[q * 4], w[q * 4 + 1], w[q * 4 + 2], w[q * 4 + 3]);
          }
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            const int cg = tj * kTile + gq * 32 + c;
            if (cg <= r) mrow[cg] = fmaf(a.scale, v[c], bias[gq * 32 + c]);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(128) : "memory");
  }
}

// The metric row of a sequence's partial last block (when it belongs to the query chunk): for every j <= r the
// mean over the anti-diagonal pairs whose two tokens exist.  One CTA per (sequence, query head); a warp takes
// 32 consecutive columns at a time, the lanes share each dot product (4 elements of d per lane).
template <int BLK>
__global__ void __launch_bounds__(256) antidiag_partial_kernel(const AntiArgs a) {
  const int seq = blockIdx.x, h = blockIdx.y, kvh = h / a.g;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nb = a.rows.seq_nblk[seq], r0 = a.rows.seq_r0[seq];
  const int r = nb - 1;
  const int ntok = a.rows.kb_ntok[a.rows.seq_kb_first[seq] + r];
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (ntok == BLK || r < r0) return;
  const int R = a.rows.seq_row_off[seq] + (r - r0);
  const __nv_bfloat16* qblk = a.Q + (int64_t)a.rows.row_tok0[R] * a.q_st + (int64_t)h * a.q_sh;
  const __nv_bfloat16* kseq = a.K + (int64_t)a.rows.seq_tok0[seq] * a.kv_st + (int64_t)kvh * a.kv_sh;
  const int stride = (nb + 31) & ~31;
  uint32_t* planes = (uint32_t*)a.M + (int64_t)h * a.mt_tot + a.rows.seq_mt_off[seq] + (int64_t)(r - r0) * stride;
  float* mrow = a.M + (int64_t)h * a.m_tot + a.rows.seq_m_off[seq] + (int64_t)(r - r0) * nb;
  const float score_scale = a.scale * (float)BLK;
  for (int j0 = warp * 32; j0 <= r; j0 += 8 * 32) {
    float mine = 0.f;  // lane c keeps the value of column j0 + c
    for (int c = 0; c < 32; ++c) {
      const int j = j0 + c;
      if (j > r) break;  // warp-uniform
      const int ktok = j == r ? ntok : BLK;
      float acc = 0.f;
      int pairs = 0;
      for (int s = 0; s < BLK; ++s) {
        const int tq = BLK - 1 - s;
        if (tq >= ntok || s >= ktok) continue;  // warp-uniform
        const uint2 qv = *(const uint2*)(qblk + (int64_t)tq * a.q_st + lane * 4);
        const uint2 kv = *(const uint2*)(kseq + (int64_t)(j * BLK + s) * a.kv_st + lane * 4);
        acc = fmaf(__uint_as_float(qv.x << 16), __uint_as_float(kv.x << 16), acc);
        acc = fmaf(__uint_as_float(qv.x & 0xffff0000u), __uint_as_float(kv.x & 0xffff0000u), acc);
        acc = fmaf(__uint_as_float(qv.y << 16), __uint_as_float(kv.y << 16), acc);
        acc = fmaf(__uint_as_float(qv.y & 0xffff0000u), __uint_as_float(kv.y & 0xffff0000u), acc);
        ++pairs;
      }
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
      const float val = score_scale * (pairs > 0 ? acc / (float)pairs : 0.f) +
                        a.beta * a.mv[(int64_t)kvh * a.KB_tot + a.rows.seq_kb_off[seq] + j];
      if (lane == c) mine = val;
    }
    if (a.as_keys) {
      // the 32 columns' keys as 32 bit planes: lane k stores plane k
      const uint32_t key = j0 + lane <= r ? metric_key(mine) : 0u;
      uint32_t word = 0u;
#pragma unroll
      for (int k = 0; k < 32; ++k) {
        const uint32_t bal = __ballot_sync(0xffffffffu, (key >> k) & 1u);
        if (lane == k) word = bal;
      }
      planes[j0 + lane] = word;
    } else if (j0 + lane <= r) {
      mrow[j0 + lane] = mine;
    }
  }
}

}  // namespace

int antidiag_max_sequences() { return kMaxSeqs; }

cudaError_t launch_antidiag_metric(const Plan& p, const void* Q, const void* K, const float* mv, float* M, bool as_keys,
                                   int32_t* status, int* launched, cudaStream_t s) {
  *launched = 0;
  const int B = p.cfg.block, batch = p.cfg.batch;
  if (batch > kMaxSeqs) return cudaErrorInvalidValue;
  MapSet maps{};
  bool any_partial = false;
  for (int b = 0; b < batch; ++b) {
    const int64_t n = p.cu[b + 1] - p.cu[b];
    const int64_t nfull = n / B;
    const int64_t r0 = p.h_seq_r0[b];
    any_partial = any_partial || (n % B != 0);
    // Maps over the FULL blocks only: (d, head, token in block, block); a block past the last full one reads as zero.
    const int64_t q_blocks = std::max<int64_t>(nfull - r0, 1), k_blocks = std::max<int64_t>(nfull, 1);
    const __nv_bfloat16* qb = (const __nv_bfloat16*)Q + (int64_t)p.h_seq_qtok0[b] * p.cfg.q_stride_tok;
    const __nv_bfloat16* kb = (const __nv_bfloat16*)K + (int64_t)p.cu[b] * p.cfg.kv_stride_tok;
    if (!make_bf16_map_4d(&maps.q[b], qb, {(uint64_t)kHeadDim, (uint64_t)p.cfg.num_q_heads, (uint64_t)B, (uint64_t)q_blocks},
                          {(uint64_t)p.cfg.q_stride_head * 2, (uint64_t)p.cfg.q_stride_tok * 2, (uint64_t)B * p.cfg.q_stride_tok * 2},
                          {64u, 1u, 1u, (uint32_t)kTile}) ||
        !make_bf16_map_4d(&maps.k[b], kb, {(uint64_t)kHeadDim, (uint64_t)p.cfg.num_kv_heads, (uint64_t)B, (uint64_t)k_blocks},
                          {(uint64_t)p.cfg.kv_stride_head * 2, (uint64_t)p.cfg.kv_stride_tok * 2, (uint64_t)B * p.cfg.kv_stride_tok * 2},
                          {64u, 1u, 1u, (uint32_t)kTile}))
      return cudaErrorInvalidValue;
  }
  for (int b = batch; b < kMaxSeqs; ++b) { maps.q[b] = maps.q[0]; maps.k[b] = maps.k[0]; }

  AntiArgs a{};
  a.tiles = p.d_gemm_tiles; a.mv = mv; a.M = M; a.status = status; a.rows = p.rows; a.m_tot = p.m_tot; a.mt_tot = p.mt_tot;
  a.Hq = p.cfg.num_q_heads; a.g = a.Hq / p.cfg.num_kv_heads; a.KB_tot = p.KB_tot; a.block = B;
  a.beta = p.cfg.beta; a.scale = p.score_scale / (float)B; a.as_keys = as_keys ? 1 : 0;
  a.Q = (const __nv_bfloat16*)Q; a.K = (const __nv_bfloat16*)K;
  a.q_st = p.cfg.q_stride_tok; a.q_sh = p.cfg.q_stride_head; a.kv_st = p.cfg.kv_stride_tok; a.kv_sh = p.cfg.kv_stride_head;
  a.batch = batch;

  static bool attr_set[64] = {};
  const int dev_slot = p.device & 63;
  if (!attr_set[dev_slot]) {
    cudaError_t e = cudaFuncSetAttribute(antidiag_metric_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(antidiag_metric_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set[dev_slot] = true;
  }
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)p.n_gemm_tiles, (unsigned)a.Hq);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = B == 128 ? cudaLaunchKernelEx(&cfg, antidiag_metric_kernel<128>, maps, a)
                           : cudaLaunchKernelEx(&cfg, antidiag_metric_kernel<64>, maps, a);
  if (e != cudaSuccess) return e;
  ++*launched;
  if (!any_partial) return e;
  // the metric rows of partial last blocks (stream-ordered behind the contraction; it waits for the pooling
  // kernel's MV through the contraction kernel)
  cudaLaunchConfig_t cfg2 = {};
  cfg2.gridDim = dim3((unsigned)batch, (unsigned)a.Hq);
  cfg2.blockDim = dim3(256);
  cfg2.stream = s;
  e = B == 128 ? cudaLaunchKernelEx(&cfg2, antidiag_partial_kernel<128>, a) : cudaLaunchKernelEx(&cfg2, antidiag_partial_kernel<64>, a);
  if (e == cudaSuccess) ++*launched;
  return e;
}

}  // namespace stem
