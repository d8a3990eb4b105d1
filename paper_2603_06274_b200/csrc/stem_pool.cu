// Alg. 1 step 1: block-wise representations.
//   Qbar, Kbar : mean over the valid tokens of each block ("Pool(Q, K, stride = B)")
//   MV         : max(0, max_t ln ||V_t||_2) per block ("MaxPool(log ||V||_2)" and the clamp of Eq. 7),
//                evaluated as 0.5 * ln(max(1, max_t ||V_t||^2)).
// One pass over Q, K and V; HBM-bound.  One CTA per (query-block row, head slot) where the head
// slots enumerate the Q heads, then the K heads, then the V heads, so that neighbouring CTAs read
// neighbouring 256-byte rows of the packed [T, H, d] tensors.
#include <cuda_bf16.h>

#include "stem_internal.h"

namespace stem {

namespace {

__device__ __forceinline__ uint4 ld_stream(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

// 128 threads: 4 warps x (2 half-warps x 16 lanes).  A half-warp reads one 256-byte token row
// (16 lanes x 16 bytes); a warp covers kTok / 4 consecutive tokens, two per step.
template <int kBlock>
__global__ void __launch_bounds__(128) pool_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                                                   const __nv_bfloat16* __restrict__ V, int64_t q_st, int64_t q_sh,
                                                   int64_t kv_st, int64_t kv_sh, int Hq, int Hkv, int R_tot,
                                                   RowTables rows, float* __restrict__ mv,
                                                   __nv_bfloat16* __restrict__ qsplit, __nv_bfloat16* __restrict__ ksplit) {
  constexpr int kTokPerWarp = kBlock / 4;
  constexpr int kSteps = kTokPerWarp / 2;
  // lets a kernel launched as a programmatic dependent set itself up during this kernel's last wave
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int slots = Hq + 2 * Hkv;
  const int R = blockIdx.x / slots;
  const int slot = blockIdx.x - R * slots;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = lane >> 4, chunk = lane & 15;

  const __nv_bfloat16* base;
  int64_t st;
  int h, kind;  // 0 = Q, 1 = K, 2 = V
  if (slot < Hq) { kind = 0; h = slot; base = Q + (int64_t)h * q_sh; st = q_st; }
  else if (slot < Hq + Hkv) { kind = 1; h = slot - Hq; base = K + (int64_t)h * kv_sh; st = kv_st; }
  else { kind = 2; h = slot - Hq - Hkv; base = V + (int64_t)h * kv_sh; st = kv_st; }

  const int tok0 = rows.row_tok0[R];
  const int ntok = rows.row_ntok[R];

  uint4 raw[kSteps];
#pragma unroll
  for (int i = 0; i < kSteps; ++i) {
    const int t = warp * kTokPerWarp + 2 * i + half;
    raw[i] = make_uint4(0, 0, 0, 0);
    if (t < ntok) raw[i] = ld_stream(base + (int64_t)(tok0 + t) * st + chunk * 8);
  }

  __shared__ float red[4][kHeadDim];
  __shared__ float redmax[4];

  if (kind < 2) {
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
    for (int i = 0; i < kSteps; ++i) {
      float f[8];
      unpack8(raw[i], f);
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[c] += f[c];
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], 16);
    if (half == 0) {
#pragma unroll
      for (int c = 0; c < 8; ++c) red[warp][chunk * 8 + c] = acc[c];
    }
    __syncthreads();
    const int c = threadIdx.x;
    const float sum = (red[0][c] + red[1][c]) + (red[2][c] + red[3][c]);
    const float mean = sum / (float)ntok;
    // mean = hi + mid + lo, each part the bf16 rounding of what the previous ones leave (the tensor-core
    // metric kernel multiplies these parts); row = global block row for both tensors
    const __nv_bfloat16 hi = __float2bfloat16_rn(mean);
    const float r1 = mean - __bfloat162float(hi);
    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
    __nv_bfloat16* dst = kind == 0 ? qsplit : ksplit;
    const int64_t plane = (int64_t)(kind == 0 ? Hq : Hkv) * R_tot * kHeadDim;
    const int64_t at = ((int64_t)h * R_tot + R) * kHeadDim + c;
    dst[at] = hi;
    dst[at + plane] = mid;
    dst[at + 2 * plane] = lo;
  } else {
    float best = 0.f;  // squared norms are >= 0
#pragma unroll
    for (int i = 0; i < kSteps; ++i) {
      float f[8];
      unpack8(raw[i], f);
      float ss = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) ss = fmaf(f[c], f[c], ss);
      ss += __shfl_xor_sync(0xffffffffu, ss, 8);
      ss += __shfl_xor_sync(0xffffffffu, ss, 4);
      ss += __shfl_xor_sync(0xffffffffu, ss, 2);
      ss += __shfl_xor_sync(0xffffffffu, ss, 1);
      best = fmaxf(best, ss);
    }
    best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, 16));
    if (lane == 0) redmax[warp] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
      const float m2 = fmaxf(fmaxf(redmax[0], redmax[1]), fmaxf(redmax[2], redmax[3]));
      mv[(int64_t)h * R_tot + R] = 0.5f * logf(fmaxf(1.f, m2));
    }
  }
}

}  // namespace

cudaError_t launch_pool(const Plan& p, const void* Q, const void* K, const void* V, float* mv, void* qsplit, void* ksplit,
                        cudaStream_t s) {
  const int slots = p.cfg.num_q_heads + 2 * p.cfg.num_kv_heads;
  const dim3 grid((unsigned)((int64_t)p.R_tot * slots));
  auto q = (const __nv_bfloat16*)Q;
  auto k = (const __nv_bfloat16*)K;
  auto v = (const __nv_bfloat16*)V;
  if (p.cfg.block == 128)
    pool_kernel<128><<<grid, 128, 0, s>>>(q, k, v, p.cfg.q_stride_tok, p.cfg.q_stride_head, p.cfg.kv_stride_tok,
                                          p.cfg.kv_stride_head, p.cfg.num_q_heads, p.cfg.num_kv_heads, p.R_tot, p.rows, mv,
                                          (__nv_bfloat16*)qsplit, (__nv_bfloat16*)ksplit);
  else
    pool_kernel<64><<<grid, 128, 0, s>>>(q, k, v, p.cfg.q_stride_tok, p.cfg.q_stride_head, p.cfg.kv_stride_tok,
                                         p.cfg.kv_stride_head, p.cfg.num_q_heads, p.cfg.num_kv_heads, p.R_tot, p.rows, mv,
                                         (__nv_bfloat16*)qsplit, (__nv_bfloat16*)ksplit);
  return cudaGetLastError();
}

}  // namespace stem
