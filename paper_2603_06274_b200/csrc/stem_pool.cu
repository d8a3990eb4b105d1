// Alg. 1 step 1: block-wise representations.
//   Qbar, Kbar : mean over the valid tokens of each block ("Pool(Q, K, stride = B)")
//   MV         : max(0, max_t ln ||V_t||_2) per block ("MaxPool(log ||V||_2)" and the clamp of Eq. 7),
//                evaluated as 0.5 * ln(max(1, max_t ||V_t||^2)).
// One pass over Q, K and V; HBM-bound.  One CTA per (block, head) of Q, of K and of V; neighbouring CTAs read
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
// CTAs 0 .. n_q - 1 pool Q: one per (query row, list head); with heads_per_list > 1 (one index list per kv
// group) a CTA averages the block over the group's query heads as well.  The CTAs after them pool K and V:
// one per (key block, kv head, K or V), over every key block of the plan or only the blocks a chunk adds.
struct PoolArgs {
  const __nv_bfloat16 *Q, *K, *V;
  int64_t q_st, q_sh, kv_st, kv_sh;
  int H_list, heads_per_list, Hkv, R_tot, KB_tot;
  int n_q;        // CTAs of the Q part (0 when Q is not pooled)
  int only_new;   // K / V part: walk kb_new instead of all key blocks
  RowTables rows;
  float* mv;
  __nv_bfloat16 *qsplit, *ksplit;
};

template <int kBlock, bool kGroupMean>
__global__ void __launch_bounds__(128) pool_kernel(const PoolArgs a) {
  constexpr int kTokPerWarp = kBlock / 4;
  constexpr int kSteps = kTokPerWarp / 2;
  // lets a kernel launched as a programmatic dependent set itself up during this kernel's last wave
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = lane >> 4, chunk = lane & 15;

  const __nv_bfloat16* base;
  int64_t st, sh;
  int h, kind, tok0, ntok, dst_row, n_heads = 1;  // kind: 0 = Q, 1 = K, 2 = V
  if ((int)blockIdx.x < a.n_q) {
    const int R = blockIdx.x / a.H_list;
    h = blockIdx.x - R * a.H_list;
    kind = 0;
    n_heads = a.heads_per_list;
    base = a.Q + (int64_t)h * n_heads * a.q_sh;
    st = a.q_st; sh = a.q_sh;
    tok0 = a.rows.row_tok0[R];
    ntok = a.rows.row_ntok[R];
    dst_row = R;
  } else {
    const int i = ((int)blockIdx.x - a.n_q) / (2 * a.Hkv);
    const int slot = ((int)blockIdx.x - a.n_q) - i * 2 * a.Hkv;
    const int kb = a.only_new ? a.rows.kb_new[i] : i;
    kind = slot < a.Hkv ? 1 : 2;
    h = kind == 1 ? slot : slot - a.Hkv;
    base = (kind == 1 ? a.K : a.V) + (int64_t)h * a.kv_sh;
    st = a.kv_st; sh = a.kv_sh;
    tok0 = a.rows.kb_tok0[kb];
    ntok = a.rows.kb_ntok[kb];
    dst_row = a.rows.kb_dst[kb];
  }

  // every load of the block (of its first head) is issued before anything else happens
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
    for (int hh = 1; kGroupMean && hh < n_heads; ++hh) {  // the other query heads of the group (one list per kv head)
#pragma unroll
      for (int i = 0; i < kSteps; ++i) {
        const int t = warp * kTokPerWarp + 2 * i + half;
        raw[i] = make_uint4(0, 0, 0, 0);
        if (t < ntok) raw[i] = ld_stream(base + (int64_t)hh * sh + (int64_t)(tok0 + t) * st + chunk * 8);
      }
#pragma unroll
      for (int i = 0; i < kSteps; ++i) {
        float f[8];
        unpack8(raw[i], f);
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[c] += f[c];
      }
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
    const float mean = sum / (float)(ntok * n_heads);
    // mean = hi + mid + lo, each part the bf16 rounding of what the previous ones leave (the tensor-core
    // metric kernel multiplies these parts)
    const __nv_bfloat16 hi = __float2bfloat16_rn(mean);
    const float r1 = mean - __bfloat162float(hi);
    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
    __nv_bfloat16* dst = kind == 0 ? a.qsplit : a.ksplit;
    const int64_t rows_tot = kind == 0 ? a.R_tot : a.KB_tot;
    const int64_t plane = (int64_t)(kind == 0 ? a.H_list : a.Hkv) * rows_tot * kHeadDim;
    const int64_t at = ((int64_t)h * rows_tot + dst_row) * kHeadDim + c;
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
      a.mv[(int64_t)h * a.KB_tot + dst_row] = 0.5f * logf(fmaxf(1.f, m2));
    }
  }
}

}  // namespace

cudaError_t launch_pool(const Plan& p, const void* Q, const void* K, const void* V, float* mv, void* qsplit, void* ksplit,
                        bool only_new, cudaStream_t s) {
  PoolArgs a{};
  a.Q = (const __nv_bfloat16*)Q; a.K = (const __nv_bfloat16*)K; a.V = (const __nv_bfloat16*)V;
  a.q_st = p.cfg.q_stride_tok; a.q_sh = p.cfg.q_stride_head; a.kv_st = p.cfg.kv_stride_tok; a.kv_sh = p.cfg.kv_stride_head;
  a.H_list = p.H_list; a.heads_per_list = p.cfg.num_q_heads / p.H_list; a.Hkv = p.cfg.num_kv_heads;
  a.R_tot = p.R_tot; a.KB_tot = p.KB_tot;
  a.n_q = Q ? p.R_tot * p.H_list : 0;
  a.only_new = only_new ? 1 : 0;
  a.rows = p.rows; a.mv = mv; a.qsplit = (__nv_bfloat16*)qsplit; a.ksplit = (__nv_bfloat16*)ksplit;
  const int64_t n_k = K ? (int64_t)(only_new ? p.n_kb_new : p.n_kb_all) * 2 * p.cfg.num_kv_heads : 0;
  const dim3 grid((unsigned)(a.n_q + n_k));
  if (grid.x == 0) return cudaSuccess;
  const bool group_mean = a.heads_per_list > 1;
  if (p.cfg.block == 128) {
    if (group_mean) pool_kernel<128, true><<<grid, 128, 0, s>>>(a);
    else pool_kernel<128, false><<<grid, 128, 0, s>>>(a);
  } else {
    if (group_mean) pool_kernel<64, true><<<grid, 128, 0, s>>>(a);
    else pool_kernel<64, false><<<grid, 128, 0, s>>>(a);
  }
  return cudaGetLastError();
}

}  // namespace stem
