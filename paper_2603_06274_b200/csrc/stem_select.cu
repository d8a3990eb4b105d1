// Alg. 1 steps 3a-3c on pooled blocks.
//   metric   M[h,r,j] = score_scale * Qbar[h,r].Kbar[kv(h),j] + beta * MV[kv(h),j],  j <= r   (Eq. 7)
//   select   forced stem/local blocks plus the top (k_eff(r) - |forced|) remaining causal blocks,
//            order (metric descending, block id ascending), emitted ascending            (Alg. 1 "TopK")
//
// One CTA owns a tile: the g query heads of one kv head times a run of consecutive rows of one
// sequence (at most 32 pooled query vectors), and walks the causal key blocks in chunks of 64.
//
// Scoring is a small fp32 GEMM on the FMA pipe (a 10-bit tensor-core mantissa would move top-k
// boundaries): Qbar^T of the tile stays in shared memory, Kbar^T (stored transposed by the pooling
// kernel, block index contiguous) streams through a double-buffered chunk, and each thread keeps
// an 8 x 2 register tile over one half of the head dimension; the two halves sit in the two lane
// halves of a warp and are added by a shuffle.  Both operands are laid out in shared memory so
// that a warp's loads of one step fall into whole 128-byte lines.
//
// Selection is streaming, so a metric row never has to exist as a whole: every row keeps a short
// list of (key, block) candidates in shared memory and a threshold tau.  A new metric value joins
// the list only if its order-preserving key is above tau; when a list runs full it is cut back
// (keeping at least the row's budget of best entries), tau rises, and the values that did not fit
// are offered again.  Because blocks arrive in ascending order, a later block with a key equal to
// tau can never displace a kept one (ties go to the smaller block id), which is why the strict
// comparison loses nothing.  At the end each row's list is cut to its budget, merged with the
// forced blocks through a bitmap and written out in ascending order.
#include "stem_internal.h"

namespace stem {

namespace {

constexpr int kThreads = 256;
constexpr int kNQ = 32;        // pooled query vector slots per tile
constexpr int kChunk = 64;     // key blocks scored per step
constexpr int kMaxWords = 64;  // bitmap words per row: at most 2048 blocks per sequence

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

// Bits of word w (blocks 32 w .. 32 w + 31) that fall into the block range [lo, hi).
__device__ __forceinline__ uint32_t range_bits(int lo, int hi, int w) {
  const int a = max(lo - w * 32, 0), b = min(hi - w * 32, 32);
  if (b <= a) return 0u;
  const uint32_t upto_b = b >= 32 ? 0xffffffffu : ((1u << b) - 1u);
  return upto_b & ~((1u << a) - 1u);  // a < 32 here
}

struct TileArgs {
  const float* qbar; const float* kbar_t; const float* mv;
  const float* M_in; float* M_out;
  int32_t* sel_idx; int32_t* sel_cnt;
  const int32_t* tiles;
  RowTables rows;
  int Hq, Hkv, g, R_tot, k_max, rows_per_tile, nq_slots, kt_width, list_cap;
  int stem, local;
  int64_t m_tot;
  float beta, score_scale;
  int mode;
};

// Per-row selection state in shared memory.
struct RowState {
  uint32_t tau;     // a candidate must have key > tau to join the list
  int cnt;          // entries in the list
  int need;         // entries the finished list must hold (0 when every candidate or none is taken)
  int n_stem;       // candidates are the blocks n_stem .. lo_local - 1
  int lo_local;
  int i;            // causal blocks of the row (r + 1)
  int take_all;     // every candidate is selected: no list is kept
  int pad;
};

// Cuts the list of one row back (in place) and raises tau.  At most max_keep entries survive and
// never fewer than the row's `need` best ones in the order (key descending, block ascending); with
// max_keep == need exactly those survive.  A loose cut (max_keep > need) needs only a few counting
// passes and is all the streaming filter asks for.  One warp.  KL > 0: the list has at most
// 32 * KL entries and is held in registers during the search; KL == 0: any length, read from
// shared memory in every pass.
template <int KL>
__device__ __forceinline__ void warp_cut_list(RowState* st, uint32_t* ckey, uint16_t* ccol, int max_keep, int lane) {
  const int n = st->cnt, need = st->need;
  if (n <= max_keep) return;
  constexpr int kRegs = KL > 0 ? KL : 1;
  uint32_t key[kRegs];
  uint32_t kmax = 0u, kmin = 0xffffffffu;
  if (KL > 0) {
#pragma unroll
    for (int q = 0; q < kRegs; ++q) {
      const int p = q * 32 + lane;
      key[q] = p < n ? ckey[p] : 0u;  // 0 is below every key and every threshold
      kmax = max(kmax, key[q]);
      kmin = min(kmin, p < n ? key[q] : 0xffffffffu);
    }
  } else {
    for (int p = lane; p < n; p += 32) { const uint32_t k = ckey[p]; kmax = max(kmax, k); kmin = min(kmin, k); }
  }
  auto count_ge = [&](uint32_t t) -> int {
    int c = 0;
    if (KL > 0) {
#pragma unroll
      for (int q = 0; q < kRegs; ++q) c += key[q] >= t ? 1 : 0;
    } else {
      for (int p = lane; p < n; p += 32) c += ckey[p] >= t ? 1 : 0;
    }
    return __reduce_add_sync(0xffffffffu, c);
  };
  uint32_t lo = __reduce_min_sync(0xffffffffu, kmin);       // f(lo) = n > max_keep, with f(t) = #{key >= t}
  uint32_t hi = __reduce_max_sync(0xffffffffu, kmax) + 1u;  // f(hi) = 0 < need (keys stay below 0xff800001)
  int c_lo = n, c_hi = 0;
  // Bracket f(lo) >= need > f(hi); thresholds alternate between the point where a linear model of
  // f reaches the middle of the wanted range and the midpoint of the bracket (which bounds the
  // number of steps); stop as soon as keeping the keys >= lo is enough of a cut, or when the
  // bracket is one key wide (a tie across the cut).
  const int aim = (need + max_keep + 1) >> 1;
#pragma unroll 1
  for (int step = 0; c_lo > max_keep && hi - lo > 1u; ++step) {
    uint32_t cand = lo + ((hi - lo) >> 1);
    if ((step & 1) == 0) {
      const float fr = (float)(c_lo - aim) / (float)(c_lo - c_hi);
      cand = lo + (uint32_t)((float)(hi - lo) * fr);
    }
    cand = min(max(cand, lo + 1u), hi - 1u);
    const int c = count_ge(cand);
    if (c >= need) { lo = cand; c_lo = c; } else { hi = cand; c_hi = c; }
  }
  // keep key > thr, plus the need_eq smallest block ids among key == thr
  uint32_t thr = lo - 1u;  // key >= lo  <=>  key > lo - 1 (lo >= 1)
  int col_thr = -1;
  if (c_lo > max_keep) {
    // lo is tied across the cut (hi == lo + 1, c_hi = keys above lo): keep exactly `need` entries
    thr = lo;
    const int need_eq = need - c_hi;
    int clo = -1, chi = 65535;  // #{tied, col <= clo} < need_eq <= #{tied, col <= chi}
    while (chi - clo > 1) {
      const int mid = (clo + chi) >> 1;
      int c = 0;
      for (int p = lane; p < n; p += 32) c += (ckey[p] == thr && (int)ccol[p] <= mid) ? 1 : 0;
      c = __reduce_add_sync(0xffffffffu, c);
      if (c >= need_eq) chi = mid; else clo = mid;
    }
    col_thr = chi;
  }
  int base = 0;
  for (int p0 = 0; p0 < n; p0 += 32) {
    const int p = p0 + lane;
    uint32_t k = 0u;
    uint16_t c = 0;
    if (p < n) { k = ckey[p]; c = ccol[p]; }
    const bool keep = p < n && (k > thr || (k == thr && (int)c <= col_thr));
    const uint32_t kb = __ballot_sync(0xffffffffu, keep);
    if (keep) {  // never behind the old position, and this pass was read before it is written
      const int q = base + __popc(kb & ((1u << lane) - 1u));
      ckey[q] = k;
      ccol[q] = c;
    }
    base += __popc(kb);
    __syncwarp();
  }
  if (lane == 0) { st->cnt = base; st->tau = thr; }
  __syncwarp();
}
__device__ __forceinline__ void cut_list(int list_cap, RowState* st, uint32_t* ckey, uint16_t* ccol, int max_keep, int lane) {
  if (list_cap <= 128) warp_cut_list<4>(st, ckey, ccol, max_keep, lane);
  else if (list_cap <= 256) warp_cut_list<8>(st, ckey, ccol, max_keep, lane);
  else warp_cut_list<0>(st, ckey, ccol, max_keep, lane);
}

__global__ void __launch_bounds__(kThreads, 2) score_select_kernel(TileArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // Element (d, x) of an operand, d = ds * 64 + dd, is stored at ((dd * G + x / W) * 2 + ds) * W + x % W
  // (G groups of W consecutive vectors / columns): the two d-halves a warp reads together are adjacent.
  float* qt = (float*)smem_raw;                        // Qbar^T of the tile: 128 d x kNQ, W = 8
  float* kt = qt + kHeadDim * kNQ;                     // Kbar^T chunk, double-buffered: 2 x (128 d x kChunk), W = 32
  RowState* rs = (RowState*)(kt + 2 * kHeadDim * kChunk);  // [kNQ]
  uint32_t* bitmap = (uint32_t*)(rs + kNQ);            // [warps][kMaxWords]
  uint32_t* ckey = bitmap + (kThreads / 32) * kMaxWords;   // [nq_slots][list_cap] candidate keys
  uint16_t* ccol = (uint16_t*)(ckey + (size_t)a.nq_slots * a.list_cap);  // [nq_slots][list_cap] candidate blocks

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
  const int n_chunks = (n_cols + kChunk - 1) / kChunk;
  const bool from_pooled = (a.mode & kFromPooled) != 0;
  const bool do_select = (a.mode & kSelect) != 0;

  const float* kb = a.kbar_t + (int64_t)kvh * kHeadDim * a.kt_width + a.rows.seq_kt_off[b];
  const float* mvb = a.mv + (int64_t)kvh * a.R_tot + row_off;
  // Kbar^T rows of this sequence start at a multiple of kChunk and are padded to a multiple of
  // kChunk, so whole chunks are in bounds.
  auto load_chunk = [&](int ch, int buf) {
    float* dst = kt + buf * kHeadDim * kChunk;
    for (int e = tid; e < kHeadDim * (kChunk / 4); e += kThreads) {
      const int d = e / (kChunk / 4), c4 = e - d * (kChunk / 4);
      const int ds = d >> 6, dd = d & 63;
      cp_async16(dst + ((dd * 2 + (c4 >> 3)) * 2 + ds) * 32 + (c4 & 7) * 4,
                 kb + (int64_t)d * a.kt_width + ch * kChunk + c4 * 4);
    }
    cp_async_commit();
  };
  if (from_pooled) {
    load_chunk(0, 0);  // in flight while the query vectors are staged
    for (int e = tid; e < kNQ * (kHeadDim / 4); e += kThreads) {
      const int v = e & (kNQ - 1), c4 = e / kNQ;
      float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
      if (v < nq) {
        const int rr = v / a.g, gh = v - rr * a.g;
        const int h = kvh * a.g + gh;
        val = *(const float4*)(a.qbar + ((int64_t)h * a.R_tot + row_off + r0 + rr) * kHeadDim + c4 * 4);
      }
      const int ds = c4 >> 4, dd = (c4 & 15) * 4;
      float* dst = qt + ((dd * 4 + (v >> 3)) * 2 + ds) * 8 + (v & 7);
      dst[0] = val.x; dst[64] = val.y; dst[128] = val.z; dst[192] = val.w;  // dd + 1 lies 4 * 2 * 8 floats further
    }
  }
  // ---- per-row selection state
  if (tid < kNQ) {
    RowState st{};
    if (tid < nq) {
      const int r = r0 + tid / a.g;
      const int i = r + 1;
      const int n_stem = min(a.stem, i);
      const int lo_local = max(0, i - a.local);
      const int n_forced = n_stem + (i - lo_local) - max(0, n_stem - lo_local);
      const int n_free = max(0, lo_local - n_stem);
      const int need = min(max(0, a.rows.row_keff[row_off + r] - n_forced), n_free);
      st.i = i; st.n_stem = n_stem; st.lo_local = lo_local;
      st.take_all = need >= n_free ? 1 : 0;
      st.need = st.take_all ? 0 : need;
      st.tau = (st.take_all || need == 0) ? 0xffffffffu : 0u;  // nothing joins a list that is not needed
    } else {
      st.tau = 0xffffffffu;
    }
    rs[tid] = st;
  }

  // thread tile: 8 vectors x 2 columns over one half of the head dimension
  const int vg = warp >> 1, cg = warp & 1;      // vectors vg * 8 .., columns cg * 32 .. of the chunk
  const int ds = lane >> 4, kp = lane & 15;
  const float* qp = qt + (vg * 2 + ds) * 8;
  for (int ch = 0; ch < n_chunks; ++ch) {
    if (from_pooled) cp_async_wait<0>();
    __syncthreads();  // chunk ch has landed, the other buffer is free, the lists are consistent
    float acc[8][2];
    uint32_t pending = 0u;  // values of this thread that found their row's list full
    const int j0 = ch * kChunk + cg * 32 + kp * 2;
    if (from_pooled) {
      if (ch + 1 < n_chunks) load_chunk(ch + 1, (ch + 1) & 1);
      const float* kp_s = kt + (ch & 1) * kHeadDim * kChunk + (cg * 2 + ds) * 32 + kp * 2;
      // packed fp32 FMAs (two vectors per instruction, same rounding as scalar FMAs): the loop is
      // bound by instruction issue, not by the FMA pipe
      float2 accp[4][2];
#pragma unroll
      for (int i = 0; i < 4; ++i) { accp[i][0] = make_float2(0.f, 0.f); accp[i][1] = make_float2(0.f, 0.f); }
#pragma unroll 8
      for (int dd = 0; dd < 64; ++dd) {
        const float4 qa = *(const float4*)(qp + dd * 64);
        const float4 qb = *(const float4*)(qp + dd * 64 + 4);
        const float2 kk = *(const float2*)(kp_s + dd * 128);
        const float2 qpair[4] = {make_float2(qa.x, qa.y), make_float2(qa.z, qa.w), make_float2(qb.x, qb.y),
                                 make_float2(qb.z, qb.w)};
        const float2 kx = make_float2(kk.x, kk.x), ky = make_float2(kk.y, kk.y);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          accp[i][0] = __ffma2_rn(qpair[i], kx, accp[i][0]);
          accp[i][1] = __ffma2_rn(qpair[i], ky, accp[i][1]);
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        acc[2 * i][0] = accp[i][0].x; acc[2 * i + 1][0] = accp[i][0].y;
        acc[2 * i][1] = accp[i][1].x; acc[2 * i + 1][1] = accp[i][1].y;
      }
      const float bias0 = (j0 < nblk) ? a.beta * mvb[j0] : 0.f;
      const float bias1 = (j0 + 1 < nblk) ? a.beta * mvb[j0 + 1] : 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        acc[i][0] += __shfl_xor_sync(0xffffffffu, acc[i][0], 16);  // lower half + upper half of d
        acc[i][1] += __shfl_xor_sync(0xffffffffu, acc[i][1], 16);
        acc[i][0] = fmaf(a.score_scale, acc[i][0], bias0);
        acc[i][1] = fmaf(a.score_scale, acc[i][1], bias1);
      }
    } else if (ds == 0) {
      // metric values come from global memory
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int v = vg * 8 + i;
        acc[i][0] = 0.f; acc[i][1] = 0.f;
        if (v < nq) {
          const int rr = v / a.g, gh = v - rr * a.g;
          const int r = r0 + rr;
          const float* src = a.M_in + (int64_t)(kvh * a.g + gh) * a.m_tot + m_off + (int64_t)r * nblk;
          if (j0 <= r) acc[i][0] = src[j0];
          if (j0 + 1 <= r) acc[i][1] = src[j0 + 1];
        }
      }
    }
    if (ds == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int v = vg * 8 + i;
        if (v >= nq) continue;
        if (a.mode & kWriteMetric) {
          const int rr = v / a.g, gh = v - rr * a.g;
          const int r = r0 + rr;
          float* dst = a.M_out + (int64_t)(kvh * a.g + gh) * a.m_tot + m_off + (int64_t)r * nblk;
          if (j0 <= r) dst[j0] = acc[i][0];
          if (j0 + 1 <= r) dst[j0 + 1] = acc[i][1];
        }
        if (do_select) {
          const uint32_t tau = rs[v].tau;
          const int n_stem = rs[v].n_stem, lo_local = rs[v].lo_local;
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            const int j = j0 + c;
            const uint32_t key = order_key(acc[i][c]);
            if (j >= n_stem && j < lo_local && key > tau) {
              const int pos = atomicAdd(&rs[v].cnt, 1);
              if (pos < a.list_cap) {
                ckey[(size_t)v * a.list_cap + pos] = key;
                ccol[(size_t)v * a.list_cap + pos] = (uint16_t)j;
              } else {
                pending |= 1u << (i * 2 + c);  // the list is full: try again after it has been cut
              }
            }
          }
        }
      }
    }
    if (do_select && __syncthreads_or(pending != 0u)) {
      // some list ran full: cut the full lists (loosely: a few counting passes), then place what was left over
      for (int v = warp; v < nq; v += kThreads / 32) {
        const int cnt_v = rs[v].cnt;
        __syncwarp();  // every lane has read the counter before lane 0 clamps it
        if (cnt_v <= a.list_cap) continue;
        if (lane == 0) rs[v].cnt = a.list_cap;
        __syncwarp();
        cut_list(a.list_cap, &rs[v], ckey + (size_t)v * a.list_cap, ccol + (size_t)v * a.list_cap,
                 (rs[v].need + a.list_cap - kChunk + 1) >> 1, lane);
      }
      __syncthreads();
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int v = vg * 8 + i;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          if (!(pending & (1u << (i * 2 + c)))) continue;
          const uint32_t key = order_key(acc[i][c]);
          if (key > rs[v].tau) {  // a cut list has room for a whole chunk
            const int pos = atomicAdd(&rs[v].cnt, 1);
            ckey[(size_t)v * a.list_cap + pos] = key;
            ccol[(size_t)v * a.list_cap + pos] = (uint16_t)(j0 + c);
          }
        }
      }
    }
  }
  if (!do_select) return;
  __syncthreads();

  // ---- finish: one warp per row cuts the list to the budget, merges it with the forced blocks
  // through a bitmap of the row's causal blocks, and writes the blocks out in ascending order
  uint32_t* bm = bitmap + warp * kMaxWords;
  for (int v = warp; v < nq; v += kThreads / 32) {
    RowState* st = &rs[v];
    uint32_t* lk = ckey + (size_t)v * a.list_cap;
    uint16_t* lc = ccol + (size_t)v * a.list_cap;
    cut_list(a.list_cap, st, lk, lc, st->need, lane);
    const int i = st->i, n_stem = st->n_stem, lo_local = st->lo_local;
    const bool take_all = st->take_all != 0;
    const int n_words = (i + 31) >> 5;
    // forced blocks [0, n_stem) and [lo_local, i); with take_all every causal block
    for (int w = lane; w < n_words; w += 32) {
      const uint32_t bits = take_all ? range_bits(0, i, w) : (range_bits(0, n_stem, w) | range_bits(lo_local, i, w));
      bm[w] = bits;
    }
    __syncwarp();
    const int n_list = take_all ? 0 : st->cnt;
    for (int p = lane; p < n_list; p += 32) atomicOr(&bm[lc[p] >> 5], 1u << (lc[p] & 31));
    __syncwarp();
    const int h = kvh * a.g + (v % a.g);
    const int R = row_off + r0 + v / a.g;
    int32_t* out = a.sel_idx + ((int64_t)h * a.R_tot + R) * a.k_max;
    int base = 0;
    for (int w0 = 0; w0 < n_words; w0 += 32) {
      const int w = w0 + lane;
      uint32_t bits = w < n_words ? bm[w] : 0u;
      const int mine = __popc(bits);
      int incl = mine;  // inclusive scan over the lanes
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
      }
      int pos = base + incl - mine;
      while (bits) {
        const int bit = __ffs(bits) - 1;
        bits &= bits - 1u;
        if (pos < a.k_max) out[pos] = w * 32 + bit;
        ++pos;
      }
      base += __shfl_sync(0xffffffffu, incl, 31);
    }
    for (int q = base + lane; q < a.k_max; q += 32) out[q] = -1;
    if (lane == 0) a.sel_cnt[(int64_t)h * a.R_tot + R] = min(base, a.k_max);
    __syncwarp();
  }
}

size_t score_select_fixed_smem() {
  return (size_t)(kHeadDim * kNQ + 2 * kHeadDim * kChunk) * sizeof(float) + kNQ * sizeof(RowState) +
         (kThreads / 32) * kMaxWords * sizeof(uint32_t);
}

}  // namespace

// Shared memory one pooled query vector needs for its candidate list.
size_t score_select_list_bytes(int k_max) {
  const size_t cap = (size_t)(k_max + kChunk + 31) / 32 * 32;
  return cap * (sizeof(uint32_t) + sizeof(uint16_t));
}
size_t score_select_smem_budget() { return 227 * 1024 - score_select_fixed_smem(); }
int score_select_max_blocks() { return kMaxWords * 32; }

cudaError_t launch_score_select(const Plan& p, int mode, const float* qbar, const float* kbar_t, const float* mv,
                                const float* M_in, float* M_out, int32_t* sel_idx, int32_t* sel_cnt, cudaStream_t s) {
  TileArgs a{};
  a.qbar = qbar; a.kbar_t = kbar_t; a.mv = mv; a.M_in = M_in; a.M_out = M_out;
  a.sel_idx = sel_idx; a.sel_cnt = sel_cnt;
  a.tiles = p.d_sel_tiles; a.rows = p.rows;
  a.Hq = p.cfg.num_q_heads; a.Hkv = p.cfg.num_kv_heads; a.g = a.Hq / a.Hkv;
  a.R_tot = p.R_tot; a.k_max = p.k_max; a.rows_per_tile = p.sel_rows_per_tile;
  a.kt_width = p.kt_width;
  a.list_cap = (p.k_max + kChunk + 31) / 32 * 32;
  a.stem = p.cfg.stem_blocks; a.local = p.cfg.local_blocks;
  a.m_tot = p.m_tot; a.beta = p.cfg.beta; a.score_scale = p.score_scale; a.mode = mode;
  a.nq_slots = (p.sel_nq + 7) / 8 * 8;
  const size_t smem = score_select_fixed_smem() + (size_t)a.nq_slots * score_select_list_bytes(p.k_max);
  if (smem > 227 * 1024 || p.max_nblk > kMaxWords * 32) return cudaErrorInvalidValue;
  // the attribute belongs to the device's context: set it once per device of this process
  static bool attr_set[64] = {};
  const int dev_slot = p.device & 63;
  if (!attr_set[dev_slot]) {
    cudaError_t e = cudaFuncSetAttribute(score_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set[dev_slot] = true;
  }
  const dim3 grid((unsigned)p.n_sel_tiles * (unsigned)a.Hkv);
  score_select_kernel<<<grid, kThreads, smem, s>>>(a);
  return cudaGetLastError();
}

}  // namespace stem
