// C ABI of libstem: argument checks, the plan (budget schedule, row maps, work orders) and the
// stage sequencing.  All arithmetic of the method on tensors happens in the kernels; the only
// method arithmetic here is the integer budget schedule of Eq. 3.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <numeric>

#include "stem_internal.h"

namespace stem {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Token Position-Decay budget in block units (Eq. 3 with N -> N_blk, i = 1-indexed block row):
//   k_blk(i) = floor(k_s - k_s (1 - mu) i / N_blk), then clamped from below by the forced blocks
//   (stem + local, counted once where they overlap) and min_blocks, and from above by the i
//   causal blocks.  Exact integer arithmetic.
static int32_t budget_row(int64_t i, int64_t n_blk, int64_t k_s, const stem_config& c) {
  const int64_t den = (int64_t)c.mu_den * n_blk;
  const int64_t num = k_s * ((int64_t)c.mu_den * n_blk - (int64_t)(c.mu_den - c.mu_num) * i);
  int64_t k = num / den;
  const int64_t n_stem = std::min<int64_t>(c.stem_blocks, i);
  const int64_t lo_local = std::max<int64_t>(0, i - c.local_blocks);
  int64_t forced = n_stem + (i - lo_local) - std::max<int64_t>(0, n_stem - lo_local);
  k = std::max<int64_t>(k, c.min_blocks);
  k = std::max<int64_t>(k, forced);
  k = std::min<int64_t>(k, i);
  return (int32_t)k;
}

static int validate(const stem_config* c) {
  if (!c || !c->cu_seqlens_host) return STEM_ERR_INVALID_ARG;
  if (c->batch < 1 || c->num_q_heads < 1 || c->num_kv_heads < 1) return STEM_ERR_INVALID_ARG;
  if (c->head_dim != kHeadDim) return STEM_ERR_UNSUPPORTED;
  if (c->block != 64 && c->block != 128) return STEM_ERR_UNSUPPORTED;
  if (c->num_q_heads % c->num_kv_heads != 0) return STEM_ERR_UNSUPPORTED;
  if (c->num_q_heads / c->num_kv_heads > 32) return STEM_ERR_UNSUPPORTED;
  if (c->mu_den <= 0 || c->mu_num <= 0 || c->mu_num > c->mu_den) return STEM_ERR_INVALID_ARG;
  if (c->stem_blocks < 0 || c->local_blocks < 1 || c->min_blocks < 0) return STEM_ERR_INVALID_ARG;
  if (c->k_start_blocks < 0 || c->budget_permille < 0 || c->budget_permille > 1000) return STEM_ERR_INVALID_ARG;
  if (c->k_start_blocks == 0 && c->budget_permille == 0 && c->min_blocks == 0 && c->stem_blocks + c->local_blocks == 0)
    return STEM_ERR_INVALID_ARG;
  if (!(c->beta == c->beta) || !(c->score_scale == c->score_scale) || !(c->softmax_scale == c->softmax_scale))
    return STEM_ERR_INVALID_ARG;
  if (c->softmax_scale < 0.f) return STEM_ERR_INVALID_ARG;
  if (c->q_stride_tok % 8 || c->q_stride_head % 8 || c->kv_stride_tok % 8 || c->kv_stride_head % 8)
    return STEM_ERR_INVALID_ARG;
  if (c->q_stride_head < kHeadDim || c->kv_stride_head < kHeadDim) return STEM_ERR_INVALID_ARG;
  if (c->q_stride_tok < kHeadDim || c->kv_stride_tok < kHeadDim) return STEM_ERR_INVALID_ARG;
  if (c->cu_seqlens_host[0] != 0) return STEM_ERR_INVALID_ARG;
  for (int b = 0; b < c->batch; ++b)
    if (c->cu_seqlens_host[b + 1] <= c->cu_seqlens_host[b]) return STEM_ERR_INVALID_ARG;
  return STEM_OK;
}

template <class T>
static size_t push(std::vector<uint8_t>& blob, const std::vector<T>& v) {
  size_t off = align_up(blob.size(), 256);
  blob.resize(off + std::max<size_t>(v.size() * sizeof(T), 1));
  if (!v.empty()) std::memcpy(blob.data() + off, v.data(), v.size() * sizeof(T));
  return off;
}

// Frees everything a plan owns (also a half-built one).
static void release_plan(stem_plan* sp) {
  Plan& p = sp->p;
  if (p.d_blob) cudaFree(p.d_blob);
  delete sp;
}

}  // namespace stem

using namespace stem;

extern "C" {

int stem_version(void) { return 100; }

const char* stem_status_string(int s) {
  switch (s) {
    case STEM_OK: return "ok";
    case STEM_ERR_INVALID_ARG: return "invalid argument";
    case STEM_ERR_UNSUPPORTED: return "unsupported configuration";
    case STEM_ERR_WORKSPACE: return "workspace missing or too small";
    case STEM_ERR_CUDA: return "CUDA error";
    case STEM_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait gave up";
    case STEM_ERR_STATIC_SCRATCH: return "problem exceeds the built-in scratch of the allocation-free entry point";
    default: return "unknown status";
  }
}

int stem_plan_create(const stem_config* cfg, stem_plan** out) { return stem_plan_create_ex(cfg, nullptr, out); }

int stem_plan_create_ex(const stem_config* cfg, const stem_options* opts, stem_plan** out) {
  if (!out) return STEM_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = validate(cfg);
  if (rc != STEM_OK) return rc;
  stem_options o{};
  if (opts) o = *opts;
  for (int i = 0; i < 3; ++i)
    if (o.reserved[i] != 0) return STEM_ERR_INVALID_ARG;
  if (o.kcache_blocks_per_seq < 0 || (o.share_group != 0 && o.share_group != 1)) return STEM_ERR_INVALID_ARG;
  if (o.score_mode != 0 && o.score_mode != 1) return STEM_ERR_INVALID_ARG;
  // anti-diagonal scoring contracts Q with K directly: no pooled-K cache to read instead, one list per query head,
  // and one tensor map per sequence (a bounded number of them ride in the kernel's parameters)
  if (o.score_mode == 1 && (o.kcache_blocks_per_seq > 0 || o.share_group != 0 || cfg->batch > antidiag_max_sequences()))
    return STEM_ERR_UNSUPPORTED;
  const int B = cfg->block, batch = cfg->batch, Hq = cfg->num_q_heads, Hkv = cfg->num_kv_heads;
  for (int b = 0; b < batch; ++b) {
    const int64_t kv_len = cfg->cu_seqlens_host[b + 1] - cfg->cu_seqlens_host[b];
    const int64_t q0 = o.q_start_host ? o.q_start_host[b] : 0;
    const int64_t tot = o.total_len_host ? o.total_len_host[b] : kv_len;
    if (q0 < 0 || q0 >= kv_len || q0 % B != 0 || tot < kv_len) return STEM_ERR_INVALID_ARG;
    if (o.kcache_blocks_per_seq > 0 && (kv_len + B - 1) / B > o.kcache_blocks_per_seq) return STEM_ERR_INVALID_ARG;
  }

  stem_plan* sp = new (std::nothrow) stem_plan();
  if (!sp) return STEM_ERR_CUDA;
  Plan& p = sp->p;
  p.cfg = *cfg;
  p.cu.assign(cfg->cu_seqlens_host, cfg->cu_seqlens_host + cfg->batch + 1);
  p.cfg.cu_seqlens_host = nullptr;
  p.score_scale = cfg->score_scale == 0.f ? 1.f : cfg->score_scale;
  p.softmax_scale = cfg->softmax_scale == 0.f ? 1.f / std::sqrt((float)kHeadDim) : cfg->softmax_scale;
  p.kcache_blocks = o.kcache_blocks_per_seq;
  p.share_group = o.share_group != 0;
  p.score_mode = o.score_mode;
  p.H_list = p.share_group ? Hkv : Hq;

  const int g = Hq / Hkv;
  p.T_kv = p.cu[batch];

  std::vector<int32_t> row_seq, row_r, row_tok0, row_ntok, seq_tok0(batch), seq_nblk(batch), seq_r0(batch),
      seq_row_off(batch), seq_kb_off(batch), seq_kb_first(batch), kb_tok0, kb_ntok, kb_dst, kb_new;
  std::vector<int64_t> seq_m_off(batch), seq_mt_off(batch);
  int64_t m_off = 0, mt_off = 0;
  int32_t q_tok = 0, kb_off = 0;
  for (int b = 0; b < batch; ++b) {
    const int32_t n = p.cu[b + 1] - p.cu[b];           // tokens of the K / V prefix
    const int32_t nb = (n + B - 1) / B;                // its blocks
    const int32_t q0 = o.q_start_host ? o.q_start_host[b] : 0;
    const int32_t r0 = q0 / B;
    const int64_t n_tot = o.total_len_host ? o.total_len_host[b] : n;
    const int64_t nb_tot = (n_tot + B - 1) / B;        // blocks of the whole sequence: N of Eq. 3
    seq_tok0[b] = p.cu[b];
    seq_nblk[b] = nb;
    seq_r0[b] = r0;
    seq_row_off[b] = (int32_t)row_seq.size();
    seq_kb_off[b] = p.kcache_blocks > 0 ? b * p.kcache_blocks : kb_off;
    seq_kb_first[b] = (int32_t)kb_tok0.size();
    p.h_seq_r0.push_back(r0);
    p.h_seq_qtok0.push_back(q_tok);
    seq_m_off[b] = m_off;
    seq_mt_off[b] = mt_off;
    mt_off += (int64_t)(nb - r0) * ((nb + 31) / 32 * 32);  // rows padded to whole 32-column groups
    m_off += (int64_t)(nb - r0) * nb;
    p.max_nblk = std::max(p.max_nblk, nb);
    const int64_t k_s = cfg->k_start_blocks > 0 ? cfg->k_start_blocks : ((int64_t)cfg->budget_permille * nb_tot) / 1000;
    for (int32_t j = 0; j < nb; ++j) {
      if (j >= r0) kb_new.push_back((int32_t)kb_tok0.size());
      kb_tok0.push_back(p.cu[b] + j * B);
      kb_ntok.push_back(std::min(B, n - j * B));
      kb_dst.push_back(seq_kb_off[b] + j);
    }
    for (int32_t r = r0; r < nb; ++r) {
      row_seq.push_back(b);
      row_r.push_back(r);
      row_tok0.push_back(q_tok + (r - r0) * B);
      const int32_t ntok = std::min(B, n - r * B);
      row_ntok.push_back(ntok);
      const int32_t ke = budget_row(r + 1, nb_tot, k_s, *cfg);
      p.k_eff.push_back(ke);
      p.k_max = std::max(p.k_max, ke);
      const int64_t diag = (int64_t)ntok * (ntok + 1) / 2;
      p.selected_blocks += ke;
      p.causal_blocks += r + 1;
      p.selected_pairs += (int64_t)(ke - 1) * ntok * B + diag;
      p.causal_pairs += (int64_t)r * ntok * B + diag;
    }
    q_tok += n - q0;
    kb_off += nb;
  }
  p.T = q_tok;
  p.R_tot = (int32_t)row_seq.size();
  p.n_kb_all = (int32_t)kb_tok0.size();
  p.n_kb_new = (int32_t)kb_new.size();
  p.KB_tot = p.kcache_blocks > 0 ? batch * p.kcache_blocks : kb_off;
  p.m_tot = m_off;
  p.mt_tot = mt_off;
  p.selected_blocks *= Hq;
  p.causal_blocks *= Hq;
  p.selected_pairs *= Hq;
  p.causal_pairs *= Hq;

  if (p.max_nblk > row_select_max_blocks()) {
    delete sp;
    return STEM_ERR_UNSUPPORTED;
  }

  // Tiles of the metric GEMM: 128 query rows x 128 key blocks, the tiles of every sequence that hold a causal
  // entry (j <= r for some row of the tile), long rows first.
  std::vector<int32_t> gemm_tiles;
  {
    int max_t = 0;
    for (int b = 0; b < batch; ++b) max_t = std::max(max_t, (seq_nblk[b] - seq_r0[b] + 127) / 128);
    for (int ti = max_t - 1; ti >= 0; --ti)
      for (int b = 0; b < batch; ++b) {
        const int rows_b = seq_nblk[b] - seq_r0[b];
        if (ti >= (rows_b + 127) / 128) continue;
        const int r_last = seq_r0[b] + std::min(rows_b, (ti + 1) * 128) - 1;  // largest global row of the tile
        for (int tj = 0; tj <= r_last / 128; ++tj) { gemm_tiles.push_back(b); gemm_tiles.push_back(ti); gemm_tiles.push_back(tj); }
      }
    p.n_gemm_tiles = (int32_t)(gemm_tiles.size() / 3);
  }

  // Attention work order: kv-head-major so that the K/V of one kv head stay hot in L2; inside a
  // kv head, rows by descending list length (longest first), the g heads of a row together.
  std::vector<int32_t> work_sparse, work_dense;
  {
    std::vector<int32_t> by_len(p.R_tot), by_r(p.R_tot);
    std::iota(by_len.begin(), by_len.end(), 0);
    std::iota(by_r.begin(), by_r.end(), 0);
    std::stable_sort(by_len.begin(), by_len.end(), [&](int a, int b) { return p.k_eff[a] > p.k_eff[b]; });
    std::stable_sort(by_r.begin(), by_r.end(), [&](int a, int b) { return row_r[a] > row_r[b]; });
    for (int kvh = 0; kvh < Hkv; ++kvh) {
      for (int32_t R : by_len)
        for (int q = 0; q < g; ++q) { work_sparse.push_back(kvh * g + q); work_sparse.push_back(R); }
      for (int32_t R : by_r)
        for (int q = 0; q < g; ++q) { work_dense.push_back(kvh * g + q); work_dense.push_back(R); }
    }
    p.n_items = p.R_tot * Hq;
  }

  // Workspace layout.  With a caller-owned cache the K-side tensors are not part of the workspace.
  {
    const bool own_k = p.kcache_blocks == 0;
    size_t off = 0;
    p.ws.status = off; off = align_up(off + kStatusWords * 4, 256);
    p.ws.mv = off;     off = align_up(off + (own_k ? (size_t)Hkv * p.KB_tot * 4 : 0), 256);
    p.ws.qsplit = off; off = align_up(off + (size_t)3 * p.H_list * p.R_tot * kHeadDim * 2, 256);
    p.ws.ksplit = off; off = align_up(off + (own_k ? (size_t)3 * Hkv * p.KB_tot * kHeadDim * 2 : 0), 256);
    p.ws.metric = off; off = align_up(off + (size_t)p.H_list * (size_t)p.mt_tot * 4, 256);
    p.ws.sel_idx = off; off = align_up(off + (size_t)p.H_list * p.R_tot * p.k_max * 4, 256);
    p.ws.sel_cnt = off; off = align_up(off + (size_t)p.H_list * p.R_tot * 4, 256);
    p.ws.total = off;
  }

  // Upload tables.
  if (cudaGetDevice(&p.device) != cudaSuccess ||
      cudaDeviceGetAttribute(&p.sm_count, cudaDevAttrMultiProcessorCount, p.device) != cudaSuccess) {
    cudaGetLastError();
    delete sp;
    return STEM_ERR_CUDA;
  }
  std::vector<uint8_t> blob;
  const size_t o_row_seq = push(blob, row_seq), o_row_r = push(blob, row_r), o_row_tok0 = push(blob, row_tok0),
               o_row_ntok = push(blob, row_ntok), o_keff = push(blob, p.k_eff), o_seq_tok0 = push(blob, seq_tok0),
               o_seq_nblk = push(blob, seq_nblk), o_seq_r0 = push(blob, seq_r0), o_seq_row_off = push(blob, seq_row_off),
               o_seq_kb_off = push(blob, seq_kb_off), o_seq_kb_first = push(blob, seq_kb_first), o_seq_m_off = push(blob, seq_m_off),
               o_seq_mt_off = push(blob, seq_mt_off), o_kb_tok0 = push(blob, kb_tok0), o_kb_ntok = push(blob, kb_ntok),
               o_kb_dst = push(blob, kb_dst), o_kb_new = push(blob, kb_new), o_gt = push(blob, gemm_tiles),
               o_ws = push(blob, work_sparse), o_wd = push(blob, work_dense);
  if (cudaMalloc(&p.d_blob, blob.size()) != cudaSuccess ||
      cudaMemcpy(p.d_blob, blob.data(), blob.size(), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    if (p.d_blob) cudaFree(p.d_blob);
    delete sp;
    return STEM_ERR_CUDA;
  }
  const uint8_t* d = (const uint8_t*)p.d_blob;
  p.rows.row_seq = (const int32_t*)(d + o_row_seq);
  p.rows.row_r = (const int32_t*)(d + o_row_r);
  p.rows.row_tok0 = (const int32_t*)(d + o_row_tok0);
  p.rows.row_ntok = (const int32_t*)(d + o_row_ntok);
  p.rows.row_keff = (const int32_t*)(d + o_keff);
  p.rows.seq_tok0 = (const int32_t*)(d + o_seq_tok0);
  p.rows.seq_nblk = (const int32_t*)(d + o_seq_nblk);
  p.rows.seq_r0 = (const int32_t*)(d + o_seq_r0);
  p.rows.seq_row_off = (const int32_t*)(d + o_seq_row_off);
  p.rows.seq_kb_off = (const int32_t*)(d + o_seq_kb_off);
  p.rows.seq_kb_first = (const int32_t*)(d + o_seq_kb_first);
  p.rows.seq_m_off = (const int64_t*)(d + o_seq_m_off);
  p.rows.seq_mt_off = (const int64_t*)(d + o_seq_mt_off);
  p.rows.kb_tok0 = (const int32_t*)(d + o_kb_tok0);
  p.rows.kb_ntok = (const int32_t*)(d + o_kb_ntok);
  p.rows.kb_dst = (const int32_t*)(d + o_kb_dst);
  p.rows.kb_new = (const int32_t*)(d + o_kb_new);
  p.d_gemm_tiles = (const int32_t*)(d + o_gt);
  p.d_work_sparse = (const int32_t*)(d + o_ws);
  p.d_work_dense = (const int32_t*)(d + o_wd);
  *out = sp;
  return STEM_OK;
}

int stem_plan_destroy(stem_plan* plan) {
  if (!plan) return STEM_ERR_INVALID_ARG;
  release_plan(plan);
  return STEM_OK;
}

int stem_plan_query(const stem_plan* plan, stem_plan_info* info) {
  if (!plan || !info) return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  info->workspace_bytes = p.ws.total;
  info->total_tokens = p.T;
  info->total_q_blocks = p.R_tot;
  info->k_max = p.k_max;
  info->metric_elems = p.m_tot;
  info->selected_blocks = p.selected_blocks;
  info->causal_blocks = p.causal_blocks;
  info->selected_pairs = p.selected_pairs;
  info->causal_pairs = p.causal_pairs;
  info->total_kv_tokens = p.T_kv;
  info->list_heads = p.H_list;
  info->kcache_bytes = p.kcache_blocks > 0 ? kcache_bytes(p) : 0;
  info->total_key_blocks = p.n_kb_all;
  info->new_key_blocks = p.n_kb_new;
  return STEM_OK;
}

int stem_plan_budget(const stem_plan* plan, int32_t* k_eff_host) {
  if (!plan || !k_eff_host) return STEM_ERR_INVALID_ARG;
  std::memcpy(k_eff_host, plan->p.k_eff.data(), plan->p.k_eff.size() * sizeof(int32_t));
  return STEM_OK;
}

int stem_budget_table(const stem_config* cfg, int32_t* k_eff_host, int64_t capacity, int32_t* r_tot) {
  int rc = validate(cfg);
  if (rc != STEM_OK) return rc;
  int64_t R = 0;
  for (int b = 0; b < cfg->batch; ++b) {
    const int64_t n = cfg->cu_seqlens_host[b + 1] - cfg->cu_seqlens_host[b];
    const int64_t nb = (n + cfg->block - 1) / cfg->block;
    const int64_t k_s = cfg->k_start_blocks > 0 ? cfg->k_start_blocks : ((int64_t)cfg->budget_permille * nb) / 1000;
    for (int64_t r = 0; r < nb; ++r, ++R)
      if (k_eff_host) {
        if (R >= capacity) return STEM_ERR_INVALID_ARG;
        k_eff_host[R] = budget_row(r + 1, nb, k_s, *cfg);
      }
  }
  if (r_tot) *r_tot = (int32_t)R;
  return STEM_OK;
}

int stem_last_launch_count(const stem_plan* plan) { return plan ? plan->p.last_launches : 0; }

static bool misaligned(const void* p) { return ((uintptr_t)p & 15) != 0; }

static int check_ws(const Plan& p, const void* ws, size_t bytes) {
  if (!ws || bytes < p.ws.total) return STEM_ERR_WORKSPACE;
  if (((uintptr_t)ws & 255) != 0) return STEM_ERR_INVALID_ARG;
  return STEM_OK;
}

static int cuda_rc(cudaError_t e) { return e == cudaSuccess ? STEM_OK : STEM_ERR_CUDA; }

// Where the K-side tensors of step 1 live: in the workspace, or in the caller's pooled-K cache.
struct KSide {
  void* ksplit;
  float* mv;
};
static KSide k_side(const Plan& p, uint8_t* w, void* kcache) {
  if (kcache) return {kcache, (float*)((uint8_t*)kcache + kcache_mv_offset(p))};
  return {w + p.ws.ksplit, (float*)(w + p.ws.mv)};
}

// Alg. 1 step 3a from what step 1 left: the product of block means on the pooled vectors, or, in the anti-diagonal
// scoring mode, the contraction of Q with K itself (MV comes from the pooling kernel in both).
static int enqueue_metric(const Plan& p, const void* Q, const void* K, uint8_t* w, const KSide& ks, float* M, bool as_keys,
                          bool dependent, cudaStream_t s) {
  int32_t* status = (int32_t*)(w + p.ws.status);
  if (p.score_mode == 1) {
    int launched = 0;
    const int rc = cuda_rc(launch_antidiag_metric(p, Q, K, ks.mv, M, as_keys, status, &launched, s));
    p.last_launches += launched;
    return rc;
  }
  const int rc = cuda_rc(launch_metric_gemm(p, w + p.ws.qsplit, ks.ksplit, ks.mv, M, as_keys, dependent, status, s));
  if (rc == STEM_OK) p.last_launches++;
  return rc;
}

// Alg. 1 steps 1-3c on one stream: pooling (one pass over Q and, unless the K side comes from a cache, over K
// and V; emits the pooled vectors as bf16 parts), the metric of every causal block on the tensor cores into
// the workspace (stored as bit planes of the selection's order-preserving keys), and the row-wise selection
// from it.  (Two ways of overlapping the HBM-bound pooling with the scoring were measured and dropped: phases
// on two streams lose more to cross-stream event waits than they gain, and one persistent kernel
// with a shared ticket list leaves too few warps per SM to stream HBM.)
static int enqueue_score_select(const Plan& p, const void* Q, const void* K, const void* V, void* kcache, uint8_t* w,
                                int32_t* idx, int32_t* cnt, cudaStream_t s) {
  const KSide ks = k_side(p, w, kcache);
  float* M = (float*)(w + p.ws.metric);  // holds the bit planes of the selection keys, not the floats
  int rc = cuda_rc(cudaMemsetAsync(w + p.ws.status + 16, 0, 16, s));  // the metric kernel's status words
  if (rc != STEM_OK) return rc;
  // (the anti-diagonal mode has no use for the pooled query vectors)
  rc = cuda_rc(launch_pool(p, p.score_mode == 1 ? nullptr : Q, K, V, ks.mv, w + p.ws.qsplit, ks.ksplit, false, s));
  if (rc != STEM_OK) return rc;
  p.last_launches++;
  rc = enqueue_metric(p, Q, K, w, ks, M, true, true, s);
  if (rc != STEM_OK) return rc;
  rc = cuda_rc(launch_select_planes(p, (const uint32_t*)M, p.score_mode != 1, idx, cnt, s));
  if (rc == STEM_OK) p.last_launches++;
  return rc;
}

int stem_score(const stem_plan* plan, const void* Q, const void* K, const void* V, float* M, void* ws, size_t ws_bytes,
               void* stream) {
  if (!plan || !Q || !K || !V) return STEM_ERR_INVALID_ARG;
  if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(M)) return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  if (p.kcache_blocks > 0) return STEM_ERR_INVALID_ARG;  // the K side of such a plan lives in the caller's cache
  int rc = check_ws(p, ws, ws_bytes);
  if (rc != STEM_OK) return rc;
  uint8_t* w = (uint8_t*)ws;
  cudaStream_t s = (cudaStream_t)stream;
  p.last_launches = 0;
  float* mv = (float*)(w + p.ws.mv);
  rc = cuda_rc(cudaMemsetAsync(w + p.ws.status + 16, 0, 16, s));  // the metric kernel's status words
  if (rc != STEM_OK) return rc;
  rc = cuda_rc(launch_pool(p, p.score_mode == 1 ? nullptr : Q, K, V, mv, w + p.ws.qsplit, w + p.ws.ksplit, false, s));
  if (rc != STEM_OK) return rc;
  p.last_launches++;
  if (M) rc = enqueue_metric(p, Q, K, w, k_side(p, w, nullptr), M, false, true, s);
  return rc;
}

int stem_select(const stem_plan* plan, const float* M, int32_t* sel_idx, int32_t* sel_cnt, void* ws, size_t ws_bytes,
                void* stream) {
  if (!plan || !sel_idx || !sel_cnt) return STEM_ERR_INVALID_ARG;
  if (misaligned(M) || ((uintptr_t)sel_idx & 3) || ((uintptr_t)sel_cnt & 3)) return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  if (!M && (p.kcache_blocks > 0 || p.score_mode == 1)) return STEM_ERR_INVALID_ARG;  // nothing pooled to recompute M from
  int rc = check_ws(p, ws, ws_bytes);
  if (rc != STEM_OK) return rc;
  uint8_t* w = (uint8_t*)ws;
  p.last_launches = 0;
  cudaStream_t s = (cudaStream_t)stream;
  if (!M) {
    // recompute the metric (as selection keys) from the pooled vectors a previous stem_score left in the workspace
    float* Mw = (float*)(w + p.ws.metric);
    rc = cuda_rc(cudaMemsetAsync(w + p.ws.status + 16, 0, 16, s));  // the metric kernel's status words
    if (rc != STEM_OK) return rc;
    rc = cuda_rc(launch_metric_gemm(p, w + p.ws.qsplit, w + p.ws.ksplit, (const float*)(w + p.ws.mv), Mw, true, false,
                                    (int32_t*)(w + p.ws.status), s));
    if (rc != STEM_OK) return rc;
    p.last_launches++;
    rc = cuda_rc(launch_select_planes(p, (const uint32_t*)Mw, true, sel_idx, sel_cnt, s));
  } else {
    rc = cuda_rc(launch_select_rows(p, M, false, sel_idx, sel_cnt, s));
  }
  if (rc == STEM_OK) p.last_launches++;
  return rc;
}

int stem_score_select(const stem_plan* plan, const void* Q, const void* K, const void* V, int32_t* sel_idx,
                      int32_t* sel_cnt, void* ws, size_t ws_bytes, void* stream) {
  if (!plan || !Q || !K || !V || !sel_idx || !sel_cnt) return STEM_ERR_INVALID_ARG;
  if (misaligned(Q) || misaligned(K) || misaligned(V) || ((uintptr_t)sel_idx & 3) || ((uintptr_t)sel_cnt & 3))
    return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  if (p.kcache_blocks > 0) return STEM_ERR_INVALID_ARG;
  int rc = check_ws(p, ws, ws_bytes);
  if (rc != STEM_OK) return rc;
  uint8_t* w = (uint8_t*)ws;
  p.last_launches = 0;
  return enqueue_score_select(p, Q, K, V, nullptr, w, sel_idx, sel_cnt, (cudaStream_t)stream);
}

int stem_pool_kv(const stem_plan* plan, const void* K, const void* V, void* kcache, void* stream) {
  if (!plan || !K || !V || !kcache) return STEM_ERR_INVALID_ARG;
  if (misaligned(K) || misaligned(V) || ((uintptr_t)kcache & 255)) return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  if (p.kcache_blocks == 0) return STEM_ERR_INVALID_ARG;
  const KSide ks = k_side(p, nullptr, kcache);
  p.last_launches = 0;
  const int rc = cuda_rc(launch_pool(p, nullptr, K, V, ks.mv, nullptr, ks.ksplit, true, (cudaStream_t)stream));
  if (rc == STEM_OK) p.last_launches++;
  return rc;
}

int stem_score_select_cached(const stem_plan* plan, const void* Q, const void* kcache, int32_t* sel_idx, int32_t* sel_cnt,
                             void* ws, size_t ws_bytes, void* stream) {
  if (!plan || !Q || !kcache || !sel_idx || !sel_cnt) return STEM_ERR_INVALID_ARG;
  if (misaligned(Q) || ((uintptr_t)kcache & 255) || ((uintptr_t)sel_idx & 3) || ((uintptr_t)sel_cnt & 3))
    return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  if (p.kcache_blocks == 0) return STEM_ERR_INVALID_ARG;
  int rc = check_ws(p, ws, ws_bytes);
  if (rc != STEM_OK) return rc;
  p.last_launches = 0;
  return enqueue_score_select(p, Q, nullptr, nullptr, const_cast<void*>(kcache), (uint8_t*)ws, sel_idx, sel_cnt,
                              (cudaStream_t)stream);
}

int stem_sparse_prefill(const stem_plan* plan, const void* Q, const void* K, const void* V, const int32_t* sel_idx,
                        const int32_t* sel_cnt, void* O, float* lse, void* ws, size_t ws_bytes, void* stream) {
  if (!plan || !Q || !K || !V || !O) return STEM_ERR_INVALID_ARG;
  if ((sel_idx == nullptr) != (sel_cnt == nullptr)) return STEM_ERR_INVALID_ARG;
  if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(O)) return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  int rc = check_ws(p, ws, ws_bytes);
  if (rc != STEM_OK) return rc;
  p.last_launches = 0;
  rc = cuda_rc(launch_sparse_attention(p, Q, K, V, sel_idx, sel_cnt, p.share_group, O, lse,
                                       (int32_t*)((uint8_t*)ws + p.ws.status), (cudaStream_t)stream));
  if (rc == STEM_OK) p.last_launches++;
  return rc;
}

// Alg. 1 on one stream: steps 1-3c, then step 3d on the lists they wrote.
static int enqueue_prefill(const Plan& p, const void* Q, const void* K, const void* V, void* O, void* kcache,
                           bool update_cache, int32_t* sel_idx, int32_t* sel_cnt, float* lse, uint8_t* w, cudaStream_t s) {
  int32_t* idx = sel_idx ? sel_idx : (int32_t*)(w + p.ws.sel_idx);
  int32_t* cnt = sel_cnt ? sel_cnt : (int32_t*)(w + p.ws.sel_cnt);
  p.last_launches = 0;
  int rc = STEM_OK;
  if (kcache && update_cache) {
    const KSide ks = k_side(p, w, kcache);
    rc = cuda_rc(launch_pool(p, nullptr, K, V, ks.mv, nullptr, ks.ksplit, true, s));
    if (rc != STEM_OK) return rc;
    p.last_launches++;
  }
  rc = enqueue_score_select(p, Q, kcache ? nullptr : K, kcache ? nullptr : V, kcache, w, idx, cnt, s);
  if (rc != STEM_OK) return rc;
  rc = cuda_rc(launch_sparse_attention(p, Q, K, V, idx, cnt, p.share_group, O, lse, (int32_t*)(w + p.ws.status), s));
  if (rc != STEM_OK) return rc;
  p.last_launches++;
  return STEM_OK;
}

int stem_prefill(const stem_plan* plan, const void* Q, const void* K, const void* V, void* O, int32_t* sel_idx,
                 int32_t* sel_cnt, float* lse, void* ws, size_t ws_bytes, void* stream) {
  if (!plan || !Q || !K || !V || !O) return STEM_ERR_INVALID_ARG;
  if ((sel_idx == nullptr) != (sel_cnt == nullptr)) return STEM_ERR_INVALID_ARG;
  if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(O)) return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  if (p.kcache_blocks > 0) return STEM_ERR_INVALID_ARG;
  int rc = check_ws(p, ws, ws_bytes);
  if (rc != STEM_OK) return rc;
  return enqueue_prefill(p, Q, K, V, O, nullptr, false, sel_idx, sel_cnt, lse, (uint8_t*)ws, (cudaStream_t)stream);
}

int stem_prefill_cached(const stem_plan* plan, const void* Q, const void* K, const void* V, void* O, void* kcache,
                        int update_cache, int32_t* sel_idx, int32_t* sel_cnt, float* lse, void* ws, size_t ws_bytes,
                        void* stream) {
  if (!plan || !Q || !K || !V || !O || !kcache) return STEM_ERR_INVALID_ARG;
  if ((sel_idx == nullptr) != (sel_cnt == nullptr)) return STEM_ERR_INVALID_ARG;
  if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(O) || ((uintptr_t)kcache & 255)) return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  if (p.kcache_blocks == 0) return STEM_ERR_INVALID_ARG;
  int rc = check_ws(p, ws, ws_bytes);
  if (rc != STEM_OK) return rc;
  return enqueue_prefill(p, Q, K, V, O, kcache, update_cache != 0, sel_idx, sel_cnt, lse, (uint8_t*)ws, (cudaStream_t)stream);
}

int stem_token_budget(int32_t n_tokens, int32_t k_start, int32_t mu_num, int32_t mu_den, int32_t stem_tokens,
                      int32_t local_tokens, int32_t* k_host) {
  if (n_tokens < 1 || k_start < 0 || mu_den <= 0 || mu_num <= 0 || mu_num > mu_den || stem_tokens < 0 || local_tokens < 1 || !k_host)
    return STEM_ERR_INVALID_ARG;
  stem_config c{};
  c.mu_num = mu_num; c.mu_den = mu_den; c.stem_blocks = stem_tokens; c.local_blocks = local_tokens; c.min_blocks = 0;
  for (int64_t t = 0; t < n_tokens; ++t) k_host[t] = budget_row(t + 1, n_tokens, k_start, c);  // Eq. 3 with one token per "block"
  return STEM_OK;
}

int stem_token_select(const float* scores, int32_t n_tokens, int32_t list_heads, const int32_t* k_tok, int32_t stem_tokens,
                      int32_t local_tokens, int32_t k_max, int32_t* sel_idx, int32_t* sel_cnt, void* stream) {
  if (!scores || !k_tok || !sel_idx || !sel_cnt) return STEM_ERR_INVALID_ARG;
  if (n_tokens < 1 || list_heads < 1 || list_heads > 65535 || k_max < 1 || stem_tokens < 0 || local_tokens < 1) return STEM_ERR_INVALID_ARG;
  return cuda_rc(launch_token_select(scores, n_tokens, list_heads, k_max, k_tok, stem_tokens, local_tokens, sel_idx, sel_cnt,
                                     (cudaStream_t)stream));
}

int stem_token_attention(const void* Q, const void* K, const void* V, int32_t n_tokens, int32_t num_q_heads,
                         int32_t num_kv_heads, int64_t q_stride_tok, int64_t q_stride_head, int64_t kv_stride_tok,
                         int64_t kv_stride_head, const int32_t* sel_idx, const int32_t* sel_cnt, int32_t k_max,
                         float softmax_scale, void* O, float* lse, void* stream) {
  if (!Q || !K || !V || !O || !sel_idx || !sel_cnt) return STEM_ERR_INVALID_ARG;
  if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(O)) return STEM_ERR_INVALID_ARG;
  if (n_tokens < 1 || num_q_heads < 1 || num_kv_heads < 1 || num_kv_heads > 65535 || k_max < 1) return STEM_ERR_INVALID_ARG;
  if (num_q_heads % num_kv_heads != 0 || num_q_heads / num_kv_heads > token_attn_max_group()) return STEM_ERR_UNSUPPORTED;
  if ((int64_t)n_tokens * num_kv_heads > 0x7fffffffLL) return STEM_ERR_UNSUPPORTED;  // work items are counted in 32 bits
  if (q_stride_tok % 8 || q_stride_head % 8 || kv_stride_tok % 8 || kv_stride_head % 8) return STEM_ERR_INVALID_ARG;
  if (q_stride_head < kHeadDim || kv_stride_head < kHeadDim) return STEM_ERR_INVALID_ARG;
  if (!(softmax_scale >= 0.f)) return STEM_ERR_INVALID_ARG;
  const float scale = softmax_scale == 0.f ? 1.f / std::sqrt((float)kHeadDim) : softmax_scale;
  return cuda_rc(launch_token_attention(Q, K, V, q_stride_tok, q_stride_head, kv_stride_tok, kv_stride_head, n_tokens, num_q_heads,
                                        num_kv_heads, k_max, sel_idx, sel_cnt, scale, O, lse, (cudaStream_t)stream));
}

int stem_token_check_status(void* stream, int32_t* detail) {
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_CUDA; }
  int32_t words[4] = {0, 0, 0, 0};
  if (token_status_words(words) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_CUDA; }
  if (detail) std::memcpy(detail, words, sizeof(words));
  return words[0] != 0 ? STEM_ERR_DEVICE_TIMEOUT : STEM_OK;
}

int stem_check_status(const stem_plan* plan, void* ws, void* stream, int32_t* detail) {
  if (!plan) return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  cudaStream_t s = (cudaStream_t)stream;
  int32_t words[kStatusWords] = {0};
  uint8_t* w = nullptr;
  if (ws) {
    w = (uint8_t*)ws + p.ws.status;
  } else {
    // no workspace: the status words of the scratch built into the library (stem_score_static)
    int device = -1;
    int32_t* st = nullptr;
    if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_CUDA; }
    const int rc = static_scratch_status_words(device, &st);
    if (rc != STEM_OK) return rc;
    w = (uint8_t*)st;
  }
  if (cudaStreamSynchronize(s) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_CUDA; }
  if (cudaMemcpy(words, w, sizeof(words), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_CUDA; }
  if (detail) std::memcpy(detail, words, 4 * sizeof(int32_t));
  if (words[0] != 0 || words[4] != 0) {
    if (detail && words[0] == 0) std::memcpy(detail, words + 4, 4 * sizeof(int32_t));  // the metric kernel's words
    cudaMemset(w, 0, sizeof(words));
    return STEM_ERR_DEVICE_TIMEOUT;
  }
  return STEM_OK;
}

int stem_selftest_wait_timeout(const stem_plan* plan, void* ws, size_t ws_bytes, void* stream) {
  if (!plan) return STEM_ERR_INVALID_ARG;
  const Plan& p = plan->p;
  const int rc = check_ws(p, ws, ws_bytes);
  if (rc != STEM_OK) return rc;
  return cuda_rc(launch_selftest_wait((int32_t*)((uint8_t*)ws + p.ws.status), (cudaStream_t)stream));
}

}  // extern "C"
