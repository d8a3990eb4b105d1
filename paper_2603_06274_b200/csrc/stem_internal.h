// Internal declarations shared by the translation units of libstem (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "stem.h"

namespace stem {

constexpr int kHeadDim = 128;

// Status words at the start of the workspace (int32 each).
//   [0] code (0 = ok, 1 = a bounded wait of the attention kernel gave up)   [1] CTA index   [2] role   [3] barrier id
//   [4] code (2 = a bounded wait of the metric kernel gave up)   [5] tile   [6] head
constexpr int kStatusWords = 8;
constexpr int kRoleSelfTest = 99;  // role recorded by stem_selftest_wait_timeout

// Device-side tables, built once per plan.  Query-block rows and key blocks are numbered separately:
// with chunked prefill the queries are a chunk of every sequence (rows r0 .. N_blk - 1 of it) while the
// keys are its whole prefix (blocks 0 .. N_blk - 1); without chunks r0 = 0 and the two coincide.
struct RowTables {
  const int32_t* row_seq;      // [R_tot] sequence of query row R
  const int32_t* row_r;        // [R_tot] row index inside its sequence (global: counts from the sequence's first block)
  const int32_t* row_tok0;     // [R_tot] first token of the row's query block in the packed Q / O
  const int32_t* row_ntok;     // [R_tot] valid tokens in that block (<= B)
  const int32_t* row_keff;     // [R_tot] budget k_eff(r)
  const int32_t* seq_tok0;     // [batch] first token of the sequence in the packed K / V
  const int32_t* seq_nblk;     // [batch] key blocks of the sequence (its prefix, with chunks)
  const int32_t* seq_r0;       // [batch] first row of the query chunk (0 without chunks)
  const int32_t* seq_row_off;  // [batch] query row R of the chunk's first row
  const int32_t* seq_kb_off;   // [batch] pooled-K row of the sequence's block 0
  const int32_t* seq_kb_first; // [batch] index of the sequence's block 0 in kb_tok0 / kb_ntok / kb_dst
  const int64_t* seq_m_off;    // [batch] offset of the sequence inside one head of M ((N_blk - r0) x N_blk entries)
  const int64_t* seq_mt_off;   // [batch] offset of the sequence inside one head of the bit-plane metric
  const int32_t* kb_tok0;      // [n_kb_all] first packed K / V token of every key block (sequence-major)
  const int32_t* kb_ntok;      // [n_kb_all] its valid tokens
  const int32_t* kb_dst;       // [n_kb_all] its pooled-K row
  const int32_t* kb_new;       // [n_kb_new] indices into the three arrays above of the blocks that the chunk adds
};

// Where things live inside the caller's workspace (byte offsets, 256-aligned).
struct WorkspaceLayout {
  size_t status = 0;
  size_t mv = 0;       // fp32 [H_kv, KB_tot]
  size_t qsplit = 0;   // bf16 [3, H_list, R_tot, d]: Qbar as hi + mid + lo parts
  size_t ksplit = 0;   // bf16 [3, H_kv, KB_tot, d]: Kbar likewise
  size_t metric = 0;   // uint32 [H_list, mt_tot]: the metric of the fused path as bit planes of its selection keys
  size_t sel_idx = 0;  // int32 [H_list, R_tot, k_max]
  size_t sel_cnt = 0;  // int32 [H_list, R_tot]
  size_t total = 0;
};

struct Plan {
  stem_config cfg{};
  std::vector<int32_t> cu;  // host copy of cu_seqlens (K / V packing)
  int device = 0;
  int sm_count = 0;
  int32_t T = 0;       // tokens of the packed Q / O
  int32_t T_kv = 0;    // tokens of the packed K / V
  int32_t R_tot = 0;   // query rows
  int32_t KB_tot = 0;  // rows of the pooled K tensors (key blocks; batch x capacity with a caller-owned cache)
  int32_t n_kb_all = 0, n_kb_new = 0;
  int32_t k_max = 0, max_nblk = 0;
  int32_t kcache_blocks = 0;  // per-sequence capacity of a caller-owned pooled-K cache (0: none)
  bool share_group = false;   // one index list per (kv head, row)
  int32_t score_mode = 0;     // 0: product of block means (Eq. 7 on pooled blocks); 1: anti-diagonal scoring
  std::vector<int32_t> h_seq_r0, h_seq_qtok0;  // host copies: first chunk row, first packed Q token of every sequence
  int32_t H_list = 0;         // heads of the metric and of the lists: H_q, or H_kv with share_group
  int64_t m_tot = 0;
  int64_t mt_tot = 0;  // words per head of the bit-plane metric: sum_b rows(b) * roundup(N_blk(b), 32)
  int64_t selected_blocks = 0, causal_blocks = 0, selected_pairs = 0, causal_pairs = 0;
  std::vector<int32_t> k_eff;  // host copy [R_tot]
  float score_scale = 1.f, softmax_scale = 0.f;

  // device blob
  void* d_blob = nullptr;
  RowTables rows{};
  const int32_t* d_gemm_tiles = nullptr;  // [n_gemm_tiles][3] (sequence, row tile, column tile) of the metric GEMM
  int32_t n_gemm_tiles = 0;
  const int32_t* d_work_sparse = nullptr;  // [n_items][2] (head, query row), attention work order
  const int32_t* d_work_dense = nullptr;
  int32_t n_items = 0;

  WorkspaceLayout ws{};
  mutable int last_launches = 0;
};

// Byte offsets inside a caller-owned pooled-K cache: Kbar parts bf16 [3, H_kv, KB_tot, d], then MV fp32 [H_kv, KB_tot].
inline size_t kcache_mv_offset(const Plan& p) {
  return ((size_t)3 * p.cfg.num_kv_heads * p.KB_tot * kHeadDim * 2 + 255) / 256 * 256;
}
inline size_t kcache_bytes(const Plan& p) { return kcache_mv_offset(p) + (size_t)p.cfg.num_kv_heads * p.KB_tot * 4; }

// Kernel launchers (each returns the cudaError_t of the launch).
// Alg. 1 step 1.  Q side (Q != null): Qbar of every query row as hi + mid + lo bf16 parts into qsplit
// [3, H_list, R_tot, d] (the mean over the heads of a kv group as well, with share_group).  K side (K, V != null):
// Kbar parts into ksplit [3, H_kv, KB_tot, d] and MV into mv [H_kv, KB_tot], for every key block of the plan or,
// with only_new, for the blocks the chunk adds.
cudaError_t launch_pool(const Plan& p, const void* Q, const void* K, const void* V, float* mv, void* qsplit, void* ksplit,
                        bool only_new, cudaStream_t s);

// Metric of every causal block (layout of stem_score's M) from the split pooled vectors, on the tensor cores.
// as_keys: instead of the floats, store bit planes of the selection's order-preserving keys: row r of sequence b at
// seq_mt_off[b] + r * roundup(N_blk(b), 32), and in it, for every group of 32 columns, 32 words, word k holding bit k
// of the 32 keys (bit t <-> column 32 * group + t).  What launch_select_planes reads.
// dependent: launch as a programmatic dependent of the kernel enqueued just before (its prologue overlaps that
// kernel's tail).  The caller clears status words 4..7 beforehand.
cudaError_t launch_metric_gemm(const Plan& p, const void* qsplit, const void* ksplit, const float* mv, float* M,
                               bool as_keys, bool dependent, int32_t* status, cudaStream_t s);

// The metric in the anti-diagonal scoring mode, straight from Q and K (mv from the pooling kernel): one tensor-core
// contraction over the full blocks plus, where a sequence ends in a partial block, a small kernel for that row.
// *launched receives the number of kernels enqueued.
int antidiag_max_sequences();
cudaError_t launch_antidiag_metric(const Plan& p, const void* Q, const void* K, const float* mv, float* M, bool as_keys,
                                   int32_t* status, int* launched, cudaStream_t s);

// Selection from a stored metric (layout of stem_score's M), one warp per (head, row).
int row_select_max_blocks();  // largest supported N_blk of a sequence
cudaError_t launch_select_rows(const Plan& p, const float* M, bool dependent, int32_t* sel_idx, int32_t* sel_cnt,
                               cudaStream_t s);
// The same selection from the bit-plane metric launch_metric_gemm(as_keys) wrote.
cudaError_t launch_select_planes(const Plan& p, const uint32_t* Mt, bool dependent, int32_t* sel_idx, int32_t* sel_cnt,
                                 cudaStream_t s);

// list_group: the lists are per kv head ([H_kv, R_tot, k_max]); every query head of a group walks its group's list.
cudaError_t launch_sparse_attention(const Plan& p, const void* Q, const void* K, const void* V,
                                    const int32_t* sel_idx, const int32_t* sel_cnt, bool list_group, void* O, float* lse,
                                    int32_t* status, cudaStream_t s);

// Token-level selection and gather attention (one sequence; lists per kv head).
int token_attn_max_group();
cudaError_t launch_token_select(const float* scores, int N, int H_list, int k_max, const int32_t* k_tok, int stem, int local,
                                int32_t* sel_idx, int32_t* sel_cnt, cudaStream_t s);
cudaError_t launch_token_attention(const void* Q, const void* K, const void* V, int64_t q_st, int64_t q_sh, int64_t kv_st,
                                   int64_t kv_sh, int N, int Hq, int Hkv, int k_max, const int32_t* sel_idx,
                                   const int32_t* sel_cnt, float softmax_scale, void* O, float* lse, cudaStream_t s);
// The status words {4, CTA, role, barrier} of the gather-attention kernel on the current device, read to the host
// and cleared when set (the caller has synchronised).
cudaError_t token_status_words(int32_t* out4);

// One thread waits 1 ms on a barrier nobody arrives at and records the time-out in status words 0..3.
cudaError_t launch_selftest_wait(int32_t* status, cudaStream_t s);

// Status words of the scratch built into the library (stem_score_static) on the current device.
int static_scratch_status_words(int device, int32_t** out);

}  // namespace stem

// The opaque handle of the C ABI.
struct stem_plan {
  stem::Plan p;
};
