/*
 * stem.h - C ABI of the Stem sparse causal prefill attention library for NVIDIA B200 (sm_100a).
 *
 * The library implements the hot path of Algorithm 1 of "Stem" (arxiv 2603.06274):
 *
 *   stem_score           Alg. 1 step 1 (block pooling of Q and K, max-pooled value magnitude)
 *                        and step 3a (Output-Aware Metric, Eq. 7) on pooled blocks
 *   stem_select          Alg. 1 steps 3b-3c: Token Position-Decay budget (Eq. 3, block units)
 *                        and per-row top-k with the forced stem / local blocks
 *   stem_sparse_prefill  Alg. 1 step 3d: exact causal softmax attention over the listed blocks
 *   stem_score_select    steps 1-3c in one call
 *   stem_prefill         all of Algorithm 1, ordered on one stream, no host synchronisation
 *   stem_plan_create_ex  the same path for a CHUNK of every sequence against its K / V prefix, with the
 *                        budget taken at the global token offset (the paper's Conclusion), with the pooled
 *                        K-side tensors in a caller-owned cache (stem_pool_kv, *_cached), and with one
 *                        index list per GQA group (the block-level top-k shared per group of Main Results)
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, 16-byte aligned.
 *     Q, K, V, O hold bf16.  Element (t, h, c) of Q is at Q[t*q_stride_tok + h*q_stride_head + c]
 *     (strides in elements, c contiguous, 0 <= c < head_dim = 128); K and V share
 *     kv_stride_tok / kv_stride_head.  O is contiguous [T, num_q_heads, head_dim].
 *     Sequences are packed along t (varlen): sequence b owns tokens
 *     cu_seqlens[b] .. cu_seqlens[b+1]-1 and never attends to another sequence.
 *   - Query-block rows are numbered globally, sequence-major: R = row_offset(b) + r,
 *     r = 0 .. N_blk(b)-1, N_blk(b) = ceil(len_b / block); R_tot = sum_b N_blk(b).
 *   - Index lists: sel_idx is int32 [num_q_heads, R_tot, k_max], sel_cnt int32
 *     [num_q_heads, R_tot] (num_kv_heads instead with share_group).  Row (h, R) holds sel_cnt valid
 *     block ids, local to the sequence, strictly ascending, each <= r; the remaining entries are -1.
 *   - `stream` is a cudaStream_t passed as void*.  Hot calls enqueue work on it and return;
 *     they never allocate, never synchronise and never throw.
 *   - Return value: STEM_OK (0) or a negative stem_status.  Nothing is enqueued when a call
 *     returns STEM_ERR_INVALID_ARG / UNSUPPORTED / WORKSPACE.
 *   - Device-side waits are bounded; a wait that gives up records a code in the workspace,
 *     the kernel returns early, and stem_check_status reports STEM_ERR_DEVICE_TIMEOUT.
 *   - Workspace: caller memory of stem_plan_info.workspace_bytes, 256-byte aligned.  Its first 32
 *     bytes are the status words: they must be ZERO before the first hot call that uses the
 *     workspace (cudaMemset them once after allocating); afterwards the library keeps them
 *     (each kernel clears its own words when it is enqueued, stem_check_status clears all of them
 *     after reporting a time-out).  The rest needs no initialisation.
 */
#ifndef STEM_H_
#define STEM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  STEM_OK = 0,
  STEM_ERR_INVALID_ARG = -1,    /* null pointer, bad size, misaligned pointer or stride           */
  STEM_ERR_UNSUPPORTED = -2,    /* head_dim != 128, block not in {64,128}, heads not divisible, ... */
  STEM_ERR_WORKSPACE = -3,      /* workspace missing or smaller than stem_plan_query reports      */
  STEM_ERR_CUDA = -4,           /* a CUDA runtime / driver call or a kernel launch failed         */
  STEM_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait gave up (see stem_check_status)     */
  STEM_ERR_STATIC_SCRATCH = -6  /* problem larger than the built-in scratch of stem_score_static  */
} stem_status;

/* Problem statement of Algorithm 1 (inputs Q, K, V; hyper-parameters k_start, mu, B, beta) plus
 * the forced-block settings of the paper's implementation details (4 initial + 4 local blocks,
 * minimum total budget). Plain data; copied by stem_plan_create. */
typedef struct {
  int32_t batch;                  /* number of packed sequences, >= 1                              */
  const int32_t* cu_seqlens_host; /* HOST pointer, [batch+1] token offsets, cu[0] = 0, increasing  */
  int32_t num_q_heads;            /* H_q                                                           */
  int32_t num_kv_heads;           /* H_kv, divides H_q; query head h reads kv head h / (H_q/H_kv)  */
  int32_t head_dim;               /* must be 128                                                   */
  int32_t block;                  /* B: 64 or 128                                                  */
  int32_t budget_permille;        /* k_start = floor(budget_permille * N_blk / 1000) blocks        */
  int32_t k_start_blocks;         /* if > 0, overrides budget_permille                             */
  int32_t mu_num, mu_den;         /* decay ratio mu = mu_num/mu_den in (0,1]; 7/10 in the paper    */
  int32_t stem_blocks;            /* initial blocks always kept (paper: 4), >= 0                   */
  int32_t local_blocks;           /* trailing blocks always kept, diagonal included (paper: 4), >= 1 */
  int32_t min_blocks;             /* lower bound of the per-row budget (paper: 54), >= 0           */
  float beta;                     /* weight of the magnitude term of Eq. 7 (paper: 0.2)            */
  float score_scale;              /* multiplies Qbar.Kbar in the metric; 0 means 1.0 (Eq. 7)       */
  float softmax_scale;            /* 0 means 1/sqrt(head_dim) (Alg. 1 step d)                      */
  int64_t q_stride_tok, q_stride_head;   /* elements; multiples of 8                               */
  int64_t kv_stride_tok, kv_stride_head; /* elements; multiples of 8                               */
} stem_config;

typedef struct stem_plan stem_plan; /* opaque; owns small host and device tables only */

/* Sizes a caller needs to allocate buffers for a plan. */
typedef struct {
  size_t workspace_bytes;       /* scratch the hot calls need (pooled tensors, metric, lists, status) */
  int32_t total_tokens;         /* tokens of Q and O (the chunk's tokens with chunked prefill)      */
  int32_t total_q_blocks;       /* R_tot: query-block rows                                         */
  int32_t k_max;                /* longest index list = max_r k_eff(r)                             */
  int64_t metric_elems;         /* per head: sum_b rows(b) * N_blk(b), the size of one head of M   */
  int64_t selected_blocks;      /* sum over query heads and rows of the list lengths (exact)       */
  int64_t causal_blocks;        /* sum over query heads and rows of r+1 (admissible blocks)        */
  int64_t selected_pairs;       /* unmasked (query, key) pairs inside the selected blocks          */
  int64_t causal_pairs;         /* unmasked (query, key) pairs of dense causal attention           */
  int32_t total_kv_tokens;      /* tokens of K and V (= total_tokens without chunks)               */
  int32_t list_heads;           /* first dimension of sel_idx / sel_cnt / M: H_q, or H_kv with share_group */
  size_t kcache_bytes;          /* size of the caller-owned pooled-K cache (0 without one)         */
  int32_t total_key_blocks;     /* key blocks of all sequences (sum_b N_blk(b))                    */
  int32_t new_key_blocks;       /* key blocks the chunk adds (what stem_pool_kv pools)             */
} stem_plan_info;

/* Extensions of the problem statement (all optional; a zeroed struct or NULL means plain Algorithm 1).
 *
 * Chunked prefill (Conclusion, "Limitations and future work": the position-decay schedule applies to chunk
 * prefill when global token offsets are kept across chunks).  cfg.cu_seqlens_host then describes K and V: the
 * first kv_len(b) tokens of every sequence.  Q and O hold only the chunk, the tokens q_start(b) ..
 * kv_len(b)-1 of every sequence, packed in sequence order.  Block row r of a chunk is the global row
 * (r >= q_start/B): its causal blocks are 0 .. r of the prefix, and its budget is Eq. 3 at row r+1 of a
 * sequence of ceil(total_len(b)/B) blocks, with k_start taken from that block count.
 *
 * Pooled-K cache (Main Results / Related Work: block-level K-side representations kept with the KV cache).
 * With kcache_blocks_per_seq > 0 the K-side tensors of step 1 (Kbar parts and MV) live in caller memory of
 * stem_plan_info.kcache_bytes: sequence b owns rows b*capacity .. of it, row j = its block j, so the layout
 * does not move while the prefix grows.  stem_pool_kv writes the rows of the blocks the plan's chunk adds;
 * the *_cached calls read rows 0 .. N_blk(b)-1 and never touch K or V for scoring.
 *
 * share_group (Main Results: integration with a block-level top-k shared by the heads of a GQA group): one
 * index list per (kv head, row).  The group's metric is the mean over its query heads of Eq. 7, i.e. Eq. 7 on
 * the group-mean pooled query; sel_idx / sel_cnt / M have num_kv_heads heads; every query head of the group
 * attends over its group's list.
 *
 * score_mode = 1, anti-diagonal scoring (Overall Algorithm: "anti-diagonal scoring", after XAttention; Alg. 1
 * step 1 comment, stride = B): the other reading of the pooling step.  The routing term of block pair (r, j)
 * is the mean of the token scores along the main anti-diagonal of the B x B score block,
 *   (1/n) sum_s q[rB + B-1-s] . k[jB + s]  over the s whose two tokens exist (n = B for full blocks),
 * in place of Qbar[h,r] . Kbar[kv(h),j]; the magnitude term, the budget and the selection are unchanged.
 * Computed as one tensor-core contraction of Q with K (inner dimension B * d).  Not combinable with the
 * pooled-K cache or share_group; at most 8 sequences per plan (STEM_ERR_UNSUPPORTED otherwise). */
typedef struct {
  const int32_t* q_start_host;    /* HOST [batch]: first query token of every sequence's chunk, a multiple of
                                     block, < kv_len(b); NULL = 0 (no chunking)                               */
  const int32_t* total_len_host;  /* HOST [batch]: full length of every sequence for Eq. 3, >= kv_len(b);
                                     NULL = kv_len(b)                                                         */
  int32_t kcache_blocks_per_seq;  /* capacity (blocks per sequence) of a caller-owned pooled-K cache; 0 = none */
  int32_t share_group;            /* 1: one index list per kv head                                            */
  int32_t score_mode;             /* 0: product of block means (Eq. 7 on pooled blocks); 1: anti-diagonal scoring */
  int32_t reserved[3];            /* must be 0                                                                */
} stem_options;

/* Builds the per-row budget table k_eff(r) (Eq. 3 in block units, i = r+1, clamped by the forced
 * blocks, min_blocks and the r+1 causal blocks), the row maps and the work order of the attention
 * kernel, and uploads them to the current CUDA device (the only allocation the library makes).
 * Host work only plus one synchronous copy; call it outside the hot path. */
int stem_plan_create(const stem_config* cfg, stem_plan** out_plan);
/* The same with the extensions above; opts == NULL is stem_plan_create. */
int stem_plan_create_ex(const stem_config* cfg, const stem_options* opts, stem_plan** out_plan);
int stem_plan_destroy(stem_plan* plan);
int stem_plan_query(const stem_plan* plan, stem_plan_info* info);

/* Copies the per-row budget table k_eff (int32 [R_tot], host memory) out of the plan. */
int stem_plan_budget(const stem_plan* plan, int32_t* k_eff_host);

/* Host-only form of the budget schedule (Eq. 3 in block units with the forced-block and
 * min_blocks clamps): validates cfg and writes k_eff for every global row into k_eff_host
 * (capacity entries; pass NULL to only count).  *r_tot receives R_tot.  Needs no CUDA device. */
int stem_budget_table(const stem_config* cfg, int32_t* k_eff_host, int64_t capacity, int32_t* r_tot);

/* Alg. 1 step 1 and step 3a.
 *   Pools Q and K (block means over the valid tokens of each block) and V
 *   (MV = max(0, max_t ln ||V_t||_2) per block) into the workspace, then, if M != NULL, writes
 *   the Output-Aware Metric of Eq. 7 on pooled blocks,
 *     M[h, m_off(b) + r*N_blk(b) + j] = score_scale * Qbar[h,r].Kbar[kv(h),j] + beta * MV[kv(h),j],
 *   for causal blocks j <= r only (entries with j > r are not written).  M is fp32
 *   [num_q_heads, metric_elems].  With M == NULL only the pooled tensors are produced. */
int stem_score(const stem_plan* plan, const void* Q, const void* K, const void* V, float* M, void* workspace,
               size_t workspace_bytes, void* stream);

/* stem_score for callers that cannot hand the library a workspace.  (The paper has no counterpart;
 * this is a packaging variant of stem_score: same two kernels, same M.)
 *
 * Who needs it: code that runs where device allocation is off limits - a plug-in called from inside
 * a serving engine whose memory pool already owns the whole GPU, a callback that must not touch the
 * allocator because the host framework forbids it there, a process running close to the memory
 * limit where a multi-megabyte request could fail.  Such a caller still owns Q, K, V and M, but has
 * nowhere to put the pooled tensors stem_score keeps in its workspace.
 *
 * Here that scratch lives in a fixed array inside the library image (STEM_STATIC_SCRATCH_BYTES,
 * resident on every GPU that loads the library until the process exits).  The call performs no
 * cudaMalloc / cudaFree and uses no allocating routine; the plan must have been created earlier
 * (plan creation does allocate its small tables).
 *
 *   - M is required.  Same layout as stem_score with a workspace, and the same values (the same
 *     pooling and metric kernels run on the same inputs).
 *   - Problems whose status words and pooled tensors exceed the array, i.e.
 *       256 + H_kv * R_tot * 4 + (H_q + H_kv) * R_tot * 128 * 6 bytes (each part rounded up to 256)
 *       > STEM_STATIC_SCRATCH_BYTES,
 *     are rejected with STEM_ERR_STATIC_SCRATCH and nothing is enqueued.
 *   - The first call on each device resolves the array's device address (a one-time set-up that
 *     talks to the CUDA runtime; with lazy module loading it is also the moment the array becomes
 *     resident on that device, so the driver's free-memory count drops by its size once); make
 *     that first call before starting any stream capture.  Later calls neither allocate nor free.
 *     The plan's device must be the current device.
 *   - All calls on a device share the one array.  Its contents are whatever the previous call
 *     left: the call clears the status words it needs at zero, and overwrites every pooled element
 *     its result depends on before reading it (metric tiles that reach past a sequence's last
 *     block do read stale rows, but only into entries that are never stored).  Two calls that
 *     overlap on the GPU (different streams, no ordering between them) race on the array:
 *     serialise them.
 *   - A bounded wait that gave up inside this call is reported by stem_check_status called with
 *     workspace == NULL. */
#define STEM_STATIC_SCRATCH_BYTES (8u * 1024u * 1024u)
int stem_score_static(const stem_plan* plan, const void* Q, const void* K, const void* V, float* M, void* stream);

/* Alg. 1 steps 3b-3c.
 *   For every (head, row): keeps the forced blocks {0..stem-1} and {r-local+1..r}, then adds the
 *   causal blocks of largest metric until the row holds k_eff(r) blocks.  Order: metric
 *   descending, block id ascending on equal metric, -0 == +0, NaN below every number.
 *   Reads M (layout above) if M != NULL, else recomputes the metric (into the workspace) from the
 *   pooled tensors a preceding stem_score left in the same workspace.  Writes sel_idx / sel_cnt. */
int stem_select(const stem_plan* plan, const float* M, int32_t* sel_idx, int32_t* sel_cnt, void* workspace,
                size_t workspace_bytes, void* stream);

/* Alg. 1 steps 1-3c in one call: block-wise representations, Output-Aware Metric (Eq. 7), Token
 * Position-Decay budget (Eq. 3) and top-k selection; the metric is kept in the workspace (as bit
 *   planes of its order-preserving selection keys, part of workspace_bytes), never handed to the caller.
 *   Same results as stem_score(M = NULL) followed by stem_select(M = NULL).
 *   Writes sel_idx / sel_cnt; leaves the pooled tensors in the workspace. */
int stem_score_select(const stem_plan* plan, const void* Q, const void* K, const void* V, int32_t* sel_idx,
                      int32_t* sel_cnt, void* workspace, size_t workspace_bytes, void* stream);

/* Alg. 1 step 3d.
 *   O[t,h,:] = softmax_k( Q[t,h].K[k,kv(h)] * softmax_scale ) V over the keys k of the listed
 *   blocks of t's row with position <= t.  sel_idx == NULL (with sel_cnt == NULL) means every
 *   causal block, i.e. dense causal attention.  Lists must be ascending and within [0, r];
 *   out-of-range ids are clamped, never dereferenced.  lse (fp32 [num_q_heads, T], natural-log
 *   sum-exp of the scaled scores) is optional (NULL to skip). */
int stem_sparse_prefill(const stem_plan* plan, const void* Q, const void* K, const void* V, const int32_t* sel_idx,
                        const int32_t* sel_cnt, void* O, float* lse, void* workspace, size_t workspace_bytes,
                        void* stream);

/* All of Algorithm 1: stem_score_select -> stem_sparse_prefill, ordered on `stream`, no host
 * synchronisation.  sel_idx / sel_cnt are optional outputs (both NULL: lists stay in the workspace). */
int stem_prefill(const stem_plan* plan, const void* Q, const void* K, const void* V, void* O, int32_t* sel_idx,
                 int32_t* sel_cnt, float* lse, void* workspace, size_t workspace_bytes, void* stream);

/* K side of Alg. 1 step 1 into a caller-owned pooled-K cache (plans created with kcache_blocks_per_seq > 0):
 * block means of K (as the three bf16 parts the metric kernel multiplies) and MV = max(0, max ln ||V||) for
 * the key blocks the plan's chunk adds (every block without chunking), read from the packed K / V of the
 * prefix.  The hook for "pool K and V once, when they are written".  kcache: DEVICE, 256-byte aligned,
 * stem_plan_info.kcache_bytes; rows of other blocks are left as they are. */
int stem_pool_kv(const stem_plan* plan, const void* K, const void* V, void* kcache, void* stream);

/* Alg. 1 steps 1-3c reading only Q: pools Q, takes Kbar and MV of blocks 0 .. N_blk(b)-1 from the cache
 * (written by earlier stem_pool_kv calls), metric, budget, selection.  Same lists as stem_score_select. */
int stem_score_select_cached(const stem_plan* plan, const void* Q, const void* kcache, int32_t* sel_idx,
                             int32_t* sel_cnt, void* workspace, size_t workspace_bytes, void* stream);

/* All of Algorithm 1 with the cache: update_cache != 0 first pools the chunk's new key blocks into it
 * (stem_pool_kv), then stem_score_select_cached and stem_sparse_prefill, ordered on `stream`. */
int stem_prefill_cached(const stem_plan* plan, const void* Q, const void* K, const void* V, void* O, void* kcache,
                        int update_cache, int32_t* sel_idx, int32_t* sel_cnt, float* lse, void* workspace,
                        size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Token Position-Decay on a token-level selector (Main Results: the integration with a sparse-attention
 * model that keeps the top 2048 tokens per query, k_start = 2048, mu = 0.7).  One sequence of n_tokens;
 * selection granularity is ONE TOKEN; one index list per (kv head, query token), shared by the query heads
 * of the group.  head_dim = 128, bf16, layouts as above.
 * ---------------------------------------------------------------------------------------------- */

/* Eq. 3 at token positions: k(t) = floor(k_start - k_start (1 - mu) (t+1) / n_tokens), raised to the number of
 * forced tokens (the first stem_tokens and the last local_tokens of the t+1 causal tokens, the token itself
 * included: local_tokens >= 1) and capped at t+1.  Host only; k_host: HOST int32 [n_tokens]. */
int stem_token_budget(int32_t n_tokens, int32_t k_start, int32_t mu_num, int32_t mu_den, int32_t stem_tokens,
                      int32_t local_tokens, int32_t* k_host);

/* Per (list head, query token t): keeps the forced tokens, then the causal tokens of largest score until the list
 * holds k_tok[t] tokens (score descending, token id ascending on equal scores, -0 == +0, NaN lowest); the list is
 * emitted ascending, -1 padded.  scores: DEVICE fp32 [list_heads, n_tokens, n_tokens] (row t: entries 0 .. t are
 * read), the indexer scores the caller computed; k_tok: DEVICE int32 [n_tokens]; sel_idx int32
 * [list_heads, n_tokens, k_max], sel_cnt int32 [list_heads, n_tokens]; k_max >= max_t k_tok[t]. */
int stem_token_select(const float* scores, int32_t n_tokens, int32_t list_heads, const int32_t* k_tok, int32_t stem_tokens,
                      int32_t local_tokens, int32_t k_max, int32_t* sel_idx, int32_t* sel_cnt, void* stream);

/* Gather-style attention over token lists: O[t,h] = softmax_s( Q[t,h].K[s,kv(h)] * softmax_scale ) V over the tokens
 * s of list (kv(h), t) (ids are clamped to [0, t], never dereferenced out of range; at most min(k_max, t+1) entries
 * of a list are used).  Lists are per kv head ([num_kv_heads, n_tokens, k_max]); at most 16 query heads per kv head
 * (STEM_ERR_UNSUPPORTED otherwise).  Strides in elements, multiples of 8; Q, K, V, O 16-byte aligned.
 * softmax_scale 0 means 1/sqrt(128).  O bf16 [n_tokens, num_q_heads, 128] (contiguous); lse fp32
 * [num_q_heads, n_tokens] or NULL.  Probabilities are rounded to bf16 before they meet V (as in stem_sparse_prefill).
 * The call only enqueues; a bounded device-side wait that gave up is reported by stem_token_check_status. */
int stem_token_attention(const void* Q, const void* K, const void* V, int32_t n_tokens, int32_t num_q_heads,
                         int32_t num_kv_heads, int64_t q_stride_tok, int64_t q_stride_head, int64_t kv_stride_tok,
                         int64_t kv_stride_head, const int32_t* sel_idx, const int32_t* sel_cnt, int32_t k_max,
                         float softmax_scale, void* O, float* lse, void* stream);

/* Synchronises `stream`, then reads (and clears, if set) the status words of the gather-attention kernel on the
 * current device.  Returns STEM_OK, STEM_ERR_DEVICE_TIMEOUT (a bounded wait in stem_token_attention gave up; the
 * outputs of that call are undefined) or STEM_ERR_CUDA.  detail (optional, HOST int32[4]) receives
 * {4, CTA index, role, barrier id}. */
int stem_token_check_status(void* stream, int32_t* detail_host);

/* Synchronises `stream`, then reads the device status words of `workspace` (workspace == NULL: of
 * the scratch built into the library, see stem_score_static) and clears them if they are set.
 * Returns STEM_OK, STEM_ERR_DEVICE_TIMEOUT (a bounded wait in a kernel gave up; outputs of that
 * call are undefined) or STEM_ERR_CUDA.  detail (optional, HOST int32[4]) receives the raw words:
 * {1, CTA index, role, barrier id} of the attention kernel, or {2, tile, kv head, 0} when
 * the wait that gave up was in the metric kernel ({3, tile, query head, 0}: its anti-diagonal form). */
int stem_check_status(const stem_plan* plan, void* workspace, void* stream, int32_t* detail_host);

/* Self-test of the time-out reporting (the paper has no counterpart).  Enqueues a one-thread kernel
 * that waits 1 ms, with the same bounded-wait routine the attention and metric kernels use, on a
 * barrier nothing ever arrives at, records {1, 0, 99, 0} in the workspace status words and returns
 * normally.  A following stem_check_status must report STEM_ERR_DEVICE_TIMEOUT; the CUDA context
 * stays usable.  Never needed in production. */
int stem_selftest_wait_timeout(const stem_plan* plan, void* workspace, size_t workspace_bytes, void* stream);

/* Number of kernels the last hot call on this plan launched (for launch accounting). */
int stem_last_launch_count(const stem_plan* plan);

const char* stem_status_string(int status);
int stem_version(void);

#ifdef __cplusplus
}
#endif
#endif /* STEM_H_ */
