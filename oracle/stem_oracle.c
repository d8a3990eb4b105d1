/*
 * CPU checker for Stem sparse causal prefill attention.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * path computes; it is used by the tests, by the smoke check and by the CPU
 * baseline leg of the benchmark.  It shares no code with the CUDA path and the
 * product never calls it.
 *
 * The method is a heuristic (it approximates dense attention), so this file
 * follows Algorithm 1 of the paper step by step, in its order and notation:
 *
 *   step 1  block-wise representations   Qbar, Kbar  (Alg. 1 "Pool", mean reading)
 *                                        MV          (Alg. 1 "MaxPool(log||V||_2)")
 *   step 2  position-decay schedule      k(i)        (Eq. 3, evaluated in block units)
 *   step 3a coarse metric                M = Qbar Kbar^T + beta * max(0, MV)   (Eq. 7)
 *   step 3c top-k block selection        I_block     (Alg. 1 "TopK")
 *   step 3d exact softmax attention over the selected blocks  (Alg. 1 step d)
 *
 * Precision: inputs are bf16 bit patterns widened exactly; every reduction
 * accumulates in double; the pooled tensors and the metric are stored as fp32
 * because the selection decision is taken on fp32 metric values (the precision
 * the kernels decide in); attention is double throughout and stored as fp32.
 *
 * Pins (see tests, "not gpu"): schedule end points / monotonicity / closed forms
 * of Eq. 2 and Eq. 4; pooled dot product equals the mean of the block's token
 * dot products; closed form of the magnitude term; beta = 0 ranking; brute-force
 * sort for selection; full budget reproduces dense causal softmax attention.
 * Chunked prefill (so_*_chunk) is pinned against the one-shot functions: the rows of any split of a
 * sequence into chunks must reproduce the one-shot lists bit for bit and the outputs to 1e-6; the
 * group-shared metric (so_metric_shared) against a numpy fp64 mean of per-head metrics.
 * The anti-diagonal scoring mode (so_metric_antidiag) is pinned against the anti-diagonal of a numpy fp64
 * score matrix and against hand-built inputs whose anti-diagonal sums are known in closed form.
 * End-task accuracy (the paper's tables) needs trained weights: parity unpinned.
 *
 * Layouts
 *   X (Q, K or V): element (t, h, c) at X[t*stride_tok + h*stride_head + c], bf16 bits.
 *   rows: global query-block row R = row_off[b] + r, sequence-major.
 *   Qbar [H, R_tot, d], MV [H_kv, R_tot] fp32.
 *   M [H_q, m_tot] fp32 with m_tot = sum_b N_blk_b^2; entry (h, b, r, j) at
 *     h*m_tot + m_off[b] + r*N_blk_b + j, defined for j <= r only.
 *   sel_idx [H_q, R_tot, k_max] int32 (block ids local to the sequence, ascending, -1 padded),
 *   sel_cnt [H_q, R_tot] int32.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline float bf16_to_f32(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }

/* ---------------------------------------------------------------------------------------------
 * Step 2: Token Position-Decay schedule (Eq. 3) in block units, with the forced blocks and the
 * minimum budget of the paper's implementation details.
 *
 *   k_blk(i) = floor( k_s - k_s (1 - mu) i / N_blk ),  i = 1..N_blk   (mu = mu_num / mu_den)
 *   forced(i) = {0 .. min(stem,i)-1}  union  {max(0,i-local) .. i-1}
 *   k_eff(i)  = min( i, max( k_blk(i), min_blocks, |forced(i)| ) )
 *
 * All integer; the floor is taken once on an exact rational.
 * k_blk_out and k_eff_out have n_blk entries (row r = i-1).
 * ------------------------------------------------------------------------------------------- */
void so_schedule(int32_t n_blk, int64_t k_s, int64_t mu_num, int64_t mu_den, int32_t stem, int32_t local,
                 int32_t min_blocks, int32_t* k_blk_out, int32_t* k_eff_out) {
    for (int64_t i = 1; i <= n_blk; ++i) {
        /* k_s - k_s (mu_den - mu_num) i / (mu_den N_blk), as one fraction */
        int64_t num = k_s * (mu_den * (int64_t)n_blk - (mu_den - mu_num) * i);
        int64_t den = mu_den * (int64_t)n_blk;
        int64_t kb = num / den; /* num >= 0, so C division is the floor */
        int64_t n_stem = stem < i ? stem : i;
        int64_t lo_local = i - local > 0 ? i - local : 0;
        /* size of the union of [0, n_stem) and [lo_local, i) */
        int64_t forced = n_stem + (i - lo_local);
        if (lo_local < n_stem) forced -= (n_stem - lo_local);
        int64_t ke = kb;
        if (min_blocks > ke) ke = min_blocks;
        if (forced > ke) ke = forced;
        if (ke > i) ke = i;
        if (k_blk_out) k_blk_out[i - 1] = (int32_t)kb;
        if (k_eff_out) k_eff_out[i - 1] = (int32_t)ke;
    }
}

/* ---------------------------------------------------------------------------------------------
 * Step 1a: mean pooling of Q or K over each block of B tokens (Alg. 1 "Pool", stride = B).
 * The last block of a sequence may be partial; the mean is over its valid tokens.
 * ------------------------------------------------------------------------------------------- */
void so_pool_mean(const uint16_t* X, int64_t stride_tok, int64_t stride_head, int32_t H, int32_t d,
                  int32_t batch, const int32_t* cu_seqlens, int32_t B, float* out /*[H,R_tot,d]*/) {
    int64_t r_tot = 0;
    for (int b = 0; b < batch; ++b) r_tot += cdiv(cu_seqlens[b + 1] - cu_seqlens[b], B);
    int64_t row_off = 0;
    for (int b = 0; b < batch; ++b) {
        int64_t t0 = cu_seqlens[b], n = cu_seqlens[b + 1] - cu_seqlens[b];
        int64_t n_blk = cdiv(n, B);
#pragma omp parallel for collapse(2) schedule(static)
        for (int h = 0; h < H; ++h) {
            for (int64_t r = 0; r < n_blk; ++r) {
                int64_t lo = r * B, hi = lo + B < n ? lo + B : n;
                float* o = out + ((int64_t)h * r_tot + row_off + r) * d;
                for (int c = 0; c < d; ++c) {
                    double acc = 0.0;
                    for (int64_t t = lo; t < hi; ++t)
                        acc += (double)bf16_to_f32(X[(t0 + t) * stride_tok + (int64_t)h * stride_head + c]);
                    o[c] = (float)(acc / (double)(hi - lo));
                }
            }
        }
        row_off += n_blk;
    }
}

/* ---------------------------------------------------------------------------------------------
 * Step 1b: value magnitude, MV[h, j] = max(0, max_{t in block j} ln ||V_t||_2)
 * (Alg. 1 "MaxPool(log||V||_2)" followed by the max(0, .) of Eq. 7).  ln 0 = -inf -> 0.
 * ------------------------------------------------------------------------------------------- */
void so_value_magnitude(const uint16_t* V, int64_t stride_tok, int64_t stride_head, int32_t H, int32_t d,
                        int32_t batch, const int32_t* cu_seqlens, int32_t B, float* mv /*[H,R_tot]*/) {
    int64_t r_tot = 0;
    for (int b = 0; b < batch; ++b) r_tot += cdiv(cu_seqlens[b + 1] - cu_seqlens[b], B);
    int64_t row_off = 0;
    for (int b = 0; b < batch; ++b) {
        int64_t t0 = cu_seqlens[b], n = cu_seqlens[b + 1] - cu_seqlens[b];
        int64_t n_blk = cdiv(n, B);
#pragma omp parallel for collapse(2) schedule(static)
        for (int h = 0; h < H; ++h) {
            for (int64_t j = 0; j < n_blk; ++j) {
                int64_t lo = j * B, hi = lo + B < n ? lo + B : n;
                double best = -INFINITY;
                for (int64_t t = lo; t < hi; ++t) {
                    double ss = 0.0;
                    for (int c = 0; c < d; ++c) {
                        double x = (double)bf16_to_f32(V[(t0 + t) * stride_tok + (int64_t)h * stride_head + c]);
                        ss += x * x;
                    }
                    double lg = log(sqrt(ss)); /* natural log of the 2-norm */
                    if (lg > best) best = lg;
                }
                if (!(best > 0.0)) best = 0.0;
                mv[(int64_t)h * r_tot + row_off + j] = (float)best;
            }
        }
        row_off += n_blk;
    }
}

/* ---------------------------------------------------------------------------------------------
 * Step 3a: Output-Aware Metric on pooled blocks (Eq. 7 / Alg. 1 step a), per query head,
 * K-side terms taken from the head's kv head (h / g), causal blocks j <= r only:
 *   M[h,r,j] = score_scale * (Qbar[h,r] . Kbar[kv(h),j]) + beta * MV[kv(h),j]
 * ------------------------------------------------------------------------------------------- */
void so_metric(const float* qbar /*[Hq,R_tot,d]*/, const float* kbar /*[Hkv,R_tot,d]*/,
               const float* mv /*[Hkv,R_tot]*/, int32_t Hq, int32_t Hkv, int32_t d, int32_t batch,
               const int32_t* n_blk /*[batch]*/, float beta, float score_scale, float* M /*[Hq,m_tot]*/) {
    int64_t r_tot = 0, m_tot = 0;
    for (int b = 0; b < batch; ++b) { r_tot += n_blk[b]; m_tot += (int64_t)n_blk[b] * n_blk[b]; }
    int g = Hq / Hkv;
    int64_t row_off = 0, m_off = 0;
    for (int b = 0; b < batch; ++b) {
        int64_t nb = n_blk[b];
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
        for (int h = 0; h < Hq; ++h) {
            for (int64_t r = 0; r < nb; ++r) {
                int kvh = h / g;
                const float* qv = qbar + ((int64_t)h * r_tot + row_off + r) * d;
                for (int64_t j = 0; j <= r; ++j) {
                    const float* kv = kbar + ((int64_t)kvh * r_tot + row_off + j) * d;
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) acc += (double)qv[c] * (double)kv[c];
                    double m = (double)score_scale * acc + (double)beta * (double)mv[(int64_t)kvh * r_tot + row_off + j];
                    M[(int64_t)h * m_tot + m_off + r * nb + j] = (float)m;
                }
            }
        }
        row_off += nb;
        m_off += nb * nb;
    }
}

/* ---------------------------------------------------------------------------------------------
 * Step 3c: selection.  For row r (i = r+1): forced = stem blocks and local blocks (the
 * diagonal block r is the last local block); the remaining k_eff - |forced| blocks are the
 * causal, non-forced candidates of largest metric, ties broken toward the smaller block id.
 * -0 is treated as +0 and NaN as -inf before comparing.  Output ascending.
 * ------------------------------------------------------------------------------------------- */
typedef struct { float m; int32_t j; } so_cand;

static int so_cand_cmp(const void* a, const void* b) {
    const so_cand* x = (const so_cand*)a;
    const so_cand* y = (const so_cand*)b;
    if (x->m > y->m) return -1;
    if (x->m < y->m) return 1;
    return (x->j > y->j) - (x->j < y->j);
}

static int so_int_cmp(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return (x > y) - (x < y);
}

void so_select(const float* M /*[Hq,m_tot]*/, int32_t Hq, int32_t batch, const int32_t* n_blk,
               const int32_t* k_eff /*[R_tot]*/, int32_t stem, int32_t local, int32_t k_max,
               int32_t* sel_idx /*[Hq,R_tot,k_max]*/, int32_t* sel_cnt /*[Hq,R_tot]*/) {
    int64_t r_tot = 0, m_tot = 0;
    for (int b = 0; b < batch; ++b) { r_tot += n_blk[b]; m_tot += (int64_t)n_blk[b] * n_blk[b]; }
    int64_t row_off = 0, m_off = 0;
    for (int b = 0; b < batch; ++b) {
        int64_t nb = n_blk[b];
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
        for (int h = 0; h < Hq; ++h) {
            for (int64_t r = 0; r < nb; ++r) {
                int64_t i = r + 1;
                int64_t n_stem = stem < i ? stem : i;
                int64_t lo_local = i - local > 0 ? i - local : 0;
                int32_t ke = k_eff[row_off + r];
                int32_t* out = sel_idx + ((int64_t)h * r_tot + row_off + r) * k_max;
                so_cand* cand = (so_cand*)malloc(sizeof(so_cand) * (size_t)i);
                int n_out = 0, n_cand = 0;
                for (int64_t j = 0; j < i; ++j) {
                    if (j < n_stem || j >= lo_local) {
                        out[n_out++] = (int32_t)j;
                    } else {
                        float m = M[(int64_t)h * m_tot + m_off + r * nb + j];
                        if (m != m) m = -INFINITY;
                        if (m == 0.0f) m = 0.0f; /* -0 -> +0 */
                        cand[n_cand].m = m;
                        cand[n_cand].j = (int32_t)j;
                        ++n_cand;
                    }
                }
                int need = ke - n_out;
                if (need > n_cand) need = n_cand;
                if (need > 0) {
                    qsort(cand, (size_t)n_cand, sizeof(so_cand), so_cand_cmp);
                    for (int q = 0; q < need; ++q) out[n_out++] = cand[q].j;
                }
                free(cand);
                qsort(out, (size_t)n_out, sizeof(int32_t), so_int_cmp);
                for (int q = n_out; q < k_max; ++q) out[q] = -1;
                sel_cnt[(int64_t)h * r_tot + row_off + r] = n_out;
            }
        }
        row_off += nb;
        m_off += nb * nb;
    }
}

/* ---------------------------------------------------------------------------------------------
 * Step 3d: exact attention over the selected blocks (Alg. 1 step d).  For every token t of
 * query-block row (b, r) and head h: keys are the tokens of the listed blocks whose position
 * is <= t (the causal mask only bites inside the diagonal block); s = (q . k) * softmax_scale;
 * softmax over exactly those keys; o = sum p v.  lse = max + ln sum exp(s - max).
 *
 * Only the rows named in `rows` ([n_rows] entries of (h, R) pairs) are computed, so large
 * inputs can be sampled.  O is [T, Hq, d] fp32, lse is [Hq, T] fp32 (may be NULL).
 * ------------------------------------------------------------------------------------------- */
void so_attention(const uint16_t* Q, int64_t q_stride_tok, int64_t q_stride_head, const uint16_t* K,
                  const uint16_t* V, int64_t kv_stride_tok, int64_t kv_stride_head, int32_t Hq, int32_t Hkv,
                  int32_t d, int32_t batch, const int32_t* cu_seqlens, int32_t B, const int32_t* sel_idx,
                  const int32_t* sel_cnt, int32_t k_max, float softmax_scale, const int32_t* rows /*[n_rows,2]*/,
                  int64_t n_rows, float* O, float* lse) {
    int64_t r_tot = 0, T = cu_seqlens[batch];
    for (int b = 0; b < batch; ++b) r_tot += cdiv(cu_seqlens[b + 1] - cu_seqlens[b], B);
    int g = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t it = 0; it < n_rows; ++it) {
        int h = rows[2 * it], R = rows[2 * it + 1];
        int kvh = h / g;
        /* locate the sequence of global row R */
        int b = 0;
        int64_t row_off = 0;
        for (;; ++b) {
            int64_t nb = cdiv(cu_seqlens[b + 1] - cu_seqlens[b], B);
            if (R < row_off + nb) break;
            row_off += nb;
        }
        int64_t t0 = cu_seqlens[b], n = cu_seqlens[b + 1] - cu_seqlens[b];
        int64_t r = R - row_off;
        const int32_t* list = sel_idx + ((int64_t)h * r_tot + R) * k_max;
        int cnt = sel_cnt[(int64_t)h * r_tot + R];
        int64_t max_keys = (int64_t)cnt * B;
        double* s = (double*)malloc(sizeof(double) * (size_t)(max_keys > 0 ? max_keys : 1));
        int64_t* kpos = (int64_t*)malloc(sizeof(int64_t) * (size_t)(max_keys > 0 ? max_keys : 1));
        double* qd = (double*)malloc(sizeof(double) * (size_t)d);
        double* acc = (double*)malloc(sizeof(double) * (size_t)d);
        int64_t q_lo = r * B, q_hi = q_lo + B < n ? q_lo + B : n;
        for (int64_t tq = q_lo; tq < q_hi; ++tq) {
            const uint16_t* qp = Q + (t0 + tq) * q_stride_tok + (int64_t)h * q_stride_head;
            for (int c = 0; c < d; ++c) qd[c] = (double)bf16_to_f32(qp[c]);
            int64_t nk = 0;
            double mx = -INFINITY;
            for (int e = 0; e < cnt; ++e) {
                int64_t j = list[e];
                int64_t k_lo = j * B, k_hi = k_lo + B < n ? k_lo + B : n;
                for (int64_t tk = k_lo; tk < k_hi && tk <= tq; ++tk) {
                    const uint16_t* kp = K + (t0 + tk) * kv_stride_tok + (int64_t)kvh * kv_stride_head;
                    double dot = 0.0;
#pragma omp simd reduction(+ : dot)
                    for (int c = 0; c < d; ++c) dot += qd[c] * (double)bf16_to_f32(kp[c]);
                    double sc = dot * (double)softmax_scale;
                    s[nk] = sc;
                    kpos[nk] = tk;
                    ++nk;
                    if (sc > mx) mx = sc;
                }
            }
            for (int c = 0; c < d; ++c) acc[c] = 0.0;
            double denom = 0.0;
            for (int64_t e = 0; e < nk; ++e) {
                double p = exp(s[e] - mx);
                denom += p;
                const uint16_t* vp = V + (t0 + kpos[e]) * kv_stride_tok + (int64_t)kvh * kv_stride_head;
#pragma omp simd
                for (int c = 0; c < d; ++c) acc[c] += p * (double)bf16_to_f32(vp[c]);
            }
            float* op = O + ((t0 + tq) * (int64_t)Hq + h) * d;
            for (int c = 0; c < d; ++c) op[c] = nk > 0 ? (float)(acc[c] / denom) : 0.0f;
            if (lse) lse[(int64_t)h * T + t0 + tq] = nk > 0 ? (float)(mx + log(denom)) : -INFINITY;
        }
        free(s); free(kpos); free(qd); free(acc);
    }
}

/* =============================================================================================
 * Chunked prefill with global token offsets (Conclusion, "Limitations and future work": the
 * position-decay schedule is applied by keeping global token offsets across chunks).
 *
 * Sequence b is prefilled in chunks.  At one chunk, K and V hold the first kv_len(b) tokens of the
 * sequence (packed by cu_kv), and Q holds only the chunk's tokens, positions q_start(b) ..
 * kv_len(b)-1 (packed by cu_q; q_start is a multiple of the block size).  Block row r of the chunk
 * is the GLOBAL row index r0(b) + local row, r0 = q_start / B; its causal blocks are 0 .. r of the
 * prefix, and its budget is Eq. 3 evaluated at the global row of a sequence of N_total blocks (the
 * caller passes k_eff already sliced to the chunk's rows).  Everything else is Algorithm 1 as above.
 *
 * Layouts: chunk rows are numbered sequence-major, RQ = rq_off(b) + (r - r0(b)); key blocks
 * KB = kb_off(b) + j.  qbar [Hq, RQ_tot, d]; kbar [Hkv, KB_tot, d]; mv [Hkv, KB_tot].
 * M [Hq, m_tot], m_tot = sum_b rows(b) * n_kv_blk(b); entry (h, b, r, j) at
 *   h*m_tot + m_off(b) + (r - r0(b)) * n_kv_blk(b) + j, defined for j <= r.
 * =========================================================================================== */
void so_metric_chunk(const float* qbar, const float* kbar, const float* mv, int32_t Hq, int32_t Hkv, int32_t d,
                     int32_t batch, const int32_t* n_kv_blk, const int32_t* r0, float beta, float score_scale,
                     float* M) {
    int64_t rq_tot = 0, kb_tot = 0, m_tot = 0;
    for (int b = 0; b < batch; ++b) {
        rq_tot += n_kv_blk[b] - r0[b];
        kb_tot += n_kv_blk[b];
        m_tot += (int64_t)(n_kv_blk[b] - r0[b]) * n_kv_blk[b];
    }
    int g = Hq / Hkv;
    int64_t rq_off = 0, kb_off = 0, m_off = 0;
    for (int b = 0; b < batch; ++b) {
        int64_t nb = n_kv_blk[b], first = r0[b];
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
        for (int h = 0; h < Hq; ++h) {
            for (int64_t r = first; r < nb; ++r) {
                int kvh = h / g;
                const float* qv = qbar + ((int64_t)h * rq_tot + rq_off + (r - first)) * d;
                for (int64_t j = 0; j <= r; ++j) {
                    const float* kv = kbar + ((int64_t)kvh * kb_tot + kb_off + j) * d;
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) acc += (double)qv[c] * (double)kv[c];
                    double m = (double)score_scale * acc + (double)beta * (double)mv[(int64_t)kvh * kb_tot + kb_off + j];
                    M[(int64_t)h * m_tot + m_off + (r - first) * nb + j] = (float)m;
                }
            }
        }
        rq_off += nb - first;
        kb_off += nb;
        m_off += (nb - first) * nb;
    }
}

void so_select_chunk(const float* M, int32_t Hq, int32_t batch, const int32_t* n_kv_blk, const int32_t* r0,
                     const int32_t* k_eff /*[RQ_tot]*/, int32_t stem, int32_t local, int32_t k_max,
                     int32_t* sel_idx /*[Hq,RQ_tot,k_max]*/, int32_t* sel_cnt /*[Hq,RQ_tot]*/) {
    int64_t rq_tot = 0, m_tot = 0;
    for (int b = 0; b < batch; ++b) {
        rq_tot += n_kv_blk[b] - r0[b];
        m_tot += (int64_t)(n_kv_blk[b] - r0[b]) * n_kv_blk[b];
    }
    int64_t rq_off = 0, m_off = 0;
    for (int b = 0; b < batch; ++b) {
        int64_t nb = n_kv_blk[b], first = r0[b];
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
        for (int h = 0; h < Hq; ++h) {
            for (int64_t r = first; r < nb; ++r) {
                int64_t i = r + 1; /* the global row decides the forced blocks and the causal range */
                int64_t n_stem = stem < i ? stem : i;
                int64_t lo_local = i - local > 0 ? i - local : 0;
                int64_t RQ = rq_off + (r - first);
                int32_t ke = k_eff[RQ];
                int32_t* out = sel_idx + ((int64_t)h * rq_tot + RQ) * k_max;
                so_cand* cand = (so_cand*)malloc(sizeof(so_cand) * (size_t)i);
                int n_out = 0, n_cand = 0;
                for (int64_t j = 0; j < i; ++j) {
                    if (j < n_stem || j >= lo_local) {
                        out[n_out++] = (int32_t)j;
                    } else {
                        float m = M[(int64_t)h * m_tot + m_off + (r - first) * nb + j];
                        if (m != m) m = -INFINITY;
                        if (m == 0.0f) m = 0.0f;
                        cand[n_cand].m = m;
                        cand[n_cand].j = (int32_t)j;
                        ++n_cand;
                    }
                }
                int need = ke - n_out;
                if (need > n_cand) need = n_cand;
                if (need > 0) {
                    qsort(cand, (size_t)n_cand, sizeof(so_cand), so_cand_cmp);
                    for (int q = 0; q < need; ++q) out[n_out++] = cand[q].j;
                }
                free(cand);
                qsort(out, (size_t)n_out, sizeof(int32_t), so_int_cmp);
                for (int q = n_out; q < k_max; ++q) out[q] = -1;
                sel_cnt[(int64_t)h * rq_tot + RQ] = n_out;
            }
        }
        rq_off += nb - first;
        m_off += (nb - first) * nb;
    }
}

/* Attention of a chunk: the query token at chunk position tq has global position q_start + tq and
 * sees the keys of its row's listed blocks with position <= its own.  O is [Tq, Hq, d] and lse
 * [Hq, Tq], packed like Q.  rows: (h, RQ) pairs in the chunk's row numbering. */
void so_attention_chunk(const uint16_t* Q, int64_t q_stride_tok, int64_t q_stride_head, const uint16_t* K,
                        const uint16_t* V, int64_t kv_stride_tok, int64_t kv_stride_head, int32_t Hq, int32_t Hkv,
                        int32_t d, int32_t batch, const int32_t* cu_q, const int32_t* cu_kv, const int32_t* q_start,
                        int32_t B, const int32_t* sel_idx, const int32_t* sel_cnt, int32_t k_max,
                        float softmax_scale, const int32_t* rows, int64_t n_rows, float* O, float* lse) {
    int64_t rq_tot = 0, Tq = cu_q[batch];
    for (int b = 0; b < batch; ++b) rq_tot += cdiv(cu_q[b + 1] - cu_q[b], B);
    int g = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t it = 0; it < n_rows; ++it) {
        int h = rows[2 * it], RQ = rows[2 * it + 1];
        int kvh = h / g;
        int b = 0;
        int64_t rq_off = 0;
        for (;; ++b) {
            int64_t nr = cdiv(cu_q[b + 1] - cu_q[b], B);
            if (RQ < rq_off + nr) break;
            rq_off += nr;
        }
        int64_t tq0 = cu_q[b], nq = cu_q[b + 1] - cu_q[b];    /* chunk tokens of the sequence */
        int64_t tk0 = cu_kv[b], nk_seq = cu_kv[b + 1] - cu_kv[b]; /* prefix tokens of the sequence */
        int64_t start = q_start[b];
        int64_t rl = RQ - rq_off;                                /* row inside the chunk */
        const int32_t* list = sel_idx + ((int64_t)h * rq_tot + RQ) * k_max;
        int cnt = sel_cnt[(int64_t)h * rq_tot + RQ];
        int64_t max_keys = (int64_t)cnt * B;
        double* s = (double*)malloc(sizeof(double) * (size_t)(max_keys > 0 ? max_keys : 1));
        int64_t* kpos = (int64_t*)malloc(sizeof(int64_t) * (size_t)(max_keys > 0 ? max_keys : 1));
        double* qd = (double*)malloc(sizeof(double) * (size_t)d);
        double* acc = (double*)malloc(sizeof(double) * (size_t)d);
        int64_t q_lo = rl * B, q_hi = q_lo + B < nq ? q_lo + B : nq;
        for (int64_t tq = q_lo; tq < q_hi; ++tq) {
            int64_t pos = start + tq; /* global position of the query token */
            const uint16_t* qp = Q + (tq0 + tq) * q_stride_tok + (int64_t)h * q_stride_head;
            for (int c = 0; c < d; ++c) qd[c] = (double)bf16_to_f32(qp[c]);
            int64_t nk = 0;
            double mx = -INFINITY;
            for (int e = 0; e < cnt; ++e) {
                int64_t j = list[e];
                int64_t k_lo = j * B, k_hi = k_lo + B < nk_seq ? k_lo + B : nk_seq;
                for (int64_t tk = k_lo; tk < k_hi && tk <= pos; ++tk) {
                    const uint16_t* kp = K + (tk0 + tk) * kv_stride_tok + (int64_t)kvh * kv_stride_head;
                    double dot = 0.0;
#pragma omp simd reduction(+ : dot)
                    for (int c = 0; c < d; ++c) dot += qd[c] * (double)bf16_to_f32(kp[c]);
                    double sc = dot * (double)softmax_scale;
                    s[nk] = sc;
                    kpos[nk] = tk;
                    ++nk;
                    if (sc > mx) mx = sc;
                }
            }
            for (int c = 0; c < d; ++c) acc[c] = 0.0;
            double denom = 0.0;
            for (int64_t e = 0; e < nk; ++e) {
                double p = exp(s[e] - mx);
                denom += p;
                const uint16_t* vp = V + (tk0 + kpos[e]) * kv_stride_tok + (int64_t)kvh * kv_stride_head;
#pragma omp simd
                for (int c = 0; c < d; ++c) acc[c] += p * (double)bf16_to_f32(vp[c]);
            }
            float* op = O + ((tq0 + tq) * (int64_t)Hq + h) * d;
            for (int c = 0; c < d; ++c) op[c] = nk > 0 ? (float)(acc[c] / denom) : 0.0f;
            if (lse) lse[(int64_t)h * Tq + tq0 + tq] = nk > 0 ? (float)(mx + log(denom)) : -INFINITY;
        }
        free(s); free(kpos); free(qd); free(acc);
    }
}

/* =============================================================================================
 * Group-shared selection (Main Results: the integration into a model whose block-level top-k is
 * shared by the query heads of a GQA group).  One index list per (kv head, row) instead of one per
 * query head.  The paper does not say how the heads' metrics are combined; the reading taken here:
 * the group's metric is the MEAN over its query heads of Eq. 7's metric,
 *   Mg[kvh, r, j] = (1/g) * sum_{h in group} ( score_scale * Qbar[h,r].Kbar[kvh,j] ) + beta * MV[kvh,j],
 * which equals Eq. 7 evaluated on the group-mean pooled query.  Layout of Mg: that of M with Hkv heads.
 * =========================================================================================== */
void so_metric_shared(const float* qbar /*[Hq,R_tot,d]*/, const float* kbar /*[Hkv,R_tot,d]*/,
                      const float* mv /*[Hkv,R_tot]*/, int32_t Hq, int32_t Hkv, int32_t d, int32_t batch,
                      const int32_t* n_blk, float beta, float score_scale, float* Mg /*[Hkv,m_tot]*/) {
    int64_t r_tot = 0, m_tot = 0;
    for (int b = 0; b < batch; ++b) { r_tot += n_blk[b]; m_tot += (int64_t)n_blk[b] * n_blk[b]; }
    int g = Hq / Hkv;
    int64_t row_off = 0, m_off = 0;
    for (int b = 0; b < batch; ++b) {
        int64_t nb = n_blk[b];
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
        for (int kvh = 0; kvh < Hkv; ++kvh) {
            for (int64_t r = 0; r < nb; ++r) {
                for (int64_t j = 0; j <= r; ++j) {
                    const float* kv = kbar + ((int64_t)kvh * r_tot + row_off + j) * d;
                    double sum = 0.0;
                    for (int q = 0; q < g; ++q) {
                        const float* qv = qbar + ((int64_t)(kvh * g + q) * r_tot + row_off + r) * d;
                        double acc = 0.0;
                        for (int c = 0; c < d; ++c) acc += (double)qv[c] * (double)kv[c];
                        sum += acc;
                    }
                    double m = (double)score_scale * (sum / (double)g) + (double)beta * (double)mv[(int64_t)kvh * r_tot + row_off + j];
                    Mg[(int64_t)kvh * m_tot + m_off + r * nb + j] = (float)m;
                }
            }
        }
        row_off += nb;
        m_off += nb * nb;
    }
}

/* =============================================================================================
 * Anti-diagonal scoring (Overall Algorithm: the pooling step is called anti-diagonal scoring, after
 * XAttention; Alg. 1 step 1 comment "Pool(Q, K, stride = B)").  The other reading of the pooling
 * step: instead of the product of block means, the routing term of block pair (r, j) is the mean
 * of the token scores ALONG THE MAIN ANTI-DIAGONAL of the B x B score block (stride B leaves one
 * anti-diagonal per block),
 *   A[h,r,j] = (1/n) * sum_{s=0..B-1, both tokens exist} q[rB + B-1-s] . k[jB + s],
 * n = number of such s (B for full blocks), and M = score_scale * A + beta * MV as in Eq. 7.
 * Layout of M as in so_metric.
 * =========================================================================================== */
void so_metric_antidiag(const uint16_t* Q, int64_t q_stride_tok, int64_t q_stride_head, const uint16_t* K,
                        int64_t kv_stride_tok, int64_t kv_stride_head, const float* mv /*[Hkv,R_tot]*/, int32_t Hq,
                        int32_t Hkv, int32_t d, int32_t batch, const int32_t* cu_seqlens, int32_t B, float beta,
                        float score_scale, float* M /*[Hq,m_tot]*/) {
    int64_t r_tot = 0, m_tot = 0;
    for (int b = 0; b < batch; ++b) {
        int64_t nb = cdiv(cu_seqlens[b + 1] - cu_seqlens[b], B);
        r_tot += nb;
        m_tot += nb * nb;
    }
    int g = Hq / Hkv;
    int64_t row_off = 0, m_off = 0;
    for (int b = 0; b < batch; ++b) {
        int64_t t0 = cu_seqlens[b], n = cu_seqlens[b + 1] - cu_seqlens[b];
        int64_t nb = cdiv(n, B);
#pragma omp parallel for collapse(2) schedule(dynamic, 4)
        for (int h = 0; h < Hq; ++h) {
            for (int64_t r = 0; r < nb; ++r) {
                int kvh = h / g;
                for (int64_t j = 0; j <= r; ++j) {
                    double acc = 0.0;
                    int64_t pairs = 0;
                    for (int64_t s = 0; s < B; ++s) {
                        int64_t tq = r * B + (B - 1 - s), tk = j * B + s;
                        if (tq >= n || tk >= n) continue;
                        const uint16_t* qp = Q + (t0 + tq) * q_stride_tok + (int64_t)h * q_stride_head;
                        const uint16_t* kp = K + (t0 + tk) * kv_stride_tok + (int64_t)kvh * kv_stride_head;
                        double dot = 0.0;
                        for (int c = 0; c < d; ++c) dot += (double)bf16_to_f32(qp[c]) * (double)bf16_to_f32(kp[c]);
                        acc += dot;
                        ++pairs;
                    }
                    double a = pairs > 0 ? acc / (double)pairs : 0.0;
                    double m = (double)score_scale * a + (double)beta * (double)mv[(int64_t)kvh * r_tot + row_off + j];
                    M[(int64_t)h * m_tot + m_off + r * nb + j] = (float)m;
                }
            }
        }
        row_off += nb;
        m_off += nb * nb;
    }
}

/* Number of OpenMP threads the loops above will use (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int so_num_threads(void) { return omp_get_max_threads(); }
#else
int so_num_threads(void) { return 1; }
#endif
