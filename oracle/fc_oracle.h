/*
 * FlowCache hot-path ORACLE — test infrastructure, not product code.
 *
 * A plain, slow, fp64 CPU statement of what the FlowCache (arXiv 2602.10825)
 * chunk pipeline computes, written from the paper's definitions.  It shares no
 * source, header, table or helper with the CUDA library and must never be
 * called from a product path: only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may load it.
 *
 * All pointers are HOST pointers.  Storage dtypes: FCO_BF16 (raw 16-bit
 * patterns) or FCO_F32; every value is widened to double before any
 * arithmetic.  Tensors are [heads, tokens, d] with explicit head / token
 * strides in elements and a contiguous last dimension.
 *
 * Every function returns 0 on success and a negative value on a bad argument.
 */
#ifndef FC_ORACLE_H_
#define FC_ORACLE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { FCO_BF16 = 0, FCO_F32 = 1 };
enum { FCO_RED_AUTO = 0, FCO_RED_PLAIN = 1, FCO_RED_MEANKEY = 2, FCO_RED_MAXSIM = 3 };

/* Per-chunk reuse decision: relative-L1 indicator (Eq. 5, the per-chunk form
 * of Eq. 4) fed to the accumulate / threshold / reset rule (Eq. 8).
 *   r_i = sum|cur - prev| / sum|prev|  over chunk i's elements (fp64), then
 *   rounded to fp32; s = acc_i + r_i in fp32.
 *   recompute iff chunk_step[i] < warmup_m, or force[i], or s > eps (strict);
 *   acc_i <- 0 on recompute, else acc_i <- s.
 * A zero denominator gives r = +inf when the numerator is positive, else 0. */
int fco_chunk_decide(const void* cur, const void* prev, int dtype,
                     const int64_t* chunk_elem_off, int n_chunks,
                     const int32_t* chunk_step, int warmup_m, float eps,
                     const uint8_t* force, float* acc, float* l1rel,
                     uint8_t* recompute, int32_t* active_ids,
                     int32_t* n_active, int n_threads);

/* The uniform ("traditional reuse") policy the paper compares with (caption of
 * Fig. 3): every chunk of a timestep shares one compute / reuse status, except
 * chunks that must be computed anyway (chunk_step[i] < warmup_m, or force[i]).
 * Over the sharing chunks S taken as one tensor:
 *   r = sum_S |cur - prev| / sum_S |prev|  (fp64, rounded to fp32);
 *   s = acc[first chunk of S] + r in fp32; all of S is recomputed iff s > eps;
 *   every acc[i] <- 0 if so, else s (all entries stay equal; 0 if S is empty).
 * l1rel[i] = r for i in S, the chunk's own indicator otherwise. */
int fco_chunk_decide_uniform(const void* cur, const void* prev, int dtype,
                             const int64_t* chunk_elem_off, int n_chunks,
                             const int32_t* chunk_step, int warmup_m, float eps,
                             const uint8_t* force, float* acc, float* l1rel,
                             uint8_t* recompute, int32_t* active_ids,
                             int32_t* n_active, int n_threads);

/* Serving skipped chunks from the activation cache (Sec. 3.2, text after Eq. 8).
 * For every element e of chunk i (same flat layout as fco_chunk_decide):
 *   recompute[i] != 0:  cache[e] <- round(y[e] - x[e])      (y: the fresh output)
 *   recompute[i] == 0:  y[e]     <- round(x[e] + cache[e])  (cache is not modified)
 * with the difference / sum taken in fp32 and rounded once to the storage type
 * (round to nearest even for bf16). */
int fco_chunk_cache_apply(const void* x_in, void* y_io, void* cache, int dtype,
                          const int64_t* chunk_elem_off, int n_chunks,
                          const uint8_t* recompute, int n_threads);

typedef struct {
  int32_t H_q, H_kv, d, W;
  int64_t q_hs, q_rs, k_hs, k_rs, v_hs, v_rs; /* element strides: head, row */
  double scale;                               /* 0 => 1/sqrt(d) */
} fco_attn_desc;

/* Chunk-causal attention of the active chunks (Sec. 3.3: the denoising group
 * attends to the clean-chunk cache plus the denoising region).  For an active
 * chunk c, head h, query row r:
 *   O = softmax_j(q . k_j * scale) V  over the first kv_visible_len[c] LOGICAL
 *   key/value tokens.  Logical token j lives at physical row
 *   kv_token_index[h_kv][j] when that map is given, else at
 *   seg_phys_off[s] + (j - seg_logical_off[s]) for the segment s holding j
 *   (seg_logical_off has n_seg+1 entries).
 * sample_rows == NULL: O is [H_q, n_rows_total, d] (strides o_hs, o_rs), lse is
 *   [H_q, n_rows_total]; rows of inactive chunks are left untouched.
 * sample_rows != NULL: global query-row ids; O is [H_q, n_sample, d] packed,
 *   lse [H_q, n_sample]; sampled rows of inactive chunks are left untouched. */
int fco_chunk_attention(const fco_attn_desc* desc, const void* Q,
                        const void* K, const void* V, int dtype,
                        const int32_t* q_chunk_row_off,
                        const int32_t* kv_visible_len,
                        const int32_t* seg_logical_off,
                        const int32_t* seg_phys_off, int n_seg,
                        const int32_t* kv_token_index, int64_t kv_index_hs,
                        const int32_t* active_ids, int n_active,
                        const int32_t* sample_rows, int n_sample, double* O,
                        int64_t o_hs, int64_t o_rs, double* lse,
                        int n_threads);

typedef struct {
  int32_t H_q, H_kv, d, L_q, L_k;
  int64_t q_hs, q_rs, k_hs, k_rs;
  double scale;  /* 0 => 1/sqrt(d) */
  double lambda; /* mixing coefficient of Eq. 12 */
  int32_t pool_k; /* odd max-pool window of Eq. 10 */
  int32_t red_mode;
} fco_score_desc;

/* Joint importance-redundancy score (Eqs. 9-12).
 *   Imp_j  = mean over the group's query heads and the L_q query rows of
 *            softmax_j(q K^T * scale)                                (Eq. 9)
 *   Imp~_j = max over |u| <= pool_k/2 of Imp_{j+u}, -inf padding     (Eq. 10)
 *   Red_j  = softmax_j( (1/L_k) sum_{i != j} khat_i . khat_j )       (Eq. 11)
 *   Score  = lambda*Imp~ - (1-lambda)*Red, rounded to fp32           (Eq. 12)
 * red_mode PLAIN builds the L_k x L_k cosine matrix, zeroes its diagonal and
 * takes column means; MEANKEY uses the appendix identity
 * (mean_i khat_i) . khat_j - |khat_j|^2 / L_k; AUTO = PLAIN up to 4096 tokens.
 * MAXSIM is a variant outside the paper that no mean key can express: the
 * softmax argument of token j is max_{i != j} khat_i . khat_j (0 if L_k = 1).
 * accum_phase: 0 single shot; 1 imp_accum += Imp, no outputs; 2 imp_accum +=
 * Imp, Imp := imp_accum / n_steps, then finalise.  Outputs other than score may
 * be NULL. */
int fco_kv_score(const fco_score_desc* desc, const void* Q_obs,
                 const void* K_cand, int dtype, double* imp_accum,
                 int accum_phase, int n_steps, double* imp, double* imp_pooled,
                 double* red, float* score, int n_threads);

/* The softmax argument of Eq. 11 for chosen columns only, by its plain
 * definition: out[h][c] = (1/L_k) sum_{i != j} khat_i . khat_j for j = cols[c]
 * (red_mode PLAIN) or max_{i != j} khat_i . khat_j (MAXSIM).  K_cand is
 * [n_heads, L_k, d] with strides k_hs, k_rs; out is [n_heads, n_cols]. */
int fco_key_similarity_columns(const void* K_cand, int dtype, int n_heads,
                               int L_k, int d, int64_t k_hs, int64_t k_rs,
                               const int32_t* cols, int n_cols, int red_mode,
                               double* out, int n_threads);

/* The softmax argument of Eq. 11 for chosen columns only, by its plain
 * definition: out[h][c] = (1/L_k) sum_{i != j} khat_i . khat_j for j = cols[c]
 * (red_mode PLAIN) or max_{i != j} khat_i . khat_j (MAXSIM).  K_cand is
 * [n_heads, L_k, d] with strides k_hs, k_rs; out is [n_heads, n_cols]. */
int fco_key_similarity_columns(const void* K_cand, int dtype, int n_heads,
                               int L_k, int d, int64_t k_hs, int64_t k_rs,
                               const int32_t* cols, int n_cols, int red_mode,
                               double* out, int n_threads);

/* Per-head top-B (Sec. 3.3, text after Eq. 12) and retention of the selected
 * K/V rows.  Total order: score descending, index ascending; NaN ranks as
 * -inf.  kept_idx[h] lists min(B, L_k) indices ascending; dst row r of head h
 * is src row kept_idx[h][r].  K/V pointers may all be NULL (select only). */
int fco_kv_select_compact(const float* score, int n_heads, int L_k, int B,
                          const void* K_src, const void* V_src, void* K_dst,
                          void* V_dst, int elem_bytes, int d, int64_t src_hs,
                          int64_t src_rs, int64_t dst_hs, int64_t dst_rs,
                          int32_t* kept_idx, int32_t* n_kept, int n_threads);

int fco_hardware_threads(void);

/* Selection at a coarser key granularity (key-granularity ablation, Table 4) and
 * with a protected tail: units of `unit` consecutive tokens (L_k and B multiples
 * of it) are kept or dropped as a whole; unit score = mean of its tokens' scores
 * (fp64 sum, rounded to fp32); the last ceil(n_protect / unit) units are always
 * kept; the others rank by (score desc, index asc), NaN as -inf.  kept_idx
 * [n_heads, min(B, L_k)] lists the kept tokens ascending.  unit = 1 and
 * n_protect = 0 is the selection of fco_kv_select_compact. */
int fco_kv_select_units(const float* score, int n_heads, int L_k, int B, int unit,
                        int n_protect, int32_t* kept_idx, int32_t* n_kept,
                        int n_threads);

#ifdef __cplusplus
}
#endif
#endif /* FC_ORACLE_H_ */
