/*
 * fc.h — C ABI of the FlowCache hot path for NVIDIA B200 (sm_100a).
 *
 * FlowCache (arXiv 2602.10825) is a chunkwise caching scheme for autoregressive
 * video diffusion transformers.  This library implements the per-denoising-step
 * chunk pipeline as four calls, all enqueued on a caller-supplied CUDA stream:
 *
 *   fc_chunk_decide       which chunks are recomputed at this step   (Eqs. 5, 8)
 *   fc_chunk_attention    attention of the recomputed chunks' queries over the
 *                         fixed-budget KV cache plus the denoising window (Sec. 3.3)
 *   fc_kv_score           importance / redundancy score of cached tokens (Eqs. 9-12)
 *   fc_kv_select_compact  per-head top-B and retention of the chosen K/V rows
 *
 * and a fifth for the step around the forward pass:
 *
 *   fc_chunk_cache_apply  chunks that were not recomputed are served from the
 *                         activation cache (Sec. 3.2)
 *
 * Conventions
 *   - Plain C types only.  Every pointer argument says whether it is a HOST or a
 *     DEVICE pointer.  The caller owns every buffer, including the workspace,
 *     whose size the matching fc_*_workspace_bytes() returns.  No call allocates
 *     or frees device memory, synchronises the host with the device, or uses a
 *     stream other than `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream).
 *   - Tensors are [heads, tokens, d] with d contiguous and explicit head / token
 *     strides counted in elements.  Device base pointers must be 16-byte aligned
 *     and every stride a multiple of 16 bytes.
 *   - dtype is the storage type of the tensors (FC_BF16 or FC_F32); sums and
 *     softmax statistics are always kept in fp32 or wider.
 *   - Return value: FC_OK (0) or a negative fc_status.  On an error nothing has
 *     been launched.  Data-dependent conditions that can only be seen on the
 *     device (a NaN score, a bounded wait that expired) set bits in the optional
 *     DEVICE word `status` (OR-ed in, never cleared by the library); the caller
 *     reads it after its own synchronisation.
 *   - The library keeps no state between calls except immutable per-device
 *     attributes inside fc_ctx.  Calls on different streams may overlap as long
 *     as their buffers and workspaces do not.
 *   - One exception to the two points above: fc_chunk_decide_static takes no
 *     workspace; its scratch is an array inside the library that all its calls
 *     on a device share (see its comment for what that implies).
 */
#ifndef FC_H_
#define FC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FC_OK = 0,
  FC_ERR_INVALID_ARG = -1, /* NULL where a pointer is required, negative size, even pool_k ... */
  FC_ERR_UNSUPPORTED = -2, /* d not in {64,128}, unknown dtype, too many chunks / segments */
  FC_ERR_MISALIGNED = -3,  /* a base pointer or stride is not a multiple of 16 bytes */
  FC_ERR_WORKSPACE = -4,   /* ws is NULL or ws_bytes is below fc_*_workspace_bytes() */
  FC_ERR_DEVICE = -5,      /* the device is not compute capability 10.x */
  FC_ERR_CUDA = -6,        /* a CUDA runtime / driver call failed (see fc_last_cuda_error) */
  FC_ERR_UNIMPLEMENTED = -7,
  FC_ERR_TOO_LARGE = -8    /* the problem needs more scratch than a no-allocation entry point holds */
} fc_status;

typedef enum { FC_BF16 = 0, FC_F32 = 1 } fc_dtype;

/* Reuse policy of fc_chunk_decide: the paper's chunkwise rule, or the uniform policy it compares with. */
typedef enum { FC_POLICY_CHUNKWISE = 0, FC_POLICY_UNIFORM = 1 } fc_policy;

/* Bits of the device status word. */
enum {
  FC_DEV_TIMEOUT = 1u,   /* a bounded in-kernel wait expired; the affected outputs are invalid */
  FC_DEV_NAN_SCORE = 2u, /* a NaN score was ranked as -inf by the selection */
  FC_DEV_BAD_INDEX = 4u  /* an index read from device memory was out of range and was skipped */
};

enum { FC_MAX_CHUNKS = 64, FC_MAX_SEGMENTS = 64 };

typedef struct fc_ctx fc_ctx;

/* Create / destroy a context for CUDA device `device` (made current by the call).  Reads the
 * device attributes (SM count, shared-memory limit) and resolves the driver entry point used to
 * encode TMA tensor maps.  Fails with FC_ERR_DEVICE unless the device is compute capability 10.x. */
int fc_create(fc_ctx** out, int device);
int fc_destroy(fc_ctx* ctx);
const char* fc_status_string(int status);
/* Text of the last CUDA error a call on this thread ran into ("" if none). */
const char* fc_last_cuda_error(void);
/* Number of SMs the context's persistent kernels size their grids by. */
int fc_sm_count(const fc_ctx* ctx);

/* Self-test of the bounded waits (no counterpart in the paper).  Every wait on a barrier inside the tensor-core
 * kernels gives up after a wall-time limit instead of spinning forever; the kernel then runs to its normal end
 * and sets FC_DEV_TIMEOUT.  This call launches one warp that waits, with the same routine and a limit of
 * `limit_ns` (clamped to 1 us .. 1 s), on a barrier nobody signals.  After the caller's synchronisation `status`
 * (DEVICE, required) has FC_DEV_TIMEOUT set and `waited_ns` (DEVICE [1] or NULL) holds how long the warp waited.
 * Nothing faults or hangs; the context stays usable. */
int fc_selftest_bounded_wait(fc_ctx* ctx, void* stream, uint64_t limit_ns, uint32_t* status, uint32_t* waited_ns);

/* ------------------------------------------------------------------------------------------
 * fc_chunk_decide — per-chunk reuse decision.
 *
 * Paper: the relative L1 distance of chunk i between consecutive denoising steps (Eq. 5, the
 * per-chunk form of Eq. 4) is accumulated per chunk and compared with a threshold (Eq. 8):
 *     r_i = sum|cur_i - prev_i| / sum|prev_i|           (the denominator is the earlier state)
 *     s_i = acc_i + r_i                                 (fp32)
 *     recompute_i = chunk_step[i] < warmup_m  ||  force[i]  ||  s_i > eps      (strict)
 *     acc_i <- 0 if recompute_i else s_i
 * A zero denominator yields r = +inf if the numerator is positive, else 0.
 *
 * policy = FC_POLICY_UNIFORM is the "traditional reuse" the paper compares with (caption of Fig. 3): all chunks of
 * a step share one compute / reuse status, except chunks that must be computed anyway (chunk_step[i] < warmup_m
 * or force[i]: a newly initialised chunk).  Over the sharing chunks S taken as one tensor (Eq. 4):
 *     r = sum_S |cur - prev| / sum_S |prev|,   s = acc[first chunk of S] + r   (fp32)
 *     recompute_i = (i not in S) || s > eps;   every acc[i] <- 0 if s > eps (or S is empty) else s
 * and l1rel[i] = r for i in S, the chunk's own indicator otherwise.
 *
 *   cur, prev        DEVICE, `dtype` elements; chunk i occupies elements
 *                    [chunk_elem_off[i], chunk_elem_off[i+1]) of both.  The vectorised path
 *                    is taken when every offset is a multiple of 16 bytes.
 *   chunk_elem_off   HOST [n_chunks+1], non-decreasing; n_chunks <= FC_MAX_CHUNKS.
 *   chunk_step       DEVICE [n_chunks]: number of steps chunk i has already taken.
 *   force            DEVICE [n_chunks] or NULL: non-zero forces a recompute (a newly
 *                    initialised chunk must be computed).
 *   acc              DEVICE [n_chunks], in/out: the accumulator f of Eq. 8.
 *   l1rel            DEVICE [n_chunks] out or NULL: r_i.
 *   recompute        DEVICE [n_chunks] out: 1 = recompute, 0 = serve from cache.
 *   active_ids       DEVICE [n_chunks] out: ids of recomputed chunks, ascending; entries at
 *                    and after n_active are set to -1.
 *   n_active         DEVICE [1] out.
 * Sums are fixed-order (run-to-run bit-reproducible): fp32 inside a thread's 32-element run,
 * fp64 above that.  Workspace: fc_chunk_decide_workspace_bytes(total elements, n_chunks). */
size_t fc_chunk_decide_workspace_bytes(int64_t total_elems, int n_chunks);
int fc_chunk_decide(fc_ctx* ctx, void* stream, const void* cur, const void* prev, int dtype,
                    const int64_t* chunk_elem_off, int n_chunks, const int32_t* chunk_step,
                    int warmup_m, float eps, const uint8_t* force, int policy, float* acc, float* l1rel,
                    uint8_t* recompute, int32_t* active_ids, int32_t* n_active,
                    uint32_t* status, void* ws, size_t ws_bytes);

/* fc_chunk_decide_static — fc_chunk_decide without a workspace argument.
 *
 * The paper has no counterpart: this entry point exists for callers that may not allocate device
 * memory at the point of the call — code running inside a memory-pool or allocator callback, a
 * real-time loop that must not touch the allocator, a host that was handed fixed buffers by
 * another runtime — and therefore have no workspace to pass.  The (num, den) slab pairs go to an
 * array of fc_chunk_decide_static_max_bytes() = 1 MiB that is part of the library image: every
 * GPU that loads the library holds it until the process exits.  Inputs, outputs and semantics are
 * exactly those of fc_chunk_decide.
 *
 *   - Limit: fc_chunk_decide_workspace_bytes(total elements, n_chunks) must not exceed the
 *     array, which holds 65,536 slab pairs: about 268 million elements over all chunks together,
 *     whatever the dtype.  Beyond it the call returns FC_ERR_TOO_LARGE and launches nothing.
 *   - The call never allocates or frees device memory.  The array's device address is looked up
 *     once per device (a driver query, made with that device current) by fc_create; should that
 *     have failed, the first call on the device repeats it, so create the context, or make that
 *     first call, before starting any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents.
 *     Nothing in it has to start at zero (each slab pair is written before it is read), but two
 *     calls that overlap on the GPU (different streams, no dependency) race on it: serialise
 *     them, or use fc_chunk_decide with separate workspaces. */
size_t fc_chunk_decide_static_max_bytes(void);
int fc_chunk_decide_static(fc_ctx* ctx, void* stream, const void* cur, const void* prev, int dtype,
                           const int64_t* chunk_elem_off, int n_chunks, const int32_t* chunk_step,
                           int warmup_m, float eps, const uint8_t* force, int policy, float* acc, float* l1rel,
                           uint8_t* recompute, int32_t* active_ids, int32_t* n_active,
                           uint32_t* status);

/* ------------------------------------------------------------------------------------------
 * fc_chunk_cache_apply — serving the chunks that were not recomputed from the activation cache.
 *
 * Paper (Sec. 3.2, text after Eq. 8): when the rule says reuse, the chunk's cached activations are
 * reused instead of a forward pass; the cache is one tensor the size of the model input (efficiency
 * appendix).  The cache holds, per chunk, the residual output - input of the chunk's last computed
 * forward; a reused chunk's output is its current input plus that residual.  For every element e of
 * chunk i (flat layout as in fc_chunk_decide):
 *     recompute[i] != 0:  cache[e] <- y[e] - x[e]       (y holds the fresh output of the forward)
 *     recompute[i] == 0:  y[e]     <- x[e] + cache[e]   (the cache is left as it is)
 * in fp32, rounded once to `dtype` (round to nearest even for bf16).  Call it after the forward of
 * the active chunks, with the recompute flags fc_chunk_decide left on the device.
 *
 *   x_in             DEVICE, `dtype`: the chunks' inputs at this step.
 *   y_io             DEVICE, `dtype`, in/out: outputs; only skipped chunks are written.
 *   cache            DEVICE, `dtype`, in/out: only computed chunks are written.
 *   chunk_elem_off   HOST [n_chunks+1]; recompute DEVICE [n_chunks].
 * The three tensors must not overlap.  Needs no workspace.  Moves 3 x (elements x element size)
 * bytes with 16-byte accesses when every offset is a multiple of 16 bytes. */
int fc_chunk_cache_apply(fc_ctx* ctx, void* stream, const void* x_in, void* y_io, void* cache, int dtype,
                         const int64_t* chunk_elem_off, int n_chunks, const uint8_t* recompute,
                         uint32_t* status);

/* ------------------------------------------------------------------------------------------
 * fc_chunk_attention — chunk-causal attention of the active chunks.
 *
 * Paper (Sec. 3.3): the chunks being denoised attend to the compressed clean-chunk region of
 * the KV buffer followed by the current denoising region; generation is causal over chunks.
 * For every active chunk c, head h and query row r of c:
 *     O[h, r, :] = softmax_j( Q[h, r, :] . K[g(h), p(j), :] * scale ) V[g(h), p(j), :],
 *     j over the first kv_visible_len[c] LOGICAL tokens, g(h) = h / (H_q / H_kv),
 * where p maps a logical token to a physical row of the K/V store: through the segment table
 * (logical range [seg_logical_off[s], seg_logical_off[s+1]) starts at physical row
 * seg_phys_off[s]) or, if given, through the per-head token map kv_token_index[g][j] (this is
 * how a cache is read through the kept-index list of fc_kv_select_compact without moving it).
 * All tokens of a chunk's own range are visible to all its rows (no mask inside a chunk).
 * Rows of chunks that are not in active_ids are never written: their cached outputs stay.
 */
typedef struct {
  int32_t H_q, H_kv, d, W;                   /* query heads, kv heads, head dim (64|128), chunks */
  int64_t q_hs, q_rs, k_hs, k_rs, v_hs, v_rs; /* element strides: head, row */
  int64_t o_hs, o_rs;
  int64_t kv_rows;                           /* physical rows per head in the K/V store */
  float scale;                               /* 0 => 1/sqrt(d) */
  int32_t impl;                              /* 0 auto; 1 force the CUDA-core kernel; 2 force the tcgen05
                                                kernel (FC_ERR_UNSUPPORTED where it does not apply) */
} fc_attn_desc;

/*   Q, O             DEVICE [H_q, rows, d]; K, V DEVICE [H_kv, kv_rows, d]; `dtype` elements.
 *   q_chunk_row_off  HOST [W+1]: chunk c owns query rows [off[c], off[c+1]).  W <= FC_MAX_CHUNKS.
 *   kv_visible_len   HOST [W].
 *   seg_logical_off  HOST [n_seg+1], seg_phys_off HOST [n_seg]; n_seg <= FC_MAX_SEGMENTS.
 *                    Ignored (may be NULL, n_seg 0) when kv_token_index is given.
 *   kv_token_index   DEVICE [H_kv, kv_index_hs] int32 or NULL.
 *   active_ids       DEVICE [<= W], n_active DEVICE [1] (as written by fc_chunk_decide): the
 *                    work list is read on the device, so no host synchronisation is needed
 *                    between the decision and the attention.
 *   lse              DEVICE [H_q, lse_hs] fp32 or NULL: natural-log sum-exp of each computed row.
 * bf16 runs on tcgen05 tensor cores (fp32 accumulation in tensor memory, TMA-fed); fp32 runs
 * on CUDA cores with fp32 accumulation.  With a token map the tensor-core kernel fetches K / V rows
 * by index (four rows per copy instruction), at roughly three quarters of the segment-table rate;
 * it needs K's and V's head strides to be whole numbers of rows, otherwise the CUDA-core kernel
 * takes the call.  An index outside [0, kv_rows) sets FC_DEV_BAD_INDEX and is not followed.
 * Physical rows that no visible logical token maps to (rows behind a segment's end, slots of
 * the store that were never written) are never used, whatever they hold.
 * Workspace: fc_chunk_attention_workspace_bytes(). */
size_t fc_chunk_attention_workspace_bytes(const fc_attn_desc* desc);
int fc_chunk_attention(fc_ctx* ctx, void* stream, const fc_attn_desc* desc, const void* Q,
                       const void* K, const void* V, int dtype, const int32_t* q_chunk_row_off,
                       const int32_t* kv_visible_len, const int32_t* seg_logical_off,
                       const int32_t* seg_phys_off, int n_seg, const int32_t* kv_token_index,
                       int64_t kv_index_hs, const int32_t* active_ids, const int32_t* n_active,
                       void* O, float* lse, int64_t lse_hs, uint32_t* status, void* ws,
                       size_t ws_bytes);

/* ------------------------------------------------------------------------------------------
 * fc_kv_score — joint importance / redundancy score of the candidate tokens.
 *
 * Paper: Imp_j = mean over the observation queries (and the query heads of a kv head's group)
 * of softmax_j(q K_cand^T * scale) (Eq. 9); Imp~ = stride-1 max-pool of width pool_k with
 * -inf padding (Eq. 10); Red_j = softmax_j of the column means of the cosine-similarity matrix
 * of the l2-normalised keys with a zeroed diagonal (Eq. 11), evaluated through the mean-key
 * identity of the paper's efficiency appendix, column mean_j = (mean_i khat_i).khat_j -
 * |khat_j|^2 / L_k, with khat = k / max(|k|, 1e-12); Score = lambda*Imp~ - (1-lambda)*Red (Eq. 12).
 *
 * Query granularity (the paper's ablation of token / frame / chunk observation queries): up to
 * 128 query rows per kv head take the streaming pipelines (the paper's setting, the last 50
 * tokens); more than that - a latent frame or a whole chunk of queries, bf16, H_q == H_kv, up
 * to 8192 - take the frame-level pipeline, in which both passes over the logits run on the
 * tensor cores.
 */
/* How the softmax argument of the redundancy (Eq. 11) is evaluated.
 *   FC_RED_MEANKEY    the mean-key identity of the efficiency appendix (default; O(L_k d) per head)
 *   FC_RED_TILED      Eq. 11 as written: 128 x 128 tiles of the cosine matrix on the tensor cores, diagonal
 *                     zeroed, column sums in the epilogue, the matrix never stored (O(L_k^2 d) per head: the
 *                     dense work the identity avoids; for checking it and as the base of the next mode)
 *   FC_RED_TILED_MAX  not in the paper: the column MAXIMUM over the other tokens instead of the column mean,
 *                     a statistic no mean key can express (same tiles, another epilogue)
 * The tiled modes need bf16 keys. */
typedef enum { FC_RED_MEANKEY = 0, FC_RED_TILED = 1, FC_RED_TILED_MAX = 2 } fc_red_mode;

typedef struct {
  int32_t H_q, H_kv, d, L_q, L_k;  /* n = L_q * (H_q/H_kv) queries per kv head: n <= 128, or bf16 with n <= 8192 and
                                      either H_q == H_kv or the query heads stored one after the other (q_hs = L_q q_rs) */
  int64_t q_hs, q_rs, k_hs, k_rs;  /* element strides */
  float scale;                     /* 0 => 1/sqrt(d) */
  float lambda;                    /* mixing coefficient (paper: 0.07) */
  int32_t pool_k;                  /* odd, >= 1 */
  int32_t impl;                    /* 0 auto; 1 force the CUDA-core kernels; 2 force tcgen05 */
  int32_t red_mode;                /* fc_red_mode */
} fc_score_desc;

/*   Q_obs            DEVICE [H_q, L_q, d]; K_cand DEVICE [H_kv, L_k, d]; `dtype` elements.
 *   imp_accum        DEVICE [H_kv, L_k] fp32 or NULL; accum_phase: 0 single shot (imp_accum
 *                    unused); 1 imp_accum += Imp of this call, nothing else is written; 2
 *                    imp_accum += Imp, then Imp := imp_accum / n_steps and the scores are
 *                    finalised (mean importance over the steps of a chunk).
 *   imp, red         DEVICE [H_kv, L_k] fp32 out, either may be NULL.
 *   score            DEVICE [H_kv, L_k] fp32 out (required unless accum_phase == 1).
 * Deterministic: no floating-point atomics.  Workspace: fc_kv_score_workspace_bytes(). */
size_t fc_kv_score_workspace_bytes(const fc_score_desc* desc);
int fc_kv_score(fc_ctx* ctx, void* stream, const fc_score_desc* desc, const void* Q_obs,
                const void* K_cand, int dtype, float* imp_accum, int accum_phase, int n_steps,
                float* imp, float* red, float* score, uint32_t* status, void* ws,
                size_t ws_bytes);

/* ------------------------------------------------------------------------------------------
 * fc_kv_select_compact — per-head top-B and retention of the selected rows.
 *
 * Paper: for each head keep the B tokens with the highest Score (text after Eq. 12); the kept
 * K/V form the compressed clean region (Sec. 3.3).  Total order: score descending, index
 * ascending (so ties keep the lowest indices); NaN ranks as -inf and sets FC_DEV_NAN_SCORE;
 * -0 equals +0.  B >= L_k keeps everything (identity).
 *
 *   score            DEVICE [n_heads, L_k] fp32.
 *   K_src, V_src     DEVICE [n_heads, L_k, d] with strides src_hs / src_rs (elements);
 *   K_dst, V_dst     DEVICE [n_heads, >= min(B,L_k), d] with strides dst_hs / dst_rs; must not
 *                    overlap the sources.  All four NULL => selection only.
 *   kept_idx         DEVICE [n_heads, min(B, L_k)] int32 out, ascending per head.
 *   n_kept           DEVICE [1] out or NULL: min(B, L_k).
 * Row r of head h of the destination is source row kept_idx[h][r], copied byte for byte with
 * 16-byte accesses; bytes outside the kept rows are not touched; dropped rows are not read. */
typedef struct {
  int64_t src_hs, src_rs, dst_hs, dst_rs;
} fc_compact_strides;

size_t fc_kv_select_compact_workspace_bytes(int n_heads, int L_k);
int fc_kv_select_compact(fc_ctx* ctx, void* stream, const float* score, int n_heads, int L_k,
                         int B, const void* K_src, const void* V_src, void* K_dst, void* V_dst,
                         int dtype, int d, const fc_compact_strides* strides, int32_t* kept_idx,
                         int32_t* n_kept, uint32_t* status, void* ws, size_t ws_bytes);

/* fc_kv_select_compact_ex — the same selection at a coarser key granularity and / or with a protected tail.
 *
 * Paper: the key-granularity ablation (Table 4) compresses with frame- or chunk-level keys instead of tokens (and
 * finds token-level keys best, which is why fc_kv_select_compact is the default).  Here a unit is `unit`
 * consecutive tokens (a latent frame, a chunk), kept or dropped as a whole; a unit's score is the mean of its
 * tokens' scores (fp64 sum, rounded to fp32); L_k and B must be whole numbers of units.  n_protect (not in the
 * paper) keeps the units of the last n_protect tokens - the newest ones - whatever their score; the others rank
 * by (score descending, index ascending), NaN as -inf.  unit = 1, n_protect = 0 is fc_kv_select_compact.
 * Workspace (only for unit > 1): fc_kv_select_compact_ex_workspace_bytes().  All other arguments as above;
 * kept_idx lists the kept tokens ascending, n_kept = min(B, L_k). */
typedef struct {
  int32_t unit;      /* tokens per selection unit, >= 1 */
  int32_t n_protect; /* newest tokens always kept, >= 0 */
} fc_select_opts;

size_t fc_kv_select_compact_ex_workspace_bytes(int n_heads, int L_k, int unit);
int fc_kv_select_compact_ex(fc_ctx* ctx, void* stream, const float* score, int n_heads, int L_k, int B,
                            const fc_select_opts* opts, const void* K_src, const void* V_src, void* K_dst,
                            void* V_dst, int dtype, int d, const fc_compact_strides* strides, int32_t* kept_idx,
                            int32_t* n_kept, uint32_t* status, void* ws, size_t ws_bytes);

#ifdef __cplusplus
}
#endif
#endif /* FC_H_ */
