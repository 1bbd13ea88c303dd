// Interface between fc_kv_score's front end (fc_score.cu) and its tensor-core kernels (fc_score_tc.cu).
#pragma once

#include <cuda_runtime.h>

#include "fc_common.cuh"

namespace fc {

constexpr int kScoreTcMaxQueries = 64;  // query rows of the tensor-core path: observation queries (at most 62, zero-
                                        // padded) and two rows for the mean key
constexpr int kScoreTcMaxSlices = 64;   // slices of key tiles per head
constexpr int kScoreFrameMaxQueries = 8192;  // observation queries of the frame-level path
constexpr int kScoreFrameMaxSlices = 16;     // slices of the key range in its row-statistics launch

struct ScoreTcArgs {
  int H, L_q, L_k, n_tiles, tiles_per_slice, n_slices;  // n_tiles = ceil(L_k / 128); slices are set by score_tc_run
  float scale_log2;                                     // softmax scale times log2(e)
  int accum_phase, n_steps;
  float2* ml_part;     // [H, n_slices, 64] running (max, sum) of pass 1, log2 domain
  float* colsum_part;  // [H, n_slices, d] sums of normalised keys
  float* norm2;        // [H, L_k] squared l2 norm of every key (pass 1 -> pass 2)
  float* imp_accum;    // caller's accumulator or NULL
  float* imp_out;      // [H, L_k]
  float* a_out;        // [H, L_k] redundancy logits
  float2* a_partial;   // [H, n_tiles * 4] softmax statistics (max, sum of exp) of a per 32 keys (one warp of a tile)
  uint32_t* status;
};

// pass 1, pass 2; the caller runs the finalize kernel afterwards (unless accum_phase == 1)
int score_tc_run(fc_ctx* ctx, cudaStream_t st, ScoreTcArgs args, int d, int64_t q_hs, int64_t q_rs, int64_t k_hs,
                 int64_t k_rs, const void* Q, const void* K);

// Redundancy from explicit tiles of the cosine-similarity matrix (fc_score_red.cu).
struct RedTiledArgs {
  int H, L_k, n_tiles;  // n_tiles = ceil(L_k / 128)
  float* inv_norm;      // [H, n_tiles * 128] scratch: 1 / max(|k|, 1e-12), 0 past the end of the cache
  float* a_out;         // [H, L_k] softmax argument of the redundancy
  float2* a_partial;    // [H, n_tiles * 4] (max, sum of exp) of a per 32 keys
  uint32_t* status;
};
// a_j = column mean of the cosine matrix with zeroed diagonal (Eq. 11), or with `max_similarity` the largest
// similarity of token j to another token; bf16 keys only
int score_red_tiled(fc_ctx* ctx, cudaStream_t st, RedTiledArgs args, int d, int64_t k_hs, int64_t k_rs, const void* K,
                    bool max_similarity);

// Frame-level query granularity on tensor cores (bf16, one query head per key head): first every query's (maximum,
// sum) over slices of the candidates into `ml_part` ([H, kScoreFrameMaxSlices, L_q] at most, log2 domain), their
// merge into `nlse` ([H, L_q], minus the log2-domain log-sum-exp), then mass[h, j] = sum_i exp(q_i . k_j * scale -
// lse[h, i]) ([H, L_k] dense).
int score_frame_mass(fc_ctx* ctx, cudaStream_t st, int H, int d, int L_q, int L_k, float scale_log2, const void* Q,
                     int64_t q_hs, int64_t q_rs, const void* K, int64_t k_hs, int64_t k_rs, float2* ml_part, float* nlse,
                     float* mass, uint32_t* status);

}  // namespace fc
