// Host side of the tensor-core attention path (bf16): TMA tensor maps over Q, K and V, merging of adjacent
// segments, and the hand-over to the warp-specialised kernel in fc_attention_ws.cu.
#include <algorithm>
#include <climits>
#include <cmath>

#include "fc_attention.cuh"

namespace {
constexpr int kBM = 128;  // rows of a TMA box = rows of a query / key tile
}  // namespace

namespace fc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [heads, rows, d] bf16 tensor, box = 64 elements (128 bytes) x 128 rows x 1 head, 128-byte swizzle.
int make_tmap(fc_ctx* ctx, CUtensorMap* map, const void* base, int d, int64_t rows, int heads, int64_t row_stride,
              int64_t head_stride, int box_rows) {
  const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)rows, (cuuint64_t)heads};
  const cuuint64_t strides[2] = {(cuuint64_t)row_stride * 2, (cuuint64_t)head_stride * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = ((EncodeTiledFn)ctx->encode_tiled)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base),
                                                  dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    fc::set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return FC_ERR_CUDA;
  }
  return FC_OK;
}


// [all rows of all heads, d] bf16 view of a [heads, rows, d] tensor whose head stride is a whole number of rows:
// box = 64 elements x 1 row, 128-byte swizzle, for the tile::gather4 loads of the token-map path.
static int make_tmap_rows(fc_ctx* ctx, CUtensorMap* map, const void* base, int d, int64_t rows_total, int64_t row_stride) {
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows_total};
  const cuuint64_t strides[1] = {(cuuint64_t)row_stride * 2};
  const cuuint32_t box[2] = {64, 1};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = ((EncodeTiledFn)ctx->encode_tiled)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
                                                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    fc::set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return FC_ERR_CUDA;
  }
  return FC_OK;
}

size_t attention_tc_workspace_bytes() { return 256; }

bool attention_tc_supported(const AttnGeom& g, int dtype) {
  if (dtype != FC_BF16) return false;
  if (g.d != 64 && g.d != 128) return false;
  if (g.tok_index) {
    // the gathered rows are addressed as rows of one 2-D tensor over all heads: the head stride must be a whole
    // number of rows, and every row coordinate must fit 32 bits
    if (g.k_hs % g.k_rs || g.v_hs % g.v_rs) return false;
    if ((g.H_kv - 1) * (g.k_hs / g.k_rs) + g.kv_rows > INT32_MAX || (g.H_kv - 1) * (g.v_hs / g.v_rs) + g.kv_rows > INT32_MAX)
      return false;
  }
  // a head stride of 0 rows (single head) is fine; TMA needs the head stride to fit 2^40 bytes
  return true;
}

int attention_tc(fc_ctx* ctx, cudaStream_t st, const AttnGeom& g_in, const void* Q, const void* K, const void* V,
                 void* O, void* ws, size_t ws_bytes) {
  if (!ws || ws_bytes < attention_tc_workspace_bytes()) return FC_ERR_WORKSPACE;
  if (!aligned16(ws)) return FC_ERR_MISALIGNED;
  AttnGeom g = g_in;
  if (g.tok_index) {  // one logical segment; its tokens are found through the map
    g.n_seg = 1;
    g.seg_log[0] = 0;
    g.seg_log[1] = (int32_t)std::min<int64_t>(g.tok_hs, INT32_MAX);
    g.seg_phys[0] = 0;
  }
  // merge logically adjacent segments that are also physically adjacent: fewer ragged tails
  int n = 0;
  for (int s = 0; s < (g.tok_index ? 0 : g_in.n_seg); ++s) {
    const int len = g_in.seg_log[s + 1] - g_in.seg_log[s];
    if (len == 0) continue;
    if (n > 0 && g.seg_phys[n - 1] + (g.seg_log[n] - g.seg_log[n - 1]) == g_in.seg_phys[s]) {
      g.seg_log[n] = g_in.seg_log[s + 1];
    } else {
      g.seg_phys[n] = g_in.seg_phys[s];
      g.seg_log[n] = g_in.seg_log[s];
      g.seg_log[n + 1] = g_in.seg_log[s + 1];
      ++n;
    }
  }
  if (!g.tok_index) g.n_seg = n;
  int64_t q_rows = g.q_row_off[g.W];
  int max_tiles = 0;
  for (int c = 0; c < g.W; ++c) max_tiles += (g.q_row_off[c + 1] - g.q_row_off[c] + kBM - 1) / kBM;
  if (max_tiles == 0 || q_rows == 0) return FC_OK;
  CUtensorMap tq, tk, tv;
  int rc;
  if ((rc = make_tmap(ctx, &tq, Q, g.d, q_rows, g.H_q, g.q_rs, g.H_q > 1 ? g.q_hs : g.q_rs * q_rows)) != FC_OK) return rc;
  if (g.tok_index) {
    if ((rc = make_tmap_rows(ctx, &tk, K, g.d, (g.H_kv - 1) * (g.k_hs / g.k_rs) + g.kv_rows, g.k_rs)) != FC_OK) return rc;
    if ((rc = make_tmap_rows(ctx, &tv, V, g.d, (g.H_kv - 1) * (g.v_hs / g.v_rs) + g.kv_rows, g.v_rs)) != FC_OK) return rc;
  } else {
    if ((rc = make_tmap(ctx, &tk, K, g.d, g.kv_rows, g.H_kv, g.k_rs, g.H_kv > 1 ? g.k_hs : g.k_rs * g.kv_rows)) != FC_OK) return rc;
    if ((rc = make_tmap(ctx, &tv, V, g.d, g.kv_rows, g.H_kv, g.v_rs, g.H_kv > 1 ? g.v_hs : g.v_rs * g.kv_rows)) != FC_OK) return rc;
  }
  return attention_ws_launch(ctx, st, g, tq, tk, tv, O, (uint32_t*)ws);
}

}  // namespace fc
