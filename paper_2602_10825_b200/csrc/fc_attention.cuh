// Geometry shared by the two attention kernels of libfc (CUDA-core and tcgen05).
#pragma once

#include <cuda.h>

#include "fc_common.cuh"

namespace fc {

struct AttnGeom {
  int32_t H_q, H_kv, d, W, group, n_seg;
  int64_t q_hs, q_rs, k_hs, k_rs, v_hs, v_rs, o_hs, o_rs, kv_rows, lse_hs, tok_hs;
  float scale;
  int32_t q_row_off[FC_MAX_CHUNKS + 1];
  int32_t vis[FC_MAX_CHUNKS];
  int32_t seg_log[FC_MAX_SEGMENTS + 1];
  int32_t seg_phys[FC_MAX_SEGMENTS];
  const int32_t* tok_index;
  const int32_t* active_ids;
  const int32_t* n_active;
  float* lse;
  uint32_t* status;
};

int attention_simt(cudaStream_t st, const AttnGeom& g, const void* Q, const void* K, const void* V,
                   int dtype, void* O);
// bf16 only: builds the tensor maps and launches the warp-specialised tcgen05 kernel.
int attention_tc(fc_ctx* ctx, cudaStream_t st, const AttnGeom& g, const void* Q, const void* K,
                 const void* V, void* O, void* ws, size_t ws_bytes);
size_t attention_tc_workspace_bytes();
// warp-specialised kernel; tensor maps as built by attention_tc, `counter` = 4 bytes of workspace
int attention_ws_launch(fc_ctx* ctx, cudaStream_t st, const AttnGeom& g, const CUtensorMap& tq,
                        const CUtensorMap& tk, const CUtensorMap& tv, void* O, uint32_t* counter);
bool attention_tc_supported(const AttnGeom& g, int dtype);
// Tensor map of a [heads, rows, d] bf16 tensor: box = 64 elements (128 bytes) x `box_rows` rows x 1 head, 128-byte
// swizzle; rows past `rows` read as zero.
int make_tmap(fc_ctx* ctx, CUtensorMap* map, const void* base, int d, int64_t rows, int heads, int64_t row_stride,
              int64_t head_stride, int box_rows = 128);

}  // namespace fc
