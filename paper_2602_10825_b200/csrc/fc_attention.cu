// fc_chunk_attention: argument validation and the choice between the tcgen05 kernel (bf16,
// segment-table addressing) and the CUDA-core kernel (fp32 tensors, token-level index maps).
#include <cmath>

#include "fc_attention.cuh"

extern "C" size_t fc_chunk_attention_workspace_bytes(const fc_attn_desc* desc) {
  (void)desc;
  return fc::attention_tc_workspace_bytes();
}

extern "C" int fc_chunk_attention(fc_ctx* ctx, void* stream, const fc_attn_desc* desc, const void* Q,
                                  const void* K, const void* V, int dtype, const int32_t* q_chunk_row_off,
                                  const int32_t* kv_visible_len, const int32_t* seg_logical_off,
                                  const int32_t* seg_phys_off, int n_seg, const int32_t* kv_token_index,
                                  int64_t kv_index_hs, const int32_t* active_ids, const int32_t* n_active,
                                  void* O, float* lse, int64_t lse_hs, uint32_t* status, void* ws,
                                  size_t ws_bytes) {
  if (!ctx || !desc || !Q || !K || !V || !O || !q_chunk_row_off || !kv_visible_len || !active_ids || !n_active)
    return FC_ERR_INVALID_ARG;
  if (dtype != FC_BF16 && dtype != FC_F32) return FC_ERR_UNSUPPORTED;
  if (desc->d != 64 && desc->d != 128) return FC_ERR_UNSUPPORTED;
  if (desc->H_q <= 0 || desc->H_kv <= 0 || desc->H_q % desc->H_kv || desc->W <= 0 || desc->kv_rows <= 0)
    return FC_ERR_INVALID_ARG;
  if (desc->W > FC_MAX_CHUNKS) return FC_ERR_UNSUPPORTED;
  if (desc->impl < 0 || desc->impl > 2) return FC_ERR_INVALID_ARG;
  if (!(desc->scale >= 0.f)) return FC_ERR_INVALID_ARG;  // 0 selects 1/sqrt(d); the kernels assume a positive scale
  if (!kv_token_index) {
    if (!seg_logical_off || !seg_phys_off || n_seg <= 0) return FC_ERR_INVALID_ARG;
    if (n_seg > FC_MAX_SEGMENTS) return FC_ERR_UNSUPPORTED;
  } else if (kv_index_hs <= 0) {
    return FC_ERR_INVALID_ARG;
  }
  const int es = fc::elem_size(dtype);
  if (!fc::aligned16(Q) || !fc::aligned16(K) || !fc::aligned16(V) || !fc::aligned16(O)) return FC_ERR_MISALIGNED;
  const int64_t strides[8] = {desc->q_hs, desc->q_rs, desc->k_hs, desc->k_rs,
                              desc->v_hs, desc->v_rs, desc->o_hs, desc->o_rs};
  for (int i = 0; i < 8; ++i)
    if (strides[i] < 0 || (strides[i] * es) % 16) return FC_ERR_MISALIGNED;
  if (desc->q_rs < desc->d || desc->k_rs < desc->d || desc->v_rs < desc->d || desc->o_rs < desc->d)
    return FC_ERR_INVALID_ARG;
  if (lse && lse_hs <= 0) return FC_ERR_INVALID_ARG;

  fc::AttnGeom g;
  g.H_q = desc->H_q; g.H_kv = desc->H_kv; g.d = desc->d; g.W = desc->W;
  g.group = desc->H_q / desc->H_kv;
  g.q_hs = desc->q_hs; g.q_rs = desc->q_rs; g.k_hs = desc->k_hs; g.k_rs = desc->k_rs;
  g.v_hs = desc->v_hs; g.v_rs = desc->v_rs; g.o_hs = desc->o_hs; g.o_rs = desc->o_rs;
  g.kv_rows = desc->kv_rows; g.lse_hs = lse_hs; g.tok_hs = kv_index_hs;
  g.scale = desc->scale != 0.f ? desc->scale : 1.f / sqrtf((float)desc->d);
  for (int c = 0; c <= g.W; ++c) {
    g.q_row_off[c] = q_chunk_row_off[c];
    if (q_chunk_row_off[c] < 0 || (c > 0 && q_chunk_row_off[c] < q_chunk_row_off[c - 1])) return FC_ERR_INVALID_ARG;
  }
  int64_t logical_len = kv_token_index ? kv_index_hs : 0;
  g.n_seg = kv_token_index ? 0 : n_seg;
  if (!kv_token_index) {
    for (int s = 0; s <= n_seg; ++s) {
      g.seg_log[s] = seg_logical_off[s];
      if (s == 0 ? seg_logical_off[0] != 0 : seg_logical_off[s] < seg_logical_off[s - 1]) return FC_ERR_INVALID_ARG;
    }
    for (int s = 0; s < n_seg; ++s) {
      g.seg_phys[s] = seg_phys_off[s];
      const int64_t len = seg_logical_off[s + 1] - seg_logical_off[s];
      if (seg_phys_off[s] < 0 || seg_phys_off[s] + len > desc->kv_rows) return FC_ERR_INVALID_ARG;
    }
    logical_len = seg_logical_off[n_seg];
  }
  for (int c = 0; c < g.W; ++c) {
    g.vis[c] = kv_visible_len[c];
    if (kv_visible_len[c] < 0 || kv_visible_len[c] > logical_len) return FC_ERR_INVALID_ARG;
  }
  g.tok_index = kv_token_index;
  g.active_ids = active_ids;
  g.n_active = n_active;
  g.lse = lse;
  g.status = status;

  cudaStream_t st = (cudaStream_t)stream;
  const bool tc_ok = fc::attention_tc_supported(g, dtype);
  if (desc->impl >= 2 && !tc_ok) return FC_ERR_UNSUPPORTED;
  if (desc->impl != 1 && tc_ok) return fc::attention_tc(ctx, st, g, Q, K, V, O, ws, ws_bytes);
  return fc::attention_simt(st, g, Q, K, V, dtype, O);
}
