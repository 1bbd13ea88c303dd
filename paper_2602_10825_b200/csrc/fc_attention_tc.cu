// Chunk-causal attention on tcgen05 tensor cores (bf16 in, fp32 accumulation in tensor memory).
//
// Work item = (head, active chunk, 128-row query tile); items are ordered head-major with the
// longest visible prefix first inside a head and are handed out through a device counter, so the
// data-dependent list of active chunks never returns to the host.  Per item the CTA walks the
// visible key/value prefix segment by segment in tiles of 128 tokens:
//   TMA (128-byte swizzle) -> shared memory -> S = Q K^T (tcgen05.mma, SS) -> tensor memory
//   -> registers: online softmax in the exp2 domain, one query row per thread
//   -> P (bf16) back to tensor memory, aliasing S -> O += P V (tcgen05.mma, A from tensor memory).
// Columns past the end of a segment get -inf before the row maximum, so P is exactly 0 there.
// Every mbarrier wait is bounded; a wait that gives up sets FC_DEV_TIMEOUT and the kernel runs on
// to its normal teardown (tensor memory is always released).
#include <cmath>

#include "fc_attention.cuh"
#include "fc_tcgen05.cuh"

namespace {

using namespace fc::sm100;

constexpr int kBM = 128;  // query rows per tile
constexpr int kBN = 128;  // key/value tokens per tile
constexpr int kThreads = 128;
constexpr uint32_t kTmemCols = 256;  // S/P: columns [0,128), O: columns [128, 128+D)

struct TcSmem {
  // tile buffers are carved from the dynamic region (1024-byte aligned); this trailer follows them
  uint64_t bar_q, bar_kv, bar_s, bar_o;
  uint32_t tmem_base;
  uint32_t abort;
  int32_t item;
  int32_t n_act;
  int32_t act_chunk[FC_MAX_CHUNKS];
  int32_t act_tile_end[FC_MAX_CHUNKS];  // running tile count over the (descending) active list
};

template <int D>
__global__ void __launch_bounds__(kThreads)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ fc::AttnGeom g,
                    __nv_bfloat16* __restrict__ O, uint32_t* __restrict__ counter) {
  constexpr uint32_t kTileBytes = kBM * D * 2;  // one Q, K or V tile
  constexpr int kAtoms = D / 64;                // 64-element (128-byte) column blocks per row
  constexpr uint32_t kAtomBytes = kBM * 128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t q_s = smem_u32(smem), k_s = q_s + kTileBytes, v_s = k_s + kTileBytes;
  TcSmem* sh = (TcSmem*)(smem + 3 * kTileBytes);
  const uint32_t bar_q = smem_u32(&sh->bar_q), bar_kv = smem_u32(&sh->bar_kv), bar_s = smem_u32(&sh->bar_s),
                 bar_o = smem_u32(&sh->bar_o);
  volatile uint32_t* abort = &sh->abort;
  const int tid = threadIdx.x, warp = tid >> 5;

  if (tid == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_kv, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_o, 1);
    mbar_fence_init();
    sh->abort = 0;
    tma_prefetch_desc(&tmap_q);
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_v);
    // active chunks, longest visible prefix (highest id) first
    const int n_in = min(max(*g.n_active, 0), g.W);
    int n = 0, tiles = 0;
    for (int a = n_in - 1; a >= 0; --a) {
      const int c = g.active_ids[a];
      if (c < 0 || c >= g.W) {
        if (g.status) atomicOr(g.status, FC_DEV_BAD_INDEX);
        continue;
      }
      tiles += (g.q_row_off[c + 1] - g.q_row_off[c] + kBM - 1) / kBM;
      sh->act_chunk[n] = c;
      sh->act_tile_end[n] = tiles;
      ++n;
    }
    sh->n_act = n;
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&sh->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh->tmem_base;
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
  const uint32_t t_s = tmem + lane_base;        // S (fp32) and, aliased, P (bf16 pairs)
  const uint32_t t_o = tmem + lane_base + 128;  // O accumulator
  const int n_act = sh->n_act;
  const int tiles_per_head = n_act > 0 ? sh->act_tile_end[n_act - 1] : 0;
  const int total_items = tiles_per_head * g.H_q;
  const float scale_log2 = g.scale * 1.4426950408889634f;
  constexpr uint32_t kIdescQK = idesc_bf16_f32(kBM, kBN, false, false);
  constexpr uint32_t kIdescPV = idesc_bf16_f32(kBM, D, false, true);
  uint32_t ph_q = 0, ph_kv = 0, ph_s = 0, ph_o = 0;

  while (true) {
    if (tid == 0) sh->item = (int)atomicAdd(counter, 1u);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const int item = sh->item;
    if (item >= total_items || *abort) break;
    const int h = item / tiles_per_head, rem = item % tiles_per_head;
    int a = 0;
    while (a + 1 < n_act && rem >= sh->act_tile_end[a]) ++a;
    const int c = sh->act_chunk[a];
    const int tile = rem - (a > 0 ? sh->act_tile_end[a - 1] : 0);
    const int row0 = g.q_row_off[c] + tile * kBM;
    const int rows_valid = min(kBM, g.q_row_off[c + 1] - row0);
    const int n_vis = g.vis[c];
    const int hk = h / g.group;

    if (tid == 0) {
      mbar_expect_tx(bar_q, kTileBytes);
      for (int x = 0; x < kAtoms; ++x) tma_load_3d(q_s + x * kAtomBytes, &tmap_q, bar_q, x * 64, row0, h);
      mbar_wait_bounded(bar_q, ph_q, abort);
      ph_q ^= 1;
    }

    float m = -INFINITY, l = 0.f;  // running max (log2 domain) and sum of this thread's row
    bool first = true;
    for (int s = 0; s < g.n_seg; ++s) {
      const int seg_vis = min(g.seg_log[s + 1], n_vis) - g.seg_log[s];
      if (seg_vis <= 0) break;
      for (int j0 = 0; j0 < seg_vis; j0 += kBN) {
        const int cols_valid = min(kBN, seg_vis - j0);
        if (tid == 0) {
          const int prow = g.seg_phys[s] + j0;
          mbar_expect_tx(bar_kv, 2 * kTileBytes);
          for (int x = 0; x < kAtoms; ++x) {
            tma_load_3d(k_s + x * kAtomBytes, &tmap_k, bar_kv, x * 64, prow, hk);
            tma_load_3d(v_s + x * kAtomBytes, &tmap_v, bar_kv, x * 64, prow, hk);
          }
          mbar_wait_bounded(bar_kv, ph_kv, abort);
          ph_kv ^= 1;
          tc_fence_after();
          // S = Q K^T: both operands K-major, 16 elements (32 bytes) of d per instruction
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = (kk / 4) * kAtomBytes + (kk % 4) * 32;
            umma_ss(tmem, smem_desc_sw128(q_s + off, 16, 1024), smem_desc_sw128(k_s + off, 16, 1024), kIdescQK,
                    kk > 0);
          }
          umma_commit(bar_s);
        }
        mbar_wait_bounded(bar_s, ph_s, abort);
        ph_s ^= 1;
        tc_fence_after();

        // ---- softmax of this thread's row over the tile
        float sv[kBN];
#pragma unroll
        for (int q4 = 0; q4 < kBN / 32; ++q4) {
          uint32_t r[32];
          tmem_ld32(t_s + q4 * 32, r);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) sv[q4 * 32 + i] = __uint_as_float(r[i]) * scale_log2;
        }
        float tile_max = -INFINITY;
#pragma unroll
        for (int j = 0; j < kBN; ++j) {
          if (j >= cols_valid) sv[j] = -INFINITY;
          tile_max = fmaxf(tile_max, sv[j]);
        }
        const float m_new = fmaxf(m, tile_max);  // cols_valid >= 1, so m_new is finite
        const float alpha = ex2(m - m_new);       // 0 on the first tile (m = -inf)
        float row_sum = 0.f;
#pragma unroll
        for (int q2 = 0; q2 < kBN / 32; ++q2) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float p0 = ex2(sv[q2 * 32 + 2 * i] - m_new), p1 = ex2(sv[q2 * 32 + 2 * i + 1] - m_new);
            row_sum += p0 + p1;
            __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
            pk[i] = *reinterpret_cast<uint32_t*>(&b);
          }
          tmem_st16(t_s + q2 * 16, pk);
        }
        l = l * alpha + row_sum;
        // ---- rescale the accumulator when some row of this warp moved its maximum
        if (!first && __any_sync(0xffffffffu, m_new > m)) {
#pragma unroll
          for (int q4 = 0; q4 < D / 32; ++q4) {
            uint32_t r[32];
            tmem_ld32(t_o + q4 * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tmem_st32(t_o + q4 * 32, r);
          }
        }
        m = m_new;
        tmem_wait_st();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
          tc_fence_after();
          // O += P V: A = P from tensor memory (16 tokens = 8 columns per instruction), B = V, MN-major:
          // 64-element column blocks kAtomBytes apart, 8-token groups 1024 bytes apart
#pragma unroll
          for (int kk = 0; kk < kBN / 16; ++kk)
            umma_ts(tmem + 128, tmem + kk * 8, smem_desc_sw128(v_s + kk * 2048, kAtomBytes, 1024), kIdescPV,
                    (!first) || kk > 0);
          umma_commit(bar_o);
        }
        mbar_wait_bounded(bar_o, ph_o, abort);
        ph_o ^= 1;
        tc_fence_after();
        first = false;
      }
    }

    // ---- epilogue: normalise and store this thread's row
    const int row = row0 + tid;
    const float inv = l > 0.f ? 1.f / l : 0.f;
    __nv_bfloat16* out = O + (int64_t)h * g.o_hs + (int64_t)row * g.o_rs;
#pragma unroll
    for (int q4 = 0; q4 < D / 32; ++q4) {
      uint32_t r[32];
      if (!first) {
        tmem_ld32(t_o + q4 * 32, r);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) r[i] = 0;
      }
      if (tid < rows_valid) {
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint4 w;
          uint32_t* wp = &w.x;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(r[v * 8 + 2 * i]) * inv,
                                                     __uint_as_float(r[v * 8 + 2 * i + 1]) * inv);
            wp[i] = *reinterpret_cast<uint32_t*>(&b);
          }
          *reinterpret_cast<uint4*>(out + q4 * 32 + v * 8) = w;
        }
      }
    }
    if (g.lse && tid < rows_valid)
      g.lse[(int64_t)h * g.lse_hs + row] = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
    // every row has left tensor memory before the next item's instructions may overwrite it
    tc_fence_before();
    __syncthreads();
  }

  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort && g.status) atomicOr(g.status, FC_DEV_TIMEOUT);
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace

namespace fc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [heads, rows, d] bf16 tensor, box = 64 elements (128 bytes) x 128 rows x 1 head, 128-byte swizzle.
int make_tmap(fc_ctx* ctx, CUtensorMap* map, const void* base, int d, int64_t rows, int heads, int64_t row_stride,
              int64_t head_stride) {
  const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)rows, (cuuint64_t)heads};
  const cuuint64_t strides[2] = {(cuuint64_t)row_stride * 2, (cuuint64_t)head_stride * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)kBM, 1};
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


size_t attention_tc_workspace_bytes() { return 256; }

bool attention_tc_supported(const AttnGeom& g, int dtype) {
  if (dtype != FC_BF16 || g.tok_index != nullptr) return false;
  if (g.d != 64 && g.d != 128) return false;
  // a head stride of 0 rows (single head) is fine; TMA needs the head stride to fit 2^40 bytes
  return true;
}

int attention_tc(fc_ctx* ctx, cudaStream_t st, const AttnGeom& g_in, const void* Q, const void* K, const void* V,
                 void* O, void* ws, size_t ws_bytes, bool basic) {
  if (!ws || ws_bytes < attention_tc_workspace_bytes()) return FC_ERR_WORKSPACE;
  if (!aligned16(ws)) return FC_ERR_MISALIGNED;
  AttnGeom g = g_in;
  // merge logically adjacent segments that are also physically adjacent: fewer ragged tails
  int n = 0;
  for (int s = 0; s < g_in.n_seg; ++s) {
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
  g.n_seg = n;
  int64_t q_rows = g.q_row_off[g.W];
  int max_tiles = 0;
  for (int c = 0; c < g.W; ++c) max_tiles += (g.q_row_off[c + 1] - g.q_row_off[c] + kBM - 1) / kBM;
  if (max_tiles == 0 || q_rows == 0) return FC_OK;
  CUtensorMap tq, tk, tv;
  int rc;
  if ((rc = make_tmap(ctx, &tq, Q, g.d, q_rows, g.H_q, g.q_rs, g.H_q > 1 ? g.q_hs : g.q_rs * q_rows)) != FC_OK) return rc;
  if ((rc = make_tmap(ctx, &tk, K, g.d, g.kv_rows, g.H_kv, g.k_rs, g.H_kv > 1 ? g.k_hs : g.k_rs * g.kv_rows)) != FC_OK) return rc;
  if ((rc = make_tmap(ctx, &tv, V, g.d, g.kv_rows, g.H_kv, g.v_rs, g.H_kv > 1 ? g.v_hs : g.v_rs * g.kv_rows)) != FC_OK) return rc;
  uint32_t* counter = (uint32_t*)ws;
  if (!basic) return attention_ws_launch(ctx, st, g, tq, tk, tv, O, counter);
  FC_CUDA_CHECK(cudaMemsetAsync(counter, 0, sizeof(uint32_t), st));
  const int64_t items = (int64_t)max_tiles * g.H_q;
  const int grid = (int)std::min<int64_t>(items, 2 * (int64_t)ctx->sm_count);
  const size_t smem = 3 * (size_t)kBM * g.d * 2 + sizeof(TcSmem) + 1024;
  if (g.d == 128) {
    FC_CUDA_CHECK(cudaFuncSetAttribute(attention_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    attention_tc_kernel<128><<<grid, kThreads, smem, st>>>(tq, tk, tv, g, (__nv_bfloat16*)O, counter);
  } else {
    // d = 64 tiles are 48 KiB per CTA; pad the request so that at most two CTAs (2 x 256 tensor-memory
    // columns) can share an SM
    const size_t smem64 = std::max<size_t>(smem, 80 * 1024);
    FC_CUDA_CHECK(cudaFuncSetAttribute(attention_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem64));
    attention_tc_kernel<64><<<grid, kThreads, smem64, st>>>(tq, tk, tv, g, (__nv_bfloat16*)O, counter);
  }
  FC_LAUNCH_CHECK("attention_tc_kernel");
  return FC_OK;
}

}  // namespace fc
