// Chunk-causal attention on CUDA cores (fp32 accumulation): the path of fp32 tensors, of caches
// read through a token-level index map, and an on-device second opinion for the tensor-core kernel.
//
// A block of 128 threads owns 32 query rows of one active chunk and one head; four threads share
// a row, each holding every fourth 4-element piece of q and of the output accumulator.  Key/value
// tiles of 32 logical tokens are staged in shared memory as fp32 through the index map; the 32
// logits of a tile are formed first, then one running-max update and one accumulation sweep.
#include <cmath>

#include "fc_attention.cuh"

namespace {

constexpr int kRows = 32, kKeys = 32, kThreads = 128;

template <typename T> __device__ __forceinline__ float4 load4(const T* p);
template <> __device__ __forceinline__ float4 load4<float>(const float* p) {
  return *reinterpret_cast<const float4*>(p);
}
template <> __device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16* p) {
  const uint2 w = *reinterpret_cast<const uint2*>(p);
  return make_float4(fc::bf16_lo(w.x), fc::bf16_hi(w.x), fc::bf16_lo(w.y), fc::bf16_hi(w.y));
}
__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 w;
  w.x = *reinterpret_cast<uint32_t*>(&a);
  w.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = w;
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
attention_simt_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                      T* __restrict__ O, const __grid_constant__ fc::AttnGeom g) {
  constexpr int P = D / 16;  // 4-element pieces per thread
  __shared__ __align__(16) float k_s[kKeys * D];
  __shared__ __align__(16) float v_s[kKeys * D];
  __shared__ int64_t phys_s[kKeys];
  __shared__ int sh_chunk, sh_tile;

  const int tid = threadIdx.x, h = blockIdx.y, hk = h / g.group;
  if (tid == 0) {
    // Map this block onto the device-side work list: active chunks, longest prefix first.
    int n_act = min(max(*g.n_active, 0), g.W);
    int item = blockIdx.x, chunk = -1, tile = 0;
    for (int a = n_act - 1; a >= 0; --a) {
      const int c = g.active_ids[a];
      if (c < 0 || c >= g.W) continue;
      const int tiles = (g.q_row_off[c + 1] - g.q_row_off[c] + kRows - 1) / kRows;
      if (item < tiles) {
        chunk = c;
        tile = item;
        break;
      }
      item -= tiles;
    }
    sh_chunk = chunk;
    sh_tile = tile;
  }
  __syncthreads();
  const int c = sh_chunk;
  if (c < 0) return;
  const int r_in = tid >> 2, t = tid & 3;
  const int row = g.q_row_off[c] + sh_tile * kRows + r_in;
  const bool row_ok = row < g.q_row_off[c + 1];
  const int n_vis = g.vis[c];

  float q[P * 4], o[P * 4];
#pragma unroll
  for (int i = 0; i < P; ++i) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row_ok) v = load4<T>(Q + (int64_t)h * g.q_hs + (int64_t)row * g.q_rs + (i * 4 + t) * 4);
    q[4 * i] = v.x * g.scale; q[4 * i + 1] = v.y * g.scale; q[4 * i + 2] = v.z * g.scale; q[4 * i + 3] = v.w * g.scale;
    o[4 * i] = o[4 * i + 1] = o[4 * i + 2] = o[4 * i + 3] = 0.f;
  }
  float m = -INFINITY, l = 0.f;

  for (int j0 = 0; j0 < n_vis; j0 += kKeys) {
    __syncthreads();  // previous tile fully consumed
    if (tid < kKeys) {
      const int j = j0 + tid;
      int64_t p = -1;
      if (j < n_vis) {
        if (g.tok_index) {
          p = g.tok_index[(int64_t)hk * g.tok_hs + j];
        } else {
          for (int s = 0; s < g.n_seg; ++s)
            if (j >= g.seg_log[s] && j < g.seg_log[s + 1]) {
              p = (int64_t)g.seg_phys[s] + (j - g.seg_log[s]);
              break;
            }
        }
        if (p < 0 || p >= g.kv_rows) {
          p = -1;
          if (g.status) atomicOr(g.status, FC_DEV_BAD_INDEX);
        }
      }
      phys_s[tid] = p;
    }
    __syncthreads();
    for (int x = tid; x < kKeys * (D / 4); x += kThreads) {
      const int jj = x / (D / 4), piece = x % (D / 4);
      const int64_t p = phys_s[jj];
      float4 kv = make_float4(0.f, 0.f, 0.f, 0.f), vv = kv;
      if (p >= 0) {
        kv = load4<T>(K + (int64_t)hk * g.k_hs + p * g.k_rs + piece * 4);
        vv = load4<T>(V + (int64_t)hk * g.v_hs + p * g.v_rs + piece * 4);
      }
      store4(k_s + jj * D + piece * 4, kv);
      store4(v_s + jj * D + piece * 4, vv);
    }
    __syncthreads();

    float s[kKeys];
    float tile_max = -INFINITY;
#pragma unroll
    for (int jj = 0; jj < kKeys; ++jj) {
      float dot = 0.f;
#pragma unroll
      for (int i = 0; i < P; ++i) {
        const float4 kk = *reinterpret_cast<const float4*>(k_s + jj * D + (i * 4 + t) * 4);
        dot = fmaf(q[4 * i], kk.x, dot);
        dot = fmaf(q[4 * i + 1], kk.y, dot);
        dot = fmaf(q[4 * i + 2], kk.z, dot);
        dot = fmaf(q[4 * i + 3], kk.w, dot);
      }
      dot += __shfl_xor_sync(0xffffffffu, dot, 1);
      dot += __shfl_xor_sync(0xffffffffu, dot, 2);
      s[jj] = (phys_s[jj] >= 0) ? dot : -INFINITY;
      tile_max = fmaxf(tile_max, s[jj]);
    }
    const float m_new = fmaxf(m, tile_max);
    if (m_new == -INFINITY) continue;  // nothing visible in this tile (uniform over the row's 4 threads)
    const float corr = expf(m - m_new);  // exp(-inf) = 0 on the first tile
    l *= corr;
#pragma unroll
    for (int e = 0; e < P * 4; ++e) o[e] *= corr;
#pragma unroll
    for (int jj = 0; jj < kKeys; ++jj) {
      const float p = expf(s[jj] - m_new);
      l += p;
#pragma unroll
      for (int i = 0; i < P; ++i) {
        const float4 vv = *reinterpret_cast<const float4*>(v_s + jj * D + (i * 4 + t) * 4);
        o[4 * i] = fmaf(p, vv.x, o[4 * i]);
        o[4 * i + 1] = fmaf(p, vv.y, o[4 * i + 1]);
        o[4 * i + 2] = fmaf(p, vv.z, o[4 * i + 2]);
        o[4 * i + 3] = fmaf(p, vv.w, o[4 * i + 3]);
      }
    }
    m = m_new;
  }
  if (!row_ok) return;
  const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
  for (int i = 0; i < P; ++i)
    store4(O + (int64_t)h * g.o_hs + (int64_t)row * g.o_rs + (i * 4 + t) * 4,
           make_float4(o[4 * i] * inv, o[4 * i + 1] * inv, o[4 * i + 2] * inv, o[4 * i + 3] * inv));
  if (g.lse && t == 0) g.lse[(int64_t)h * g.lse_hs + row] = l > 0.f ? m + logf(l) : -INFINITY;
}

}  // namespace

namespace fc {

int attention_simt(cudaStream_t st, const AttnGeom& g, const void* Q, const void* K, const void* V,
                   int dtype, void* O) {
  int max_tiles = 0;
  for (int c = 0; c < g.W; ++c) max_tiles += (g.q_row_off[c + 1] - g.q_row_off[c] + kRows - 1) / kRows;
  if (max_tiles == 0) return FC_OK;
  dim3 grid(max_tiles, g.H_q);
#define FC_SIMT_LAUNCH(T, D)                                                                      \
  attention_simt_kernel<T, D><<<grid, kThreads, 0, st>>>((const T*)Q, (const T*)K, (const T*)V, (T*)O, g)
  if (dtype == FC_F32) {
    if (g.d == 128) FC_SIMT_LAUNCH(float, 128); else FC_SIMT_LAUNCH(float, 64);
  } else {
    if (g.d == 128) FC_SIMT_LAUNCH(__nv_bfloat16, 128); else FC_SIMT_LAUNCH(__nv_bfloat16, 64);
  }
#undef FC_SIMT_LAUNCH
  FC_LAUNCH_CHECK("attention_simt_kernel");
  return FC_OK;
}

}  // namespace fc
