// fc_kv_score: importance (Eq. 9), max-pool (Eq. 10), redundancy (Eq. 11, through the mean-key
// identity of the paper's efficiency appendix) and the mixed score (Eq. 12).
//
// Two pipelines, both deterministic (no floating-point atomics).  bf16 inputs with one query head per key head
// and at most 62 observation queries take the tensor-core kernels of fc_score_tc.cu followed by the finalize
// kernel below; everything else (fp32, more queries, grouped query heads whose rows are not contiguous) takes the
// CUDA-core pipeline (below).  Grouped query heads stored head after head are folded into one head of group * L_q
// queries first, so they take whichever pipeline that number of queries takes.  bf16 inputs with more than 128 observation queries per key head (a latent frame
// or a whole chunk of them) take the frame-level pipeline: sums of normalised keys and the mean key by
// frame_key_sums_kernel and score_mean_key_kernel (below), every query's log-sum-exp over the candidates and then the
// attention mass of every key by the tensor-core kernel of fc_score_frame.cu (two launches), then frame_finish_kernel
// (below: importance from that mass, redundancy argument) and the finalize kernel.
// The CUDA-core pipeline, five launches per call:
//   pass1     one thread per key: raw logits of all observation queries against its key,
//             written to the workspace; normalised key summed per 128-key tile (mean key)
//   row_lse   one block per (head, query): log-sum-exp of that query's logits over all keys
//   mean_key  one block per head: tile sums -> mean normalised key
//   pass2     one thread per key: attention mass of the key (mean over queries of
//             exp(logit - lse)), and its redundancy logit a_j = meankey.khat_j - |khat_j|^2/L_k;
//             per-tile softmax statistics of a
//   finalize  softmax of a over the head, max-pool of the importance, lambda-mix
#include <cmath>

#include "fc_common.cuh"
#include "fc_score.cuh"

namespace {

constexpr int kTile = 128;  // keys per block, one thread each
constexpr int kCoreMaxQueries = 128;  // query rows per key head that the CUDA-core pipeline holds in shared memory

template <typename T, int D>
__device__ __forceinline__ void load_row(const T* __restrict__ row, float (&x)[D]) {
  if constexpr (sizeof(T) == 2) {
#pragma unroll
    for (int v = 0; v < D / 8; ++v) {
      const uint4 w = *reinterpret_cast<const uint4*>(row + v * 8);
      const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        x[v * 8 + 2 * i] = fc::bf16_lo(ww[i]);
        x[v * 8 + 2 * i + 1] = fc::bf16_hi(ww[i]);
      }
    }
  } else {
#pragma unroll
    for (int v = 0; v < D / 4; ++v) {
      const float4 w = *reinterpret_cast<const float4*>(row + v * 4);
      x[v * 4] = w.x;
      x[v * 4 + 1] = w.y;
      x[v * 4 + 2] = w.z;
      x[v * 4 + 3] = w.w;
    }
  }
}

struct ScoreGeom {
  int H_q, H_kv, d, L_q, L_k, group, n_q, n_tiles;
  int n_partials;  // softmax statistics of a per head handed to the finalize kernel (one per tile, or per warp of a tile)
  int64_t q_hs, q_rs, k_hs, k_rs;
  float scale, lambda;
  int pool_k;
};

// smem: q_s [n_q][D] then khat_s [kTile][D+1]
template <typename T, int D>
__global__ void __launch_bounds__(kTile)
score_pass1_kernel(const T* __restrict__ Q, const T* __restrict__ K, ScoreGeom g,
                   float* __restrict__ S, float* __restrict__ mk_partial) {
  extern __shared__ float sm[];
  float* q_s = sm;
  float* khat_s = sm + (size_t)g.n_q * D;
  const int hk = blockIdx.y, tile = blockIdx.x, tid = threadIdx.x;
  for (int t = tid; t < g.n_q * D; t += kTile) {
    const int i = t / D, e = t % D;
    const int hq = hk * g.group + i / g.L_q, r = i % g.L_q;
    q_s[t] = fc::to_float(Q[(int64_t)hq * g.q_hs + (int64_t)r * g.q_rs + e]);
  }
  const int j = tile * kTile + tid;
  const bool valid = j < g.L_k;
  float k[D];
  if (valid) {
    load_row<T, D>(K + (int64_t)hk * g.k_hs + (int64_t)j * g.k_rs, k);
  } else {
#pragma unroll
    for (int e = 0; e < D; ++e) k[e] = 0.f;
  }
  float n2 = 0.f;
#pragma unroll
  for (int e = 0; e < D; ++e) n2 = fmaf(k[e], k[e], n2);
  const float inv = valid ? 1.f / fmaxf(sqrtf(n2), 1e-12f) : 0.f;
#pragma unroll
  for (int e = 0; e < D; ++e) khat_s[tid * (D + 1) + e] = k[e] * inv;
  __syncthreads();
  if (valid) {
    float* s_out = S + ((int64_t)hk * g.n_q) * g.L_k + j;
    for (int i = 0; i < g.n_q; ++i) {
      const float4* q4 = reinterpret_cast<const float4*>(q_s + i * D);
      float dot = 0.f;
#pragma unroll
      for (int v = 0; v < D / 4; ++v) {
        const float4 q = q4[v];
        dot = fmaf(q.x, k[4 * v], dot);
        dot = fmaf(q.y, k[4 * v + 1], dot);
        dot = fmaf(q.z, k[4 * v + 2], dot);
        dot = fmaf(q.w, k[4 * v + 3], dot);
      }
      s_out[(int64_t)i * g.L_k] = dot * g.scale;
    }
  }
  if (tid < D) {
    float acc = 0.f;
    for (int r = 0; r < kTile; ++r) acc += khat_s[r * (D + 1) + tid];
    mk_partial[((int64_t)hk * g.n_tiles + tile) * D + tid] = acc;
  }
}

// Fixed-tree block reduction of an online-softmax pair (m, l); result valid in thread 0.
template <int kThreads>
__device__ __forceinline__ void reduce_ml(float& m, float& l, float* sm_m, float* sm_l) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_down_sync(0xffffffffu, m, o), l2 = __shfl_down_sync(0xffffffffu, l, o);
    const float mn = fmaxf(m, m2);
    l = (m == -INFINITY ? 0.f : l * expf(m - mn)) + (m2 == -INFINITY ? 0.f : l2 * expf(m2 - mn));
    m = mn;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) {
    sm_m[warp] = m;
    sm_l[warp] = l;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    m = sm_m[0];
    l = sm_l[0];
    for (int w = 1; w < kThreads / 32; ++w) {
      const float m2 = sm_m[w], l2 = sm_l[w];
      const float mn = fmaxf(m, m2);
      l = (m == -INFINITY ? 0.f : l * expf(m - mn)) + (m2 == -INFINITY ? 0.f : l2 * expf(m2 - mn));
      m = mn;
    }
  }
}

__global__ void __launch_bounds__(256)
score_row_lse_kernel(const float* __restrict__ S, int L_k, float* __restrict__ lse) {
  __shared__ float sm_m[8], sm_l[8];
  const int64_t row = (int64_t)blockIdx.y * gridDim.x + blockIdx.x;  // (head, query)
  const float* s = S + row * L_k;
  float m = -INFINITY, l = 0.f;
  for (int j = threadIdx.x; j < L_k; j += 256) {
    const float x = s[j];
    if (x > m) {
      l = l * expf(m - x) + 1.f;  // expf(-inf) = 0 on the first element
      m = x;
    } else {
      l += expf(x - m);
    }
  }
  reduce_ml<256>(m, l, sm_m, sm_l);
  if (threadIdx.x == 0) lse[row] = m + logf(l);
}

// Mean normalised key of a head from the per-tile sums.  One block per head, kMkGroups x 128 threads: group r adds
// the tiles r, r + kMkGroups, ... (eight loads in flight; one thread per component walking all tiles waited for one
// load after the other, 342 of them on 43680 keys), the groups are added in group order.  Fixed order throughout.
constexpr int kMkGroups = 8;
__global__ void __launch_bounds__(kMkGroups * 128)
score_mean_key_kernel(const float* __restrict__ mk_partial, int n_tiles, int d, int L_k,
                      float* __restrict__ mean_key) {
  __shared__ float part[kMkGroups][128];
  const int hk = blockIdx.x, e = threadIdx.x & 127, r = threadIdx.x >> 7;
  float acc = 0.f;
  if (e < d) {
    const float* src = mk_partial + (int64_t)hk * n_tiles * d + e;
    for (int t0 = r; t0 < n_tiles; t0 += 8 * kMkGroups) {
      float v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int t = t0 + k * kMkGroups;
        v[k] = t < n_tiles ? src[(int64_t)t * d] : 0.f;
      }
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (t0 + k * kMkGroups < n_tiles) acc += v[k];
    }
  }
  part[r][e] = acc;
  __syncthreads();
  if (r == 0 && e < d) {
    float t = 0.f;
#pragma unroll
    for (int q = 0; q < kMkGroups; ++q) t += part[q][e];
    mean_key[hk * d + e] = t / (float)L_k;
  }
}

// ---- frame-level pipeline: the two sweeps over the keys around the tensor-core launches (bf16) ----------------
// A warp reads whole rows with one instruction: a key row is D / 8 chunks of 16 bytes, one per lane, so a warp
// instruction covers 32 / (D / 8) consecutive rows (512 contiguous bytes).  What a row needs as a whole (its squared
// norm, its product with the mean key) is a sum over the lanes that hold it: log2(D / 8) shuffle steps.
template <int D>
struct RowLanes {
  static constexpr int kLanes = D / 8;        // lanes per row
  static constexpr int kRows = 32 / kLanes;   // rows per warp instruction
};

__device__ __forceinline__ void unpack8(const uint4& w, float (&x)[8]) {
  const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    x[2 * i] = fc::bf16_lo(ww[i]);
    x[2 * i + 1] = fc::bf16_hi(ww[i]);
  }
}

// Sums of the l2-normalised keys of one tile: mk_partial[head, tile, D] (what score_pass1_kernel leaves, without
// its logits).  128 threads, warp w takes rows 32 w .. 32 w + 31 of the tile.  Three steps: the squared norm of every
// row (lanes of a row added by shuffles) into shared memory; one reciprocal norm per thread (the square root and
// the division once per row, all lanes busy); the rows, still in registers, scaled and added up per column.
template <int D>
__global__ void __launch_bounds__(kTile)
frame_key_sums_kernel(const __nv_bfloat16* __restrict__ K, ScoreGeom g, float* __restrict__ mk_partial) {
  constexpr int kLanes = RowLanes<D>::kLanes, kRows = RowLanes<D>::kRows, kIters = 32 / kRows;
  __shared__ float part[kTile / 32][D];
  __shared__ float n2_s[kTile];  // squared norms, then reciprocal norms
  const int hk = blockIdx.y, tile = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane % kLanes, rsel = lane / kLanes;
  const __nv_bfloat16* base = K + (int64_t)hk * g.k_hs + sub * 8;
  uint4 w[kIters];
#pragma unroll
  for (int it = 0; it < kIters; ++it) {  // all loads of the warp's 32 rows first
    const int row = tile * kTile + warp * 32 + it * kRows + rsel;
    w[it] = row < g.L_k ? __ldg(reinterpret_cast<const uint4*>(base + (int64_t)row * g.k_rs)) : make_uint4(0u, 0u, 0u, 0u);
  }
#pragma unroll
  for (int it = 0; it < kIters; ++it) {
    float x[8];
    unpack8(w[it], x);
    float n2 = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) n2 = fmaf(x[e], x[e], n2);
#pragma unroll
    for (int o = kLanes / 2; o > 0; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
    if (sub == 0) n2_s[warp * 32 + it * kRows + rsel] = n2;
  }
  __syncthreads();
  n2_s[threadIdx.x] = 1.f / fmaxf(sqrtf(n2_s[threadIdx.x]), 1e-12f);  // rows past the end are zeros: 0 * 1e12 = 0
  __syncthreads();
  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll
  for (int it = 0; it < kIters; ++it) {
    float x[8];
    unpack8(w[it], x);
    const float inv = n2_s[warp * 32 + it * kRows + rsel];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = fmaf(x[e], inv, acc[e]);
  }
  // the lanes that hold the same chunk of different rows, then the warps, in a fixed order
#pragma unroll
  for (int o = kLanes; o < 32; o <<= 1)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
  if (rsel == 0)
#pragma unroll
    for (int e = 0; e < 8; ++e) part[warp][sub * 8 + e] = acc[e];
  __syncthreads();
  if (threadIdx.x < D) {
    float t = 0.f;
#pragma unroll
    for (int q = 0; q < kTile / 32; ++q) t += part[q][threadIdx.x];
    mk_partial[((int64_t)hk * g.n_tiles + tile) * D + threadIdx.x] = t;
  }
}

// After the mass launch: importance = mass / n_q (with the accumulation over steps), redundancy argument
// a_j = meankey . khat_j - |khat_j|^2 / L_k and its per-tile softmax statistics (what score_pass2_kernel does with
// one key per thread and uncoalesced row loads).  Two steps: the warps sweep the rows (squared norm and product with
// the mean key of every row, by shuffles, into shared memory); then one key per thread, so that the square root,
// the division and every access to the per-key arrays are done by all threads at once.
template <int D>
__global__ void __launch_bounds__(kTile)
frame_finish_kernel(const __nv_bfloat16* __restrict__ K, ScoreGeom g, const float* __restrict__ mean_key,
                    const float* __restrict__ mass_in, float* __restrict__ imp_accum, int accum_phase, int n_steps,
                    float* __restrict__ imp_out, float* __restrict__ a_out, float2* __restrict__ a_partial) {
  constexpr int kLanes = RowLanes<D>::kLanes, kRows = RowLanes<D>::kRows, kIters = 32 / kRows;
  __shared__ float sm_m[kTile / 32], sm_l[kTile / 32];
  __shared__ float n2_s[kTile], dot_s[kTile];
  const int hk = blockIdx.y, tile = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int j = tile * kTile + tid;
  const bool valid = j < g.L_k;
  const int64_t o = (int64_t)hk * g.L_k + j;
  if (valid) {
    const float ms = mass_in[o] / (float)g.n_q;
    if (accum_phase == 1) {
      imp_accum[o] += ms;
    } else if (accum_phase == 2) {
      const float t = imp_accum[o] + ms;
      imp_accum[o] = t;
      imp_out[o] = t / (float)n_steps;
    } else {
      imp_out[o] = ms;
    }
  }
  if (accum_phase == 1) return;
  {
    const int sub = lane % kLanes, rsel = lane / kLanes;
    const __nv_bfloat16* base = K + (int64_t)hk * g.k_hs + sub * 8;
    float mk[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) mk[e] = mean_key[hk * D + sub * 8 + e];
    uint4 w[kIters];
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
      const int row = tile * kTile + warp * 32 + it * kRows + rsel;
      w[it] = row < g.L_k ? __ldg(reinterpret_cast<const uint4*>(base + (int64_t)row * g.k_rs)) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int it = 0; it < kIters; ++it) {
      float x[8];
      unpack8(w[it], x);
      float n2 = 0.f, dot = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        n2 = fmaf(x[e], x[e], n2);
        dot = fmaf(mk[e], x[e], dot);
      }
#pragma unroll
      for (int o2 = kLanes / 2; o2 > 0; o2 >>= 1) {
        n2 += __shfl_xor_sync(0xffffffffu, n2, o2);
        dot += __shfl_xor_sync(0xffffffffu, dot, o2);
      }
      if (sub == 0) {
        n2_s[warp * 32 + it * kRows + rsel] = n2;
        dot_s[warp * 32 + it * kRows + rsel] = dot;
      }
    }
  }
  __syncthreads();
  float a = -INFINITY;
  if (valid) {
    const float n2 = n2_s[tid];
    const float inv = 1.f / fmaxf(sqrtf(n2), 1e-12f);
    a = dot_s[tid] * inv - (n2 * inv * inv) / (float)g.L_k;
    a_out[o] = a;
  }
  float m = a, l = valid ? 1.f : 0.f;
  reduce_ml<kTile>(m, l, sm_m, sm_l);
  if (tid == 0) a_partial[hk * g.n_tiles + tile] = make_float2(m, l);
}

template <typename T, int D>
__global__ void __launch_bounds__(kTile)
score_pass2_kernel(const T* __restrict__ K, ScoreGeom g, const float* __restrict__ S,
                   const float* __restrict__ lse, const float* __restrict__ mean_key,
                   const float* __restrict__ mass_in,  // frame-level path: sum over the queries already taken
                   float* __restrict__ imp_accum, int accum_phase, int n_steps,
                   float* __restrict__ imp_out, float* __restrict__ a_out, float2* __restrict__ a_partial) {
  __shared__ float mk_s[D];
  __shared__ float lse_s[128];
  __shared__ float sm_m[kTile / 32], sm_l[kTile / 32];
  const int hk = blockIdx.y, tile = blockIdx.x, tid = threadIdx.x;
  if (tid < D) mk_s[tid] = mean_key[hk * D + tid];
  if (!mass_in && tid < g.n_q) lse_s[tid] = lse[hk * g.n_q + tid];
  __syncthreads();
  const int j = tile * kTile + tid;
  const bool valid = j < g.L_k;
  float a = -INFINITY;
  if (valid) {
    const int64_t o = (int64_t)hk * g.L_k + j;
    float mass = 0.f;
    if (mass_in) {
      mass = mass_in[o];
    } else {
      const float* s = S + ((int64_t)hk * g.n_q) * g.L_k + j;
      for (int i = 0; i < g.n_q; ++i) mass += expf(s[(int64_t)i * g.L_k] - lse_s[i]);
    }
    mass /= (float)g.n_q;
    if (accum_phase == 1) {
      imp_accum[o] += mass;
    } else if (accum_phase == 2) {
      const float t = imp_accum[o] + mass;
      imp_accum[o] = t;
      imp_out[o] = t / (float)n_steps;
    } else {
      imp_out[o] = mass;
    }
    if (accum_phase != 1) {
      float k[D];
      load_row<T, D>(K + (int64_t)hk * g.k_hs + (int64_t)j * g.k_rs, k);
      float n2 = 0.f, dot = 0.f;
#pragma unroll
      for (int e = 0; e < D; ++e) {
        n2 = fmaf(k[e], k[e], n2);
        dot = fmaf(mk_s[e], k[e], dot);
      }
      const float inv = 1.f / fmaxf(sqrtf(n2), 1e-12f);
      a = dot * inv - (n2 * inv * inv) / (float)g.L_k;
      a_out[o] = a;
    }
  }
  if (accum_phase == 1) return;
  float m = a, l = valid ? 1.f : 0.f;
  reduce_ml<kTile>(m, l, sm_m, sm_l);
  if (tid == 0) a_partial[hk * g.n_tiles + tile] = make_float2(m, l);
}

// One block finalises kFinKeys keys of a head: it first merges the head's partial softmax statistics of a (every
// block of the head does, in the same fixed order), then writes redundancy, pooled importance and the score.
constexpr int kFinThreads = 256, kFinKeys = 1024;

__global__ void __launch_bounds__(kFinThreads)
score_finalize_kernel(ScoreGeom g, const float* __restrict__ imp_in, const float* __restrict__ a_in,
                      const float2* __restrict__ a_partial, float* __restrict__ red_out,
                      float* __restrict__ score) {
  __shared__ float sm_m[kFinThreads / 32], sm_l[kFinThreads / 32];
  __shared__ float sh_m, sh_l;
  const int hk = blockIdx.y, tid = threadIdx.x;
  fc::pdl_wait();  // launched under the tail of the kernel that writes imp, a and the softmax statistics
  float m = -INFINITY, l = 0.f;
  for (int t0 = tid; t0 < g.n_partials; t0 += 8 * kFinThreads) {  // eight loads in flight, merged in the same order
    float2 p[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int t = t0 + k * kFinThreads;
      p[k] = t < g.n_partials ? a_partial[hk * g.n_partials + t] : make_float2(-INFINITY, 0.f);
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (t0 + k * kFinThreads >= g.n_partials) break;
      const float mn = fmaxf(m, p[k].x);
      l = (m == -INFINITY ? 0.f : l * expf(m - mn)) + (p[k].x == -INFINITY ? 0.f : p[k].y * expf(p[k].x - mn));
      m = mn;
    }
  }
  reduce_ml<kFinThreads>(m, l, sm_m, sm_l);
  if (tid == 0) {
    sh_m = m;
    sh_l = l;
  }
  __syncthreads();
  const int64_t base = (int64_t)hk * g.L_k;
  const int half = g.pool_k / 2;
  const float inv_l = 1.f / sh_l;
#pragma unroll
  for (int i = 0; i < kFinKeys / kFinThreads; ++i) {
    const int j = blockIdx.x * kFinKeys + i * kFinThreads + tid;
    if (j >= g.L_k) break;
    const float red = expf(a_in[base + j] - sh_m) * inv_l;
    float pooled = -INFINITY;
    for (int u = max(j - half, 0); u <= min(j + half, g.L_k - 1); ++u) pooled = fmaxf(pooled, imp_in[base + u]);
    if (red_out) red_out[base + j] = red;
    score[base + j] = g.lambda * pooled - (1.f - g.lambda) * red;
  }
}

struct ScoreWs {
  float *S, *mk_partial, *lse, *mean_key, *a, *imp_tmp;
  float2* a_partial;
  float2* tc_ml;      // tensor-core path: per-slice (max, sum) of every query
  float* tc_colsum;   // per-slice sums of normalised keys
  float* tc_lse2;
  float* tc_norm2;
  // frame-level path
  float* inv_norm;     // tiled redundancy: [H, n_tiles * 128] reciprocal key norms
  float* fr_mass;      // [H, L_k] sum over the queries of exp(logit - lse)
  float2* fr_ml;       // [H, slices, L_q] (maximum, sum) of every query over a slice of the keys
  size_t total;
};

ScoreWs carve(const ScoreGeom& g, void* ws) {
  ScoreWs w;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    void* p = ws ? (char*)ws + off : nullptr;
    off += fc::align_up(bytes, 256);
    return p;
  };
  const bool frame = g.n_q > kCoreMaxQueries;
  w.S = (float*)take(frame ? 0 : (size_t)g.H_kv * g.n_q * g.L_k * 4);
  w.mk_partial = (float*)take((size_t)g.H_kv * g.n_tiles * g.d * 4);
  w.lse = (float*)take((size_t)g.H_kv * g.n_q * 4);
  w.mean_key = (float*)take((size_t)g.H_kv * g.d * 4);
  w.a = (float*)take((size_t)g.H_kv * g.L_k * 4);
  w.imp_tmp = (float*)take((size_t)g.H_kv * g.L_k * 4);
  w.a_partial = (float2*)take((size_t)g.H_kv * g.n_tiles * 4 * 8);  // room for one entry per warp of a tile
  w.tc_ml = (float2*)take((size_t)g.H_kv * fc::kScoreTcMaxSlices * fc::kScoreTcMaxQueries * 8);
  w.tc_colsum = (float*)take((size_t)g.H_kv * fc::kScoreTcMaxSlices * g.d * 4);
  w.tc_lse2 = (float*)take((size_t)g.H_kv * fc::kScoreTcMaxQueries * 4);
  w.tc_norm2 = (float*)take((size_t)g.H_kv * g.L_k * 4);
  w.inv_norm = (float*)take((size_t)g.H_kv * g.n_tiles * kTile * 4);
  w.fr_mass = (float*)take(frame ? (size_t)g.H_kv * g.L_k * 4 : 0);
  w.fr_ml = (float2*)take(frame ? (size_t)g.H_kv * fc::kScoreFrameMaxSlices * g.L_q * 8 : 0);
  w.total = off;
  return w;
}

int make_geom(const fc_score_desc* d, ScoreGeom& g) {
  if (!d) return FC_ERR_INVALID_ARG;
  if (d->H_q <= 0 || d->H_kv <= 0 || d->H_q % d->H_kv || d->L_q <= 0 || d->L_k <= 0) return FC_ERR_INVALID_ARG;
  if (d->pool_k < 1 || d->pool_k % 2 == 0) return FC_ERR_INVALID_ARG;
  if (d->d != 64 && d->d != 128) return FC_ERR_UNSUPPORTED;
  g.H_q = d->H_q; g.H_kv = d->H_kv; g.d = d->d; g.L_q = d->L_q; g.L_k = d->L_k;
  g.q_hs = d->q_hs; g.q_rs = d->q_rs;
  g.group = d->H_q / d->H_kv;
  // Grouped query heads whose rows follow each other in memory (head stride = L_q rows) are one key head's worth of
  // group * L_q observation queries: the importance is the mean over all of them (the group's heads and their rows)
  // either way, and every pipeline, the tensor-core ones included, then sees one query head per key head.
  if (g.group > 1 && d->q_hs == (int64_t)d->L_q * d->q_rs && (int64_t)g.group * d->L_q <= fc::kScoreFrameMaxQueries) {
    g.L_q = g.group * d->L_q;
    g.q_hs = (int64_t)g.group * d->q_hs;
    g.H_q = d->H_kv;
    g.group = 1;
  }
  g.n_q = g.group * g.L_q;
  if (g.n_q > kCoreMaxQueries && (g.group != 1 || g.L_q > fc::kScoreFrameMaxQueries)) return FC_ERR_UNSUPPORTED;
  g.n_tiles = (d->L_k + kTile - 1) / kTile;
  g.n_partials = g.n_tiles;
  g.k_hs = d->k_hs; g.k_rs = d->k_rs;
  g.scale = d->scale != 0.f ? d->scale : 1.f / sqrtf((float)d->d);
  g.lambda = d->lambda;
  g.pool_k = d->pool_k;
  return FC_OK;
}

template <typename T, int D>
int run(cudaStream_t st, const ScoreGeom& g, const ScoreWs& w, const void* Q, const void* K,
        float* imp_accum, int phase, int n_steps, float* imp_buf) {
  const size_t smem1 = ((size_t)g.n_q * D + (size_t)kTile * (D + 1)) * 4;
  FC_CUDA_CHECK(cudaFuncSetAttribute(score_pass1_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem1));
  dim3 grid(g.n_tiles, g.H_kv);
  score_pass1_kernel<T, D><<<grid, kTile, smem1, st>>>((const T*)Q, (const T*)K, g, w.S, w.mk_partial);
  FC_LAUNCH_CHECK("score_pass1_kernel");
  score_row_lse_kernel<<<dim3(g.n_q, g.H_kv), 256, 0, st>>>(w.S, g.L_k, w.lse);
  FC_LAUNCH_CHECK("score_row_lse_kernel");
  score_mean_key_kernel<<<g.H_kv, kMkGroups * 128, 0, st>>>(w.mk_partial, g.n_tiles, D, g.L_k, w.mean_key);
  FC_LAUNCH_CHECK("score_mean_key_kernel");
  score_pass2_kernel<T, D><<<grid, kTile, 0, st>>>((const T*)K, g, w.S, w.lse, w.mean_key, nullptr, imp_accum, phase,
                                                   n_steps, imp_buf, w.a, w.a_partial);
  FC_LAUNCH_CHECK("score_pass2_kernel");
  return FC_OK;
}

// Frame-level pipeline (bf16, one query head per key head, any number of queries up to kScoreFrameMaxQueries).
template <int D>
int run_frame(fc_ctx* ctx, cudaStream_t st, const ScoreGeom& g, const ScoreWs& w, const void* Q, const void* K,
              float* imp_accum, int phase, int n_steps, float* imp_buf, uint32_t* status) {
  using T = __nv_bfloat16;
  dim3 grid(g.n_tiles, g.H_kv);
  // 1. sums of normalised keys per tile, then the head's mean key
  frame_key_sums_kernel<D><<<grid, kTile, 0, st>>>((const T*)K, g, w.mk_partial);
  FC_LAUNCH_CHECK("frame_key_sums_kernel");
  score_mean_key_kernel<<<g.H_kv, kMkGroups * 128, 0, st>>>(w.mk_partial, g.n_tiles, D, g.L_k, w.mean_key);
  FC_LAUNCH_CHECK("score_mean_key_kernel");
  // 2., 3. log-sum-exp of every query over the candidates, then the attention mass of every key
  int rc = fc::score_frame_mass(ctx, st, g.H_kv, g.d, g.L_q, g.L_k, g.scale * 1.4426950408889634f, Q, g.q_hs, g.q_rs, K,
                                g.k_hs, g.k_rs, w.fr_ml, w.lse, w.fr_mass, status);
  if (rc != FC_OK) return rc;
  // 4. mean over the queries, accumulation over steps, redundancy logits
  frame_finish_kernel<D><<<grid, kTile, 0, st>>>((const T*)K, g, w.mean_key, w.fr_mass, imp_accum, phase, n_steps, imp_buf,
                                                 w.a, w.a_partial);
  FC_LAUNCH_CHECK("frame_finish_kernel");
  return FC_OK;
}

}  // namespace

extern "C" size_t fc_kv_score_workspace_bytes(const fc_score_desc* desc) {
  ScoreGeom g;
  if (make_geom(desc, g) != FC_OK) return 0;
  return carve(g, nullptr).total;
}

extern "C" int fc_kv_score(fc_ctx* ctx, void* stream, const fc_score_desc* desc, const void* Q_obs,
                           const void* K_cand, int dtype, float* imp_accum, int accum_phase, int n_steps,
                           float* imp, float* red, float* score, uint32_t* status, void* ws,
                           size_t ws_bytes) {
  if (!ctx || !Q_obs || !K_cand) return FC_ERR_INVALID_ARG;
  ScoreGeom g;
  int rc = make_geom(desc, g);
  if (rc != FC_OK) return rc;
  if (dtype != FC_BF16 && dtype != FC_F32) return FC_ERR_UNSUPPORTED;
  if (accum_phase < 0 || accum_phase > 2) return FC_ERR_INVALID_ARG;
  if (accum_phase != 0 && (!imp_accum || n_steps <= 0)) return FC_ERR_INVALID_ARG;
  if (accum_phase != 1 && !score) return FC_ERR_INVALID_ARG;
  const int es = fc::elem_size(dtype);
  if (!fc::aligned16(Q_obs) || !fc::aligned16(K_cand)) return FC_ERR_MISALIGNED;
  if ((g.k_hs * es) % 16 || (g.k_rs * es) % 16 || (g.q_hs * es) % 16 || (g.q_rs * es) % 16)
    return FC_ERR_MISALIGNED;
  if (g.k_rs < g.d || g.q_rs < g.d) return FC_ERR_INVALID_ARG;
  const ScoreWs w = carve(g, ws);
  if (!ws || ws_bytes < w.total) return FC_ERR_WORKSPACE;
  if (!fc::aligned16(ws)) return FC_ERR_MISALIGNED;
  cudaStream_t st = (cudaStream_t)stream;
  if (desc->impl < 0 || desc->impl > 2) return FC_ERR_INVALID_ARG;
  if (desc->red_mode < FC_RED_MEANKEY || desc->red_mode > FC_RED_TILED_MAX) return FC_ERR_INVALID_ARG;
  if (desc->red_mode != FC_RED_MEANKEY && dtype != FC_BF16) return FC_ERR_UNSUPPORTED;  // the tiles are bf16 MMAs
  float* imp_buf = imp ? imp : w.imp_tmp;
  // 1. importance (and the mean-key redundancy argument) by one of the three pipelines
  if (g.n_q > kCoreMaxQueries) {
    if (dtype != FC_BF16 || desc->impl == 1) return FC_ERR_UNSUPPORTED;
    rc = g.d == 128 ? run_frame<128>(ctx, st, g, w, Q_obs, K_cand, imp_accum, accum_phase, n_steps, imp_buf, status)
                    : run_frame<64>(ctx, st, g, w, Q_obs, K_cand, imp_accum, accum_phase, n_steps, imp_buf, status);
  } else {
    const bool tc_ok = dtype == FC_BF16 && g.group == 1 && g.L_q <= fc::kScoreTcMaxQueries - 2;
    if (desc->impl == 2 && !tc_ok) return FC_ERR_UNSUPPORTED;
    if (tc_ok && desc->impl != 1) {
      fc::ScoreTcArgs a;
      a.H = g.H_kv; a.L_q = g.L_q; a.L_k = g.L_k; a.n_tiles = g.n_tiles; a.tiles_per_slice = 0; a.n_slices = 0;
      a.scale_log2 = g.scale * 1.4426950408889634f;
      a.accum_phase = accum_phase; a.n_steps = n_steps;
      a.ml_part = w.tc_ml; a.colsum_part = w.tc_colsum; a.norm2 = w.tc_norm2;
      a.imp_accum = imp_accum; a.imp_out = imp_buf; a.a_out = w.a; a.a_partial = w.a_partial;
      a.status = status;
      rc = fc::score_tc_run(ctx, st, a, g.d, g.q_hs, g.q_rs, g.k_hs, g.k_rs, Q_obs, K_cand);
      g.n_partials = g.n_tiles * 4;  // the tensor-core pass leaves one entry per warp of a tile
    } else if (dtype == FC_BF16) {
      rc = g.d == 128 ? run<__nv_bfloat16, 128>(st, g, w, Q_obs, K_cand, imp_accum, accum_phase, n_steps, imp_buf)
                      : run<__nv_bfloat16, 64>(st, g, w, Q_obs, K_cand, imp_accum, accum_phase, n_steps, imp_buf);
    } else {
      rc = g.d == 128 ? run<float, 128>(st, g, w, Q_obs, K_cand, imp_accum, accum_phase, n_steps, imp_buf)
                      : run<float, 64>(st, g, w, Q_obs, K_cand, imp_accum, accum_phase, n_steps, imp_buf);
    }
  }
  if (rc != FC_OK || accum_phase == 1) return rc;
  // 2. optionally the redundancy argument from explicit similarity tiles, in place of the mean-key form
  if (desc->red_mode != FC_RED_MEANKEY) {
    fc::RedTiledArgs r;
    r.H = g.H_kv; r.L_k = g.L_k; r.n_tiles = g.n_tiles;
    r.inv_norm = w.inv_norm; r.a_out = w.a; r.a_partial = w.a_partial; r.status = status;
    rc = fc::score_red_tiled(ctx, st, r, g.d, g.k_hs, g.k_rs, K_cand, desc->red_mode == FC_RED_TILED_MAX);
    if (rc != FC_OK) return rc;
    g.n_partials = g.n_tiles * 4;
  }
  // 3. softmax of the redundancy argument, max-pool of the importance, lambda-mix
  FC_CUDA_CHECK(fc::launch_pdl(score_finalize_kernel, dim3((g.L_k + kFinKeys - 1) / kFinKeys, g.H_kv), dim3(kFinThreads), 0,
                               st, g, (const float*)imp_buf, (const float*)w.a, (const float2*)w.a_partial, red, score));
  return FC_OK;
}
