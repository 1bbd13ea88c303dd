// Redundancy from explicit tiles of the cosine-similarity matrix on tcgen05 tensor cores (bf16 keys).
//
// Eq. 11 asks for a statistic of every column of S = Khat Khat^T with the diagonal zeroed.  The default path
// of fc_kv_score never forms S (the column MEAN collapses to a dot product with the mean key, the identity of the
// paper's efficiency appendix); this file is the dense form, for checking that identity at scale and for
// statistics that do not collapse (here: the column maximum over the other tokens).  S is symmetric, so the
// statistic of column j is taken along ROW j, which keeps the reduction inside one thread:
//   a CTA owns two tiles J0, J1 of 128 keys each (the A operands, loaded once) and streams every tile I of the head
//   past them (the B operand, 4-stage TMA ring, L2 hits after the head's first CTA): D[j, i] = k_j . k_i (raw bf16
//   keys: the products are exact, accumulation is fp32 in tensor memory); the thread of row j folds D[j, i] / |k_i|
//   over i (sum or maximum), skipping i = j, and scales by 1 / |k_j| at the end.  S is never stored.  Two resident
//   tiles because the streamed operand is what costs: with one, every 128 x 128 x 128 MMA group needs 32 KB from L2
//   (26.9 GB per launch on 24 heads x 23400 keys, tensor pipe 36 % busy, bound by the L2-to-SM path); with two, half.
// Normalising in the epilogue instead of feeding normalised bf16 keys keeps 1e-4 accuracy on Red with one MMA per
// tile (normalised keys rounded to bf16 would need a high / low split: three MMAs per tile).
// Roles (288 threads): warps 0-3 read the accumulators of J0, warps 4-7 those of J1 (two 128-column accumulators per
// resident tile, alternating by streamed tile: all 512 columns), warp 8 issues the copies and the MMAs.  Measured on
// 24 heads x 23400 keys: 3.4 ms = 0.99 PFLOP/s, tensor pipe 47 % busy (4.25 ms and 36 % with one resident tile).  What
// is left is the round trip accumulator-free -> MMA -> accumulator-full -> load through two barriers with only two
// accumulators per resident tile in flight; prefetching the norms, one 128-column load and pinned MMA groups each
// changed it by less than 2 %.
// Fixed summation order: bit-reproducible.  Every mbarrier wait is bounded; tensor memory is always released.
#include <cmath>

#include "fc_attention.cuh"
#include "fc_score.cuh"
#include "fc_tcgen05.cuh"
#include "fc_tcgen05_ld.cuh"

namespace {

using namespace fc::sm100;

constexpr int kKeys = 128;  // keys per tile
constexpr int kRing = 4;    // streamed tiles in flight
constexpr int kThreads = 288;
constexpr int kCopyWarp = 8;

struct RedSmem {
  uint64_t a_full, k_full[kRing], k_free[kRing];
  uint64_t s_full[2][2], s_free[2][2];  // [resident tile][accumulator = parity of the streamed tile]
  uint32_t tmem_base, abort;
  alignas(8) float inv_s[2][2][kKeys];  // [group][parity of the streamed tile] 1 / |k_i| of the streamed tile
};

__device__ __forceinline__ void group_barrier(int grp) { asm volatile("bar.sync %0, 128;" ::"r"(1 + grp) : "memory"); }

template <typename T, int D>
__global__ void __launch_bounds__(128)
key_inv_norm_kernel(const T* __restrict__ K, int L_k, int L_pad, int64_t k_hs, int64_t k_rs, float* __restrict__ inv_norm) {
  // one key per thread; entries past the end of the cache are 0, so that they add nothing to a sum
  const int h = blockIdx.y, j = blockIdx.x * 128 + threadIdx.x;
  float inv = 0.f;
  if (j < L_k) {
    const T* row = K + (int64_t)h * k_hs + (int64_t)j * k_rs;
    float n4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int v = 0; v < D / 8; ++v) {
      const uint4 w = *reinterpret_cast<const uint4*>(row + v * 8);
      const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float lo = fc::bf16_lo(ww[e]), hi = fc::bf16_hi(ww[e]);
        n4[e] = fmaf(lo, lo, n4[e]);
        n4[e] = fmaf(hi, hi, n4[e]);
      }
    }
    inv = 1.f / fmaxf(sqrtf((n4[0] + n4[1]) + (n4[2] + n4[3])), 1e-12f);
  }
  inv_norm[(int64_t)h * L_pad + j] = inv;  // j < L_pad: the grid covers exactly the padded length
}

// kMax = false: a_j = (1 / L_k) sum_{i != j} cos(i, j)   (Eq. 11 before its softmax)
// kMax = true:  a_j = max_{i != j} cos(i, j)              (0 when there is no other token)
template <int D, bool kMax>
__global__ void __launch_bounds__(kThreads, 1)
red_tiled_kernel(const __grid_constant__ CUtensorMap tmap_k, const fc::RedTiledArgs g) {
  constexpr uint32_t kTileBytes = kKeys * D * 2;
  constexpr int kAtoms = D / 64;
  constexpr uint32_t kAtomBytes = kKeys * 128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* a_tiles = smem;                  // J0, J1
  uint8_t* k_tiles = smem + 2 * kTileBytes;
  RedSmem* sh = (RedSmem*)(smem + (2 + kRing) * kTileBytes);
  volatile uint32_t* abort = &sh->abort;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int hk = blockIdx.y, n = g.n_tiles;
  const int L_pad = g.n_tiles * kKeys;

  if (tid == 0) {
    mbar_init(smem_u32(&sh->a_full), 1);
    for (int s = 0; s < kRing; ++s) {
      mbar_init(smem_u32(&sh->k_full[s]), 1);
      mbar_init(smem_u32(&sh->k_free[s]), 1);  // the MMA's commit
    }
    for (int jj = 0; jj < 2; ++jj)
      for (int b = 0; b < 2; ++b) {
        mbar_init(smem_u32(&sh->s_full[jj][b]), 1);
        mbar_init(smem_u32(&sh->s_free[jj][b]), 4);  // the four warps of the group that reads it
      }
    mbar_fence_init();
    sh->abort = 0;
    tma_prefetch_desc(&tmap_k);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&sh->tmem_base), 4 * kKeys);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh->tmem_base;

  if (warp == kCopyWarp) {
    // ---------------------------------------------------------------- copies and MMAs (one thread)
    if (lane == 0) {
      auto load_k = [&](int i) {  // tile i of the head into stage i % kRing
        const int st = i % kRing;
        const uint32_t bar = smem_u32(&sh->k_full[st]);
        mbar_expect_tx(bar, kTileBytes);
        for (int x = 0; x < kAtoms; ++x)
          tma_load_3d(smem_u32(k_tiles + st * kTileBytes + x * kAtomBytes), &tmap_k, bar, x * 64, i * kKeys, hk);
      };
      mbar_expect_tx(smem_u32(&sh->a_full), 2 * kTileBytes);  // a resident tile past the cache reads as zeros
      for (int jj = 0; jj < 2; ++jj)
        for (int x = 0; x < kAtoms; ++x)
          tma_load_3d(smem_u32(a_tiles + jj * kTileBytes + x * kAtomBytes), &tmap_k, smem_u32(&sh->a_full), x * 64,
                      (2 * blockIdx.x + jj) * kKeys, hk);
      for (int i = 0; i < min(n, kRing - 1); ++i) load_k(i);
      mbar_wait_bounded(smem_u32(&sh->a_full), 0, abort);
      const uint64_t da0 = smem_desc_sw128(smem_u32(a_tiles), 16, 1024);
      constexpr uint32_t kIdesc = idesc_bf16_f32(kKeys, kKeys, false, false);
      // The issuing thread does not run ahead of the tensor pipe: whatever it executes between two MMAs is time the
      // pipe idles.  So the descriptors of a group are computed and pinned in registers before the waits, and a
      // group is one block of instructions.
      constexpr int kSteps = D / 16;
      uint64_t a0[kSteps], a1[kSteps], kb[kSteps];
#pragma unroll
      for (int kk = 0; kk < kSteps; ++kk) {
        const uint64_t off = ((kk / 4) * kAtomBytes + (kk % 4) * 32) >> 4;
        a0[kk] = da0 + off;
        a1[kk] = da0 + off + (uint64_t)(kTileBytes >> 4);
      }
      pin(a0);
      pin(a1);
      const uint64_t dk0 = smem_desc_sw128(smem_u32(k_tiles), 16, 1024);
      for (int i = 0; i < n; ++i) {
        const int st = i % kRing, b = i & 1;
        const uint32_t par_free = ((i >> 1) & 1) ^ 1;
#pragma unroll
        for (int kk = 0; kk < kSteps; ++kk)
          kb[kk] = dk0 + (uint64_t)((st * kTileBytes + (kk / 4) * kAtomBytes + (kk % 4) * 32) >> 4);
        pin(kb);
        mbar_wait_bounded(smem_u32(&sh->k_full[st]), (i / kRing) & 1, abort);
        mbar_wait_bounded(smem_u32(&sh->s_free[0][b]), par_free, abort);
        tc_fence_after();
        umma_ss_group<kSteps>(tmem + b * kKeys, a0, kb, kIdesc);  // D[j, i] = k_j . k_i for the first resident tile
        umma_commit(smem_u32(&sh->s_full[0][b]));
        mbar_wait_bounded(smem_u32(&sh->s_free[1][b]), par_free, abort);
        tc_fence_after();
        umma_ss_group<kSteps>(tmem + (2 + b) * kKeys, a1, kb, kIdesc);  // ... and the second
        umma_commit(smem_u32(&sh->s_full[1][b]));
        umma_commit(smem_u32(&sh->k_free[st]));
        if (i + kRing - 1 < n) {  // refill the stage tile i-1 has left
          if (i >= 1) mbar_wait_bounded(smem_u32(&sh->k_free[(i - 1) % kRing]), ((i - 1) / kRing) & 1, abort);
          load_k(i + kRing - 1);
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- accumulators out of tensor memory
    const int grp = warp >> 2, row = tid & 127;  // group = resident tile
    const int tj = 2 * blockIdx.x + grp;
    const uint32_t t_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16) + grp * 2 * kKeys;
    const float* inv_h = g.inv_norm + (int64_t)hk * L_pad;
    float acc = kMax ? -INFINITY : 0.f;
    uint64_t acc2[2] = {0ull, 0ull};  // the sum's fast path: two independent two-wide chains
    float next_inv = inv_h[row];  // reciprocal norm of this thread's key of the first streamed tile
    for (int i = 0; i < n; ++i) {
      const int b = i & 1, par = (i >> 1) & 1;
      const float my_inv = next_inv;
      if (i + 1 < n) next_inv = inv_h[(i + 1) * kKeys + row];  // a tile ahead: its latency hides behind this tile's work
      mbar_wait_bounded(smem_u32(&sh->s_full[grp][b]), par, abort);
      tc_fence_after();
      sh->inv_s[grp][b][row] = my_inv;
      uint32_t sv[kKeys];
      tmem_ld128_wait(t_lane + b * kKeys, sv);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sh->s_free[grp][b]));  // the accumulator can take the tile after next
      group_barrier(grp);  // the tile's 128 reciprocal norms are in place (the other buffer is still being read)
      const float* inv_t = sh->inv_s[grp][b];
      const bool special = i == tj || (i + 1) * kKeys > g.L_k;  // the diagonal tile, or a ragged last tile
      if (special) {
        const int cols_valid = min(kKeys, g.L_k - i * kKeys);
#pragma unroll
        for (int col = 0; col < kKeys; ++col) {
          const bool skip = (i == tj && col == row) || col >= cols_valid;  // S_jj, and columns past the cache
          const float x = __uint_as_float(sv[col]) * inv_t[col];
          if (kMax) acc = skip ? acc : fmaxf(acc, x);
          else acc += skip ? 0.f : x;
        }
      } else if (kMax) {
#pragma unroll
        for (int c = 0; c < kKeys; c += 2) {
          const uint64_t i2 = *reinterpret_cast<const uint64_t*>(&inv_t[c]);
          float x0, x1;
          unpack2(fma2(pack2(__uint_as_float(sv[c]), __uint_as_float(sv[c + 1])), i2, 0ull), x0, x1);
          acc = max3(acc, x0, x1);
        }
      } else {
#pragma unroll
        for (int c = 0; c < kKeys; c += 2) {
          const uint64_t i2 = *reinterpret_cast<const uint64_t*>(&inv_t[c]);
          acc2[(c >> 1) & 1] = fma2(pack2(__uint_as_float(sv[c]), __uint_as_float(sv[c + 1])), i2, acc2[(c >> 1) & 1]);
        }
      }
    }
    if (!kMax) {
      float s0, s1, s2, s3;
      unpack2(acc2[0], s0, s1);
      unpack2(acc2[1], s2, s3);
      acc += (s0 + s1) + (s2 + s3);
    }
    if (tj < g.n_tiles) {  // (warp-uniform: the second resident tile of the last CTA may lie past the cache)
      const int j = tj * kKeys + row;
      const bool valid = j < g.L_k;
      float a = -INFINITY;
      if (valid) {
        const float inv_j = inv_h[j];
        if (kMax) a = g.L_k > 1 ? acc * inv_j : 0.f;
        else a = acc * inv_j / (float)g.L_k;
        g.a_out[(int64_t)hk * g.L_k + j] = a;
      }
      // softmax statistics (max, sum of exp) of a over this warp's 32 keys, fixed order
      float m = a;
#pragma unroll
      for (int w = 16; w > 0; w >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, w));
      float l = valid ? expf(a - m) : 0.f;
#pragma unroll
      for (int w = 16; w > 0; w >>= 1) l += __shfl_xor_sync(0xffffffffu, l, w);
      if (lane == 0) g.a_partial[((int64_t)hk * g.n_tiles + tj) * 4 + (warp & 3)] = make_float2(m, l);
    }
  }

  if (*abort) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let copies and MMAs in flight land before teardown
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort && g.status) atomicOr(g.status, FC_DEV_TIMEOUT);
  if (warp == 0) tmem_dealloc(tmem, 4 * kKeys);
}

}  // namespace

namespace fc {

int score_red_tiled(fc_ctx* ctx, cudaStream_t st, RedTiledArgs g, int d, int64_t k_hs, int64_t k_rs, const void* K,
                    bool max_similarity) {
  CUtensorMap tk;
  int rc;
  if ((rc = make_tmap(ctx, &tk, K, d, g.L_k, g.H, k_rs, g.H > 1 ? k_hs : k_rs * g.L_k)) != FC_OK) return rc;
  const int L_pad = g.n_tiles * kKeys;
  const dim3 grid(g.n_tiles, g.H), grid2((g.n_tiles + 1) / 2, g.H);  // the similarity kernel: two resident tiles per CTA
  auto* Kb = (const __nv_bfloat16*)K;
  if (d == 128) key_inv_norm_kernel<__nv_bfloat16, 128><<<grid, 128, 0, st>>>(Kb, g.L_k, L_pad, k_hs, k_rs, g.inv_norm);
  else key_inv_norm_kernel<__nv_bfloat16, 64><<<grid, 128, 0, st>>>(Kb, g.L_k, L_pad, k_hs, k_rs, g.inv_norm);
  FC_LAUNCH_CHECK("key_inv_norm_kernel");
  const size_t smem = (size_t)(2 + kRing) * kKeys * d * 2 + sizeof(RedSmem) + 1024;
  auto launch = [&](auto kernel) -> int {
    FC_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kernel<<<grid2, kThreads, smem, st>>>(tk, g);
    FC_LAUNCH_CHECK("red_tiled_kernel");
    return FC_OK;
  };
  if (d == 128) return max_similarity ? launch(red_tiled_kernel<128, true>) : launch(red_tiled_kernel<128, false>);
  return max_similarity ? launch(red_tiled_kernel<64, true>) : launch(red_tiled_kernel<64, false>);
}

}  // namespace fc
