// Attention mass of every candidate key under many observation queries (a latent frame or a whole chunk of
// them) on tcgen05 tensor cores: the importance of Eq. 9 at frame-level query granularity, where the score stage
// is a dense contraction instead of a streaming read.
//
//   mass[h, j] = sum_i exp(q_i . k_j * scale - lse_i)        lse_i = log sum_j exp(q_i . k_j * scale)
//
// Two launches of one kernel, which recomputes the logits instead of storing them and picks the orientation whose
// reduction stays inside a thread:
//   row statistics   S[query, key] = Q K^T, one query row per thread: running (max, sum) over all keys -> lse
//   masses           S[key, query] = K Q^T, one key row per thread: the sum over the queries
// Below, the tile that a CTA holds is the "own" tile (queries for the statistics, keys for the masses) and the
// other operand streams past it.  A CTA owns one head and every gridDim.x-th tile of 128 keys of it (set-up, the
// head's log-sum-exps in shared memory and the tensor-memory allocation are paid once per CTA); per key tile the
// keys are loaded once and the
// head's query tiles stream through a 2-stage TMA ring (they stay in L2: every CTA of the head reads them), one
// thread issues the MMAs into two 128-column accumulators and four warps turn them into masses.  Two CTAs share
// an SM (2 x 256 tensor-memory columns, 2 x 97 KiB of shared memory; one CTA when the head has more than about
// 3000 queries, whose log-sum-exps sit in shared memory), which puts two exponentiating warps on every
// scheduler: the special-function unit, 16 exponentials per clock, is what bounds the kernel.
// Sums are fixed-order: results are bit-reproducible from run to run.  Every mbarrier wait is bounded.
#include <cmath>

#include "fc_attention.cuh"
#include "fc_score.cuh"
#include "fc_tcgen05.cuh"
#include "fc_tcgen05_ld.cuh"

namespace {

using namespace fc::sm100;

constexpr int kKeys = 128, kQueries = 128;  // tile: MMA M and N
constexpr int kRing = 4;     // streamed tiles in flight = logit accumulators in tensor memory (4 x 128 columns)
constexpr int kFmaShare = 1;  // of every four column pairs, how many take their exponential on the fma pipe
constexpr int kGroups = 4;   // consumer warpgroups; group g takes every fourth streamed tile
constexpr int kThreads = 32 * (4 * kGroups + 2);  // 16 consumer warps, one copy warp, one MMA warp

struct MassSmem {
  uint64_t own_full[2], own_free[2], q_full[kRing], q_free[kRing], s_full[kRing], s_free[kRing];
  uint64_t merge_bar;  // all consumer warps, once per own tile
  uint32_t tmem_base, abort;
  float2 part[2][kGroups][kKeys];  // per own tile (double-buffered), group and row: partial mass or (maximum, sum)
};

// minus the log2-domain log-sum-exp of every query: the slices' (maximum, sum) pairs merged in slice order
__global__ void score_frame_lse_kernel(const float2* __restrict__ ml, int n_slices, int L_q, float* __restrict__ nlse) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x, hk = blockIdx.y;
  if (i >= L_q) return;
  float m = -INFINITY, l = 0.f;
  for (int sl = 0; sl < n_slices; ++sl) {
    const float2 p = ml[((int64_t)hk * n_slices + sl) * L_q + i];
    const float mn = fmaxf(m, p.x);
    l = (m == -INFINITY ? 0.f : l * exp2f(m - mn)) + (p.x == -INFINITY ? 0.f : p.y * exp2f(p.x - mn));
    m = mn;
  }
  nlse[(int64_t)hk * L_q + i] = -(m + log2f(l));
}

template <int D, bool kStats>
__global__ void __launch_bounds__(kThreads, 1)
score_mass_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k, int L_q,
                  int L_k, float scale_log2, const float* __restrict__ nlse_in, float2* __restrict__ ml_out,
                  float* __restrict__ mass, uint32_t* __restrict__ status) {
  constexpr uint32_t kTileBytes = kKeys * D * 2;
  constexpr int kAtoms = D / 64;
  constexpr uint32_t kAtomBytes = kKeys * 128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t k_s = smem_u32(smem), q_s = k_s + 2 * kTileBytes;  // own tiles (2), then the ring of streamed tiles
  MassSmem* sh = (MassSmem*)(smem + (2 + kRing) * kTileBytes);
  // minus the log-sum-exp of every query of the head in the log2 domain, padded to whole tiles with -inf
  float* nlse_s = (float*)(sh + 1);
  volatile uint32_t* abort = &sh->abort;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int hk = blockIdx.y;
  const int n_qt = (L_q + kQueries - 1) / kQueries, n_kt = (L_k + kKeys - 1) / kKeys;
  // streamed tiles of this CTA (a slice of them in the statistics launch)
  const int per_slice = (n_qt + (int)gridDim.z - 1) / (int)gridDim.z;
  const int t_begin = blockIdx.z * per_slice, t_end = min(n_qt, t_begin + per_slice);

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&sh->own_full[s]), 1);
      mbar_init(smem_u32(&sh->own_free[s]), 1);
    }
    for (int s = 0; s < kRing; ++s) {
      mbar_init(smem_u32(&sh->q_full[s]), 1);
      mbar_init(smem_u32(&sh->q_free[s]), 1);
      mbar_init(smem_u32(&sh->s_full[s]), 1);
      mbar_init(smem_u32(&sh->s_free[s]), 4);  // the four warps of the group that reads accumulator s
    }
    mbar_init(smem_u32(&sh->merge_bar), 4 * kGroups);
    mbar_fence_init();
    sh->abort = 0;
    tma_prefetch_desc(&tmap_q);
    tma_prefetch_desc(&tmap_k);
  }
  if (!kStats) {
    for (int i = tid; i < n_qt * kQueries; i += kThreads)
      nlse_s[i] = i < L_q ? nlse_in[(int64_t)hk * L_q + i] : -INFINITY;  // padding queries: 2^-inf = 0
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&sh->tmem_base), kRing * kQueries);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh->tmem_base;

  if (warp == 4 * kGroups) {
    // ------------------------------------------------------------------ copies
    if (lane == 0) {
      uint32_t tq = 0, it = 0;  // streamed tiles and own tiles loaded so far (ring phases)
      for (int tile = blockIdx.x; tile < n_kt && !*abort; tile += gridDim.x, ++it) {
        const int o = it & 1;
        if (!mbar_wait_bounded(smem_u32(&sh->own_free[o]), ((it >> 1) & 1) ^ 1, abort)) break;
        mbar_expect_tx(smem_u32(&sh->own_full[o]), kTileBytes);
        for (int x = 0; x < kAtoms; ++x)
          tma_load_3d(k_s + o * kTileBytes + x * kAtomBytes, &tmap_k, smem_u32(&sh->own_full[o]), x * 64, tile * kKeys, hk);
        for (int t = t_begin; t < t_end; ++t, ++tq) {
          const int st = tq % kRing, ph = (tq / kRing) & 1;
          if (!mbar_wait_bounded(smem_u32(&sh->q_free[st]), ph ^ 1, abort)) break;
          mbar_expect_tx(smem_u32(&sh->q_full[st]), kTileBytes);
          for (int x = 0; x < kAtoms; ++x)
            tma_load_3d(q_s + st * kTileBytes + x * kAtomBytes, &tmap_q, smem_u32(&sh->q_full[st]), x * 64,
                        t * kQueries, hk);
        }
      }
    }
  } else if (warp == 4 * kGroups + 1) {
    // ------------------------------------------------------------------ MMAs: S[own row, streamed row]
    if (lane == 0) {
      constexpr uint32_t kIdesc = idesc_bf16_f32(kKeys, kQueries, false, false);
      constexpr int kSteps = D / 16;
      const uint64_t dk = smem_desc_sw128(k_s, 16, 1024), dq = smem_desc_sw128(q_s, 16, 1024);
      // The issuing thread does not run ahead of the tensor pipe, so the operand descriptors of a tile are computed
      // and pinned in registers before the waits, and its MMAs go out as one block of instructions.
      uint64_t da[kSteps], db[kSteps];
      uint32_t tq = 0, it = 0;
      for (int tile = blockIdx.x; tile < n_kt && !*abort; tile += gridDim.x, ++it) {
        const int o = it & 1;
#pragma unroll
        for (int kk = 0; kk < kSteps; ++kk)
          da[kk] = dk + (uint64_t)((o * kTileBytes + (kk / 4) * kAtomBytes + (kk % 4) * 32) >> 4);
        pin(da);
        if (!mbar_wait_bounded(smem_u32(&sh->own_full[o]), (it >> 1) & 1, abort)) break;
        for (int t = t_begin; t < t_end; ++t, ++tq) {
          const int st = tq % kRing, ph = (tq / kRing) & 1;  // ring slot = accumulator
#pragma unroll
          for (int kk = 0; kk < kSteps; ++kk)
            db[kk] = dq + (uint64_t)((st * kTileBytes + (kk / 4) * kAtomBytes + (kk % 4) * 32) >> 4);
          pin(db);
          if (!mbar_wait_bounded(smem_u32(&sh->q_full[st]), ph, abort)) break;
          if (!mbar_wait_bounded(smem_u32(&sh->s_free[st]), ph ^ 1, abort)) break;
          tc_fence_after();
          umma_ss_group<kSteps>(tmem + st * kQueries, da, db, kIdesc);
          umma_commit(smem_u32(&sh->s_full[st]));
          umma_commit(smem_u32(&sh->q_free[st]));
        }
        umma_commit(smem_u32(&sh->own_free[o]));  // the own tile has been read by every MMA issued for it
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers: one own row per thread; group grp
    // takes the streamed tiles whose ring slot is grp
    const int grp = warp >> 2, quad = warp & 3;
    const uint32_t t_acc = tmem + ((uint32_t)(quad * 32) << 16) + grp * kQueries;
    const uint64_t sc2 = pack2(scale_log2, scale_log2);
    const uint32_t b_sfull = smem_u32(&sh->s_full[grp]), b_sfree = smem_u32(&sh->s_free[grp]);
    uint32_t tq = 0, it = 0;
    for (int tile = blockIdx.x; tile < n_kt && !*abort; tile += gridDim.x, ++it) {
      uint64_t acc[2] = {0ull, 0ull};
      float m_run = -INFINITY, l_run = 0.f;  // kStats: running reference maximum (log2 domain) and sum against it
      for (int t = t_begin; t < t_end; ++t, ++tq) {
        if ((int)(tq % kRing) != grp) continue;
        if (!mbar_wait_bounded(b_sfull, (tq / kRing) & 1, abort)) break;
        tc_fence_after();
        if constexpr (kStats) {
          // one query row against 128 keys: the reference moves only when the tile maximum exceeds it by 2^8, so
          // the exponents stay below 2^8 and the sum is rescaled a few times per row at most
          const int cols_valid = min(kQueries, L_q - t * kQueries);
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t sv[64];
            tmem_ld64_wait(t_acc + half * 64, sv);
            if (cols_valid < half * 64 + 64) {
#pragma unroll
              for (int i = 0; i < 64; ++i)
                if (half * 64 + i >= cols_valid) sv[i] = 0xff800000u;  // -inf
            }
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int i = 0; i < 64; i += 8) {
#pragma unroll
              for (int c4 = 0; c4 < 4; ++c4)
                mx[c4] = max3(mx[c4], __uint_as_float(sv[i + 2 * c4]), __uint_as_float(sv[i + 2 * c4 + 1]));
            }
            const float tile_max = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2;  // scale > 0
            if (tile_max > m_run + 8.f) {
              l_run *= ex2(m_run - tile_max);  // 0 on the first tile (m_run = -inf)
              m_run = tile_max;
            }
            const uint64_t nm2 = pack2(-m_run, -m_run);
            uint64_t sum2[2] = {0ull, 0ull};
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const uint64_t x = fma2(pack2(__uint_as_float(sv[2 * i]), __uint_as_float(sv[2 * i + 1])), sc2, nm2);
              float p0, p1;
              if (kFmaShare > 0 && (i & 3) >= 4 - kFmaShare) {
                ex2_fma_pair(x, p0, p1);  // x <= 8 here
              } else {
                float x0, x1;
                unpack2(x, x0, x1);
                p0 = ex2(x0);
                p1 = ex2(x1);
              }
              sum2[i & 1] = add2(sum2[i & 1], pack2(p0, p1));
            }
            float a0, a1, a2, a3;
            unpack2(sum2[0], a0, a1);
            unpack2(sum2[1], a2, a3);
            l_run += (a0 + a1) + (a2 + a3);
          }
        } else {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t sv[64];
            tmem_ld64_wait(t_acc + half * 64, sv);
            const float2* nl = reinterpret_cast<const float2*>(nlse_s + t * kQueries + half * 64);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float2 n2 = nl[i];  // the same address in every lane: a broadcast
              const uint64_t x =
                  fma2(pack2(__uint_as_float(sv[2 * i]), __uint_as_float(sv[2 * i + 1])), sc2, pack2(n2.x, n2.y));
              float p0, p1;
              if (kFmaShare > 0 && (i & 3) >= 4 - kFmaShare) {
                ex2_fma_pair(x, p0, p1);  // one pair in four on the fma pipe: the special-function unit is the bound
              } else {
                float x0, x1;
                unpack2(x, x0, x1);
                p0 = ex2(x0);
                p1 = ex2(x1);
              }
              acc[i & 1] = add2(acc[i & 1], pack2(p0, p1));  // padding queries: 2^-inf = 0 (2^-125 on the fma pipe)
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(b_sfree);
      }
      // the four groups' partial results of this own tile, merged by group 0 in group order
      const int row = quad * 32 + lane;
      if constexpr (kStats) {
        sh->part[it & 1][grp][row] = make_float2(m_run, l_run);
      } else {
        float a0, a1, a2, a3;
        unpack2(acc[0], a0, a1);
        unpack2(acc[1], a2, a3);
        sh->part[it & 1][grp][row] = make_float2((a0 + a1) + (a2 + a3), 0.f);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sh->merge_bar));
      // every consumer warp waits: no warp may arrive for the next own tile before this phase is complete
      if (!mbar_wait_bounded(smem_u32(&sh->merge_bar), it & 1, abort)) break;
      if (grp == 0) {
        const int j = tile * kKeys + row;
        if (j < L_k) {
          if constexpr (kStats) {
            float m = -INFINITY, l = 0.f;
#pragma unroll
            for (int gq = 0; gq < kGroups; ++gq) {
              const float2 p = sh->part[it & 1][gq][row];
              const float mn = fmaxf(m, p.x);
              l = (m == -INFINITY ? 0.f : l * exp2f(m - mn)) + (p.x == -INFINITY ? 0.f : p.y * exp2f(p.x - mn));
              m = mn;
            }
            ml_out[((int64_t)hk * gridDim.z + blockIdx.z) * L_k + j] = make_float2(m, l);
          } else {
            float sum = 0.f;
#pragma unroll
            for (int gq = 0; gq < kGroups; ++gq) sum += sh->part[it & 1][gq][row].x;
            mass[(int64_t)hk * L_k + j] = sum;
          }
        }
      }
    }
  }

  if (*abort) {
    // something never arrived: give copies and instructions still in flight time to land before the
    // shared and tensor memory of this CTA are handed back
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort && status) atomicOr(status, FC_DEV_TIMEOUT);
  if (warp == 0) tmem_dealloc(tmem, kRing * kQueries);
}

}  // namespace

namespace fc {

namespace {
template <int D, bool kStats>
int launch(fc_ctx* ctx, cudaStream_t st, const CUtensorMap& t_stream, const CUtensorMap& t_own, int H, int n_stream,
           int n_own, float scale_log2, const float* nlse, float2* ml, int n_slices, float* mass, uint32_t* status) {
  const int n_st = (n_stream + kQueries - 1) / kQueries, n_ot = (n_own + kKeys - 1) / kKeys;
  // at least 120 KiB, so that a second CTA (and its 512 columns) never joins the SM
  const size_t need = (2 + kRing) * (size_t)kKeys * D * 2 + sizeof(MassSmem) + (kStats ? 0 : (size_t)n_st * kQueries * 4) + 1024;
  const size_t smem = std::max<size_t>(need, 120 * 1024);
  if (smem > 227 * 1024) return FC_ERR_UNSUPPORTED;
  // one CTA per SM over all heads; every CTA stays inside one head.  The statistics launch has few own tiles per
  // head and slices the streamed range instead (every CTA one own tile).
  dim3 grid(kStats ? n_ot : std::max(1, std::min(n_ot, ctx->sm_count / H)), H, kStats ? n_slices : 1);
  FC_CUDA_CHECK(cudaFuncSetAttribute(score_mass_kernel<D, kStats>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  score_mass_kernel<D, kStats><<<grid, kThreads, smem, st>>>(t_stream, t_own, n_stream, n_own, scale_log2, nlse, ml, mass,
                                                             status);
  FC_LAUNCH_CHECK("score_mass_kernel");
  return FC_OK;
}
}  // namespace

int score_frame_slices(fc_ctx* ctx, int H, int L_q, int L_k) {
  // Slices of the key range in the statistics launch: with few query tiles per head the (head, query tile) pairs
  // alone do not fill the CTA slots evenly.  Cost model: waves of CTAs x (key tiles per slice + 3 tiles' worth of
  // set-up per CTA).
  const int n_qt = (L_q + kKeys - 1) / kKeys, n_kt = (L_k + kQueries - 1) / kQueries, slots = ctx->sm_count;
  int best = 1;
  int64_t best_cost = INT64_MAX;
  for (int sl = 1; sl <= kScoreFrameMaxSlices && sl <= n_kt; ++sl) {
    const int64_t ctas = (int64_t)n_qt * H * sl;
    const int64_t cost = ((ctas + slots - 1) / slots) * ((n_kt + sl - 1) / sl + 3);
    if (cost < best_cost) {
      best_cost = cost;
      best = sl;
    }
  }
  return best;
}

int score_frame_mass(fc_ctx* ctx, cudaStream_t st, int H, int d, int L_q, int L_k, float scale_log2, const void* Q,
                     int64_t q_hs, int64_t q_rs, const void* K, int64_t k_hs, int64_t k_rs, float2* ml_part, float* nlse,
                     float* mass, uint32_t* status) {
  if (L_q > kScoreFrameMaxQueries) return FC_ERR_UNSUPPORTED;
  CUtensorMap tq, tk;
  int rc;
  if ((rc = make_tmap(ctx, &tq, Q, d, L_q, H, q_rs, H > 1 ? q_hs : q_rs * L_q)) != FC_OK) return rc;
  if ((rc = make_tmap(ctx, &tk, K, d, L_k, H, k_rs, H > 1 ? k_hs : k_rs * L_k)) != FC_OK) return rc;
  const int n_slices = score_frame_slices(ctx, H, L_q, L_k);
  // (max, sum) of every query over the slices of the candidates, their merge, then the mass of every key
  if (d == 128) rc = launch<128, true>(ctx, st, tk, tq, H, L_k, L_q, scale_log2, nullptr, ml_part, n_slices, nullptr, status);
  else rc = launch<64, true>(ctx, st, tk, tq, H, L_k, L_q, scale_log2, nullptr, ml_part, n_slices, nullptr, status);
  if (rc != FC_OK) return rc;
  score_frame_lse_kernel<<<dim3((L_q + 255) / 256, H), 256, 0, st>>>(ml_part, n_slices, L_q, nlse);
  FC_LAUNCH_CHECK("score_frame_lse_kernel");
  if (d == 128) return launch<128, false>(ctx, st, tq, tk, H, L_q, L_k, scale_log2, nlse, nullptr, 1, mass, status);
  return launch<64, false>(ctx, st, tq, tk, H, L_q, L_k, scale_log2, nlse, nullptr, 1, mass, status);
}

}  // namespace fc
