// fc_kv_score on tcgen05 tensor cores (bf16 keys and queries, one query head per key head, at most 64
// observation queries).
//
// The importance of a key is a column sum of a row-normalised matrix (Eq. 9), so the logits are needed
// twice: once to get every query's log-sum-exp over all candidates, once to add up exp(logit - lse) per key.
// Both passes recompute the logits on the tensor cores instead of storing them (50 x L_k fp32 per head would be
// five times the keys themselves), and each pass picks the orientation whose reduction stays inside a thread:
//   pass 1  S[query, key] = Q K^T   one query row per thread: running (max, sum) over the keys of the slice;
//                                   the same pass adds up the l2-normalised keys (the mean key of the
//                                   paper's efficiency appendix)
//           (every pass-2 CTA first merges its head's slice results: (max, sum) -> log-sum-exp per query, slice
//           sums -> mean normalised key)
//   pass 2  S[key, query] = K Q^T   one key row per thread: attention mass of the key; redundancy logit
//                                   a_j = meankey . khat_j - |khat_j|^2 / L_k and its per-tile softmax statistics.
//                                   The mean key rides along as two more query rows (its bf16 high and low
//                                   parts: the keys are bf16, so the products are exact and the sum carries 16
//                                   bits of the mean), and |k_j|^2 comes from pass 1: no key is read twice
//                                   by CUDA cores
// The finalize step (softmax of a, max-pool, lambda-mix) is the one the CUDA-core path uses.
//
// A CTA owns one (head, slice of key tiles).  Pass 1 (640 threads): two warpgroups read the logits from tensor
// memory and two read the key tile from shared memory (norms, column sums), each pair taking alternate tiles; one
// warp streams key tiles through a 4-stage TMA ring and issues the MMAs into a 2-deep tensor-memory ring (one
// accumulator per logit warpgroup).  Pass 2 (288 threads): no key-vector work, two logit warpgroups on alternate
// tiles.  The second pass walks heads, slices and tiles in the reverse of the first pass's order, so it starts on
// what the first pass left in L2 (all of it while the candidates of all heads fit there: a head is a few MB).
// Sums are fixed-order: results are bit-reproducible from run to run.  Every mbarrier wait is bounded.
#include <cmath>

#include "fc_attention.cuh"
#include "fc_score.cuh"
#include "fc_tcgen05.cuh"
#include "fc_tcgen05_ld.cuh"

namespace {

using namespace fc::sm100;

constexpr int kKeys = 128;     // keys per tile
constexpr int kRing = 4;       // key tiles in flight
// pass 1: warps 0-3 and 4-7 logits, warps 8-11 and 12-15 key vectors (each pair of warpgroups takes alternate
//         tiles: one warp per scheduler doing either job alone is bound by the latency of its own instruction
//         stream), warp 16 copies and MMAs, warps 17-19 idle (whole warpgroups only)
// pass 2: warps 0-3 and 4-7 logits (alternate tiles), warp 8 copies and MMAs
template <int PASS>
constexpr int kThreadsOf = PASS == 1 ? 640 : 288;
template <int PASS>
constexpr int kCopyWarp = PASS == 1 ? 16 : 8;
constexpr int kNQ = fc::kScoreTcMaxQueries;  // queries of pass 2 (MMA N), zero-padded

struct TcSmem {
  uint64_t q_full, q_patched, k_full[kRing], k_free[kRing], s_full[2], s_free[2];
  uint32_t tmem_base, abort;
  float inv_s[2][kKeys];   // 1 / |k| of the current tile's keys, per key-vector warpgroup (= tile parity)
  float2 ml_s[kNQ];        // pass 1: (max, sum) of the second logit warpgroup, merged by the first
  alignas(8) float lse_s[kNQ];  // pass 2: minus the log2-domain log-sum-exp per query (-inf for padding queries)
  float colsum_s[2][16][128];  // pass 1: per warpgroup and row group, column sums at the end of the slice
};

// 16-byte chunk `c` of key row `r` inside a 128-byte-swizzled tile of 64-element column blocks
template <int D>
__device__ __forceinline__ uint4 lds_key_chunk(const uint8_t* tile, int r, int c) {
  const int x = c >> 3, cc = c & 7;
  return *reinterpret_cast<const uint4*>(tile + x * (kKeys * 128) + r * 128 + ((cc ^ (r & 7)) << 4));
}

__device__ __forceinline__ void named_barrier_128(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }

// PASS 1: ml_part [H, n_slices, kNQ] (max, sum) in the log2 domain; colsum_part [H, n_slices, D]
// PASS 2: imp / a / a_partial as in the CUDA-core path
template <int D, int PASS>
__global__ void __launch_bounds__(kThreadsOf<PASS>, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                const fc::ScoreTcArgs g) {
  constexpr uint32_t kTileBytes = kKeys * D * 2;
  constexpr int kAtoms = D / 64;
  constexpr uint32_t kAtomBytes = kKeys * 128;
  constexpr int kCols = PASS == 1 ? kKeys : kNQ;  // tensor-memory columns of one logit buffer
  constexpr int kChunks = D / 8;                  // 16-byte chunks per key row
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* q_tile = smem;
  uint8_t* k_tiles = smem + kTileBytes;
  TcSmem* sh = (TcSmem*)(smem + (1 + kRing) * kTileBytes);
  volatile uint32_t* abort = &sh->abort;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Pass 2 walks heads, slices and tiles in the reverse of pass 1's order: what pass 1 read last is still in L2.
  const int hk = PASS == 1 ? blockIdx.y : gridDim.y - 1 - blockIdx.y;
  const int slice = PASS == 1 ? blockIdx.x : gridDim.x - 1 - blockIdx.x;
  const int t0 = slice * g.tiles_per_slice, t1 = min(g.n_tiles, t0 + g.tiles_per_slice), n = t1 - t0;
  // i-th tile of this CTA
  auto tile_of = [&](int i) { return PASS == 1 ? t0 + i : t1 - 1 - i; };

  if (tid == 0) {
    mbar_init(smem_u32(&sh->q_full), 1);
    mbar_init(smem_u32(&sh->q_patched), 128);
    for (int s = 0; s < kRing; ++s) {
      mbar_init(smem_u32(&sh->k_full[s]), 1);
      mbar_init(smem_u32(&sh->k_free[s]), PASS == 1 ? 5 : 1);  // the MMA's commit and, in pass 1, warps 4-7
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&sh->s_full[b]), 1);
      mbar_init(smem_u32(&sh->s_free[b]), 4);  // warps 0-3
    }
    mbar_fence_init();
    sh->abort = 0;
    tma_prefetch_desc(&tmap_q);
    tma_prefetch_desc(&tmap_k);
  }
  // Both passes let their successor (pass 2, the finalize kernel) be scheduled under their tail.
  fc::pdl_launch_dependents();
  if (warp == 0) {
    tmem_alloc(smem_u32(&sh->tmem_base), 2 * kCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // Pass 2 is such a successor itself.  Its copy warp touches nothing that pass 1 writes (keys and queries are the
  // call's inputs), so it starts filling the key ring at once, under pass 1's tail; every other warp waits here for
  // pass 1's results to be complete and visible.
  if (PASS == 2 && warp != kCopyWarp<PASS>) fc::pdl_wait();
  if (PASS == 2 && tid < kNQ) {
    // log-sum-exp of query `tid` over the whole head: pass 1's per-slice (max, sum) pairs, merged in slice order
    // (loaded eight at a time: one dependent round trip per slice would cost microseconds before the first tile)
    float lse = INFINITY;  // padding queries: exp2(anything - inf) = 0
    if (tid < g.L_q) {
      float m = -INFINITY, l = 0.f;
      for (int s0 = 0; s0 < g.n_slices; s0 += 8) {
        float2 p[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
          p[k] = s0 + k < g.n_slices ? g.ml_part[((int64_t)hk * g.n_slices + s0 + k) * kNQ + tid] : make_float2(-INFINITY, 0.f);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          if (s0 + k >= g.n_slices) break;
          const float mn = fmaxf(m, p[k].x);
          l = (m == -INFINITY ? 0.f : l * exp2f(m - mn)) + (p[k].x == -INFINITY ? 0.f : p[k].y * exp2f(p[k].x - mn));
          m = mn;
        }
      }
      lse = m + log2f(l);
    }
    sh->lse_s[tid] = -lse;
  }
  const uint32_t tmem = sh->tmem_base;

  if (warp == kCopyWarp<PASS>) {
    // ---------------------------------------------------------------- copies and MMAs (one thread)
    if (lane == 0 && n > 0) {
      auto load_k = [&](int i) {  // i-th tile of the CTA into stage i % kRing
        const int st = i % kRing;
        const uint32_t bar = smem_u32(&sh->k_full[st]);
        mbar_expect_tx(bar, kTileBytes);
        for (int x = 0; x < kAtoms; ++x)
          tma_load_3d(smem_u32(k_tiles + st * kTileBytes + x * kAtomBytes), &tmap_k, bar, x * 64, tile_of(i) * kKeys, hk);
      };
      // The query box is 64 rows high (at most 62 queries).  Pass 1 puts the queries into rows 0-63 AND rows 64-127
      // of its A operand: the two logit warpgroups, which take alternate tiles, then read the same logits from
      // different lane quadrants, i.e. with warps that sit on different schedulers (warps 0, 1 and warps 6, 7).
      // With one copy, warps 0, 1 and 4, 5 did all the exponentials on two of the four schedulers.
      mbar_expect_tx(smem_u32(&sh->q_full), PASS == 1 ? kTileBytes : kTileBytes / 2);
      for (int x = 0; x < kAtoms; ++x)
        for (int rep = 0; rep < (PASS == 1 ? 2 : 1); ++rep)
          tma_load_3d(smem_u32(q_tile + x * kAtomBytes + rep * 64 * 128), &tmap_q, smem_u32(&sh->q_full), x * 64, 0, hk);
      for (int i = 0; i < min(n, kRing - 1); ++i) load_k(i);
      mbar_wait_bounded(smem_u32(&sh->q_full), 0, abort);
      if (PASS == 2) mbar_wait_bounded(smem_u32(&sh->q_patched), 0, abort);
      const uint64_t dq = smem_desc_sw128(smem_u32(q_tile), 16, 1024);
      constexpr uint32_t kIdesc = PASS == 1 ? idesc_bf16_f32(128, kKeys, false, false) : idesc_bf16_f32(kKeys, kNQ, false, false);
      for (int i = 0; i < n; ++i) {
        const int st = i % kRing, b = i & 1;
        mbar_wait_bounded(smem_u32(&sh->k_full[st]), (i / kRing) & 1, abort);
        mbar_wait_bounded(smem_u32(&sh->s_free[b]), ((i >> 1) & 1) ^ 1, abort);
        tc_fence_after();
        const uint64_t dk = smem_desc_sw128(smem_u32(k_tiles + st * kTileBytes), 16, 1024);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint64_t off = ((kk / 4) * kAtomBytes + (kk % 4) * 32) >> 4;
          if (PASS == 1) umma_ss(tmem + b * kCols, dq + off, dk + off, kIdesc, kk > 0);  // S[query, key]
          else umma_ss(tmem + b * kCols, dk + off, dq + off, kIdesc, kk > 0);            // S[key, query]
        }
        umma_commit(smem_u32(&sh->s_full[b]));
        umma_commit(smem_u32(&sh->k_free[st]));
        if (i + kRing - 1 < n) {  // refill the stage tile i-1 has left
          if (i >= 1) mbar_wait_bounded(smem_u32(&sh->k_free[(i - 1) % kRing]), ((i - 1) / kRing) & 1, abort);
          load_k(i + kRing - 1);
        }
      }
    }
  } else if (warp < 8) {
    // ---------------------------------------------------------------- logits out of tensor memory
    // (pass 2 has no key-vector work, so warps 4-7 are a second logit warpgroup: the two take alternate tiles,
    // each the tensor-memory buffer of its own parity)
    const uint32_t t_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    if (PASS == 1) {
      const int grp = warp >> 2;  // this warpgroup takes the tiles of its parity and the accumulator of that parity
      const int q = (tid & 127) - grp * 64;  // query row: group 0 reads rows 0-63 of the accumulator, group 1 rows 64-127
      const bool row_ok = q >= 0 && q < g.L_q;
      const int q_warp = (warp & 3) * 32 - grp * 64;  // first query of this warp's lane quadrant
      const bool warp_ok = q_warp >= 0 && q_warp < g.L_q;
      float m = -INFINITY, l = 0.f;
      for (int i = grp; i < n; i += 2) {
        const int b = grp;
        mbar_wait_bounded(smem_u32(&sh->s_full[b]), (i >> 1) & 1, abort);
        tc_fence_after();
        const int cols_valid = min(kKeys, g.L_k - tile_of(i) * kKeys);
        // 64 columns at a time (a 128-column row per thread does not fit the registers of a 640-thread CTA)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t sv[64];
          if (warp_ok) tmem_ld64_wait(t_lane + b * kCols + half * 64, sv);
          if (half == 1) {  // the accumulator can take this warpgroup's next tile
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->s_free[b]));
          }
          if (!warp_ok) continue;
          if (cols_valid < half * 64 + 64) {
#pragma unroll
            for (int c = 0; c < 64; ++c)
              if (half * 64 + c >= cols_valid) sv[c] = 0xff800000u;  // -inf
          }
          float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < 64; c += 8) {
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4)
              mx[c4] = max3(mx[c4], __uint_as_float(sv[c + 2 * c4]), __uint_as_float(sv[c + 2 * c4 + 1]));
          }
          const float tile_max = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * g.scale_log2;  // scale > 0
          if (tile_max > m) {
            l *= ex2(m - tile_max);  // 0 on the first tile
            m = tile_max;
          }
          const uint64_t sc2 = pack2(g.scale_log2, g.scale_log2), nm2 = pack2(-m, -m);
          uint64_t sum2[2] = {0ull, 0ull};
#pragma unroll
          for (int c = 0; c < 64; c += 2) {
            const uint64_t x = fma2(pack2(__uint_as_float(sv[c]), __uint_as_float(sv[c + 1])), sc2, nm2);
            float x0, x1;
            unpack2(x, x0, x1);
            sum2[(c >> 1) & 1] = add2(sum2[(c >> 1) & 1], pack2(ex2(x0), ex2(x1)));
          }
          float a0, a1, a2, a3;
          unpack2(sum2[0], a0, a1);
          unpack2(sum2[1], a2, a3);
          l += (a0 + a1) + (a2 + a3);
        }
      }
      // the two warpgroups' results of the slice, merged in group order
      if (grp == 1 && q >= 0 && q < kNQ) sh->ml_s[q] = make_float2(m, l);
      asm volatile("bar.sync 4, 256;" ::: "memory");
      if (grp == 0 && row_ok) {
        const float2 p = sh->ml_s[q];
        const float mn = fmaxf(m, p.x);
        const float lm = (m == -INFINITY ? 0.f : l * exp2f(m - mn)) + (p.x == -INFINITY ? 0.f : p.y * exp2f(p.x - mn));
        g.ml_part[((int64_t)hk * g.n_slices + slice) * kNQ + q] = make_float2(mn, lm);
      }
    } else {
      // The mean key joins the queries as rows kNQ-2 (bf16 high part) and kNQ-1 (low part) of the Q tile, which
      // the copy zero-filled: generic-proxy writes, made visible to the tensor cores by the proxy fence.
      const int wg = warp >> 2, row = tid & 127;
      asm volatile("bar.sync 5, 256;" ::: "memory");  // lse_s, written by warps 0 and 1 above, is read by all eight
      if (wg == 0) mbar_wait_bounded(smem_u32(&sh->q_full), 0, abort);
      if (tid < D) {
        float mk = 0.f;  // mean normalised key: pass 1's per-slice column sums, added in slice order
        for (int s0 = 0; s0 < g.n_slices; s0 += 8) {
          float v[8];
#pragma unroll
          for (int k = 0; k < 8; ++k)
            v[k] = s0 + k < g.n_slices ? g.colsum_part[((int64_t)hk * g.n_slices + s0 + k) * D + tid] : 0.f;
#pragma unroll
          for (int k = 0; k < 8; ++k)
            if (s0 + k < g.n_slices) mk += v[k];
        }
        mk /= (float)g.L_k;
        const __nv_bfloat16 hi = __float2bfloat16_rn(mk), lo = __float2bfloat16_rn(mk - __bfloat162float(hi));
        const int c = tid >> 3, x = c >> 3, cc = c & 7, e = tid & 7;
#pragma unroll
        for (int part = 0; part < 2; ++part) {
          const int r = kNQ - 2 + part;
          *reinterpret_cast<__nv_bfloat16*>(q_tile + x * kAtomBytes + r * 128 + ((cc ^ (r & 7)) << 4) + e * 2) = part ? lo : hi;
        }
      }
      if (wg == 0) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(smem_u32(&sh->q_patched));
      }
      const float inv_nq = 1.f / (float)g.L_q, inv_lk = 1.f / (float)g.L_k;
      const uint64_t sc2 = pack2(g.scale_log2, g.scale_log2);
      for (int i = wg; i < n; i += 2) {
        const int b = i & 1;
        const int tile_id = tile_of(i), j = tile_id * kKeys + row;  // this thread's key
        const bool valid = j < g.L_k && fc::bounds_ok(j >= 0 && hk >= 0 && hk < g.H && tile_id < g.n_tiles, g.status);
        const int64_t o = (int64_t)hk * g.L_k + j;
        const float n2 = valid && g.accum_phase != 1 ? g.norm2[o] : 0.f;  // in flight while the logits arrive
        mbar_wait_bounded(smem_u32(&sh->s_full[b]), (i >> 1) & 1, abort);
        tc_fence_after();
        uint32_t sv[kNQ];
        tmem_ld64_wait(t_lane + b * kCols, sv);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh->s_free[b]));
        // exp2(s * scale - lse) two queries at a time; lse_s holds -lse, and -inf for the padding queries (-> 0)
        uint64_t ms2[2] = {0ull, 0ull};
#pragma unroll
        for (int q = 0; q < kNQ - 2; q += 2) {
          const uint64_t nl = *reinterpret_cast<const uint64_t*>(&sh->lse_s[q]);
          float x0, x1;
          unpack2(fma2(pack2(__uint_as_float(sv[q]), __uint_as_float(sv[q + 1])), sc2, nl), x0, x1);
          ms2[(q >> 1) & 1] = add2(ms2[(q >> 1) & 1], pack2(ex2(x0), ex2(x1)));
        }
        float m0, m1, m2, m3;
        unpack2(ms2[0], m0, m1);
        unpack2(ms2[1], m2, m3);
        const float mass = ((m0 + m1) + (m2 + m3)) * inv_nq;
        if (valid) {
          if (g.accum_phase == 1) {
            g.imp_accum[o] += mass;
          } else if (g.accum_phase == 2) {
            const float t = g.imp_accum[o] + mass;
            g.imp_accum[o] = t;
            g.imp_out[o] = t / (float)g.n_steps;
          } else {
            g.imp_out[o] = mass;
          }
        }
        if (g.accum_phase == 1) continue;
        float a = -INFINITY;
        if (valid) {
          const float dot = __uint_as_float(sv[kNQ - 2]) + __uint_as_float(sv[kNQ - 1]);
          const float inv = 1.f / fmaxf(sqrtf(n2), 1e-12f);
          a = dot * inv - (n2 * inv * inv) * inv_lk;
          g.a_out[o] = a;
        }
        // softmax statistics (max, sum of exp) of a over this warp's 32 keys, fixed order
        float m = a;
#pragma unroll
        for (int w = 16; w > 0; w >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, w));
        float l = valid ? expf(a - m) : 0.f;
#pragma unroll
        for (int w = 16; w > 0; w >>= 1) l += __shfl_xor_sync(0xffffffffu, l, w);
        if (lane == 0) g.a_partial[((int64_t)hk * g.n_tiles + tile_id) * 4 + (warp & 3)] = make_float2(m, l);
      }
    }
  } else if (PASS == 1 && warp < 16) {
    // ---------------------------------------------------------------- key vectors out of shared memory
    const int vg = (tid - 256) >> 7;  // warpgroup 0 or 1: the tiles of its parity
    const int u = (tid - 256) & 127;  // 0..127
    {
      // column sums of the normalised keys: this thread owns 16-byte chunk `c` of the rows r = rg (mod kGroups)
      constexpr int kGroups = 128 / kChunks;  // 8 for d = 128, 16 for d = 64
      const int c = u % kChunks, rg = u / kChunks;
      uint64_t acc2[4] = {0ull, 0ull, 0ull, 0ull};  // columns (2e, 2e + 1) of this thread's chunk
      for (int i = vg; i < n; i += 2) {
        const int st = i % kRing;
        mbar_wait_bounded(smem_u32(&sh->k_full[st]), (i / kRing) & 1, abort);
        const uint8_t* tile = k_tiles + st * kTileBytes;
        uint64_t n4[4] = {0ull, 0ull, 0ull, 0ull};  // two-wide fp32: (low element, high element) of each 32-bit word
#pragma unroll
        for (int cc = 0; cc < kChunks; ++cc) {
          const uint4 w = lds_key_chunk<D>(tile, u, cc);
          const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const uint64_t p2 = pack2(fc::bf16_lo(ww[e]), fc::bf16_hi(ww[e]));
            n4[e] = fma2(p2, p2, n4[e]);
          }
        }
        float n2;
        {
          float a0, a1, b0, b1, c0, c1, d0, d1;
          unpack2(n4[0], a0, a1);
          unpack2(n4[1], b0, b1);
          unpack2(n4[2], c0, c1);
          unpack2(n4[3], d0, d1);
          n2 = ((a0 + a1) + (b0 + b1)) + ((c0 + c1) + (d0 + d1));
        }
        const int j = tile_of(i) * kKeys + u;
        if (j < g.L_k) g.norm2[(int64_t)hk * g.L_k + j] = n2;  // pass 2 takes |k|^2 from here
        // rows past the end of the cache are zero-filled: 0 * (1 / 1e-12) = 0, they add nothing
        sh->inv_s[vg][u] = 1.f / fmaxf(sqrtf(n2), 1e-12f);
        named_barrier_128(1 + vg);
        for (int r = rg; r < kKeys; r += kGroups) {
          const uint4 w = lds_key_chunk<D>(tile, r, c);
          const float inv = sh->inv_s[vg][r];
          const uint64_t inv2 = pack2(inv, inv);
          const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) acc2[e] = fma2(pack2(fc::bf16_lo(ww[e]), fc::bf16_hi(ww[e])), inv2, acc2[e]);
        }
        named_barrier_128(1 + vg);  // inv_s[vg] is rewritten for this warpgroup's next tile
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh->k_free[st]));
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float lo, hi;
        unpack2(acc2[e], lo, hi);
        sh->colsum_s[vg][rg][c * 8 + 2 * e] = lo;
        sh->colsum_s[vg][rg][c * 8 + 2 * e + 1] = hi;
      }
      asm volatile("bar.sync 3, 256;" ::: "memory");  // both key-vector warpgroups
      if (vg == 0 && u < D) {
        float t = 0.f;
        for (int v = 0; v < 2; ++v)
          for (int r = 0; r < kGroups; ++r) t += sh->colsum_s[v][r][u];
        g.colsum_part[((int64_t)hk * g.n_slices + slice) * D + u] = t;
      }
    }
  }

  if (*abort) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let copies and MMAs in flight land before teardown
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort && g.status) atomicOr(g.status, FC_DEV_TIMEOUT);
  if (warp == 0) tmem_dealloc(tmem, 2 * kCols);
}

}  // namespace

namespace fc {

int score_tc_run(fc_ctx* ctx, cudaStream_t st, ScoreTcArgs g, int d, int64_t q_hs, int64_t q_rs, int64_t k_hs,
                 int64_t k_rs, const void* Q, const void* K) {
  CUtensorMap tq, tk;
  int rc;
  if ((rc = make_tmap(ctx, &tq, Q, d, g.L_q, g.H, q_rs, g.H > 1 ? q_hs : q_rs * g.L_q, 64)) != FC_OK) return rc;
  if ((rc = make_tmap(ctx, &tk, K, d, g.L_k, g.H, k_rs, g.H > 1 ? k_hs : k_rs * g.L_k)) != FC_OK) return rc;
  // slices: one CTA per SM over all heads (a single wave), at most kScoreTcMaxSlices per head
  const int want = std::max(1, ctx->sm_count / g.H);
  g.n_slices = std::min(std::min(want, kScoreTcMaxSlices), g.n_tiles);
  g.tiles_per_slice = (g.n_tiles + g.n_slices - 1) / g.n_slices;
  g.n_slices = (g.n_tiles + g.tiles_per_slice - 1) / g.tiles_per_slice;  // no empty slice
  const size_t smem = (size_t)(1 + kRing) * kKeys * d * 2 + sizeof(TcSmem) + 1024;
  const dim3 grid(g.n_slices, g.H);
  auto launch = [&](auto kernel, int threads, bool dependent) -> int {
    FC_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    if (dependent) {
      FC_CUDA_CHECK(launch_pdl(kernel, grid, dim3(threads), smem, st, tq, tk, g));
    } else {
      kernel<<<grid, threads, smem, st>>>(tq, tk, g);
      FC_LAUNCH_CHECK("score_tc_kernel");
    }
    return FC_OK;
  };
  if ((rc = d == 128 ? launch(score_tc_kernel<128, 1>, kThreadsOf<1>, false)
                     : launch(score_tc_kernel<64, 1>, kThreadsOf<1>, false)) != FC_OK)
    return rc;
  return d == 128 ? launch(score_tc_kernel<128, 2>, kThreadsOf<2>, true) : launch(score_tc_kernel<64, 2>, kThreadsOf<2>, true);
}

}  // namespace fc
