// Chunk-causal attention on tcgen05 tensor cores, warp-specialised (bf16 in, fp32 accumulation).
//
// One persistent CTA per SM (384 threads, all 512 tensor-memory columns).  A work item is
// (active chunk, head, pair of 128-row query tiles A and B).  Items are ordered by the length of
// the chunk's visible prefix, longest first, and handed out through a device counter, so the
// last items to start are the shortest ones and the SMs finish together.  Roles:
//   warps 0-3  softmax of tile A     one query row per thread, online softmax in the exp2 domain
//   warps 4-7  softmax of tile B
//   warp  8    scheduler + TMA       takes the next item off the counter, publishes it to the
//                                    other warps through a 2-slot ring, then loads the Q pair and
//                                    streams K and V tiles into 2-stage rings (segment table: one tiled
//                                    load per 64-column block; per-head token map: every lane gathers four
//                                    rows at a time by index, tile::gather4, into the same swizzled tile)
//   warps 9,10 MMA issuers           one thread per query tile
//   warp  11   tail patcher          zeroes the rows of a V stage that lie past the end of a segment (with a token
//                                    map it also gathers the V rows, so that two warps share the copy instructions)
// Tensor memory: S_A [0,128) S_B [128,256) O_A [256,384) O_B [384,512).
// A key tile of 128 tokens is worked through as two halves of 64: S_x is two 64-column accumulators, each with
// its own "full" and "P ready" barriers, and P (bf16) of a half overwrites the first 32 columns of that half.
// The order of one MMA thread is S0(0) S1(0) | PV0(0) S0(1) PV1(0) S1(1) | PV0(1) S0(2) ..., so the S of the
// next key tile's first half is issued as soon as P of this tile's first half has been handed to the tensor pipe,
// while the softmax is still busy with the second half.  A softmax warp therefore normally finds its next half
// already computed instead of waiting for a round trip through the tensor pipe; what bounds it then is the
// special-function unit (2 tiles x 128 x 128 exponentials at 16 per clock = 2048 clocks per pair of tiles, the
// same as the tensor pipe's 2048).  With whole-tile S accumulators the chain S -> softmax -> PV -> S of one tile was the
// critical path (about 3800 clocks per pair of tiles, measured).  The price: an S instruction with N = 64 reads
// the whole 128-row Q operand from shared memory for half the columns and takes about 45 clocks instead of 32
// (measured), so the tensor pipe needs about 1240 clocks per tile instead of 1024.
// tcgen05.mma executes in issue order, so S_u(j+1) cannot overtake PV_u(j), which still reads P_u(j).
// The rescale is lazy: a row keeps its reference maximum until the true maximum exceeds it by more
// than 2^8, so P stays below 256 and O is rescaled only a few times per row; a softmax warp that has to rescale
// O_x first waits for the PV instructions issued so far (barrier pv_done: one phase per half).
// The softmax is written for issue slots: three-input max, two-wide fp32 fma / add, one bf16x2
// convert per pair.  Two softmax warps share a scheduler (the same lane quadrant of tiles A and B), and together
// they saturate the special-function unit (measured: 1115 clocks per half tile per warp when both run, 640 when
// one runs alone).  One column pair in four therefore takes its exponential on the fma pipe (range reduction and a
// cubic): 900 clocks per half tile in isolation; a larger share costs more fma-pipe time than it saves.
// As measured with clock probes, a softmax warp now spends about 75 % of its time in exponentials and 10 % waiting
// for S; the tensor pipe has work about 75 % of the time.
// Tails.  A segment's last key tile may be ragged: the TMA box still brings 128 physical rows, and the rows past the
// segment's end are whatever the K/V store holds there (another segment, or slots of the buffer that were never
// written).  Their logits are replaced by -inf before the row maximum and their P is exactly 0 (a ragged half takes
// every exponential on the special-function unit, and masked columns are forced to 0); the V rows themselves are
// overwritten with zeros in shared memory by warp 11 before the PV instructions of that tile are issued, so that not
// even a NaN or an infinity in such a row can reach an output (0 x inf would).
// Every mbarrier wait is bounded (see mbar_wait_bounded); tensor memory is always released.
#include <cmath>

#include "fc_attention.cuh"
#include "fc_tcgen05.cuh"
#include "fc_tcgen05_ld.cuh"

namespace {

using namespace fc::sm100;

constexpr int kBM = 128, kBN = 128;
constexpr int kHalf = kBN / 2;  // key columns per S accumulator
constexpr int kThreads = 384;  // 3 warpgroups: softmax A, softmax B, {copy warp, two MMA warps, the tail patcher}
constexpr int kStages = 2;  // the MMA issuer computes stage and phase with masks: keep at 2
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.f;  // log2 units
// Registers per thread after the split: softmax warpgroups / the warpgroup of the copy and MMA warps.
// The CTA owns 384 x 168 registers from launch (168 = what the launch bounds allow); setmaxnreg only moves
// registers inside that pool, and an increase that the pool cannot cover would wait forever.
constexpr int kRegsHi = 200, kRegsLo = 104;
static_assert(256 * kRegsHi + 128 * kRegsLo <= 384 * 168, "register split exceeds the CTA's pool");
static_assert(kRegsHi % 8 == 0 && kRegsLo % 8 == 0, "setmaxnreg takes multiples of 8");
// Of every four column pairs, how many take their exponential on the fma pipe instead of the special-function unit
// (measured: 0 -> 1115 clocks per half tile per warp, 1 -> 900, 2 -> 970, 4 -> 1410).
constexpr int kPolyOf4 = 1;

struct WsSmem {
  uint64_t q_full, q_empty;
  uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint64_t v_fixed[kStages];             // the tail patcher is done with the stage (one phase per tile, like v_full)
  uint64_t s_full[2][2], p_ready[2][2];  // [query tile][half of the key tile]
  uint64_t pv_done[2];                   // per query tile: one phase per PV half, in issue order
  uint64_t o_done[2];                    // per query tile: one phase per item, after its last PV
  uint64_t it_full[2], it_empty[2];
  int32_t it_slot[2];
  uint32_t tmem_base;
  uint32_t abort;
  int32_t n_act, total_items;
  int32_t act_chunk[FC_MAX_CHUNKS];     // active chunks, longest visible prefix first
  int32_t act_item_end[FC_MAX_CHUNKS];  // running item count over that list (all heads)
};

struct Item {
  int h, hk, c, row0, n_vis;
  bool b_valid;  // tile B has at least one row of the chunk (false for the ragged last item of a chunk)
};

// P = 2^(S * scale - m) for one row of a 64-column half tile, written as bf16 to tensor-memory columns
// [t_p, t_p + 32); returns the row sum.  kRagged: only the first n_valid columns are visible; the others get P = 0
// exactly and every exponential is taken on the special-function unit (2^-inf = 0 there, 2^-125 on the fma pipe).
template <bool kRagged>
__device__ __forceinline__ float exp_half(const uint32_t (&sv)[kHalf], float scale_log2, float m, uint32_t t_p,
                                          int n_valid) {
  const uint64_t sc2 = pack2(scale_log2, scale_log2), nm2 = pack2(-m, -m);
  uint64_t sum2[2] = {0ull, 0ull};
#pragma unroll
  for (int q2 = 0; q2 < kHalf / 32; ++q2) {
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint64_t x = fma2(pack2(__uint_as_float(sv[q2 * 32 + 2 * i]), __uint_as_float(sv[q2 * 32 + 2 * i + 1])),
                              sc2, nm2);
      float p0, p1;
      if (!kRagged && kPolyOf4 > 0 && (i & 3) >= 4 - kPolyOf4) {
        // the special-function unit is what bounds the softmax warps: a share of the pairs goes to the fma pipe
        ex2_fma_pair(x, p0, p1);
      } else {
        float x0, x1;
        unpack2(x, x0, x1);
        p0 = ex2(x0);
        p1 = ex2(x1);
      }
      if (kRagged) {
        if (q2 * 32 + 2 * i >= n_valid) p0 = 0.f;
        if (q2 * 32 + 2 * i + 1 >= n_valid) p1 = 0.f;
      }
      sum2[i & 1] = add2(sum2[i & 1], pack2(p0, p1));
      pk[i] = cvt_bf16x2(p0, p1);
    }
    tmem_st16(t_p + q2 * 16, pk);
  }
  float a, b, c, d;
  unpack2(sum2[0], a, b);
  unpack2(sum2[1], c, d);
  return (a + b) + (c + d);
}

// A wait by every lane of a warp (softmax and copy warps).  Measured alternatives: lane 0 polling with the
// others parked at a warp barrier, and polls separated by nanosleep; both were slower or no faster.
__device__ __forceinline__ void warp_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort) {
  mbar_wait_bounded(bar, parity, abort);
}

// kGather: the logical key/value tokens are reached through the per-head token map g.tok_index (tmap_k / tmap_v are
// then 2-D maps over all rows of all heads, box one row high) instead of the segment table.
template <int D, bool kGather>
__global__ void __launch_bounds__(kThreads, 1)
attention_ws_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ fc::AttnGeom g,
                    __nv_bfloat16* __restrict__ O, uint32_t* __restrict__ counter) {
  constexpr uint32_t kTileBytes = kBM * D * 2;
  constexpr int kAtoms = D / 64;
  constexpr uint32_t kAtomBytes = kBM * 128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t q_s = smem_u32(smem);                 // Q_A, Q_B
  const uint32_t k_s = q_s + 2 * kTileBytes;           // K ring
  const uint32_t v_s = k_s + kStages * kTileBytes;     // V ring
  WsSmem* sh = (WsSmem*)(smem + (2 + 2 * kStages) * kTileBytes);
  volatile uint32_t* abort = &sh->abort;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(smem_u32(&sh->q_full), 1);
    mbar_init(smem_u32(&sh->q_empty), 2);  // both MMA threads
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sh->k_full[s]), 1);
      mbar_init(smem_u32(&sh->k_empty[s]), 2);  // both MMA threads
      mbar_init(smem_u32(&sh->v_full[s]), 1);
      mbar_init(smem_u32(&sh->v_empty[s]), 3);  // both MMA threads and the tail patcher
      mbar_init(smem_u32(&sh->v_fixed[s]), 1);
    }
    for (int x = 0; x < 2; ++x) {
      for (int u = 0; u < 2; ++u) {
        mbar_init(smem_u32(&sh->s_full[x][u]), 1);
        mbar_init(smem_u32(&sh->p_ready[x][u]), 4);  // one arrival per softmax warp
      }
      mbar_init(smem_u32(&sh->pv_done[x]), 1);
      mbar_init(smem_u32(&sh->o_done[x]), 1);
      mbar_init(smem_u32(&sh->it_full[x]), 1);
      mbar_init(smem_u32(&sh->it_empty[x]), 11);  // the two MMA threads, the eight softmax warps, the tail patcher
      sh->it_slot[x] = -1;
    }
    mbar_fence_init();
    sh->abort = 0;
    tma_prefetch_desc(&tmap_q);
    tma_prefetch_desc(&tmap_k);
    tma_prefetch_desc(&tmap_v);
    // active chunks sorted by visible length, longest first (insertion sort, at most 64 entries)
    const int n_in = min(max(*g.n_active, 0), g.W);
    int n = 0;
    for (int a = 0; a < n_in; ++a) {
      const int c = g.active_ids[a];
      if (c < 0 || c >= g.W) {
        if (g.status) atomicOr(g.status, FC_DEV_BAD_INDEX);
        continue;
      }
      int p = n++;
      while (p > 0 && g.vis[sh->act_chunk[p - 1]] < g.vis[c]) {
        sh->act_chunk[p] = sh->act_chunk[p - 1];
        --p;
      }
      sh->act_chunk[p] = c;
    }
    int items = 0;
    for (int a = 0; a < n; ++a) {
      const int c = sh->act_chunk[a];
      items += g.H_q * ((g.q_row_off[c + 1] - g.q_row_off[c] + 2 * kBM - 1) / (2 * kBM));
      sh->act_item_end[a] = items;
    }
    sh->n_act = n;
    sh->total_items = items;
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&sh->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh->tmem_base;
  const int n_act = sh->n_act;
  const int total_items = sh->total_items;

  auto decode = [&](int item) {
    Item it;
    int a = 0;
    while (a + 1 < n_act && item >= sh->act_item_end[a]) ++a;
    const int start = a > 0 ? sh->act_item_end[a - 1] : 0;
    const int pairs = (sh->act_item_end[a] - start) / g.H_q;
    it.c = sh->act_chunk[a];
    it.h = (item - start) / pairs;
    it.row0 = g.q_row_off[it.c] + ((item - start) % pairs) * 2 * kBM;
    it.n_vis = g.vis[it.c];
    it.hk = it.h / g.group;
    it.b_valid = it.row0 + kBM < g.q_row_off[it.c + 1];
    return it;
  };
  // consumer side of the item ring; -1 once the list is exhausted or the CTA has given up
  auto next_item = [&](uint32_t n) {
    const int slot = n & 1;
    warp_wait(smem_u32(&sh->it_full[slot]), (n >> 1) & 1, abort);
    int item = sh->it_slot[slot];
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&sh->it_empty[slot]));
    if (*abort || item >= total_items) item = -1;
    return item;
  };

  auto count_tiles = [&](const Item& it) {
    int n = 0;
    for (int s = 0; s < g.n_seg; ++s) {
      const int seg_vis = min(g.seg_log[s + 1], it.n_vis) - g.seg_log[s];
      if (seg_vis <= 0) break;
      n += (seg_vis + kBN - 1) / kBN;
    }
    return n;
  };

  // Registers move from the third warpgroup, which only issues copies and MMAs, to the softmax
  // warpgroups, which hold a 128-column row of S per thread.
  if (warp >= 8) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsLo));
  if (warp == 8) {
    // ------------------------------------------------------------------ scheduler + TMA producer
    uint32_t kv = 0, it_n = 0;
    int next = 0;
    if (lane == 0) next = (int)atomicAdd(counter, 1u);
    while (true) {
      int item = __shfl_sync(0xffffffffu, next, 0);
      if (item >= total_items) item = -1;
      const int slot = it_n & 1;
      warp_wait(smem_u32(&sh->it_empty[slot]), ((it_n >> 1) & 1) ^ 1, abort);
      if (lane == 0) {
        sh->it_slot[slot] = item < 0 ? total_items : item;
        mbar_arrive(smem_u32(&sh->it_full[slot]));
      }
      if (item < 0 || *abort) break;
      if (lane == 0) next = (int)atomicAdd(counter, 1u);  // in flight while this item's tiles are loaded
      const Item it = decode(item);
      warp_wait(smem_u32(&sh->q_empty), (it_n & 1) ^ 1, abort);
      if (lane == 0) {
        mbar_expect_tx(smem_u32(&sh->q_full), 2 * kTileBytes);
        for (int t = 0; t < 2; ++t)
          for (int x = 0; x < kAtoms; ++x)
            tma_load_3d(q_s + t * kTileBytes + x * kAtomBytes, &tmap_q, smem_u32(&sh->q_full), x * 64,
                        it.row0 + t * kBM, it.h);
      }
      if constexpr (kGather) {
        // One logical segment [0, n_vis) whose token j of head hk lives in physical row tok[j].  Lane L brings rows
        // 4L .. 4L+3 of every tile; positions past the visible prefix repeat its last token (their logits are masked
        // and their V rows zeroed like any other tail).  A row index outside the store is reported and replaced by 0.
        const int32_t* tok = g.tok_index + (int64_t)it.hk * g.tok_hs;
        const int k_base = (int)(it.hk * (g.k_hs / g.k_rs));
        for (int j0 = 0; j0 < it.n_vis; j0 += kBN, ++kv) {
          const int st = kv % kStages, ph = (kv / kStages) & 1;
          int r[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            r[e] = __ldg(tok + min(j0 + 4 * lane + e, it.n_vis - 1));  // in flight during the wait for the stage
          }
          warp_wait(smem_u32(&sh->k_empty[st]), ph ^ 1, abort);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            if (r[e] < 0 || r[e] >= g.kv_rows) {
              if (g.status) atomicOr(g.status, FC_DEV_BAD_INDEX);
              r[e] = 0;
            }
          }
          if (lane == 0) mbar_expect_tx(smem_u32(&sh->k_full[st]), kTileBytes);
          __syncwarp();
          for (int x = 0; x < kAtoms; ++x)
            tma_gather4_2d(k_s + st * kTileBytes + x * kAtomBytes + lane * 512, &tmap_k, smem_u32(&sh->k_full[st]), x * 64,
                           k_base + r[0], k_base + r[1], k_base + r[2], k_base + r[3]);
          __syncwarp();  // (the V rows of the tile are gathered by warp 11: two warps issue the copies)
        }
      } else {
      for (int s = 0; s < g.n_seg; ++s) {
        const int seg_vis = min(g.seg_log[s + 1], it.n_vis) - g.seg_log[s];
        if (seg_vis <= 0) break;
        for (int j0 = 0; j0 < seg_vis; j0 += kBN, ++kv) {
          const int st = kv % kStages, ph = (kv / kStages) & 1, prow = g.seg_phys[s] + j0;
          warp_wait(smem_u32(&sh->k_empty[st]), ph ^ 1, abort);
          if (lane == 0) {
            mbar_expect_tx(smem_u32(&sh->k_full[st]), kTileBytes);
            for (int x = 0; x < kAtoms; ++x)
              tma_load_3d(k_s + st * kTileBytes + x * kAtomBytes, &tmap_k, smem_u32(&sh->k_full[st]), x * 64, prow,
                          it.hk);
          }
          warp_wait(smem_u32(&sh->v_empty[st]), ph ^ 1, abort);
          if (lane == 0) {
            mbar_expect_tx(smem_u32(&sh->v_full[st]), kTileBytes);
            for (int x = 0; x < kAtoms; ++x)
              tma_load_3d(v_s + st * kTileBytes + x * kAtomBytes, &tmap_v, smem_u32(&sh->v_full[st]), x * 64, prow,
                          it.hk);
          }
          __syncwarp();
        }
      }
      }
      ++it_n;
    }
  } else if (warp == 9 || warp == 10) {
    // ------------------------------------------------------------------ MMA issuers (one thread per query tile)
    // Lane 0 of warp 9 issues S_A and PV_A, lane 0 of warp 10 issues S_B and PV_B.  The tensor pipe takes
    // instructions in arrival order; the order that matters, S_u(j+1) after PV_u(j), is program order of one
    // thread.  While one thread sits in a wait or a commit the other keeps the pipe fed.
    if (lane == 0) {
    const int x = warp - 9;
    constexpr uint32_t kIdescQK = idesc_bf16_f32(kBM, kHalf, false, false);
    constexpr uint32_t kIdescPV = idesc_bf16_f32(kBM, D, false, true);
    // descriptors are built once; a k-step only moves the 14-bit address field (units of 16 bytes)
    const uint64_t dq = smem_desc_sw128(q_s + x * kTileBytes, 16, 1024), dk = smem_desc_sw128(k_s, 16, 1024),
                   dv = smem_desc_sw128(v_s, kAtomBytes, 1024);
    const uint32_t t_s = tmem + x * 128, t_o = tmem + 256 + x * 128;
    constexpr int kSteps = D / 16;
    uint64_t qa[kSteps], kb[kSteps], vb[4];  // operand descriptors of the next S group (Q_x fixed) and PV group
    uint32_t pa[4];                          // tensor-memory addresses of P for the next PV group
#pragma unroll
    for (int kk = 0; kk < kSteps; ++kk) qa[kk] = dq + (uint64_t)(((kk / 4) * kAtomBytes + (kk % 4) * 32) >> 4);
    pin(qa);
    // S_x[:, half u] = Q_x K[half u]^T; a key row is 128 bytes of each atom
    auto prep_s = [&](uint32_t st, int u) {
      const uint64_t b0 = dk + (uint64_t)((st * kTileBytes + u * (kHalf * 128)) >> 4);
#pragma unroll
      for (int kk = 0; kk < kSteps; ++kk) kb[kk] = b0 + (uint64_t)(((kk / 4) * kAtomBytes + (kk % 4) * 32) >> 4);
      pin(kb);
    };
    auto issue_s = [&](int u) { umma_ss_group<kSteps>(t_s + u * kHalf, qa, kb, kIdescQK); };
    // O_x (+)= P_x[:, half u] V[half u]
    auto prep_pv = [&](uint32_t st, int u) {
      const uint64_t b0 = dv + (uint64_t)((st * kTileBytes + u * (kHalf / 16) * 2048) >> 4);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        vb[kk] = b0 + (uint64_t)(kk * (2048 >> 4));
        pa[kk] = t_s + u * kHalf + kk * 8;
      }
      pin(vb);
      pin(pa);
    };
    auto issue_pv = [&](bool accumulate) { umma_ts_group(t_o, pa, vb, kIdescPV, accumulate); };
    // barrier addresses as plain registers: the issue loop should be little more than the MMAs themselves
    const uint32_t b_kfull = smem_u32(&sh->k_full[0]), b_kempty = smem_u32(&sh->k_empty[0]);
    const uint32_t b_vfull = smem_u32(&sh->v_full[0]), b_vempty = smem_u32(&sh->v_empty[0]);
    const uint32_t b_vfixed = smem_u32(&sh->v_fixed[0]);
    const uint32_t b_sfull = smem_u32(&sh->s_full[x][0]), b_pready = smem_u32(&sh->p_ready[x][0]);
    const uint32_t b_pvdone = smem_u32(&sh->pv_done[x]);
    // Barrier phases are counted per use: tile B sits out the items in which it has no rows (the last item of a
    // chunk whose length is not a multiple of 256), so its barriers see fewer phases than tile A's.
    uint32_t kv = 0, uses = 0;
    for (uint32_t it_n = 0;; ++it_n) {
      const int slot = it_n & 1;
      mbar_wait_bounded(smem_u32(&sh->it_full[slot]), (it_n >> 1) & 1, abort);
      const int item = sh->it_slot[slot];
      mbar_arrive(smem_u32(&sh->it_empty[slot]));
      if (*abort || item >= total_items) break;
      const Item it = decode(item);
      const int n_tiles = count_tiles(it);
      mbar_wait_bounded(smem_u32(&sh->q_full), it_n & 1, abort);
      tc_fence_after();
      if (x == 1 && !it.b_valid) {
        // Nothing to compute for tile B.  Its arrivals on the ring barriers are still due, one stage at a time
        // (waiting for the stage to be full keeps them in the right phase).
        for (int j = 0; j < n_tiles; ++j, ++kv) {
          const uint32_t st = kv & 1, ph = (kv >> 1) & 1;
          mbar_wait_bounded(b_kfull + 8 * st, ph, abort);
          mbar_arrive(b_kempty + 8 * st);
          mbar_wait_bounded(b_vfull + 8 * st, ph, abort);
          mbar_arrive(b_vempty + 8 * st);
        }
        mbar_arrive(smem_u32(&sh->q_empty));
        continue;
      }
      if (n_tiles > 0) {  // both halves of S for the first key tile
        const uint32_t st = kv & 1, ph = (kv >> 1) & 1;  // kStages == 2
        prep_s(st, 0);
        mbar_wait_bounded(b_kfull + 8 * st, ph, abort);
        tc_fence_after();
        issue_s(0);
        umma_commit(b_sfull);
        prep_s(st, 1);
        issue_s(1);
        umma_commit(b_sfull + 8);
        umma_commit(b_kempty + 8 * st);
      }
      // the walk over the segments, to know which tiles are ragged (their V stage is patched before PV)
      int seg = 0, seg_left = n_tiles > 0 ? min(g.seg_log[1], it.n_vis) - g.seg_log[0] : 0;
      for (int j = 0; j < n_tiles; ++j, ++kv, ++uses) {
        const uint32_t st = kv & 1, ph = (kv >> 1) & 1;
        const uint32_t st2 = st ^ 1, ph2 = ((kv + 1) >> 1) & 1;  // the next key tile's stage
        const bool more = j + 1 < n_tiles;
        const bool ragged = seg_left < kBN;
        seg_left -= kBN;
        if (seg_left <= 0 && more) {
          ++seg;
          seg_left = min(g.seg_log[seg + 1], it.n_vis) - g.seg_log[seg];
        }
        prep_pv(st, 0);
        if (more) prep_s(st2, 0);
        mbar_wait_bounded(b_vfull + 8 * st, ph, abort);
        if (ragged) mbar_wait_bounded(b_vfixed + 8 * st, ph, abort);
        mbar_wait_bounded(b_pready, uses & 1, abort);
        tc_fence_after();
        issue_pv(j > 0);
        umma_commit(b_pvdone);
        if (more) {
          mbar_wait_bounded(b_kfull + 8 * st2, ph2, abort);
          tc_fence_after();
          issue_s(0);
          umma_commit(b_sfull);
        }
        prep_pv(st, 1);
        if (more) prep_s(st2, 1);
        mbar_wait_bounded(b_pready + 8, uses & 1, abort);
        tc_fence_after();
        issue_pv(true);
        umma_commit(b_pvdone);
        umma_commit(b_vempty + 8 * st);
        if (more) {
          issue_s(1);
          umma_commit(b_sfull + 8);
          umma_commit(b_kempty + 8 * st2);
        }
      }
      umma_commit(smem_u32(&sh->q_empty));  // every read of this thread's Q tile has been issued
      umma_commit(smem_u32(&sh->o_done[x]));
    }
    }
  } else {
    // ------------------------------------------------------------------ tail patcher (warp 11)
    // Follows the V ring tile by tile.  On a ragged tile it writes zeros over the rows past the segment's end
    // (row r of a stage is 128 bytes at r * 128 in every 64-column block, whatever the swizzle does inside them),
    // makes the writes visible to the tensor cores' proxy and only then reports the stage as fixed.  It takes
    // part in the ring's flow control (v_empty), so the copy warp cannot refill a stage that is being patched and
    // the phases of v_fixed stay in step with those of v_full.
    uint8_t* v_tiles = smem + (2 + kStages) * kTileBytes;
    uint32_t kv = 0;
    for (uint32_t it_n = 0;; ++it_n) {
      const int item = next_item(it_n);
      if (item < 0) break;
      const Item it = decode(item);
      for (int s = 0; s < g.n_seg; ++s) {
        const int seg_vis = min(g.seg_log[s + 1], it.n_vis) - g.seg_log[s];
        if (seg_vis <= 0) break;
        for (int j0 = 0; j0 < seg_vis; j0 += kBN, ++kv) {
          const int st = kv % kStages, ph = (kv / kStages) & 1;
          const int cols_valid = min(kBN, seg_vis - j0);
          if constexpr (kGather) {
            // token map: this warp also brings the tile's V rows (lane L rows 4L .. 4L+3, as the copy warp does for K)
            const int32_t* tok = g.tok_index + (int64_t)it.hk * g.tok_hs;
            const int v_base = (int)(it.hk * (g.v_hs / g.v_rs));
            int r[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) r[e] = __ldg(tok + min(j0 + 4 * lane + e, it.n_vis - 1));
            warp_wait(smem_u32(&sh->v_empty[st]), ph ^ 1, abort);
#pragma unroll
            for (int e = 0; e < 4; ++e)
              if (r[e] < 0 || r[e] >= g.kv_rows) r[e] = 0;  // reported by the copy warp, which reads the same indices
            if (lane == 0) mbar_expect_tx(smem_u32(&sh->v_full[st]), kTileBytes);
            __syncwarp();
            for (int x = 0; x < kAtoms; ++x)
              tma_gather4_2d(v_s + st * kTileBytes + x * kAtomBytes + lane * 512, &tmap_v, smem_u32(&sh->v_full[st]),
                             x * 64, v_base + r[0], v_base + r[1], v_base + r[2], v_base + r[3]);
          }
          warp_wait(smem_u32(&sh->v_full[st]), ph, abort);
          if (cols_valid < kBN) {
            uint8_t* vt = v_tiles + st * kTileBytes;
            const int n16 = (kBN - cols_valid) * kAtoms * 8;  // 16-byte pieces to clear
            for (int i = lane; i < n16; i += 32) {
              const int r = cols_valid + i / (kAtoms * 8), x = (i / 8) % kAtoms, c = i % 8;
              *reinterpret_cast<uint4*>(vt + x * kAtomBytes + r * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          }
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(smem_u32(&sh->v_fixed[st]));
            mbar_arrive(smem_u32(&sh->v_empty[st]));
          }
        }
      }
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsHi));
    // ------------------------------------------------------------------ softmax + epilogue, tile x
    const int x = warp >> 2;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t t_s = tmem + lane_base + x * 128;
    const uint32_t t_o = tmem + lane_base + 256 + x * 128;
    const int r_in = (warp & 3) * 32 + lane;  // row inside the tile
    const float scale_log2 = g.scale * 1.4426950408889634f;
    // tiles seen; tiles, half tiles and items actually processed (barrier phases)
    uint32_t kv = 0, uses = 0, sub = 0, items = 0;
    // Before O_x is rescaled in place: every PV instruction that this warp has released so far (the first `sub`
    // phases of pv_done) has completed.  A parity wait tells two states apart, and there are only two here: the
    // half tile being worked on was computed after PV of two halves ago, so at least sub - 1 phases are over.
    auto wait_pv = [&]() {
      warp_wait(smem_u32(&sh->pv_done[x]), (sub - 1) & 1, abort);
      tc_fence_after();
    };
    auto rescale_o = [&](float alpha) {
#pragma unroll
      for (int q4 = 0; q4 < D / 32; ++q4) {
        uint32_t r[32];
        tmem_ld32_wait(t_o + q4 * 32, r);
#pragma unroll
        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
        tmem_st32(t_o + q4 * 32, r);
      }
    };
    for (uint32_t it_n = 0;; ++it_n) {
      const int item = next_item(it_n);
      if (item < 0) break;
      const Item it = decode(item);
      if (x == 1 && !it.b_valid) {  // no row of the chunk in tile B: its MMA thread sits the item out too
        kv += count_tiles(it);
        continue;
      }
      float m = -INFINITY, l = 0.f;
      int j = 0;
      for (int s = 0; s < g.n_seg; ++s) {
        const int seg_vis = min(g.seg_log[s + 1], it.n_vis) - g.seg_log[s];
        if (seg_vis <= 0) break;
        for (int j0 = 0; j0 < seg_vis; j0 += kBN, ++kv, ++j, ++uses) {
          const int cols_valid = min(kBN, seg_vis - j0);
#pragma unroll
          for (int u = 0; u < 2; ++u, ++sub) {
            const int mine_valid = min(max(cols_valid - u * kHalf, 0), kHalf);
            const uint32_t t_su = t_s + u * kHalf;  // S of this half; its first 32 columns take P
            const bool first = j == 0 && u == 0;
            warp_wait(smem_u32(&sh->s_full[x][u]), uses & 1, abort);
            tc_fence_after();
            uint32_t sv[kHalf];
            tmem_ld64_wait(t_su, sv);
            auto row_max = [&]() {
              float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
              for (int i = 0; i < kHalf; i += 8) {
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4)
                  mx[c4] = max3(mx[c4], __uint_as_float(sv[i + 2 * c4]), __uint_as_float(sv[i + 2 * c4 + 1]));
              }
              return fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2;  // scale > 0
            };
            if (mine_valid < kHalf) {
#pragma unroll
              for (int i = 0; i < kHalf; ++i)
                if (i >= mine_valid) sv[i] = 0xff800000u;  // -inf
            }
            const float tile_max = row_max();  // -inf if the half holds no visible token: then nothing moves
            // Lazy reference update: move only when the maximum grew by more than the threshold.  Either way the
            // exponent below is at most 2^kRescaleThreshold, which is what lets a share of the exponentials run on
            // the fma pipe (ex2_fma_pair has no upper clamp).
            const bool move = tile_max > m + kRescaleThreshold;  // always true on an item's first half (m = -inf)
            float alpha = 1.f;
            if (move) {
              alpha = ex2(m - tile_max);
              m = tile_max;
            }
            if (!first && __any_sync(0xffffffffu, move)) {
              wait_pv();
              rescale_o(alpha);
            }
            const float row_sum = mine_valid < kHalf ? exp_half<true>(sv, scale_log2, m, t_su, mine_valid)
                                                     : exp_half<false>(sv, scale_log2, m, t_su, kHalf);
            l = l * alpha + row_sum;
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->p_ready[x][u]));
          }
        }
      }
      // epilogue
      warp_wait(smem_u32(&sh->o_done[x]), items & 1, abort);
      ++items;
      tc_fence_after();
      const int row = it.row0 + x * kBM + r_in;
      const bool row_ok = row < g.q_row_off[it.c + 1] &&
                          fc::bounds_ok(row >= 0 && row < g.q_row_off[g.W] && it.h >= 0 && it.h < g.H_q, g.status);
      const float inv = l > 0.f ? 1.f / l : 0.f;
      __nv_bfloat16* out = O + (int64_t)it.h * g.o_hs + (int64_t)row * g.o_rs;
#pragma unroll
      for (int q4 = 0; q4 < D / 32; ++q4) {
        uint32_t r[32];
        if (j > 0) {
          tmem_ld32_wait(t_o + q4 * 32, r);
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = 0;
        }
        if (row_ok) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint4 w;
            uint32_t* wp = &w.x;
#pragma unroll
            for (int i = 0; i < 4; ++i)
              wp[i] = cvt_bf16x2(__uint_as_float(r[v * 8 + 2 * i]) * inv, __uint_as_float(r[v * 8 + 2 * i + 1]) * inv);
            *reinterpret_cast<uint4*>(out + q4 * 32 + v * 8) = w;
          }
        }
      }
      if (g.lse && row_ok)
        g.lse[(int64_t)it.h * g.lse_hs + row] = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
      tc_fence_before();  // O_x has been read before this warp's next p_ready arrival lets PV_x overwrite it
    }
  }

  if (*abort) {
    // something never arrived: give copies and instructions still in flight time to land before the
    // shared and tensor memory of this CTA are handed back
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort && g.status) atomicOr(g.status, FC_DEV_TIMEOUT);
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace

namespace fc {

int attention_ws_launch(fc_ctx* ctx, cudaStream_t st, const AttnGeom& g, const CUtensorMap& tq,
                        const CUtensorMap& tk, const CUtensorMap& tv, void* O, uint32_t* counter) {
  int max_items = 0;
  for (int c = 0; c < g.W; ++c) max_items += (g.q_row_off[c + 1] - g.q_row_off[c] + 2 * kBM - 1) / (2 * kBM);
  const int64_t items = (int64_t)max_items * g.H_q;
  if (items == 0) return FC_OK;
  FC_CUDA_CHECK(cudaMemsetAsync(counter, 0, sizeof(uint32_t), st));
  const int grid = (int)std::min<int64_t>(items, (int64_t)ctx->sm_count);
  // at least half of the shared memory, so that a second CTA (and its 512 columns) never joins the SM
  const size_t need = (2 + 2 * kStages) * (size_t)kBM * g.d * 2 + sizeof(WsSmem) + 1024;
  const size_t smem = std::max<size_t>(need, 120 * 1024);
  auto launch = [&](auto kernel) -> int {
    FC_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kernel<<<grid, kThreads, smem, st>>>(tq, tk, tv, g, (__nv_bfloat16*)O, counter);
    return FC_OK;
  };
  int rc;
  if (g.tok_index) rc = g.d == 128 ? launch(attention_ws_kernel<128, true>) : launch(attention_ws_kernel<64, true>);
  else rc = g.d == 128 ? launch(attention_ws_kernel<128, false>) : launch(attention_ws_kernel<64, false>);
  if (rc != FC_OK) return rc;
  FC_LAUNCH_CHECK("attention_ws_kernel");
  return FC_OK;
}

}  // namespace fc
