// fc_kv_select_compact: per-head top-B of the selection score (text after Eq. 12) and the
// retention of the selected K/V rows (Sec. 3.3).
//
// Selection: one cluster of up to four 1024-thread blocks per head, each holding its share of the head's keys.
// Scores become order-preserving 32-bit keys (NaN ranks as -inf, -0 as +0) held in shared memory when they fit; an
// 11-bit-digit radix select over the bits in which the head's keys differ (at most 3 passes, one cluster barrier
// each) finds the key T of the B-th largest score and how many keys exceed it; one ordered
// compaction then keeps every key above T plus the lowest-index keys equal to T, so the kept
// set is exactly the first B elements of the total order (score descending, index ascending),
// written in ascending index order (by warps, 32 neighbouring entries at a time, positions from ballots).  Integer
// work only: bit-exact.
//
// Compaction: a separate streaming kernel moves whole rows with 16-byte accesses, several
// independent loads in flight per thread; rows that were dropped are never read.  It is launched as a programmatic
// dependent of the selection: its blocks take their places on the SMs while the selection still runs and start
// copying the moment it has ended.
#include <algorithm>
#include <cstdint>

#include <cooperative_groups.h>

#include "fc_common.cuh"

namespace {

constexpr int kSelThreads = 1024;

__device__ __forceinline__ uint32_t score_key(float s, bool& is_nan) {
  uint32_t u = __float_as_uint(s);
  is_nan = (u & 0x7fffffffu) > 0x7f800000u;
  if (is_nan) u = 0xff800000u;              // -inf
  if ((u << 1) == 0) u = 0;                 // -0 -> +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // larger float <=> larger key
}

// One cluster of CTAs per head (1, 2 or 4 of them: as many as keep the whole grid within one wave); CTA r of the
// cluster owns the contiguous index range [r * chunk, (r + 1) * chunk) of the head.  The CTAs exchange their partial
// results (minimum / maximum, digit histograms, counts of kept keys) by storing them into each other's shared
// memory before a cluster barrier.
constexpr int kDigitBits = 11, kBins = 1 << kDigitBits;  // at most three passes over 32 bits
constexpr int kMaxCluster = 4;  // measured: a cluster of 8 is slower (16.6 us against 13.2 on 12 heads x 20400 keys)

struct SelShared {
  uint32_t hist[2][kBins];  // this CTA's histogram of the current digit; two copies (even / odd warps) to spread the atomics
  // Every CTA's histogram of the current digit, written into this CTA's shared memory by its owner (rank = second
  // index) before the pass's cluster barrier and read locally after it.  Passes alternate between the two buffers, so
  // one cluster barrier per pass is enough.
  uint32_t hist_all[2][kMaxCluster][kBins];
  uint32_t red_min[kSelThreads / 32], red_max[kSelThreads / 32];
  uint32_t warp_gt[kSelThreads / 32], warp_eq[kSelThreads / 32], scan_w[kSelThreads / 32];
  uint32_t in_min[kMaxCluster], in_max[kMaxCluster];  // written by every CTA of the cluster: its smallest / largest key
  uint32_t in_gt[kMaxCluster], in_eq[kMaxCluster];    // written by the CTAs that own lower indices: their kept counts
  uint32_t prefix, remaining;
};

// Dynamic shared memory: SelShared, then (kSmemKeys) this CTA's keys.  No CTA reads another's shared memory: what the
// others need is stored into THEIR shared memory before a cluster barrier, so the cost of the exchange is a store that
// nobody waits for instead of a load across the cluster, and no CTA has to outlive its last barrier.
template <bool kSmemKeys>
__global__ void __launch_bounds__(kSelThreads)
select_topb_kernel(const float* __restrict__ score, int L_k, int B, int chunk, int protect_from,
                   int32_t* __restrict__ kept_idx, int32_t* __restrict__ n_kept, uint32_t* __restrict__ status) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) uint8_t sel_smem[];
  SelShared& sh = *reinterpret_cast<SelShared*>(sel_smem);
  uint32_t* smem_keys = reinterpret_cast<uint32_t*>(sel_smem + sizeof(SelShared));
  const int cs = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank(), h = blockIdx.x / cs, tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int begin = min(rank * chunk, L_k), n = min(begin + chunk, L_k) - begin;  // this CTA's keys: begin + [0, n)
  const float* s = score + (size_t)h * L_k + begin;
  int32_t* out = kept_idx + (size_t)h * B;  // B <= L_k here (the identity case is handled apart)

  fc::pdl_launch_dependents();  // the gather's blocks may take their places; they wait for this grid to end
  fc::pdl_wait();               // the scores are complete and visible from here on
  if (tid == 0 && blockIdx.x == 0 && n_kept) *n_kept = B;
  // the digit histograms start at zero; after that every pass clears what it has read
  for (int b = tid; b < 2 * kBins; b += kSelThreads) (&sh.hist[0][0])[b] = 0;
  bool any_nan = false;
  // Keys, and their range.  The scores of a head sit in a narrow band, so their keys share the leading bits;
  // digits taken from the raw keys would send almost every key of the first passes to one histogram bin (and
  // one shared-memory atomic at a time).  The select therefore works on key - min(key), which keeps the order,
  // and starts at the highest bit in which the keys of this head differ.
  uint32_t kmin = 0xffffffffu, kmax = 0;
  constexpr int kLoads = 12;  // loads in flight per thread: a quarter of a 44k-key head in one round
  for (int j0 = tid; j0 < n; j0 += kLoads * kSelThreads) {
    float v[kLoads];
#pragma unroll
    for (int u = 0; u < kLoads; ++u) {
      const int j = j0 + u * kSelThreads;
      v[u] = j < n ? s[j] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < kLoads; ++u) {
      const int j = j0 + u * kSelThreads;
      if (j < n) {
        bool nn;
        uint32_t k = score_key(v[u], nn);
        any_nan |= nn;
        if (begin + j >= protect_from) k = 0xffffffffu;  // protected tail: above every score's key (+inf is 0xff800000)
        if (kSmemKeys) smem_keys[j] = k;
        kmin = min(kmin, k);
        kmax = max(kmax, k);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
  }
  if (lane == 0) {
    sh.red_min[warp] = kmin;
    sh.red_max[warp] = kmax;
  }
  __syncthreads();
  if (warp == 0) {
    kmin = sh.red_min[lane];
    kmax = sh.red_max[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
      kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    }
    if (lane < cs) {  // lane q tells CTA q
      SelShared* other = cluster.map_shared_rank(&sh, lane);
      other->in_min[rank] = kmin;
      other->in_max[rank] = kmax;
    }
  }
  cluster.sync();
  kmin = 0xffffffffu;
  kmax = 0;
  for (int q = 0; q < cs; ++q) {
    kmin = min(kmin, sh.in_min[q]);
    kmax = max(kmax, sh.in_max[q]);
  }
  const uint32_t base = kmin;
  const int n_bits = kmax >= kmin ? 32 - __clz(kmax - kmin) : 0;  // 0 when all keys are equal
  auto key_at = [&](int j) -> uint32_t {  // key relative to the head's minimum; j is local to this CTA
    if (kSmemKeys) return smem_keys[j] - base;
    bool nn;
    return (begin + j >= protect_from ? 0xffffffffu : score_key(s[j], nn)) - base;
  };

  // Radix select, most significant digit first, kDigitBits at a time over the n_bits that vary.  Invariant: the
  // B-th largest key has the bits of `prefix` above bit `hi`, and `remaining` of the keys with that prefix
  // (counted from the largest) are still to be taken.  Every CTA adds up all CTAs' histograms and takes the
  // same decision.
  uint32_t prefix = 0, remaining = (uint32_t)B;
  int pass = 0;
  for (int hi = n_bits; hi > 0; ++pass) {
    const int lo = max(hi - kDigitBits, 0);
    const uint32_t digit_mask = (1u << (hi - lo)) - 1u;
    for (int j = tid; j < n; j += kSelThreads) {
      const uint32_t k = key_at(j);
      const bool candidate = hi >= 32 || (k >> hi) == (prefix >> hi);
      if (candidate) atomicAdd(&sh.hist[warp & 1][(k >> lo) & digit_mask], 1u);
    }
    __syncthreads();
    for (int b = tid; b < kBins; b += kSelThreads) {
      const uint32_t v = sh.hist[0][b] + sh.hist[1][b];
      sh.hist[0][b] = 0;  // for the next pass, whose atomics come after the barriers below
      sh.hist[1][b] = 0;
      for (int q = 0; q < cs; ++q) cluster.map_shared_rank(&sh, q)->hist_all[pass & 1][rank][b] = v;
    }
    cluster.sync();
    {
      // digits from the largest downwards, two per thread; the digit of the B-th largest key is where the running
      // count first reaches `remaining`
      const int d0 = kBins - 1 - 2 * tid, d1 = d0 - 1;
      uint32_t c0 = 0, c1 = 0;
      for (int q = 0; q < cs; ++q) {
        c0 += sh.hist_all[pass & 1][q][d0];
        c1 += sh.hist_all[pass & 1][q][d1];
      }
      const uint32_t tot = c0 + c1;
      uint32_t inc = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += v;
      }
      if (lane == 31) sh.scan_w[warp] = inc;
      __syncthreads();
      uint32_t before = lane < warp ? sh.scan_w[lane] : 0u;  // totals of the warps in front of this one
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
      const uint32_t exc = before + inc - tot;
      if (exc < remaining && remaining <= exc + tot) {
        uint32_t rem = remaining - exc;
        int digit = d0;
        if (c0 < rem) {
          rem -= c0;
          digit = d1;
        }
        sh.prefix = prefix | ((uint32_t)digit << lo);
        sh.remaining = rem;
      }
      __syncthreads();
    }
    prefix = sh.prefix;
    remaining = sh.remaining;
    hi = lo;
  }
  const uint32_t T = prefix;           // key (relative to the minimum) of the B-th largest score
  const uint32_t need_eq = remaining;  // how many keys equal to T are kept (lowest indices)

  // Ordered compaction.  Warp w owns the contiguous local range [w * wper, (w + 1) * wper) and walks it 32 keys at a
  // time: a ballot gives every kept key its rank among the 32, so the lanes of a warp write neighbouring entries of
  // the output (one thread writing a run of entries of its own made every store instruction touch 32 sectors).
  const int wper = (((n + 31) / 32 + 31) / 32) * 32;
  const int w0 = min(warp * wper, n), w1 = min(w0 + wper, n);
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t n_gt = 0, n_eq = 0;  // of this warp's range (the same in every lane)
  for (int j = w0 + lane; j - lane < w1; j += 32) {
    const uint32_t k = j < w1 ? key_at(j) : 0u;
    n_gt += __popc(__ballot_sync(0xffffffffu, j < w1 && k > T));
    n_eq += __popc(__ballot_sync(0xffffffffu, j < w1 && k == T));
  }
  if (lane == 0) {
    sh.warp_gt[warp] = n_gt;
    sh.warp_eq[warp] = n_eq;
  }
  __syncthreads();
  // kept keys above T / equal to T in front of this warp: the warps before it, then the CTAs before this one
  uint32_t gt_before = lane < warp ? sh.warp_gt[lane] : 0u, eq_before = lane < warp ? sh.warp_eq[lane] : 0u;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    gt_before += __shfl_xor_sync(0xffffffffu, gt_before, o);
    eq_before += __shfl_xor_sync(0xffffffffu, eq_before, o);
  }
  if (warp == kSelThreads / 32 - 1 && lane > rank && lane < cs) {
    // This CTA's totals go into the shared memory of the CTAs that own higher indices (lane q tells CTA q).  Written
    // before the barrier and read by their owner after it: no CTA touches another's shared memory after this barrier,
    // so none has to wait for the others before it leaves.
    SelShared* other = cluster.map_shared_rank(&sh, lane);
    other->in_gt[rank] = gt_before + n_gt;
    other->in_eq[rank] = eq_before + n_eq;
  }
  cluster.sync();
  for (int q = 0; q < rank; ++q) {
    gt_before += sh.in_gt[q];
    eq_before += sh.in_eq[q];
  }
  for (int j = w0 + lane; j - lane < w1; j += 32) {
    const uint32_t k = j < w1 ? key_at(j) : 0u;
    const bool gt = j < w1 && k > T, eq = j < w1 && k == T;
    const uint32_t m_gt = __ballot_sync(0xffffffffu, gt), m_eq = __ballot_sync(0xffffffffu, eq);
    const uint32_t gt_mine = gt_before + __popc(m_gt & lt), eq_mine = eq_before + __popc(m_eq & lt);
    if (gt) {
      const uint32_t pos = gt_mine + min(eq_mine, need_eq);
      if (fc::bounds_ok(pos < (uint32_t)B, status)) out[pos] = begin + j;
    } else if (eq && eq_mine < need_eq) {
      if (fc::bounds_ok(gt_mine + eq_mine < (uint32_t)B, status)) out[gt_mine + eq_mine] = begin + j;
    }
    gt_before += __popc(m_gt);
    eq_before += __popc(m_eq);
  }
  if (__any_sync(0xffffffffu, any_nan) && lane == 0 && status) atomicOr(status, FC_DEV_NAN_SCORE);
}

__global__ void select_identity_kernel(int32_t* __restrict__ kept_idx, int n_heads, int L_k,
                                       const float* __restrict__ score, int32_t* __restrict__ n_kept,
                                       uint32_t* __restrict__ status) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i == 0 && n_kept) *n_kept = L_k;
  if (i >= (int64_t)n_heads * L_k) return;
  kept_idx[i] = (int32_t)(i % L_k);
  if (status) {
    const uint32_t u = __float_as_uint(score[i]);
    if ((u & 0x7fffffffu) > 0x7f800000u) atomicOr(status, FC_DEV_NAN_SCORE);
  }
}


// Row gather.  The copy of one head is a flat list of 16-byte pieces: piece p of the head
// belongs to kept row p / pieces_per_row.  A block moves kUnroll * blockDim pieces of K and of V;
// all loads of a thread are issued before its first store.
constexpr int kCopyThreads = 256;
constexpr int kUnroll = 4;

__global__ void __launch_bounds__(kCopyThreads)
gather_rows_kernel(const uint8_t* __restrict__ K_src, const uint8_t* __restrict__ V_src,
                   uint8_t* __restrict__ K_dst, uint8_t* __restrict__ V_dst,
                   const int32_t* __restrict__ kept_idx, int n_keep, int L_k, int pieces_per_row, int ppr_shift,
                   int64_t src_hs_b, int64_t src_rs_b, int64_t dst_hs_b, int64_t dst_rs_b,
                   uint32_t* __restrict__ status) {
  const int h = blockIdx.y;
  fc::pdl_wait();  // the kept indices are complete and visible from here on
  // piece numbers fit 32 bits (the launcher checks), and a row is a power of two of pieces for every power-of-two head
  // dimension (ppr_shift >= 0): a shift and a mask instead of divisions, which cost more than the copy's own
  // instructions and show once the clocks are low
  const uint32_t n_pieces = (uint32_t)n_keep * (uint32_t)pieces_per_row;
  const uint32_t p0 = blockIdx.x * (uint32_t)(kCopyThreads * kUnroll) + threadIdx.x;
  const int32_t* idx = kept_idx + (size_t)h * n_keep;
  uint4 kv[kUnroll], vv[kUnroll];
  int64_t dst_off[kUnroll];
  bool ok[kUnroll];
#pragma unroll
  for (int u = 0; u < kUnroll; ++u) {
    const uint32_t p = p0 + (uint32_t)u * kCopyThreads;
    ok[u] = p < n_pieces;
    if (ok[u]) {
      const int r = (int)(ppr_shift >= 0 ? p >> ppr_shift : p / (uint32_t)pieces_per_row);
      const int c = (int)(p - (uint32_t)r * (uint32_t)pieces_per_row);
      const int32_t src_row = idx[r];
      if (src_row < 0 || src_row >= L_k) {  // never produced by the selection kernel
        ok[u] = false;
        if (status) atomicOr(status, FC_DEV_BAD_INDEX);
        continue;
      }
      const int64_t so = (int64_t)h * src_hs_b + (int64_t)src_row * src_rs_b + c * 16;
      dst_off[u] = (int64_t)h * dst_hs_b + (int64_t)r * dst_rs_b + c * 16;
      if (!fc::bounds_ok(r < n_keep && c < pieces_per_row, status)) {
        ok[u] = false;
        continue;
      }
      kv[u] = fc::ld_stream16(K_src + so);
      vv[u] = fc::ld_stream16(V_src + so);
    }
  }
#pragma unroll
  for (int u = 0; u < kUnroll; ++u)
    if (ok[u]) {
      fc::st_stream16(K_dst + dst_off[u], kv[u]);
      fc::st_stream16(V_dst + dst_off[u], vv[u]);
    }
}


// Selection units (a latent frame, a chunk): mean score of the `unit` consecutive tokens of every unit.  One warp per
// unit: each lane adds every 32nd score in fp64, the lanes are combined in a fixed tree; fp64 sums of fp32 scores of
// one head are exact for any realistic spread of magnitudes, so the order of summation does not show in the result.
__global__ void __launch_bounds__(256)
unit_mean_kernel(const float* __restrict__ score, int L_k, int unit, int n_units, int n_heads,
                 float* __restrict__ unit_score) {
  const int w = (int)((blockIdx.x * 256 + threadIdx.x) >> 5), lane = threadIdx.x & 31;
  if (w >= n_heads * n_units) return;
  const int h = w / n_units, u = w % n_units;
  const float* s = score + (size_t)h * L_k + (size_t)u * unit;
  double acc = 0.0;
  for (int t = lane; t < unit; t += 32) acc += (double)s[t];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
  if (lane == 0) unit_score[w] = (float)(acc / (double)unit);
}

// kept units -> kept tokens (ascending, as the units are)
__global__ void expand_units_kernel(const int32_t* __restrict__ unit_idx, int keep_units, int unit, int n_heads,
                                    int32_t* __restrict__ kept_idx, int32_t* __restrict__ n_kept) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t per_head = (int64_t)keep_units * unit;
  if (i == 0 && n_kept) *n_kept = (int32_t)per_head;
  if (i >= per_head * n_heads) return;
  const int h = (int)(i / per_head), r = (int)((i % per_head) / unit), t = (int)(i % unit);
  kept_idx[i] = unit_idx[(size_t)h * keep_units + r] * unit + t;
}

// Top-B of [n_heads, L] scores into out_idx [n_heads, min(B, L)]; entries at or after `protect_from` are kept first.
int launch_select(fc_ctx* ctx, cudaStream_t st, const float* score, int n_heads, int L, int B, int protect_from,
                  int32_t* out_idx, int32_t* n_kept, uint32_t* status) {
  if (B >= L) {
    const int64_t n = (int64_t)n_heads * L;
    select_identity_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(out_idx, n_heads, L, score, n_kept, status);
    FC_LAUNCH_CHECK("select_identity_kernel");
    return FC_OK;
  }
  // cluster size: as many CTAs per head as keep all heads within one wave of the SMs
  int cs = 1;
  while (cs < kMaxCluster && n_heads * cs * 2 <= ctx->sm_count) cs *= 2;
  const int chunk = (L + cs - 1) / cs;
  const size_t key_bytes = (size_t)chunk * 4;
  const bool smem_keys = key_bytes + sizeof(SelShared) + 1024 <= (size_t)ctx->smem_optin;
  const size_t smem_bytes = sizeof(SelShared) + (smem_keys ? key_bytes : 0);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)n_heads * cs);
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // may be scheduled under the previous kernel's tail
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (smem_keys) {
    FC_CUDA_CHECK(cudaFuncSetAttribute(select_topb_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes));
    FC_CUDA_CHECK(cudaLaunchKernelEx(&cfg, select_topb_kernel<true>, score, L, B, chunk, protect_from, out_idx, n_kept, status));
  } else {
    FC_CUDA_CHECK(cudaFuncSetAttribute(select_topb_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes));
    FC_CUDA_CHECK(cudaLaunchKernelEx(&cfg, select_topb_kernel<false>, score, L, B, chunk, protect_from, out_idx, n_kept, status));
  }
  FC_LAUNCH_CHECK("select_topb_kernel");
  return FC_OK;
}

struct CopyArgs {
  const void *K_src, *V_src;
  void *K_dst, *V_dst;
  int dtype, d;
  const fc_compact_strides* strides;
};

int check_copy(const CopyArgs& c, bool& copy) {
  copy = c.K_src || c.V_src || c.K_dst || c.V_dst;
  if (!copy) return FC_OK;
  if (!c.K_src || !c.V_src || !c.K_dst || !c.V_dst || !c.strides) return FC_ERR_INVALID_ARG;
  if (c.dtype != FC_BF16 && c.dtype != FC_F32) return FC_ERR_UNSUPPORTED;
  if (c.d <= 0) return FC_ERR_INVALID_ARG;
  const int es = fc::elem_size(c.dtype);
  if ((c.d * es) % 16) return FC_ERR_UNSUPPORTED;
  if (!fc::aligned16(c.K_src) || !fc::aligned16(c.V_src) || !fc::aligned16(c.K_dst) || !fc::aligned16(c.V_dst))
    return FC_ERR_MISALIGNED;
  const int64_t st[4] = {c.strides->src_hs, c.strides->src_rs, c.strides->dst_hs, c.strides->dst_rs};
  for (int i = 0; i < 4; ++i)
    if (st[i] < 0 || (st[i] * es) % 16) return FC_ERR_MISALIGNED;
  if (c.strides->src_rs < c.d || c.strides->dst_rs < c.d) return FC_ERR_INVALID_ARG;
  return FC_OK;
}

int launch_gather(cudaStream_t st, const CopyArgs& c, const int32_t* kept_idx, int n_heads, int n_keep, int L_k,
                  uint32_t* status) {
  const int es = fc::elem_size(c.dtype);
  const int ppr = c.d * es / 16;
  const int64_t n_pieces = (int64_t)n_keep * ppr;
  if (n_pieces + kCopyThreads * kUnroll > (int64_t)UINT32_MAX) return FC_ERR_UNSUPPORTED;  // 64 GB of rows per head and tensor
  int ppr_shift = -1;
  for (int sft = 0; sft < 16; ++sft)
    if ((1 << sft) == ppr) ppr_shift = sft;
  dim3 grid((unsigned)((n_pieces + kCopyThreads * kUnroll - 1) / (kCopyThreads * kUnroll)), n_heads);
  FC_CUDA_CHECK(fc::launch_pdl(gather_rows_kernel, grid, dim3(kCopyThreads), 0, st, (const uint8_t*)c.K_src,
                               (const uint8_t*)c.V_src, (uint8_t*)c.K_dst, (uint8_t*)c.V_dst, kept_idx, n_keep, L_k, ppr,
                               ppr_shift,
                               c.strides->src_hs * es, c.strides->src_rs * es, c.strides->dst_hs * es,
                               c.strides->dst_rs * es, status));
  FC_LAUNCH_CHECK("gather_rows_kernel");
  return FC_OK;
}

}  // namespace

extern "C" size_t fc_kv_select_compact_workspace_bytes(int n_heads, int L_k) {
  (void)n_heads;
  (void)L_k;
  return 16;  // the selection works in shared memory; a token size keeps the calling convention uniform
}

extern "C" int fc_kv_select_compact(fc_ctx* ctx, void* stream, const float* score, int n_heads, int L_k,
                                    int B, const void* K_src, const void* V_src, void* K_dst, void* V_dst,
                                    int dtype, int d, const fc_compact_strides* strides, int32_t* kept_idx,
                                    int32_t* n_kept, uint32_t* status, void* ws, size_t ws_bytes) {
  (void)ws;
  (void)ws_bytes;
  if (!ctx || !score || !kept_idx || n_heads <= 0 || L_k <= 0 || B <= 0) return FC_ERR_INVALID_ARG;
  const CopyArgs c = {K_src, V_src, K_dst, V_dst, dtype, d, strides};
  bool copy;
  int rc = check_copy(c, copy);
  if (rc != FC_OK) return rc;
  if (L_k > (1 << 20)) return FC_ERR_UNSUPPORTED;  // keeps the packed 16-bit scan counters exact
  cudaStream_t st = (cudaStream_t)stream;
  if ((rc = launch_select(ctx, st, score, n_heads, L_k, B, L_k, kept_idx, n_kept, status)) != FC_OK) return rc;
  if (copy) return launch_gather(st, c, kept_idx, n_heads, B < L_k ? B : L_k, L_k, status);
  return FC_OK;
}

extern "C" size_t fc_kv_select_compact_ex_workspace_bytes(int n_heads, int L_k, int unit) {
  if (n_heads <= 0 || L_k <= 0 || unit <= 1) return 16;
  const size_t n_units = (size_t)(L_k / unit);
  return fc::align_up(n_heads * n_units * sizeof(float), 256) + fc::align_up(n_heads * n_units * sizeof(int32_t), 256);
}

extern "C" int fc_kv_select_compact_ex(fc_ctx* ctx, void* stream, const float* score, int n_heads, int L_k, int B,
                                       const fc_select_opts* opts, const void* K_src, const void* V_src, void* K_dst,
                                       void* V_dst, int dtype, int d, const fc_compact_strides* strides,
                                       int32_t* kept_idx, int32_t* n_kept, uint32_t* status, void* ws, size_t ws_bytes) {
  if (!ctx || !score || !kept_idx || !opts || n_heads <= 0 || L_k <= 0 || B <= 0) return FC_ERR_INVALID_ARG;
  const int unit = opts->unit, n_protect = opts->n_protect;
  if (unit <= 0 || n_protect < 0) return FC_ERR_INVALID_ARG;
  if (L_k % unit || B % unit) return FC_ERR_INVALID_ARG;  // whole units only
  const CopyArgs c = {K_src, V_src, K_dst, V_dst, dtype, d, strides};
  bool copy;
  int rc = check_copy(c, copy);
  if (rc != FC_OK) return rc;
  if (L_k > (1 << 20)) return FC_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  const int n_keep = B < L_k ? B : L_k;
  if (unit == 1) {
    const int protect = n_protect < n_keep ? n_protect : n_keep;
    if ((rc = launch_select(ctx, st, score, n_heads, L_k, B, L_k - protect, kept_idx, n_kept, status)) != FC_OK) return rc;
  } else {
    const int n_units = L_k / unit, keep_units = n_keep / unit;
    const int protect_units = std::min((n_protect + unit - 1) / unit, keep_units);
    if (!ws || ws_bytes < fc_kv_select_compact_ex_workspace_bytes(n_heads, L_k, unit)) return FC_ERR_WORKSPACE;
    if (!fc::aligned16(ws)) return FC_ERR_MISALIGNED;
    float* unit_score = (float*)ws;
    int32_t* unit_idx = (int32_t*)((char*)ws + fc::align_up((size_t)n_heads * n_units * sizeof(float), 256));
    const int64_t warps = (int64_t)n_heads * n_units;
    unit_mean_kernel<<<(unsigned)((warps * 32 + 255) / 256), 256, 0, st>>>(score, L_k, unit, n_units, n_heads, unit_score);
    FC_LAUNCH_CHECK("unit_mean_kernel");
    if ((rc = launch_select(ctx, st, unit_score, n_heads, n_units, keep_units, n_units - protect_units, unit_idx, nullptr,
                            status)) != FC_OK)
      return rc;
    const int64_t n = (int64_t)n_heads * keep_units * unit;
    expand_units_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(unit_idx, keep_units, unit, n_heads, kept_idx, n_kept);
    FC_LAUNCH_CHECK("expand_units_kernel");
  }
  if (copy) return launch_gather(st, c, kept_idx, n_heads, n_keep, L_k, status);
  return FC_OK;
}
