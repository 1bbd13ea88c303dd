// fc_chunk_decide: per-chunk relative-L1 indicator (Eq. 5) and the accumulate / threshold /
// reset rule (Eq. 8); as a switch, the uniform policy the paper compares with (caption of Fig. 3): one shared
// decision for all chunks of a step except those that must be computed anyway.
//
// Two launches, the second one programmatically dependent on the first (it is scheduled under the first one's
// tail and waits there).  (1) A streaming segmented reduction: the chunks are cut into slabs of 16 KiB
// per tensor, one block per slab; every thread sums |cur-prev| and |prev| of 4 interleaved
// 16-byte vectors in fp32, the block combines them in fp64 in a fixed tree and writes one
// (num, den) pair per slab.  (2) One block: its 32 warps are shared out over the chunks; they add a chunk's slab
// pairs in a fixed order in fp64 (eight loads in flight per thread), form r, apply the rule in fp32 and compact the
// active ids.
// No atomics: results are bit-reproducible from run to run.
#include <atomic>

#include "fc_common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kVecPerThread = 4;
constexpr int kSlabBytes = kThreads * kVecPerThread * 16;  // per tensor

struct DecideGeom {
  int64_t elem_off[FC_MAX_CHUNKS + 1];
  int32_t slab_off[FC_MAX_CHUNKS + 1];
  int32_t n_chunks;
};

__device__ __forceinline__ void accum_vec(const uint4& c, const uint4& p, __nv_bfloat16*, float& num,
                                          float& den) {
  const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, pw[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float c0 = fc::bf16_lo(cw[i]), c1 = fc::bf16_hi(cw[i]);
    float p0 = fc::bf16_lo(pw[i]), p1 = fc::bf16_hi(pw[i]);
    num += fabsf(c0 - p0);
    den += fabsf(p0);
    num += fabsf(c1 - p1);
    den += fabsf(p1);
  }
}
__device__ __forceinline__ void accum_vec(const uint4& c, const uint4& p, float*, float& num, float& den) {
  const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, pw[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float cf = __uint_as_float(cw[i]), pf = __uint_as_float(pw[i]);
    num += fabsf(cf - pf);
    den += fabsf(pf);
  }
}

template <typename T, bool kVec>
__global__ void __launch_bounds__(kThreads)
decide_partial_kernel(const T* __restrict__ cur, const T* __restrict__ prev, DecideGeom g,
                      double2* __restrict__ partial) {
  constexpr int kElemPerVec = 16 / (int)sizeof(T);
  constexpr int kSlabElems = kSlabBytes / (int)sizeof(T);
  fc::pdl_launch_dependents();  // the finalising block may take its place on an SM; it waits for this grid to end
  const int b = blockIdx.x;
  int c = 0;
  while (c + 1 < g.n_chunks && b >= g.slab_off[c + 1]) ++c;
  const int64_t begin = g.elem_off[c] + (int64_t)(b - g.slab_off[c]) * kSlabElems;
  const int64_t end = min(begin + (int64_t)kSlabElems, g.elem_off[c + 1]);
  float num = 0.f, den = 0.f;
  if (kVec) {
    uint4 cv[kVecPerThread], pv[kVecPerThread];
    bool ok[kVecPerThread];
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
      const int64_t e = begin + (int64_t)(k * kThreads + threadIdx.x) * kElemPerVec;
      ok[k] = e < end;  // chunk lengths are vector multiples on this path
      if (ok[k]) {
        cv[k] = fc::ld_stream16(cur + e);
        pv[k] = fc::ld_stream16(prev + e);
      }
    }
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k)
      if (ok[k]) accum_vec(cv[k], pv[k], (T*)nullptr, num, den);
  } else {
    for (int64_t e = begin + threadIdx.x; e < end; e += kThreads) {
      float cf = fc::to_float(cur[e]), pf = fc::to_float(prev[e]);
      num += fabsf(cf - pf);
      den += fabsf(pf);
    }
  }
  double dn = (double)num, dd = (double)den;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    dn += __shfl_down_sync(0xffffffffu, dn, o);
    dd += __shfl_down_sync(0xffffffffu, dd, o);
  }
  __shared__ double2 warp_sum[kThreads / 32];
  if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = make_double2(dn, dd);
  __syncthreads();
  if (threadIdx.x == 0) {
    double2 s = warp_sum[0];
    for (int w = 1; w < kThreads / 32; ++w) {
      s.x += warp_sum[w].x;
      s.y += warp_sum[w].y;
    }
    partial[b] = s;
  }
}

// Eq. 5's ratio; a zero denominator yields +inf if anything changed, else 0
__device__ __forceinline__ double ratio(double num, double den) {
  if (den > 0.0) return num / den;
  return num > 0.0 ? (double)INFINITY : 0.0;
}

__global__ void __launch_bounds__(1024)
decide_finalize_kernel(DecideGeom g, const double2* __restrict__ partial,
                       const int32_t* __restrict__ chunk_step, int warmup_m, float eps,
                       const uint8_t* __restrict__ force, int policy, float* __restrict__ acc,
                       float* __restrict__ l1rel, uint8_t* __restrict__ recompute,
                       int32_t* __restrict__ active_ids, int32_t* __restrict__ n_active) {
  __shared__ uint8_t flag[FC_MAX_CHUNKS];
  __shared__ double2 part[32];
  __shared__ double2 chunk_sum[FC_MAX_CHUNKS];  // uniform policy: every chunk's (num, den)
  fc::pdl_wait();  // launched under the reduction's tail: its slab pairs are complete and visible from here on
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // The 32 warps are shared out over the chunks, a power of two of them per chunk (all 32 for one chunk, one each
  // for 32 or more): every warp adds up a fixed subset of the chunk's slabs, the warps of a chunk are combined in
  // warp order.  Fixed order throughout: bit-reproducible.
  int wpc = 32;
  while (wpc > 1 && wpc * min(g.n_chunks, 32) > 32) wpc >>= 1;
  const int per_round = 32 / wpc;  // chunks handled at a time
  for (int c0 = 0; c0 < g.n_chunks; c0 += per_round) {
    const int c = c0 + warp / wpc, sub = warp % wpc;
    double num = 0.0, den = 0.0;
    if (c < g.n_chunks) {
      // eight loads in flight at a time (one after the other, every iteration waited for its own load: 37 round trips
      // on 16 chunks of 2340 slabs); the additions keep their order
      constexpr int kBatch = 8;
      const int end = g.slab_off[c + 1], stride = wpc * 32;
      for (int s0 = g.slab_off[c] + sub * 32 + lane; s0 < end; s0 += kBatch * stride) {
        double2 v[kBatch];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          const int s = s0 + k * stride;
          v[k] = s < end ? partial[s] : make_double2(0.0, 0.0);
        }
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
          if (s0 + k * stride < end) {
            num += v[k].x;
            den += v[k].y;
          }
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      num += __shfl_down_sync(0xffffffffu, num, o);
      den += __shfl_down_sync(0xffffffffu, den, o);
    }
    if (lane == 0) part[warp] = make_double2(num, den);
    __syncthreads();
    if (sub == 0 && lane == 0 && c < g.n_chunks) {
      num = 0.0;
      den = 0.0;
      for (int w = 0; w < wpc; ++w) {
        num += part[warp + w].x;
        den += part[warp + w].y;
      }
      if (policy == FC_POLICY_UNIFORM) {
        chunk_sum[c] = make_double2(num, den);
      } else {
        const float rf = (float)ratio(num, den);
        const float s = __fadd_rn(acc[c], rf);
        const bool rec = chunk_step[c] < warmup_m || (force && force[c]) || s > eps;
        if (l1rel) l1rel[c] = rf;
        recompute[c] = rec ? 1 : 0;
        acc[c] = rec ? 0.f : s;
        flag[c] = rec ? 1 : 0;
      }
    }
    __syncthreads();  // part[] is reused by the next round
  }
  __syncthreads();
  if (threadIdx.x == 0 && policy == FC_POLICY_UNIFORM) {
    // One decision for the chunks that share it (those neither in warm-up nor forced): Eq. 4 over them as one
    // tensor, sums taken in chunk order, then Eq. 8 on the shared accumulator (read from the first sharing chunk,
    // written to every entry so that they stay equal).
    double num = 0.0, den = 0.0;
    int first = -1;
    for (int c = 0; c < g.n_chunks; ++c) {
      const bool own = chunk_step[c] < warmup_m || (force && force[c]);
      flag[c] = own ? 2 : 0;
      if (own) continue;
      if (first < 0) first = c;
      num += chunk_sum[c].x;
      den += chunk_sum[c].y;
    }
    bool shared_compute = true;
    float acc_next = 0.f, r_shared = 0.f;
    if (first >= 0) {
      r_shared = (float)ratio(num, den);
      const float s = __fadd_rn(acc[first], r_shared);
      shared_compute = s > eps;
      acc_next = shared_compute ? 0.f : s;
    }
    for (int c = 0; c < g.n_chunks; ++c) {
      const bool own = flag[c] == 2;
      if (l1rel) l1rel[c] = own ? (float)ratio(chunk_sum[c].x, chunk_sum[c].y) : r_shared;
      const bool rec = own || shared_compute;
      recompute[c] = rec ? 1 : 0;
      acc[c] = acc_next;
      flag[c] = rec ? 1 : 0;
    }
  }
  if (threadIdx.x == 0) {
    int n = 0;
    for (int c = 0; c < g.n_chunks; ++c)
      if (flag[c]) active_ids[n++] = c;
    *n_active = n;
    for (int c = n; c < g.n_chunks; ++c) active_ids[c] = -1;
  }
}

int64_t slab_elems(int dtype) { return kSlabBytes / fc::elem_size(dtype); }

}  // namespace

extern "C" size_t fc_chunk_decide_workspace_bytes(int64_t total_elems, int n_chunks) {
  if (total_elems < 0 || n_chunks < 0) return 0;
  // one (num, den) pair per slab; slabs never straddle chunks, sized for the narrower dtype
  const int64_t slabs = total_elems / slab_elems(FC_F32) + n_chunks + 1;
  return (size_t)slabs * sizeof(double2);
}

extern "C" int fc_chunk_decide(fc_ctx* ctx, void* stream, const void* cur, const void* prev, int dtype,
                               const int64_t* chunk_elem_off, int n_chunks, const int32_t* chunk_step,
                               int warmup_m, float eps, const uint8_t* force, int policy, float* acc,
                               float* l1rel, uint8_t* recompute, int32_t* active_ids, int32_t* n_active,
                               uint32_t* status, void* ws, size_t ws_bytes) {
  (void)status;
  if (policy != FC_POLICY_CHUNKWISE && policy != FC_POLICY_UNIFORM) return FC_ERR_INVALID_ARG;
  if (!ctx || !chunk_elem_off || !chunk_step || !acc || !recompute || !active_ids || !n_active)
    return FC_ERR_INVALID_ARG;
  if (n_chunks <= 0) return FC_ERR_INVALID_ARG;
  if (n_chunks > FC_MAX_CHUNKS) return FC_ERR_UNSUPPORTED;
  if (dtype != FC_BF16 && dtype != FC_F32) return FC_ERR_UNSUPPORTED;
  const int es = fc::elem_size(dtype);
  DecideGeom g;
  g.n_chunks = n_chunks;
  const int64_t se = slab_elems(dtype);
  bool vec = fc::aligned16(cur) && fc::aligned16(prev);
  int64_t slabs = 0;
  for (int c = 0; c <= n_chunks; ++c) {
    g.elem_off[c] = chunk_elem_off[c];
    if (chunk_elem_off[c] < 0 || (c > 0 && chunk_elem_off[c] < chunk_elem_off[c - 1]))
      return FC_ERR_INVALID_ARG;
    if ((chunk_elem_off[c] * es) % 16) vec = false;
    g.slab_off[c] = (int32_t)slabs;
    if (c < n_chunks) slabs += (chunk_elem_off[c + 1] - chunk_elem_off[c] + se - 1) / se;
    if (slabs > INT32_MAX / 2) return FC_ERR_UNSUPPORTED;
  }
  const int64_t total = chunk_elem_off[n_chunks];
  if (total > 0 && (!cur || !prev)) return FC_ERR_INVALID_ARG;
  if (!ws || ws_bytes < (size_t)slabs * sizeof(double2) ||
      ws_bytes < fc_chunk_decide_workspace_bytes(total, n_chunks))
    return FC_ERR_WORKSPACE;
  if (!fc::aligned16(ws)) return FC_ERR_MISALIGNED;
  cudaStream_t st = (cudaStream_t)stream;
  double2* partial = (double2*)ws;
  if (slabs > 0) {
    if (dtype == FC_BF16) {
      auto* c = (const __nv_bfloat16*)cur;
      auto* p = (const __nv_bfloat16*)prev;
      if (vec)
        decide_partial_kernel<__nv_bfloat16, true><<<(unsigned)slabs, kThreads, 0, st>>>(c, p, g, partial);
      else
        decide_partial_kernel<__nv_bfloat16, false><<<(unsigned)slabs, kThreads, 0, st>>>(c, p, g, partial);
    } else {
      auto* c = (const float*)cur;
      auto* p = (const float*)prev;
      if (vec)
        decide_partial_kernel<float, true><<<(unsigned)slabs, kThreads, 0, st>>>(c, p, g, partial);
      else
        decide_partial_kernel<float, false><<<(unsigned)slabs, kThreads, 0, st>>>(c, p, g, partial);
    }
    FC_LAUNCH_CHECK("decide_partial_kernel");
  }
  FC_CUDA_CHECK(fc::launch_pdl(decide_finalize_kernel, dim3(1), dim3(1024), 0, st, g, (const double2*)partial,
                               chunk_step, warmup_m, eps, force, policy, acc, l1rel, recompute, active_ids,
                               n_active));
  return FC_OK;
}

// ---------------------------------------------------------------------------------------------
// fc_chunk_decide_static: the same decision for callers that cannot allocate device memory.
//
// The slab partials live in a fixed array inside the library image instead of a caller workspace.
// In host code the array's name is only a handle; its device address is looked up once per
// device, with that device current, and that address is what the kernels receive.
namespace {

constexpr size_t kStaticScratchBytes = 1u << 20;  // 65,536 slabs of 16 KiB per tensor
static __device__ __align__(256) unsigned char g_decide_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
// device address of g_decide_scratch on each device (null = not looked up yet)
std::atomic<void*> g_scratch_addr[kMaxDevices];

// Look the address up once per device (fc_create does it; the first call does if that did not happen).  Not an allocation: the array is part of the
// module image every device already holds.  Concurrent first calls may both do the lookup; they
// get the same answer and store the same value.
int static_scratch(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return FC_ERR_UNSUPPORTED;
  void* known = g_scratch_addr[device].load(std::memory_order_acquire);
  if (!known) {
    int current = -1;
    FC_CUDA_CHECK(cudaGetDevice(&current));
    if (current != device) FC_CUDA_CHECK(cudaSetDevice(device));
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_decide_scratch);
    if (current != device) cudaSetDevice(current);
    if (e != cudaSuccess || !p) {
      fc::set_cuda_error(e, "cudaGetSymbolAddress(g_decide_scratch)");
      return FC_ERR_CUDA;
    }
    g_scratch_addr[device].store(p, std::memory_order_release);
    known = p;
  }
  *out = known;
  return FC_OK;
}

}  // namespace

namespace fc {
// Called by fc_create with `device` current: looks the array's address up ahead of the first static call, so that
// callers who may not touch the driver where they call do not pay for it there.  A failure here is not an error of
// fc_create; the first fc_chunk_decide_static call then tries again and reports it.
void decide_static_setup(int device) {
  void* p = nullptr;
  (void)static_scratch(device, &p);
}
}  // namespace fc

extern "C" size_t fc_chunk_decide_static_max_bytes(void) { return kStaticScratchBytes; }

extern "C" int fc_chunk_decide_static(fc_ctx* ctx, void* stream, const void* cur, const void* prev, int dtype,
                                      const int64_t* chunk_elem_off, int n_chunks, const int32_t* chunk_step,
                                      int warmup_m, float eps, const uint8_t* force, int policy, float* acc,
                                      float* l1rel, uint8_t* recompute, int32_t* active_ids, int32_t* n_active,
                                      uint32_t* status) {
  if (!ctx || !chunk_elem_off || n_chunks <= 0) return FC_ERR_INVALID_ARG;
  if (n_chunks > FC_MAX_CHUNKS) return FC_ERR_UNSUPPORTED;
  const int64_t total = chunk_elem_off[n_chunks];
  if (total < 0) return FC_ERR_INVALID_ARG;
  if (fc_chunk_decide_workspace_bytes(total, n_chunks) > kStaticScratchBytes) return FC_ERR_TOO_LARGE;
  void* scratch = nullptr;
  const int rc = static_scratch(ctx->device, &scratch);
  if (rc != FC_OK) return rc;
  // Every slab pair is written by the reduction before the finalising kernel reads it, so the
  // array needs no clearing between calls even though it keeps the previous call's contents.
  return fc_chunk_decide(ctx, stream, cur, prev, dtype, chunk_elem_off, n_chunks, chunk_step, warmup_m, eps, force,
                         policy, acc, l1rel, recompute, active_ids, n_active, status, scratch, kStaticScratchBytes);
}
