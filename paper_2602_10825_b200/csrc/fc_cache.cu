// fc_chunk_cache_apply: serving skipped chunks from the activation cache (Sec. 3.2, text after Eq. 8).
//
// One streaming launch over the chunks' elements.  The chunks are cut into slabs of 16 KiB per tensor that never
// straddle a chunk, one block per slab, so a block reads one recompute flag (from device memory: the decision
// never returns to the host) and then does one of two things with 16-byte accesses, four vectors in flight per
// thread and tensor:
//   computed chunk:  cache <- y - x      (x, y read; cache written)
//   skipped chunk:   y     <- x + cache  (x, cache read; y written)
// Either way three tensors' worth of bytes move: the roofline is 3 * elements * element size over the HBM rate.
// Arithmetic is fp32, rounded once to the storage type (round to nearest even for bf16).
#include "fc_common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kVecPerThread = 4;
constexpr int kSlabBytes = kThreads * kVecPerThread * 16;  // per tensor

struct CacheGeom {
  int64_t elem_off[FC_MAX_CHUNKS + 1];
  int32_t slab_off[FC_MAX_CHUNKS + 1];
  int32_t n_chunks;
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// out = a + sign * b, element by element, on one 16-byte vector
template <typename T>
__device__ __forceinline__ uint4 combine(const uint4& a, const uint4& b, float sign);
template <>
__device__ __forceinline__ uint4 combine<__nv_bfloat16>(const uint4& a, const uint4& b, float sign) {
  const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
    o[i] = pack_bf16(__fmaf_rn(sign, fc::bf16_lo(bw[i]), fc::bf16_lo(aw[i])),
                     __fmaf_rn(sign, fc::bf16_hi(bw[i]), fc::bf16_hi(aw[i])));
  return make_uint4(o[0], o[1], o[2], o[3]);
}
template <>
__device__ __forceinline__ uint4 combine<float>(const uint4& a, const uint4& b, float sign) {
  const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = __float_as_uint(__fmaf_rn(sign, __uint_as_float(bw[i]), __uint_as_float(aw[i])));
  return make_uint4(o[0], o[1], o[2], o[3]);
}
__device__ __forceinline__ void store_elem(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_elem(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// sign * b + a with sign = +-1 is exactly a +- b rounded once: the product is exact.
template <typename T, bool kVec>
__global__ void __launch_bounds__(kThreads)
cache_apply_kernel(const T* __restrict__ x, T* __restrict__ y, T* __restrict__ cache, CacheGeom g,
                   const uint8_t* __restrict__ recompute) {
  constexpr int kElemPerVec = 16 / (int)sizeof(T);
  constexpr int kSlabElems = kSlabBytes / (int)sizeof(T);
  const int b = blockIdx.x;
  int c = 0;
  while (c + 1 < g.n_chunks && b >= g.slab_off[c + 1]) ++c;
  const int64_t begin = g.elem_off[c] + (int64_t)(b - g.slab_off[c]) * kSlabElems;
  const int64_t end = min(begin + (int64_t)kSlabElems, g.elem_off[c + 1]);
  const bool computed = recompute[c] != 0;
  // computed: cache = y - x (first operand y, second x, sign -1); skipped: y = x + cache
  const T* first = computed ? y : x;
  const T* second = computed ? x : cache;
  T* dst = computed ? cache : y;
  const float sign = computed ? -1.f : 1.f;
  if (kVec) {
    uint4 av[kVecPerThread], bv[kVecPerThread];
    bool ok[kVecPerThread];
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
      const int64_t e = begin + (int64_t)(k * kThreads + threadIdx.x) * kElemPerVec;
      ok[k] = e < end;  // chunk lengths are vector multiples on this path
      if (ok[k]) {
        av[k] = fc::ld_stream16(first + e);
        bv[k] = fc::ld_stream16(second + e);
      }
    }
#pragma unroll
    for (int k = 0; k < kVecPerThread; ++k) {
      const int64_t e = begin + (int64_t)(k * kThreads + threadIdx.x) * kElemPerVec;
      if (ok[k]) fc::st_stream16(dst + e, combine<T>(av[k], bv[k], sign));
    }
  } else {
    for (int64_t e = begin + threadIdx.x; e < end; e += kThreads)
      store_elem(dst + e, __fmaf_rn(sign, fc::to_float(second[e]), fc::to_float(first[e])));
  }
}

}  // namespace

extern "C" int fc_chunk_cache_apply(fc_ctx* ctx, void* stream, const void* x_in, void* y_io, void* cache, int dtype,
                                    const int64_t* chunk_elem_off, int n_chunks, const uint8_t* recompute,
                                    uint32_t* status) {
  (void)status;
  if (!ctx || !chunk_elem_off || !recompute || n_chunks <= 0) return FC_ERR_INVALID_ARG;
  if (n_chunks > FC_MAX_CHUNKS) return FC_ERR_UNSUPPORTED;
  if (dtype != FC_BF16 && dtype != FC_F32) return FC_ERR_UNSUPPORTED;
  const int es = fc::elem_size(dtype);
  const int64_t se = kSlabBytes / es;
  CacheGeom g;
  g.n_chunks = n_chunks;
  bool vec = fc::aligned16(x_in) && fc::aligned16(y_io) && fc::aligned16(cache);
  int64_t slabs = 0;
  for (int c = 0; c <= n_chunks; ++c) {
    g.elem_off[c] = chunk_elem_off[c];
    if (chunk_elem_off[c] < 0 || (c > 0 && chunk_elem_off[c] < chunk_elem_off[c - 1])) return FC_ERR_INVALID_ARG;
    if ((chunk_elem_off[c] * es) % 16) vec = false;
    g.slab_off[c] = (int32_t)slabs;
    if (c < n_chunks) slabs += (chunk_elem_off[c + 1] - chunk_elem_off[c] + se - 1) / se;
    if (slabs > INT32_MAX / 2) return FC_ERR_UNSUPPORTED;
  }
  if (chunk_elem_off[n_chunks] > 0 && (!x_in || !y_io || !cache)) return FC_ERR_INVALID_ARG;
  {  // the three tensors must not overlap
    const uintptr_t n = (uintptr_t)chunk_elem_off[n_chunks] * es;
    const uintptr_t p[3] = {(uintptr_t)x_in, (uintptr_t)y_io, (uintptr_t)cache};
    for (int a = 0; a < 3; ++a)
      for (int b = a + 1; b < 3; ++b)
        if (p[a] < p[b] + n && p[b] < p[a] + n) return FC_ERR_INVALID_ARG;
  }
  if (slabs == 0) return FC_OK;
  cudaStream_t st = (cudaStream_t)stream;
  const unsigned grid = (unsigned)slabs;
  if (dtype == FC_BF16) {
    auto *x = (const __nv_bfloat16*)x_in;
    auto *y = (__nv_bfloat16*)y_io, *c = (__nv_bfloat16*)cache;
    if (vec) cache_apply_kernel<__nv_bfloat16, true><<<grid, kThreads, 0, st>>>(x, y, c, g, recompute);
    else cache_apply_kernel<__nv_bfloat16, false><<<grid, kThreads, 0, st>>>(x, y, c, g, recompute);
  } else {
    auto *x = (const float*)x_in;
    auto *y = (float*)y_io, *c = (float*)cache;
    if (vec) cache_apply_kernel<float, true><<<grid, kThreads, 0, st>>>(x, y, c, g, recompute);
    else cache_apply_kernel<float, false><<<grid, kThreads, 0, st>>>(x, y, c, g, recompute);
  }
  FC_LAUNCH_CHECK("cache_apply_kernel");
  return FC_OK;
}
