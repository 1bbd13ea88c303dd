// Internal helpers shared by the kernels of libfc (never by the CPU oracle).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "fc.h"

struct fc_ctx {
  int device;
  int sm_count;
  int smem_optin;       // max dynamic shared memory per block (opt-in), bytes
  void* encode_tiled;   // cuTensorMapEncodeTiled, resolved through the runtime
};

namespace fc {

void set_cuda_error(cudaError_t e, const char* where);
void decide_static_setup(int device);  // fc_decide.cu: address of the built-in scratch of fc_chunk_decide_static

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int elem_size(int dtype) { return dtype == FC_F32 ? 4 : 2; }

#define FC_CUDA_CHECK(expr)                         \
  do {                                              \
    cudaError_t e__ = (expr);                       \
    if (e__ != cudaSuccess) {                       \
      fc::set_cuda_error(e__, #expr);               \
      return FC_ERR_CUDA;                           \
    }                                               \
  } while (0)

#define FC_LAUNCH_CHECK(name)                       \
  do {                                              \
    cudaError_t e__ = cudaGetLastError();           \
    if (e__ != cudaSuccess) {                       \
      fc::set_cuda_error(e__, name);                \
      return FC_ERR_CUDA;                           \
    }                                               \
  } while (0)

// Bounds-checking build (-DFC_DEBUG_BOUNDS, libfc_debug.so): every store whose address is computed from data read on
// the device, or from a tile / slice walk, is guarded; a violated guard sets FC_DEV_BAD_INDEX in the status word and
// skips the store (nothing traps).  In the normal build the guard is the constant `true`.
#ifdef FC_DEBUG_BOUNDS
__device__ __forceinline__ bool bounds_ok(bool inside, uint32_t* status) {
  if (!inside && status) atomicOr(status, (uint32_t)FC_DEV_BAD_INDEX);
  return inside;
}
#else
__device__ __forceinline__ bool bounds_ok(bool, uint32_t*) { return true; }
#endif

// Programmatic dependent launch.  launch_pdl() starts `kernel` so that its blocks may become resident while the
// previous kernel of the stream is still running (once every block of that kernel has executed
// pdl_launch_dependents() or exited); the kernel must execute pdl_wait() before it reads or writes anything the
// previous kernel touches: the wait returns when that kernel has completed and its writes are visible.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Storage element -> float.
template <typename T> __device__ __forceinline__ float to_float(T x);
template <> __device__ __forceinline__ float to_float<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 x) {
  return __bfloat162float(x);
}

// Two bf16 packed in a 32-bit word -> two floats (exact: bf16 is the top half of an fp32).
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream16(void* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}

}  // namespace fc
