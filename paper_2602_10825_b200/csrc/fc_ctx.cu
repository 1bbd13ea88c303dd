// Context, status strings and the CUDA error record of libfc.
#include <cstdio>
#include <cstring>
#include <new>

#include "fc_common.cuh"

namespace fc {
static thread_local char g_cuda_error[256] = "";
void set_cuda_error(cudaError_t e, const char* where) {
  std::snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", where, cudaGetErrorString(e));
}
}  // namespace fc

extern "C" const char* fc_last_cuda_error(void) { return fc::g_cuda_error; }

extern "C" const char* fc_status_string(int status) {
  switch (status) {
    case FC_OK: return "ok";
    case FC_ERR_INVALID_ARG: return "invalid argument";
    case FC_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case FC_ERR_MISALIGNED: return "pointer or stride not 16-byte aligned";
    case FC_ERR_WORKSPACE: return "workspace missing or too small";
    case FC_ERR_DEVICE: return "device is not compute capability 10.x";
    case FC_ERR_CUDA: return "CUDA call failed";
    case FC_ERR_UNIMPLEMENTED: return "not implemented";
    case FC_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
    default: return "unknown status";
  }
}

extern "C" int fc_create(fc_ctx** out, int device) {
  if (!out) return FC_ERR_INVALID_ARG;
  *out = nullptr;
  int n_dev = 0;
  FC_CUDA_CHECK(cudaGetDeviceCount(&n_dev));
  if (device < 0 || device >= n_dev) return FC_ERR_INVALID_ARG;
  FC_CUDA_CHECK(cudaSetDevice(device));
  cudaDeviceProp prop;
  FC_CUDA_CHECK(cudaGetDeviceProperties(&prop, device));
  if (prop.major != 10) return FC_ERR_DEVICE;
  fc_ctx* ctx = new (std::nothrow) fc_ctx();
  if (!ctx) return FC_ERR_INVALID_ARG;
  ctx->device = device;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->smem_optin = (int)prop.sharedMemPerBlockOptin;
  ctx->encode_tiled = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ctx->encode_tiled,
                                          cudaEnableDefault, &qres);
  if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !ctx->encode_tiled) {
    fc::set_cuda_error(e, "cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)");
    delete ctx;
    return FC_ERR_CUDA;
  }
  fc::decide_static_setup(device);
  *out = ctx;
  return FC_OK;
}

extern "C" int fc_destroy(fc_ctx* ctx) {
  delete ctx;
  return FC_OK;
}

extern "C" int fc_sm_count(const fc_ctx* ctx) { return ctx ? ctx->sm_count : 0; }
