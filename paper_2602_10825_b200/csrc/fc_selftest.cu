// fc_selftest_bounded_wait: shows, without faulting or hanging anything, what the tcgen05 kernels do when a
// barrier they wait on is never signalled.  One warp waits with mbar_wait_bounded (the wait every such kernel uses)
// on an mbarrier that nobody will ever arrive at, with a short limit; the wait gives up, the kernel runs on to its
// end, FC_DEV_TIMEOUT is set in the status word and the context stays usable.
#include <algorithm>

#include "fc_common.cuh"
#include "fc_tcgen05.cuh"

namespace {

using namespace fc::sm100;

__global__ void __launch_bounds__(32)
bounded_wait_selftest_kernel(uint64_t limit_ns, uint32_t* __restrict__ status, uint32_t* __restrict__ waited_ns) {
  __shared__ uint64_t bar;
  __shared__ uint32_t gave_up;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);  // one arrival would complete the phase; none ever comes
    mbar_fence_init();
    gave_up = 0;
  }
  __syncthreads();
  const uint64_t t0 = global_timer_ns();
  mbar_wait_bounded(smem_u32(&bar), 0, &gave_up, limit_ns);
  const uint64_t t1 = global_timer_ns();
  __syncthreads();
  if (threadIdx.x == 0) {
    if (gave_up && status) atomicOr(status, FC_DEV_TIMEOUT);
    if (waited_ns) *waited_ns = (uint32_t)min(t1 - t0, (uint64_t)0xffffffffu);
  }
}

}  // namespace

extern "C" int fc_selftest_bounded_wait(fc_ctx* ctx, void* stream, uint64_t limit_ns, uint32_t* status,
                                        uint32_t* waited_ns) {
  if (!ctx || !status) return FC_ERR_INVALID_ARG;
  limit_ns = std::min<uint64_t>(std::max<uint64_t>(limit_ns, 1000ull), 1000000000ull);  // 1 us .. 1 s
  bounded_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(limit_ns, status, waited_ns);
  FC_LAUNCH_CHECK("bounded_wait_selftest_kernel");
  return FC_OK;
}
