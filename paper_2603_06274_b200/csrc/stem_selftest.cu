// stem_selftest_wait_timeout: exercises the bounded-wait machinery of the library without touching
// the production kernels.  One thread waits, with a 1 ms limit, on an mbarrier that nothing ever
// arrives at, using the same helper the attention and metric kernels wait with; when the limit runs
// out it records a status code the way those kernels do and returns normally.  The context stays
// usable; stem_check_status then reports STEM_ERR_DEVICE_TIMEOUT.
#include "stem_internal.h"
#include "stem_ptx.cuh"

namespace stem {
namespace {

constexpr uint64_t kSelfTestLimitNs = 1000ull * 1000;  // 1 ms

__global__ void selftest_wait_kernel(int32_t* status) {
  __shared__ __align__(8) uint64_t bar;
  const uint32_t bar_addr = (uint32_t)__cvta_generic_to_shared(&bar);
  ptx::mbar_init(bar_addr, 1);
  ptx::mbar_init_fence();
  // phase 0 of a barrier that expects one arrival and never gets it
  if (!ptx::mbar_wait_bounded(bar_addr, 0, kSelfTestLimitNs)) {
    if (atomicCAS(status, 0, 1) == 0) {
      status[1] = (int32_t)blockIdx.x;
      status[2] = kRoleSelfTest;
      status[3] = 0;
    }
  }
}

}  // namespace

cudaError_t launch_selftest_wait(int32_t* status, cudaStream_t s) {
  selftest_wait_kernel<<<1, 1, 0, s>>>(status);
  return cudaGetLastError();
}

}  // namespace stem
