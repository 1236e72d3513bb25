// Self-test of the bounded device-side waits.  Every wait on an mbarrier in this library gives up after a
// cycle limit, sets the plan's status word and lets the kernel return, so that a copy or a tensor-core
// commit that never completes ends in NGC_ERR_TIMEOUT instead of a hung GPU.  This file exercises that
// path without anything going wrong: one warp waits, with a short limit, on a barrier that has no copy in
// flight and that nobody arrives on.  Nothing faults, traps or spins without end, and no copy needs draining.
#include "ngc_device.h"
#include "ngc_tc.cuh"

namespace ngc {

namespace {

__global__ void __launch_bounds__(32) wait_timeout_kernel(long long limit_cycles, int *status) {
  __shared__ uint64_t bar;
  const uint32_t b = tc::smem_u32(&bar);
  if (threadIdx.x == 0) {
    tc::mbar_init(b, 1);
    tc::mbar_fence_init();
  }
  __syncwarp();
  // phase 0 of a freshly initialised barrier never completes without an arrival
  if (threadIdx.x == 0 && !tc::mbar_wait(b, 0u, limit_cycles)) atomicExch(status, 1);
}

}  // namespace

cudaError_t launch_wait_timeout(long long limit_cycles, int *status, cudaStream_t stream) {
  wait_timeout_kernel<<<1, 32, 0, stream>>>(limit_cycles, status);
  return cudaGetLastError();
}

}  // namespace ngc
