// Self-test of the bounded device-side waits (kvc_selftest_bounded_wait): a wait that nothing completes must give
// up after WAIT_SPIN_LIMIT polls and report KVC_ERR_TIMEOUT instead of hanging the GPU.
#include "kvc_async.cuh"
#include "kvc_internal.cuh"

namespace kvc {

__global__ void wait_selftest_kernel(int* status) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);                       // one arrival expected; none is ever made
    fence_mbar_init();
  }
  __syncwarp();
  const bool completed = mbar_wait_bounded(&bar, 0);
  __syncwarp();
  if (threadIdx.x == 0) *status = completed ? (int)KVC_OK : (int)KVC_ERR_TIMEOUT;
}

void launch_wait_selftest(int* status, cudaStream_t st) { wait_selftest_kernel<<<1, 32, 0, st>>>(status); }

}  // namespace kvc
