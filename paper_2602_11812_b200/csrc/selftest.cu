// Self-test of the bounded wait every pipeline kernel of this library relies on: a block waits on an
// mbarrier that nobody will ever signal, the wait gives up after its (here: short) limit, and the
// kernel reports EGTP_ERR_DEVICE_TIMEOUT through the status word and returns normally.  Nothing
// traps, nothing hangs, the CUDA context stays usable.
#include "kernels.h"
#include "sm100_ptx.cuh"
#include "../../include/egtp.h"

namespace egtp {

namespace {

__global__ void wait_timeout_selftest_kernel(uint64_t limit_ns, int32_t* status) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);      // one arrival expected; none will come
    abort_flag = 0u;
    mbar_fence_init();
  }
  __syncthreads();
  const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, limit_ns);
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || abort_flag != 0u)) atomicCAS(status, 0, EGTP_ERR_DEVICE_TIMEOUT);
}

}  // namespace

cudaError_t launch_wait_timeout_selftest(uint64_t limit_ns, int32_t* status, cudaStream_t stream) {
  wait_timeout_selftest_kernel<<<1, 64, 0, stream>>>(limit_ns, status);
  return cudaGetLastError();
}

}  // namespace egtp
