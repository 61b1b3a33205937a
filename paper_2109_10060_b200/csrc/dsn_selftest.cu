// Self-test of the bounded device waits: a one-CTA kernel that waits, with the library's own wait
// routine, on a barrier that nothing ever arrives at.  The wait must run out after the context's limit,
// record DSN_ERR_TIMEOUT in the status word and let the kernel return, leaving the context usable.
// No fault, trap or endless loop is involved: the kernel always ends by itself.
#include "dsn_gemm_device.cuh"

namespace {
using namespace dsn_gemm;

__global__ void __launch_bounds__(32) selftest_wait_kernel(int32_t* status) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t abort_flag;
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);  // one arrival expected, none will come
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, &abort_flag, status, /*where=*/9001);
  __syncwarp();
}
}  // namespace

cudaError_t dsn_launch_selftest_wait(int32_t* status, cudaStream_t s) {
  return dsn_launch(selftest_wait_kernel, dim3(1), dim3(32), 0, s, 1, status);
}
