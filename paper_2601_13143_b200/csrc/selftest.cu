// Self-test of the bounded waits the tensor-core and bulk-copy kernels rely on: a block waits on an
// mbarrier that nothing will ever complete and must come back by itself with the error bit set.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace fastav {
namespace {

__global__ void __launch_bounds__(64) bounded_wait_selftest_kernel(unsigned long long limit_ns, int32_t* device_status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  // Phase 0 of `bar` never completes: every thread's wait has to give up (the first one to time out tells the rest).
  const bool completed = ptx::mbar_wait_bounded(ptx::smem_u32(&bar), 0, &abort_flag, limit_ns);
  if (!completed && threadIdx.x == 0 && device_status) atomicOr(device_status, FASTAV_DEV_WAIT_EXPIRED);
}

}  // namespace
}  // namespace fastav

extern "C" int32_t fastav_selftest_bounded_wait(int32_t limit_ms, int32_t* device_status, void* stream) {
  using namespace fastav;
  if (limit_ms < 1 || limit_ms > 1000) return FASTAV_ERR_INVALID_ARG;
  bounded_wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>((unsigned long long)limit_ms * 1000000ull, device_status);
  count_launches(1);
  return cudaGetLastError() == cudaSuccess ? FASTAV_OK : FASTAV_ERR_CUDA;
}
