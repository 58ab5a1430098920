// Kernels and entry points that exist only in the test library (see testing.h).
#ifdef SPECEXT_TESTING
#include "common.cuh"
#include "sm100.cuh"
#include "testing.h"

namespace {

// The waiting path of the attention kernels, exercised in isolation: a barrier that expects two
// arrivals gets one, so the phase never completes and the bounded wait has to give up.
__global__ void __launch_bounds__(32) wait_timeout_kernel(long long limit_cycles, int32_t* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    sm100::mbar_init(&bar, 2);
    sm100::fence_mbar_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) sm100::mbar_arrive(&bar);
  __syncwarp();
  const bool ok = sm100::mbar_wait(&bar, 0, &abort_flag, limit_cycles);
  if (!ok && threadIdx.x == 0) spx_raise(status, SPECEXT_ERR_TIMEOUT);
}

}  // namespace

extern "C" int specext_test_wait_timeout(int64_t limit_cycles, int32_t* device_status, void* cuda_stream) {
  if (!device_status || limit_cycles < 1 || limit_cycles > 4000000000ll) return SPECEXT_ERR_INVALID_ARG;
  wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>((long long)limit_cycles, device_status);
  if (cudaGetLastError() != cudaSuccess) return SPECEXT_ERR_CUDA;
  return SPECEXT_OK;
}
#endif  // SPECEXT_TESTING
