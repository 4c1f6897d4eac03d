// Self-test of the bounded waits: a kernel whose only job is to let a wait run out and report it.
//
// The warp-specialised kernels never spin without a limit: mbar_wait_abortable gives up after a number of clock
// ticks, raises the CTA's abort flag, every other role's wait sees the flag and returns, all roles reach the common
// exit, and one thread writes BDLM_ERR_DEVICE_TIMEOUT into the device status word.  This file exercises exactly
// that chain -- the wait primitive with a short limit, the flag, a second role that leaves because of the flag, the
// status word and bdlm_get_device_status -- in a one-CTA kernel that holds no tensor memory and has no copy or MMA
// in flight, so that nothing is left half finished when the wait gives up.
#include "tc_common.cuh"
#include "tc_launch.h"

namespace bdlm {
namespace {

using namespace tc;

__global__ void __launch_bounds__(64, 1)
wait_timeout_selftest_kernel(long long limit_ticks, int* __restrict__ status) {
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ int abort_word;
  const uint32_t bar = smem_u32(&bar_storage);
  volatile int* abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);      // one arrival expected; nobody arrives
    abort_word = 0;
    fence_mbar_init();
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5;
  if (warp == 0) (void)mbar_wait_abortable(bar, 0, abort_flag, limit_ticks);   // runs out, raises the flag
  else (void)mbar_wait_abortable(bar, 0, abort_flag);                          // leaves when it sees the flag
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, (int)BDLM_ERR_DEVICE_TIMEOUT);
}

}  // namespace
}  // namespace bdlm

extern "C" int bdlm_selftest_wait_timeout(int64_t limit_ticks, void* cuda_stream) {
  if (limit_ticks < 1 || limit_ticks > (int64_t)bdlm::tc::WAIT_LIMIT_TICKS) return BDLM_ERR_INVALID_ARG;
  int* status = bdlm::device_status_ptr();
  if (status == nullptr) return BDLM_ERR_CUDA;
  bdlm::wait_timeout_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(cuda_stream)>>>((long long)limit_ticks, status);
  return cudaGetLastError() == cudaSuccess ? BDLM_OK : BDLM_ERR_CUDA;
}
