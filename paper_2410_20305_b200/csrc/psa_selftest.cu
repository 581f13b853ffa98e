// Failure-detection self test and the host-side reading of the device status word.
// No counterpart in the paper.
//
// The attention kernels never wait without a limit: every mbarrier wait goes through
// dev::mbar_wait, which gives up after a number of SM clocks, raises a CTA-wide abort flag,
// ORs PSA_DEVSTAT_WAIT_EXPIRED into the caller's status word and lets the kernel run to its
// normal end.  psa_selftest_wait_expiry exercises exactly that code on a barrier that nothing
// completes, with a short limit, so that the expiry path can be tested without any fault.
#include <cuda_runtime.h>

#include "psa_device.cuh"
#include "psa_internal.h"

namespace psa {
namespace {

__global__ void __launch_bounds__(32)
psa_wait_expiry_kernel(int32_t* status, long long limit_clocks, long long* waited_out) {
  __shared__ __align__(8) unsigned long long barrier_word;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    dev::mbar_init(dev::smem_u32(&barrier_word), 1);   // one arrival expected; none will come
    dev::fence_mbar_init();
  }
  __syncwarp();
  const dev::WaitCtx ctx{&abort_flag, status, limit_clocks};
  if (threadIdx.x == 0) {
    const long long t0 = clock64();
    dev::mbar_wait(dev::smem_u32(&barrier_word), 0, ctx);   // expires: sets the flag and the status bit
    if (waited_out) *waited_out = clock64() - t0;
  }
  __syncwarp();
  // A second waiter of the same CTA sees the abort flag and returns at its first poll.
  if (threadIdx.x == 1) dev::mbar_wait(dev::smem_u32(&barrier_word), 0, ctx);
}

// One index inside and one outside a 4-element tensor through the checked-index macro.
__global__ void psa_bounds_selftest_kernel(int32_t* status, int32_t* result) {
  int32_t r = 0;
  if (PSA_IN_BOUNDS(3, 4, status)) r |= 1;    // accepted in both libraries
  if (PSA_IN_BOUNDS(4, 4, status)) r |= 2;    // accepted only where the macro is the constant true
  *result = r;
}

}  // namespace
}  // namespace psa

extern "C" psa_status_t psa_selftest_bounds(int32_t* device_status, int32_t* result, void* stream) {
  if (!device_status || !result) return PSA_ERR_INVALID_ARG;
  psa::psa_bounds_selftest_kernel<<<1, 1, 0, cudaStream_t(stream)>>>(device_status, result);
  return psa::check_last_cuda_error("psa_selftest_bounds launch");
}

extern "C" psa_status_t psa_selftest_wait_expiry(int32_t* device_status, int64_t limit_clocks, int64_t* spins_out,
                                                 void* stream) {
  if (!device_status) return PSA_ERR_INVALID_ARG;
  long long limit = limit_clocks;
  if (limit < 1000) limit = 1000;
  if (limit > psa::dev::kWaitLimitClocks) limit = psa::dev::kWaitLimitClocks;
  psa::psa_wait_expiry_kernel<<<1, 32, 0, cudaStream_t(stream)>>>(device_status, limit,
                                                                  reinterpret_cast<long long*>(spins_out));
  return psa::check_last_cuda_error("psa_selftest_wait_expiry launch");
}

extern "C" psa_status_t psa_check_device_status(int32_t word) {
  if (word == 0) return PSA_OK;
  if (word & PSA_DEVSTAT_WAIT_EXPIRED) return PSA_ERR_TIMEOUT;
  return PSA_ERR_DEVICE_STATUS;
}
