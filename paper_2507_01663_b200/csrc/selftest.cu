// af_selftest_bounded_wait: shows, on the device, that a wait nothing will ever satisfy ends by
// itself.  Every mbarrier wait of the library goes through umma::mbar_wait, which gives up after a
// time limit, raises the CTA's abort flag and lets the kernel set AF_DEVERR_WATCHDOG and return.
// This kernel runs that same wait on a barrier no one arrives at, with a limit of one millisecond
// instead of the kernels' four seconds.  Nothing traps, faults or spins without bound.
#include "common.cuh"
#include "umma.cuh"

namespace af {
namespace {

__global__ void __launch_bounds__(32) bounded_wait_kernel(unsigned int* d_err, unsigned long long limit_ns,
                                                          unsigned int* waited_us) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    umma::mbar_init(umma::smem_u32(&bar), 1);
    umma::fence_mbar_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    const unsigned long long t0 = umma::globaltimer_ns();
    const bool arrived = umma::mbar_wait(umma::smem_u32(&bar), 0u, &abort_flag, limit_ns);   // phase 0 never completes
    *waited_us = (unsigned int)((umma::globaltimer_ns() - t0) / 1000ull);
    if (!arrived && abort_flag) atomicOr(d_err, umma::kWatchdogBit);
  }
}

}  // namespace

cudaError_t launch_bounded_wait_selftest(unsigned int* d_err, unsigned int* waited_us, cudaStream_t s) {
  bounded_wait_kernel<<<1, 32, 0, s>>>(d_err, 1000000ull, waited_us);
  return cudaGetLastError();
}

}  // namespace af
