// Self-test of the bounded-wait exit: the one path of the tensor-core kernels that a correct run never takes.
//
// Every mbarrier wait in those kernels gives up after a time limit, records a code in the device status word,
// raises a CTA-wide abort flag that makes every later wait return at once, and lets the kernel leave through its
// normal exit, so that a kernel that cannot make progress costs a second instead of the device.  Making that
// happen inside a GEMM would mean breaking its protocol with copies in flight; this kernel runs the SAME wait
// routine on a barrier nobody ever arrives at, with a limit of about a millisecond, and nothing else: no TMA, no
// TMEM, one CTA.  The host then sees what it would see after a real expiry.
#include "kernels.h"
#include "tc_common.cuh"

namespace mk {
namespace {

// out[0]: what the first waiter's wait returned (0 = gave up); out[1]: the same for a second warp whose wait
// started before the expiry; out[2], out[3]: cycles each of them spent; out[4]: what a wait returned that
// started after the expiry; out[5]: cycles it spent (the abort flag must end it at once)
__global__ void __launch_bounds__(64) bounded_wait_selftest_kernel(long long limit_cycles, unsigned int* status, long long* out) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);       // one arrival expected; nobody arrives
    abort_flag = 0;
    tc::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0 || threadIdx.x == 32) {
    const long long t0 = clock64();
    // the second warp's own limit is far away: it must be released by the first one's abort flag
    const bool ok = tc::mbar_wait_slow(&bar, 0, &abort_flag, status, tc::WAIT_SELFTEST,
                                       threadIdx.x == 0 ? limit_cycles : 1000 * limit_cycles);
    out[threadIdx.x == 0 ? 0 : 1] = ok ? 1 : 0;
    out[threadIdx.x == 0 ? 2 : 3] = clock64() - t0;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const long long t0 = clock64();
    const bool ok = tc::mbar_wait(&bar, 0, &abort_flag, status, tc::WAIT_SELFTEST);
    out[4] = ok ? 1 : 0;
    out[5] = clock64() - t0;
  }
}

}  // namespace
}  // namespace mk

namespace mk {
cudaError_t launch_bounded_wait_selftest(long long limit_cycles, long long* out6, cudaStream_t s) {
  unsigned int* status = kernel_status_ptr();
  if (!status) return cudaErrorInvalidSymbol;
  bounded_wait_selftest_kernel<<<1, 64, 0, s>>>(limit_cycles, status, out6);
  return cudaGetLastError();
}
}  // namespace mk
