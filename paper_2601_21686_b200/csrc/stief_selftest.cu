// stief_selftest_wait_limit: runs the library's bounded device-side waits to their limit, on purpose and
// harmlessly, so that the give-up branch every kernel relies on is exercised: the status word must say
// STIEF_ERR_TIMEOUT, the CTA's abort flag must cut every later wait short, and the kernel must end normally.
//
// One CTA of three warps.  Thread 0 initialises an mbarrier that expects one arrival which nobody ever makes.
//   warp 0: mbar_wait on it with the caller's small poll limit     -> gives up, raises the abort flag, reports
//   warp 1: mbar_wait_poll on it with the kernels' full limit      -> must return at its first look at the flag
//   warp 2: wait_count on a counter nobody increments, full limit  -> the same
// Nothing here can fault or wait without bound: every loop has its iteration limit, and the barrier is simply
// abandoned (an mbarrier is a shared-memory word; leaving a phase incomplete at kernel exit is legal).
#include "stief_common.cuh"

namespace stief {

__global__ void __launch_bounds__(96, 1) selftest_wait_kernel(int32_t* status, int32_t* rep, uint32_t limit) {
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ int abort_flag, counter;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t bar = smem_u32(&bar_storage);
  if (tid == 0) {
    mbar_init(bar, 1);
    mbar_fence_init();
    abort_flag = 0;
    counter = 0;
  }
  __syncthreads();
  volatile int* af = &abort_flag;
  if (warp == 0 && lane == 0) {
    const long long t0 = clock64();
    const bool ok = mbar_wait(bar, 0, af, status, limit);
    rep[0] = ok ? 1 : 0;                                   // 0: the wait gave up, as it must
    rep[1] = (int32_t)min((long long)0x7fffffff, clock64() - t0);
    rep[2] = *af;                                          // 1: the abort flag is up
  }
  __syncthreads();
  if (warp == 1 && lane == 0) {
    const long long t0 = clock64();
    const bool ok = mbar_wait_poll(bar, 0, af, status);    // full limit: only the abort flag can end it early
    rep[3] = ok ? 1 : 0;
    rep[4] = (int32_t)min((long long)0x7fffffff, clock64() - t0);
  }
  if (warp == 2 && lane == 0) {
    const long long t0 = clock64();
    const bool ok = wait_count(&counter, 1, af, status);   // full limit again
    rep[5] = ok ? 1 : 0;
    rep[6] = (int32_t)min((long long)0x7fffffff, clock64() - t0);
  }
  __syncthreads();
  if (tid == 0) rep[7] = 0x600d;                           // the kernel reached its normal end
}

}  // namespace stief

extern "C" int stief_selftest_wait_limit(int32_t* status, int32_t* report, int32_t poll_limit, void* stream) {
  if (!status || !report || poll_limit < 1 || poll_limit > (1 << 20)) return STIEF_ERR_INVALID_ARG;
  stief::selftest_wait_kernel<<<1, 96, 0, static_cast<cudaStream_t>(stream)>>>(status, report, (uint32_t)poll_limit);
  return cudaGetLastError() == cudaSuccess ? STIEF_OK : STIEF_ERR_CUDA;
}
