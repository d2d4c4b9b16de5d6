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

// ---------------------------------------------------------------------------------------------------------------------
// stief_measure_read_stream: a read-only pass over a device buffer, for the roofline's context.  The usual denominator
// is a copy (which reads AND writes); the decode kernels only read.  This is their streaming skeleton with the
// arithmetic taken out: one persistent CTA per SM, four lanes of three 16 KiB stages each, every lane fed by its own
// producer warp with 1-D bulk async copies that complete on an mbarrier, a consumer warp per lane that only waits for a
// stage and hands it back.  Chunk i of the buffer goes to CTA i mod grid.  Nothing is written to global memory; every
// wait is bounded.
// ---------------------------------------------------------------------------------------------------------------------
namespace stief {

constexpr int kRsLanes = 4, kRsStages = 3, kRsChunk = 16384;

__global__ void __launch_bounds__(2 * kRsLanes * 32, 1) read_stream_kernel(const uint8_t* __restrict__ p, long long n_chunks, int32_t* status) {
  extern __shared__ uint8_t rs_smem[];
  __shared__ __align__(8) unsigned long long bars[2 * kRsLanes * kRsStages];
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t ring = (smem_u32(rs_smem) + 127u) & ~127u;
  auto full_bar = [&](int s) { return smem_u32(&bars[s]); };
  auto empty_bar = [&](int s) { return smem_u32(&bars[kRsLanes * kRsStages + s]); };
  if (tid == 0) {
    for (int s = 0; s < kRsLanes * kRsStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  volatile int* af = &abort_flag;
  const int pl = warp % kRsLanes;
  const bool producer = warp >= kRsLanes;
  if (lane != 0) return;
  // the CTA's chunks are c, c + grid, ...; its k-th chunk belongs to lane k % kRsLanes
  long long k = 0;
  for (long long i = blockIdx.x; i < n_chunks; i += gridDim.x, ++k) {
    if ((int)(k % kRsLanes) != pl) continue;
    const long long kw = k / kRsLanes;
    const int slot = pl * kRsStages + (int)(kw % kRsStages);
    const uint32_t phase = (uint32_t)((kw / kRsStages) & 1);
    if (producer) {
      if (kw >= kRsStages) mbar_wait(empty_bar(slot), phase ^ 1u, af, status);
      mbar_arrive_expect_tx(full_bar(slot), kRsChunk);
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(ring + slot * kRsChunk), "l"(reinterpret_cast<uint64_t>(p + i * kRsChunk)), "r"(kRsChunk), "r"(full_bar(slot))
                   : "memory");
    } else {
      mbar_wait(full_bar(slot), phase, af, status);
      mbar_arrive(empty_bar(slot));
    }
  }
}

}  // namespace stief

extern "C" int stief_measure_read_stream(const void* buffer, size_t bytes, int32_t* status, void* stream) {
  if (!buffer || bytes < (size_t)stief::kRsChunk || (reinterpret_cast<uintptr_t>(buffer) & 15u)) return STIEF_ERR_INVALID_ARG;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    sms = 148;
  }
  const int smem = stief::kRsLanes * stief::kRsStages * stief::kRsChunk + 128;
  static bool configured[64] = {};
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    if (cudaFuncSetAttribute(stief::read_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return STIEF_ERR_CUDA;
    configured[dev] = true;
  }
  stief::read_stream_kernel<<<sms, 2 * stief::kRsLanes * 32, smem, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint8_t*>(buffer), (long long)(bytes / stief::kRsChunk), status);
  return cudaGetLastError() == cudaSuccess ? STIEF_OK : STIEF_ERR_CUDA;
}
