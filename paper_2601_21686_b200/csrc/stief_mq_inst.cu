// Instantiations of the multi-query attention kernel for one key rank (STIEF_RK, given on the command line) and
// every supported value rank.  Compiled once per key rank so the build parallelises.
#include "stief_mq.cuh"

#ifndef STIEF_RK
#error "compile with -DSTIEF_RK=<key rank>"
#endif

namespace stief {

template <int RK, int RV>
static cudaError_t launch_one(const mq::Launch& l, cudaStream_t st) {
  auto kern = mq::mq_attention_kernel<RK, RV>;
  static bool configured[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, mq::kSmemLimit);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  kern<<<l.grid, mq::kThreads, l.smem, st>>>(l.tmQ, l.tmUk, l.tmUv, l.tmK, l.tmV, l.a);
  return cudaGetLastError();
}

#define STIEF_CAT_(a, b) a##b
#define STIEF_CAT(a, b) STIEF_CAT_(a, b)

cudaError_t STIEF_CAT(launch_mq_rk, STIEF_RK)(const mq::Launch& l, cudaStream_t st) {
  switch (l.a.L.r_v) {
    case 32: return launch_one<STIEF_RK, 32>(l, st);
    case 48: return launch_one<STIEF_RK, 48>(l, st);
    case 64: return launch_one<STIEF_RK, 64>(l, st);
    case 96: return launch_one<STIEF_RK, 96>(l, st);
    case 128: return launch_one<STIEF_RK, 128>(l, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace stief
