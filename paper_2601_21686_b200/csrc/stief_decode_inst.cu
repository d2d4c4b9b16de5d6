// Instantiations of the persistent decode kernel for one key rank (STIEF_RK, given on the command
// line) and every supported value rank.  Compiled once per key rank so the build parallelises.
#include "stief_decode.cuh"
#include "stief_kernels.h"

#ifndef STIEF_RK
#error "compile with -DSTIEF_RK=<key rank>"
#endif

namespace stief {

template <int RK, int RV>
static cudaError_t launch_one(const DecodeLaunch& a, const CUtensorMap& tmK, const CUtensorMap& tmV, cudaStream_t st) {
  using C = DecodeCfg<RK, RV>;
  auto kern = decode_persistent_kernel<RK, RV>;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    // Every rank pair asks for the same (largest) shared-memory carve-out, whatever its ring needs: a kernel whose
    // carve-out differs from its predecessor's cannot enter an SM before that SM has drained and been reconfigured,
    // which undoes the overlap of consecutive layers when their ranks differ.
    e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.n_cta);
  cfg.blockDim = dim3(C::THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.overlap_previous ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, tmK, tmV, a.args);
}

#define STIEF_CAT_(a, b) a##b
#define STIEF_CAT(a, b) STIEF_CAT_(a, b)

cudaError_t STIEF_CAT(launch_decode_rk, STIEF_RK)(const DecodeLaunch& a, const CUtensorMap& tmK, const CUtensorMap& tmV,
                                                  cudaStream_t st) {
  switch (a.args.L.r_v) {
    case 32: return launch_one<STIEF_RK, 32>(a, tmK, tmV, st);
    case 48: return launch_one<STIEF_RK, 48>(a, tmK, tmV, st);
    case 64: return launch_one<STIEF_RK, 64>(a, tmK, tmV, st);
    case 96: return launch_one<STIEF_RK, 96>(a, tmK, tmV, st);
    case 128: return launch_one<STIEF_RK, 128>(a, tmK, tmV, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace stief
