// Instantiations of the quantised decode kernel for one key rank (STIEF_RK) and one code width (STIEF_QBITS), given on
// the command line, and every value rank.  One translation unit per pair so the build parallelises.
#include "stief_decode_q.cuh"
#include "stief_kernels.h"

#if !defined(STIEF_RK) || !defined(STIEF_QBITS)
#error "compile with -DSTIEF_RK=<key rank> -DSTIEF_QBITS=<8 or 4>"
#endif

namespace stief {

template <int RK, int RV, int BITS>
static cudaError_t launch_one_q(const DecodeQArgs& a, int n_cta, bool overlap_previous, cudaStream_t st) {
  using C = DecodeQCfg<RK, RV, BITS>;
  auto kern = decode_q_kernel<RK, RV, BITS>;
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
  cfg.gridDim = dim3(n_cta);
  cfg.blockDim = dim3(C::THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap_previous ? 1 : 0;
  // Key codes: [tiles * 64 token rows][KROW bytes], one box per tile, in the form qtile_chunk<KROW> expects:
  //   16, 48 bytes: dense rows; 32: 32-byte swizzle; 64: 64-byte swizzle; 128: 128-byte swizzle;
  //   96: the tile as 192 lines of 32 bytes with the 32-byte swizzle on the linear offset.
  // Value codes: [tiles * RV channel rows][VROW bytes]: 64-byte rows with the 64-byte swizzle, 32-byte rows with the 32-byte one.
  constexpr int KROW = C::KROW, VROW = C::VROW;
  const unsigned long long tiles = (unsigned long long)a.L.num_pages * a.L.Hkv;
  CUtensorMap tmK, tmV;
  {
    constexpr bool linear = KROW == 96;
    const unsigned long long dims[2] = {(unsigned long long)(linear ? 32 : KROW), tiles * (linear ? 192 : kPage)};
    const unsigned long long strides[1] = {(unsigned long long)(linear ? 32 : KROW)};
    const unsigned box[2] = {(unsigned)(linear ? 32 : KROW), (unsigned)(linear ? 192 : kPage)};
    const CUtensorMapSwizzle sw = (KROW == 16 || KROW == 48) ? CU_TENSOR_MAP_SWIZZLE_NONE
                                  : (KROW == 32 || KROW == 96) ? CU_TENSOR_MAP_SWIZZLE_32B
                                  : KROW == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
    if (!encode_u8_map(&tmK, a.k_codes, 2, dims, strides, box, sw)) return cudaErrorInvalidValue;
  }
  {
    const unsigned long long dims[2] = {(unsigned long long)VROW, tiles * RV}, strides[1] = {(unsigned long long)VROW};
    const unsigned box[2] = {(unsigned)VROW, (unsigned)RV};
    if (!encode_u8_map(&tmV, a.v_codes, 2, dims, strides, box, VROW == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B))
      return cudaErrorInvalidValue;
  }
  return cudaLaunchKernelEx(&cfg, kern, tmK, tmV, a);
}

#define STIEF_CAT3_(a, b, c, d) a##b##c##d
#define STIEF_CAT3(a, b, c, d) STIEF_CAT3_(a, b, c, d)

cudaError_t STIEF_CAT3(launch_decode_q_rk, STIEF_RK, _b, STIEF_QBITS)(const DecodeQArgs& a, int n_cta, bool overlap_previous,
                                                                      cudaStream_t st) {
  switch (a.L.r_v) {
    case 32: return launch_one_q<STIEF_RK, 32, STIEF_QBITS>(a, n_cta, overlap_previous, st);
    case 48: return launch_one_q<STIEF_RK, 48, STIEF_QBITS>(a, n_cta, overlap_previous, st);
    case 64: return launch_one_q<STIEF_RK, 64, STIEF_QBITS>(a, n_cta, overlap_previous, st);
    case 96: return launch_one_q<STIEF_RK, 96, STIEF_QBITS>(a, n_cta, overlap_previous, st);
    case 128: return launch_one_q<STIEF_RK, 128, STIEF_QBITS>(a, n_cta, overlap_previous, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace stief
