// Prefill compression (Eq. 1 for a whole prompt): X_down = rnd_bf16(X U) for X = K or V, written to
// the paged pool.  A streaming GEMM with tokens as M, the rank as N and d_h = 128 as K: every input
// row is read once from HBM (16-byte loads straight into MMA A-fragments), the basis sits in shared
// memory for the whole CTA, products run on the tensor cores (mma.sync m16n8k16, fp32 accumulate),
// and results leave through a per-warp shared-memory staging tile as fully coalesced 16-byte stores.
//
// grid = (token blocks of 512, Hkv, 2B): blockIdx.z & 1 selects keys or values.
#include "stief_kernels.h"

namespace stief {

constexpr int kPfThreads = 128;       // 4 warps x 32 tokens = 128 tokens per pass
constexpr int kPfTokens = 512;        // tokens per CTA (4 passes)

template <int R>
struct PfCfg {
  static constexpr int PITCH_U = (R <= 64) ? 128 : 256;          // bytes per basis row in smem (power of two)
  static constexpr int U_BYTES = kD * PITCH_U;
  static constexpr int PITCH_S = R * 2 + 16;                     // staging row pitch, bytes
  static constexpr int STAGE_BYTES = 32 * PITCH_S;               // per warp
  static constexpr int SMEM = U_BYTES + 4 * STAGE_BYTES;
};
constexpr int kPfSmemMax = PfCfg<128>::SMEM;

// 16-byte chunk swizzle of basis row d: distinct for the 8 rows {8a + e + const : a < 4, e < 2} one
// transposed ldmatrix tile touches
__device__ __forceinline__ int u_swz(int d) { return (((d >> 3) & 3) << 1) | (d & 1); }

template <int R>
__device__ __forceinline__ void prefill_body(uint8_t* smem, const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ U,
                                             __nv_bfloat16* __restrict__ pool, const PrefillArgs& a, int b, int h, int len) {
  using C = PfCfg<R>;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tid4 = lane & 3;
  const uint32_t ubase = smem_u32(smem);
  uint8_t* stage = smem + C::U_BYTES + warp * C::STAGE_BYTES;
  const uint32_t sbase = smem_u32(stage);

  // basis -> shared memory, chunk-swizzled
  for (int idx = tid; idx < kD * (R / 8); idx += kPfThreads) {
    const int d = idx / (R / 8), c = idx % (R / 8);
    const uint4 v = *reinterpret_cast<const uint4*>(U + (size_t)d * R + 8 * c);
    *reinterpret_cast<uint4*>(smem + d * C::PITCH_U + ((c ^ u_swz(d)) << 4)) = v;
  }
  __syncthreads();

  const __nv_bfloat16* Xb = X + (size_t)b * a.stride_b + (size_t)h * kD;

  for (int it = 0; it < kPfTokens / 128; ++it) {
    const int tb = blockIdx.x * kPfTokens + it * 128 + warp * 32;     // first token of this warp's 32
    if (tb >= len) break;                                              // warp-uniform
    const int pi = tb / kPage;
    int page = (pi < a.Bt.max_pages) ? a.Bt.block_table[(size_t)b * a.Bt.max_pages + pi] : -1;
    if (page < 0 || page >= a.L.num_pages) {
      if (lane == 0) report(a.status, STIEF_ERR_BOUNDS);
      continue;
    }
    const size_t rowbase = ((size_t)page * a.L.Hkv + h) * kPage + (tb % kPage);

    // A operands: xa[mt][half][q] = 8 consecutive d (32q + 8*tid4 ..) of token tb + 16mt + gid + 8half
    uint4 xa[2][2][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int t = tb + 16 * mt + gid + 8 * hf;
        const uint4* src = reinterpret_cast<const uint4*>(Xb + (size_t)t * a.stride_t + 8 * tid4);
#pragma unroll
        for (int q = 0; q < 4; ++q) xa[mt][hf][q] = (t < len) ? __ldg(src + 4 * q) : make_uint4(0u, 0u, 0u, 0u);
      }

#pragma unroll 1
    for (int np = 0; np < R / 16; ++np) {
      float acc[2][2][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) acc[mt][nt][0] = acc[mt][nt][1] = acc[mt][nt][2] = acc[mt][nt][3] = 0.f;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          // contraction slots of this step: (2c,2c+1) <-> d = 32q+8c+4e+{0,1}; (2c+8,2c+9) <-> +2
          const int mi = lane >> 3, rho = lane & 7;
          const int d = 32 * q + 8 * (rho >> 1) + 4 * e + 2 * (mi & 1) + (rho & 1);
          const int chunk = 2 * np + (mi >> 1);
          uint32_t r0, r1, r2, r3;
          ldsm_x4_t(ubase + d * C::PITCH_U + ((chunk ^ u_swz(d)) << 4), r0, r1, r2, r3);
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            const uint32_t* w0 = reinterpret_cast<const uint32_t*>(&xa[mt][0][q]);
            const uint32_t* w1 = reinterpret_cast<const uint32_t*>(&xa[mt][1][q]);
            const uint32_t af[4] = {w0[2 * e], w1[2 * e], w0[2 * e + 1], w1[2 * e + 1]};
            mma_bf16(acc[mt][0], af, r0, r1);
            mma_bf16(acc[mt][1], af, r2, r3);
          }
        }
      }
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const int col = 16 * np + 8 * nt + 2 * tid4;
          const int r = 16 * mt + gid;
          *reinterpret_cast<uint32_t*>(stage + r * C::PITCH_S + col * 2) = pack_bf16(acc[mt][nt][0], acc[mt][nt][1]);
          *reinterpret_cast<uint32_t*>(stage + (r + 8) * C::PITCH_S + col * 2) = pack_bf16(acc[mt][nt][2], acc[mt][nt][3]);
        }
    }
    __syncwarp();
    // staging -> pool: the warp's 32 rows are contiguous in the pool
    uint8_t* dst = reinterpret_cast<uint8_t*>(pool + rowbase * R);
    const int nvalid = min(32, len - tb);
    for (int idx = lane; idx < nvalid * (R / 8); idx += 32) {
      const int r = idx / (R / 8), c = idx % (R / 8);
      *reinterpret_cast<uint4*>(dst + (size_t)idx * 16) = *reinterpret_cast<const uint4*>(stage + r * C::PITCH_S + 16 * c);
    }
    __syncwarp();
  }
  (void)sbase;
}

// rows kept full rank (no basis): the cache stores the bf16 rows unchanged
__device__ void prefill_copy(const __nv_bfloat16* X, __nv_bfloat16* pool, const PrefillArgs& a, int b, int h, int len) {
  const int t0 = blockIdx.x * kPfTokens;
  const __nv_bfloat16* Xb = X + (size_t)b * a.stride_b + (size_t)h * kD;
  for (int idx = threadIdx.x; idx < kPfTokens * 16; idx += kPfThreads) {
    const int t = t0 + idx / 16, c = idx % 16;
    if (t >= len) break;
    const int pi = t / kPage;
    const int page = (pi < a.Bt.max_pages) ? a.Bt.block_table[(size_t)b * a.Bt.max_pages + pi] : -1;
    if (page < 0 || page >= a.L.num_pages) {
      report(a.status, STIEF_ERR_BOUNDS);
      continue;
    }
    const size_t row = ((size_t)page * a.L.Hkv + h) * kPage + (t % kPage);
    reinterpret_cast<uint4*>(pool + row * kD)[c] = __ldg(reinterpret_cast<const uint4*>(Xb + (size_t)t * a.stride_t) + c);
  }
}

__global__ void __launch_bounds__(kPfThreads, 3)
prefill_kernel(const PrefillArgs a) {
  extern __shared__ __align__(16) uint8_t pf_smem[];
  const int h = blockIdx.y, b = blockIdx.z >> 1, which = blockIdx.z & 1;
  int len = a.Bt.seq_lens[b];
  if (len > a.T_max) len = a.T_max;
  if ((int)blockIdx.x * kPfTokens >= len) return;
  const __nv_bfloat16* X = which ? a.V : a.K;
  const __nv_bfloat16* Ub = which ? a.L.U_v : a.L.U_k;
  const __nv_bfloat16* U = Ub ? Ub + (size_t)h * (which ? a.L.uv_stride : a.L.uk_stride) : nullptr;
  __nv_bfloat16* pool = which ? a.L.v_pool : a.L.k_pool;
  const int R = which ? a.L.r_v : a.L.r_k;
  if (U == nullptr) {
    prefill_copy(X, pool, a, b, h, len);
    return;
  }
  switch (R) {
    case 32: prefill_body<32>(pf_smem, X, U, pool, a, b, h, len); break;
    case 48: prefill_body<48>(pf_smem, X, U, pool, a, b, h, len); break;
    case 64: prefill_body<64>(pf_smem, X, U, pool, a, b, h, len); break;
    case 96: prefill_body<96>(pf_smem, X, U, pool, a, b, h, len); break;
    case 128: prefill_body<128>(pf_smem, X, U, pool, a, b, h, len); break;
    default: break;
  }
}

cudaError_t launch_prefill(const PrefillArgs& a, cudaStream_t st) {
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPfSmemMax);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  const int rmax = a.L.r_k > a.L.r_v ? a.L.r_k : a.L.r_v;
  const int smem = (rmax <= 64 ? kD * 128 : kD * 256) + 4 * 32 * (rmax * 2 + 16);
  dim3 grid((a.T_max + kPfTokens - 1) / kPfTokens, a.L.Hkv, 2 * a.Bt.B);
  prefill_kernel<<<grid, kPfThreads, smem, st>>>(a);
  return cudaGetLastError();
}

}  // namespace stief
