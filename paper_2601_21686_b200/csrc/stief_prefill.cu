// Full-rank side of the prefill: a layer may keep keys or values uncompressed (Algorithm 2), in which case
// the cache stores the bf16 rows unchanged.  A plain paged copy; the projecting sides are handled by the
// tensor-core kernel in stief_prefill_tc.cu.
#include "stief_kernels.h"

namespace stief {

constexpr int kPfThreads = 128;
constexpr int kPfTokens = 512;        // tokens per CTA

// rows kept full rank (no basis): the cache stores the bf16 rows unchanged
__device__ void prefill_copy(const __nv_bfloat16* X, __nv_bfloat16* pool, const PrefillArgs& a, int b, int h, int len, int R,
                             long long stride_b, long long stride_t) {
  const int t0 = blockIdx.x * kPfTokens;
  const int cpr = R / 8;                                   // 16-byte pieces per row of R elements
  const __nv_bfloat16* Xb = X + (size_t)b * stride_b + (size_t)h * R;
  for (int idx = threadIdx.x; idx < kPfTokens * cpr; idx += kPfThreads) {
    const int t = t0 + idx / cpr, c = idx % cpr;
    if (t >= len) break;
    const int pi = t / kPage;
    const int page = (pi < a.Bt.max_pages) ? a.Bt.block_table[(size_t)b * a.Bt.max_pages + pi] : -1;
    if (page < 0 || page >= a.L.num_pages) {
      report(a.status, STIEF_ERR_BOUNDS);
      continue;
    }
    const size_t row = ((size_t)page * a.L.Hkv + h) * kPage + (t % kPage);
    reinterpret_cast<uint4*>(pool + row * R)[c] = __ldg(reinterpret_cast<const uint4*>(Xb + (size_t)t * stride_t) + c);
  }
}

__global__ void __launch_bounds__(kPfThreads)
prefill_copy_kernel(const PrefillArgs a, const int side) {
  const int h = blockIdx.y, b = blockIdx.z;
  int len = a.Bt.seq_lens[b];
  if (len > a.T_max) len = a.T_max;
  if ((int)blockIdx.x * kPfTokens >= len) return;
  if (side) prefill_copy(a.V, a.L.v_pool, a, b, h, len, a.L.r_v, a.v_stride_b, a.v_stride_t);
  else prefill_copy(a.K, a.L.k_pool, a, b, h, len, a.L.r_k, a.stride_b, a.stride_t);
}

cudaError_t launch_prefill_copy(const PrefillArgs& a, int side, cudaStream_t st) {
  dim3 grid((a.T_max + kPfTokens - 1) / kPfTokens, a.L.Hkv, a.Bt.B);
  prefill_copy_kernel<<<grid, kPfThreads, 0, st>>>(a, side);
  return cudaGetLastError();
}

}  // namespace stief
