// The small stand-alone kernels of the library:
//   append_kernel   -- per (sequence, KV head): projects the new token's k, v and stores the rows in the
//                      paged cache (Eq. 1 for one token); used by stief_append (the decode step fuses
//                      the same work into its persistent kernel).
//   combine_kernel  -- per unit (sequence, KV head, query tile): log-sum-exp merge of the unit's segment
//                      partials, then the back-projection o = o_down U_v^T (Eq. 7); used by
//                      stief_split_combine (the decode kernel fuses the same work when given `out`).
//   advance_kernel  -- seq_lens += delta.
#include "stief_kernels.h"
#include "stief_partition.cuh"

namespace stief {

// ---------------------------------------------------------------------------------------------
// append_kernel
// ---------------------------------------------------------------------------------------------
constexpr int kAppThreads = 256;          // 8 warps, warp w contracts d in [16w, 16w+16)

// out[j] = sum_d x[d] * U[d][j], j < R.  x: shared fp32 [128]; red: shared fp32 [8 warps][128];
// result left in red[0][j].
__device__ void project_row(const float* x, const __nv_bfloat16* U, int R, float* red) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int cp = lane; cp < R / 2; cp += 32) {
    float a0 = 0.f, a1 = 0.f;
    uint32_t u[16];
#pragma unroll
    for (int dd = 0; dd < 16; ++dd) u[dd] = *reinterpret_cast<const uint32_t*>(U + (size_t)(16 * warp + dd) * R + 2 * cp);
#pragma unroll
    for (int dd = 0; dd < 16; ++dd) {
      const float xv = x[16 * warp + dd];
      a0 = fmaf(xv, bf16_lo(u[dd]), a0);
      a1 = fmaf(xv, bf16_hi(u[dd]), a1);
    }
    *reinterpret_cast<float2*>(red + warp * kD + 2 * cp) = make_float2(a0, a1);
  }
  __syncthreads();
  for (int j = threadIdx.x; j < R; j += kAppThreads) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += red[w * kD + j];
    red[j] = s;
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kAppThreads)
append_kernel(const AppendArgs a) {
  __shared__ float x[kD];
  __shared__ float red[8 * kD];
  const int h = blockIdx.x, b = blockIdx.y, which = blockIdx.z;     // which: 0 = key, 1 = value
  const int pos = a.Bt.seq_lens[b];
  const int pi = pos / kPage;
  int page = -1;
  if (pos >= 0 && pi < a.Bt.max_pages) page = a.Bt.block_table[(size_t)b * a.Bt.max_pages + pi];
  if (page < 0 || page >= a.L.num_pages) {
    if (threadIdx.x == 0) report(a.status, STIEF_ERR_BOUNDS);
    return;
  }
  const size_t row = ((size_t)page * a.L.Hkv + h) * kPage + (pos % kPage);
  const __nv_bfloat16* Ub = which ? a.L.U_v : a.L.U_k;
  const __nv_bfloat16* U = Ub ? Ub + (size_t)h * (which ? a.L.uv_stride : a.L.uk_stride) : nullptr;
  const int R = which ? a.L.r_v : a.L.r_k;
  const int d_in = U ? kD : R;                             // a side without a basis arrives in its own dimension
  const __nv_bfloat16* src = (which ? a.v_new : a.k_new) + ((size_t)b * a.L.Hkv + h) * d_in;
  __nv_bfloat16* dst = (which ? a.L.v_pool : a.L.k_pool) + row * R;
  if (threadIdx.x < d_in) x[threadIdx.x] = __bfloat162float(src[threadIdx.x]);
  __syncthreads();
  const float* res = x;                                    // no basis: the row is stored as it is
  if (U) {
    project_row(x, U, R, red);
    res = red;
  }
  for (int j = threadIdx.x; j < R; j += kAppThreads) dst[j] = __float2bfloat16_rn(res[j]);
}

// ---------------------------------------------------------------------------------------------
// append_chunk_kernel: the same projection for a run of new tokens per sequence (the cache-write half of chunked
// prefill).  A block takes kChunkTok consecutive tokens of one (sequence, KV head, side); the basis stays in L1
// across them.  The work is tiny next to the attention that follows (128 r MACs per row), so it stays on the FMA
// pipe with the accumulation order of the single-token kernel: a token appended alone or inside a chunk gets the
// same bits.
// ---------------------------------------------------------------------------------------------
constexpr int kChunkTok = 8;

__global__ void __launch_bounds__(kAppThreads)
append_chunk_kernel(const AppendChunkArgs a) {
  __shared__ float x[kD];
  __shared__ float red[8 * kD];
  const int h = blockIdx.x, tile = blockIdx.y, b = blockIdx.z >> 1, which = blockIdx.z & 1;
  int len = a.chunk_lens ? a.chunk_lens[b] : a.T_chunk;
  len = min(max(len, 0), a.T_chunk);
  const int t0 = tile * kChunkTok;
  if (t0 >= len) return;
  const int sl = a.Bt.seq_lens[b];
  const int pos0 = a.ends_at_len ? sl - len : sl;          // position of the chunk's row 0
  if (pos0 < 0 || sl < 0) {
    if (threadIdx.x == 0) report(a.status, STIEF_ERR_BOUNDS);
    return;
  }
  const __nv_bfloat16* Ub = which ? a.L.U_v : a.L.U_k;
  const __nv_bfloat16* U = Ub ? Ub + (size_t)h * (which ? a.L.uv_stride : a.L.uk_stride) : nullptr;
  const int R = which ? a.L.r_v : a.L.r_k;
  const int d_in = U ? kD : R;
  const __nv_bfloat16* X = which ? a.V : a.K;
  const long long sb = which ? a.v_stride_b : a.k_stride_b, stt = which ? a.v_stride_t : a.k_stride_t;
  for (int t = t0; t < min(t0 + kChunkTok, len); ++t) {
    const int pos = pos0 + t, pi = pos / kPage;
    int page = -1;
    if (pi < a.Bt.max_pages) page = a.Bt.block_table[(size_t)b * a.Bt.max_pages + pi];
    if (page < 0 || page >= a.L.num_pages) {              // uniform over the block
      if (threadIdx.x == 0) report(a.status, STIEF_ERR_BOUNDS);
      return;
    }
    const __nv_bfloat16* src = X + (size_t)b * sb + (size_t)t * stt + (size_t)h * d_in;
    __nv_bfloat16* dst = (which ? a.L.v_pool : a.L.k_pool) + (((size_t)page * a.L.Hkv + h) * kPage + (pos % kPage)) * R;
    __syncthreads();                                       // the previous token's results have been read
    if (threadIdx.x < d_in) x[threadIdx.x] = __bfloat162float(src[threadIdx.x]);
    __syncthreads();
    const float* res = x;
    if (U) {
      project_row(x, U, R, red);
      res = red;
    }
    for (int j = threadIdx.x; j < R; j += kAppThreads) dst[j] = __float2bfloat16_rn(res[j]);
  }
}

// ---------------------------------------------------------------------------------------------
// combine_kernel
// ---------------------------------------------------------------------------------------------
constexpr int kCombThreads = 128;

__global__ void __launch_bounds__(kCombThreads)
combine_kernel(const CombineArgs a) {
  __shared__ int pref[kMaxBatch + 1];
  __shared__ __align__(16) float od[kCombineScratchFloats];
  const int j = blockIdx.x, b = blockIdx.y;
  const int upb = a.L.Hkv * a.QT;
  const int pad = seg_pad_pages(a.L.r_k, a.L.r_v);
  build_page_prefix(pref, a.Bt, a.len_add, pad, nullptr);
  const int total = pref[a.Bt.B] * upb;
  const int P = pages_per_cta(total, a.n_cta);
  const int h = j / a.QT, qt = j % a.QT;
  int first = 0, nseg = 0;
  if (pref[b + 1] != pref[b]) {
    int last;
    unit_cta_span(pref, upb, pad, P, b, j, &first, &last);
    nseg = last - first + 1;
  }
  const int slot0 = first + b * upb + j;
  switch (a.L.r_v) {
    case 32: combine_unit<32>(a.L, b, h, qt, slot0, nseg, a.partial_o, a.partial_lse, a.out, a.out_lse, od, threadIdx.x, kCombThreads); break;
    case 48: combine_unit<48>(a.L, b, h, qt, slot0, nseg, a.partial_o, a.partial_lse, a.out, a.out_lse, od, threadIdx.x, kCombThreads); break;
    case 64: combine_unit<64>(a.L, b, h, qt, slot0, nseg, a.partial_o, a.partial_lse, a.out, a.out_lse, od, threadIdx.x, kCombThreads); break;
    case 96: combine_unit<96>(a.L, b, h, qt, slot0, nseg, a.partial_o, a.partial_lse, a.out, a.out_lse, od, threadIdx.x, kCombThreads); break;
    case 128: combine_unit<128>(a.L, b, h, qt, slot0, nseg, a.partial_o, a.partial_lse, a.out, a.out_lse, od, threadIdx.x, kCombThreads); break;
    default: break;
  }
}

__global__ void advance_kernel(int32_t* seq_lens, int B, int delta) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < B) seq_lens[i] += delta;
}

// ---------------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------------
cudaError_t launch_append(const AppendArgs& a, cudaStream_t st) {
  append_kernel<<<dim3(a.L.Hkv, a.Bt.B, 2), kAppThreads, 0, st>>>(a);
  return cudaGetLastError();
}
cudaError_t launch_append_chunk(const AppendChunkArgs& a, cudaStream_t st) {
  append_chunk_kernel<<<dim3(a.L.Hkv, (a.T_chunk + kChunkTok - 1) / kChunkTok, a.Bt.B * 2), kAppThreads, 0, st>>>(a);
  return cudaGetLastError();
}
cudaError_t launch_combine(const CombineArgs& a, cudaStream_t st) {
  combine_kernel<<<dim3(a.L.Hkv * a.QT, a.Bt.B), kCombThreads, 0, st>>>(a);
  return cudaGetLastError();
}
cudaError_t launch_advance(int32_t* seq_lens, int B, int delta, cudaStream_t st) {
  advance_kernel<<<(B + 127) / 128, 128, 0, st>>>(seq_lens, B, delta);
  return cudaGetLastError();
}

}  // namespace stief
