// The latency-bound ends of a decode step:
//   pre_kernel      -- per (sequence, KV head): projects the group's queries (q' = q U_k, scaled) into
//                      the workspace and, when asked, projects the new token's k, v and stores the
//                      rows in the paged cache (Eq. 1 for one token).
//   combine_kernel  -- per (sequence, KV head): log-sum-exp merge of the chunk partials of every
//                      query head of the group, then the back-projection o = o_down U_v^T (Eq. 7).
//   advance_kernel  -- seq_lens += delta.
#include "stief_kernels.h"

namespace stief {

// ---------------------------------------------------------------------------------------------
// pre_kernel
// ---------------------------------------------------------------------------------------------
constexpr int kPreThreads = 256;          // 8 warps, warp w contracts d in [16w, 16w+16)
constexpr int kRowTile = 8;               // rows (vectors to project) handled per pass

// out[r][j] = sum_d rows[r][d] * U[d][j] for r < nrows (<= kRowTile), j < R.  rows: shared fp32
// [kRowTile][128]; red: shared fp32 [8 warps][kRowTile][128]; result left in red[0][r][j].
__device__ void project_rows(const float* rows, int nrows, const __nv_bfloat16* U, int R, float* red) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int cp = lane; cp < R / 2; cp += 32) {
    float acc[kRowTile][2];
#pragma unroll
    for (int r = 0; r < kRowTile; ++r) acc[r][0] = acc[r][1] = 0.f;
    uint32_t u[16];
#pragma unroll
    for (int dd = 0; dd < 16; ++dd)
      u[dd] = *reinterpret_cast<const uint32_t*>(U + (size_t)(16 * warp + dd) * R + 2 * cp);
#pragma unroll
    for (int dd = 0; dd < 16; ++dd) {
      const float u0 = bf16_lo(u[dd]), u1 = bf16_hi(u[dd]);
#pragma unroll
      for (int r = 0; r < kRowTile; ++r) {
        const float x = rows[r * kD + 16 * warp + dd];
        acc[r][0] = fmaf(x, u0, acc[r][0]);
        acc[r][1] = fmaf(x, u1, acc[r][1]);
      }
    }
#pragma unroll
    for (int r = 0; r < kRowTile; ++r) {
      if (r < nrows) *reinterpret_cast<float2*>(red + ((warp * kRowTile + r) * kD) + 2 * cp) = make_float2(acc[r][0], acc[r][1]);
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < nrows * R; idx += kPreThreads) {
    const int r = idx / R, j = idx % R;
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += red[(w * kRowTile + r) * kD + j];
    red[r * kD + j] = s;       // warp-0 slot of (r, j): read above by this thread only
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kPreThreads)
pre_kernel(const PreArgs a) {
  __shared__ float rows[kRowTile * kD];
  __shared__ float red[8 * kRowTile * kD];
  const int h = blockIdx.x, b = blockIdx.y;
  const int G = a.L.G, RK = a.L.r_k, RV = a.L.r_v;
  const float qscale = kLog2e * 0.08838834764831845f;    // log2(e) / sqrt(128)
  const __nv_bfloat16* Uk = a.L.U_k ? a.L.U_k + (size_t)h * a.L.uk_stride : nullptr;
  const __nv_bfloat16* Uv = a.L.U_v ? a.L.U_v + (size_t)h * a.L.uv_stride : nullptr;

  // where the new token goes
  bool do_append = a.k_new != nullptr;
  size_t row_index = 0;                                  // (page*Hkv + h)*64 + pos%64
  if (do_append) {
    const int pos = a.Bt.seq_lens[b];
    const int pi = pos / kPage;
    int page = -1;
    if (pos >= 0 && pi < a.Bt.max_pages) page = a.Bt.block_table[(size_t)b * a.Bt.max_pages + pi];
    if (page < 0 || page >= a.L.num_pages) {
      if (threadIdx.x == 0) report(a.status, STIEF_ERR_BOUNDS);
      do_append = false;
    } else {
      row_index = ((size_t)page * a.L.Hkv + h) * kPage + (pos % kPage);
    }
  }

  // vectors contracted with U_k: the group's queries, then the new key
  const int nq = a.q ? G : 0;
  const int nk = nq + (do_append ? 1 : 0);
  for (int r0 = 0; r0 < nk; r0 += kRowTile) {
    const int nr = min(kRowTile, nk - r0);
    __syncthreads();
    for (int idx = threadIdx.x; idx < kRowTile * kD; idx += kPreThreads) {
      const int r = idx / kD, d = idx % kD;
      float x = 0.f;
      if (r < nr) {
        const int v = r0 + r;
        x = __bfloat162float(v < nq ? a.q[((size_t)b * a.L.Hq + (size_t)h * G + v) * kD + d]
                                    : a.k_new[((size_t)b * a.L.Hkv + h) * kD + d]);
      }
      rows[idx] = x;
    }
    __syncthreads();
    const float* res = rows;                             // identity basis: the vector itself
    if (Uk) {
      project_rows(rows, nr, Uk, RK, red);
      res = red;
    }
    for (int idx = threadIdx.x; idx < nr * RK; idx += kPreThreads) {
      const int r = idx / RK, j = idx % RK, v = r0 + r;
      const float x = res[r * kD + j];
      if (v < nq) a.q_proj[((size_t)b * a.L.Hq + (size_t)h * G + v) * RK + j] = x * qscale;
      else a.L.k_pool[row_index * RK + j] = __float2bfloat16_rn(x);
    }
  }
  if (do_append) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < kRowTile * kD; idx += kPreThreads)
      rows[idx] = idx < kD ? __bfloat162float(a.v_new[((size_t)b * a.L.Hkv + h) * kD + idx]) : 0.f;
    __syncthreads();
    const float* res = rows;
    if (Uv) {
      project_rows(rows, 1, Uv, RV, red);
      res = red;
    }
    for (int j = threadIdx.x; j < RV; j += kPreThreads) a.L.v_pool[row_index * RV + j] = __float2bfloat16_rn(res[j]);
  }
}

// ---------------------------------------------------------------------------------------------
// combine_kernel
// ---------------------------------------------------------------------------------------------
constexpr int kCombThreads = 128;

__global__ void __launch_bounds__(kCombThreads)
combine_kernel(const CombineArgs a) {
  __shared__ float od[kRowTile * kD];                    // merged o_down of up to 8 heads, [r][RV]
  const int h = blockIdx.x, b = blockIdx.y;
  const int G = a.L.G, RV = a.L.r_v, S = a.S;
  const int tid = threadIdx.x;
  int len = a.Bt.seq_lens[b] + a.len_add;
  if (len < 0) len = 0;
  int npages = (len + kPage - 1) / kPage;
  if (npages > a.Bt.max_pages) npages = a.Bt.max_pages;
  const int live = min(S, (npages + a.chunk_pages - 1) / a.chunk_pages);   // chunks that hold tokens
  const __nv_bfloat16* Uv = a.L.U_v ? a.L.U_v + (size_t)h * a.L.uv_stride : nullptr;

  for (int g0 = 0; g0 < G; g0 += kRowTile) {
    const int ng = min(kRowTile, G - g0);
    __syncthreads();
    // ---- merge: thread j handles column j of every head of the tile
    for (int idx = tid; idx < ng * RV; idx += kCombThreads) {
      const int r = idx / RV, j = idx % RV;
      const size_t row = ((size_t)b * a.L.Hq + (size_t)h * G + g0 + r) * S;
      float M = -INFINITY;
      for (int s = 0; s < live; ++s) M = fmaxf(M, a.partial_lse[row + s]);
      float num = 0.f, den = 0.f;
      for (int s = 0; s < live; ++s) {
        const float w = __expf(a.partial_lse[row + s] - M);
        num = fmaf(w, a.partial_o[(row + s) * RV + j], num);
        den += w;
      }
      od[r * kD + j] = live > 0 ? num / den : 0.f;
      if (j == 0 && a.out_lse) a.out_lse[(size_t)b * a.L.Hq + (size_t)h * G + g0 + r] = live > 0 ? M + __logf(den) : -INFINITY;
    }
    __syncthreads();
    // ---- back-projection: thread dd owns output coordinate dd; row dd of U_v is read once for all heads
    const int dd = tid;
    float acc[kRowTile];
#pragma unroll
    for (int r = 0; r < kRowTile; ++r) acc[r] = 0.f;
    if (Uv) {
      const uint4* urow = reinterpret_cast<const uint4*>(Uv + (size_t)dd * RV);
      for (int c = 0; c < RV / 8; ++c) {
        const uint4 u = urow[c];
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float u0 = bf16_lo(w[e]), u1 = bf16_hi(w[e]);
#pragma unroll
          for (int r = 0; r < kRowTile; ++r) {
            acc[r] = fmaf(od[r * kD + 8 * c + 2 * e], u0, acc[r]);
            acc[r] = fmaf(od[r * kD + 8 * c + 2 * e + 1], u1, acc[r]);
          }
        }
      }
    } else {
#pragma unroll
      for (int r = 0; r < kRowTile; ++r) acc[r] = od[r * kD + dd];
    }
#pragma unroll
    for (int r = 0; r < kRowTile; ++r)
      if (r < ng) a.out[((size_t)b * a.L.Hq + (size_t)h * G + g0 + r) * kD + dd] = __float2bfloat16_rn(acc[r]);
  }
}

__global__ void advance_kernel(int32_t* seq_lens, int B, int delta) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < B) seq_lens[i] += delta;
}

// ---------------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------------
cudaError_t launch_pre(const PreArgs& a, cudaStream_t st) {
  pre_kernel<<<dim3(a.L.Hkv, a.Bt.B), kPreThreads, 0, st>>>(a);
  return cudaGetLastError();
}
cudaError_t launch_combine(const CombineArgs& a, cudaStream_t st) {
  combine_kernel<<<dim3(a.L.Hkv, a.Bt.B), kCombThreads, 0, st>>>(a);
  return cudaGetLastError();
}
cudaError_t launch_advance(int32_t* seq_lens, int B, int delta, cudaStream_t st) {
  advance_kernel<<<(B + 127) / 128, 128, 0, st>>>(seq_lens, B, delta);
  return cudaGetLastError();
}

}  // namespace stief
