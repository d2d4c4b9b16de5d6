// stief_mq_attention: argument checks, tensor maps and launch shape of the multi-query attention kernel
// (the kernel itself is in stief_mq.cuh, instantiated per rank pair in stief_mq_inst.cu).
#include <cstring>

#include "stief_host_util.h"
#include "stief_mq.cuh"

namespace stief {
namespace {

CUtensorMapSwizzle swizzle_of(int span) {
  return span == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : span == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
}

bool rank_ok(int r) { return r == 32 || r == 48 || r == 64 || r == 96 || r == 128; }

}  // namespace
}  // namespace stief

using namespace stief;

namespace stief {
cudaError_t launch_mq_combine(const mq::Args& a, cudaStream_t st) {
  mq::mq_combine_kernel<0><<<dim3(a.n_q, a.L.Hkv, a.Bt.B), mq::kCombineThreads, 0, st>>>(a);
  return cudaGetLastError();
}
}  // namespace stief

extern "C" int32_t stief_mq_num_splits(int32_t B, int32_t n_q, int32_t Hq, int32_t Hkv, int32_t max_pages_per_seq) {
  if (B <= 0 || n_q <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || max_pages_per_seq <= 0) return 0;
  const int G = Hq / Hkv;
  if (G > mq::kRows || mq::kRows % G != 0) return 0;
  const int TT = mq::kRows / G;
  const long long base = (long long)((n_q + 2 * TT - 1) / (2 * TT)) * B * Hkv;      // units without splitting
  long long s = host::sm_count() / base;                                           // parts so that the units about fill the GPU
  if (s > 32) s = 32;
  if (s > max_pages_per_seq / 4) s = max_pages_per_seq / 4;                        // at least a few pages per part
  return (int32_t)(s < 1 ? 1 : s);
}

extern "C" size_t stief_mq_workspace_bytes(int32_t B, int32_t n_q, int32_t Hq, int32_t r_v, int32_t num_splits) {
  if (B <= 0 || n_q <= 0 || Hq <= 0 || r_v <= 0 || num_splits < 1) return 0;
  if (num_splits == 1) return 0;
  // two result slots per part: with few query rows a CTA runs two softmax streams over alternate pages of its part
  return host::align_up((size_t)B * n_q * Hq * 2 * num_splits * (r_v + 2) * sizeof(float), 128);
}

extern "C" int stief_mq_attention(const stief_layer* layer, const stief_batch* batch, const uint16_t* q, int64_t q_stride_b,
                                  int64_t q_stride_t, int32_t n_q, const int32_t* q_lens, void* workspace,
                                  size_t workspace_bytes, int32_t num_splits, uint16_t* out, int64_t out_stride_b,
                                  int64_t out_stride_t, float* out_lse, uint32_t flags, int32_t* status, void* stream) {
  if (!layer || !q || !out || flags != 0u || num_splits < 1 || num_splits > 32) return STIEF_ERR_INVALID_ARG;
  if (num_splits > 1) {
    if (!workspace || !host::aligned(workspace, 128)) return STIEF_ERR_INVALID_ARG;
    if (workspace_bytes < stief_mq_workspace_bytes(batch ? batch->B : 0, n_q, layer->Hq, layer->r_v, num_splits) ||
        n_q > 65535 || (batch && batch->B > 65535))
      return STIEF_ERR_WORKSPACE;
  }
  const int rc = host::check_batch(batch);
  if (rc != STIEF_OK) return rc;
  if (layer->Hq <= 0 || layer->Hkv <= 0 || layer->Hq % layer->Hkv != 0 || layer->num_pages <= 0 || !layer->k_pool || !layer->v_pool ||
      n_q <= 0)
    return STIEF_ERR_INVALID_ARG;
  if (layer->d != kD || !rank_ok(layer->r_k) || !rank_ok(layer->r_v)) return STIEF_ERR_UNSUPPORTED;
  const int G = layer->Hq / layer->Hkv;
  if (G > mq::kRows || mq::kRows % G != 0) return STIEF_ERR_UNSUPPORTED;       // a tile holds whole tokens
  const int RK = layer->r_k, RV = layer->r_v;
  const bool fold_k = layer->U_k == nullptr, fold_v = layer->U_v == nullptr;
  const int dk = fold_k ? RK : kD, d_out = fold_v ? RV : kD;
  const long long q_row = (long long)layer->Hq * dk, o_row = (long long)layer->Hq * d_out;
  if (q_stride_t < q_row || q_stride_b < q_stride_t || q_stride_t % 8 || q_stride_b % 8 || out_stride_t < o_row ||
      out_stride_b < out_stride_t || out_stride_t % 8 || out_stride_b % 8)
    return STIEF_ERR_INVALID_ARG;
  if (!host::aligned(q, 16) || !host::aligned(out, 16) || !host::aligned(layer->k_pool, 128) || !host::aligned(layer->v_pool, 128) ||
      (layer->U_k && !host::aligned(layer->U_k, 16)) || (layer->U_v && !host::aligned(layer->U_v, 16)) ||
      layer->uk_head_stride % 8 || layer->uv_head_stride % 8 || layer->uk_head_stride < 0 || layer->uv_head_stride < 0)
    return STIEF_ERR_INVALID_ARG;
  // the kernels compute pool rows (page * Hkv + head) * 64 in int
  if ((long long)layer->num_pages * layer->Hkv * kPage >= (1ll << 31)) return STIEF_ERR_INVALID_ARG;

  const tc::Blocks bk = tc::blocks_of(RK), bv = tc::blocks_of(RV);
  const int TT = mq::kRows / G;
  mq::Launch L;
  memset(&L, 0, sizeof(L));
  CUtensorMap &tmQ = L.tmQ, &tmUk = L.tmUk, &tmUv = L.tmUv, &tmK = L.tmK, &tmV = L.tmV;
  {
    const unsigned long long dims[4] = {(unsigned long long)dk, (unsigned long long)layer->Hq, (unsigned long long)n_q, (unsigned long long)batch->B};
    const unsigned long long strides[3] = {(unsigned long long)dk * 2, (unsigned long long)q_stride_t * 2, (unsigned long long)q_stride_b * 2};
    const unsigned box[4] = {(unsigned)(fold_k ? bk.bw : 64), (unsigned)G, (unsigned)TT, 1u};
    if (!encode_bf16_map(&tmQ, q, 4, dims, strides, box, fold_k ? swizzle_of(bk.span) : CU_TENSOR_MAP_SWIZZLE_128B)) return STIEF_ERR_CUDA;
  }
  auto basis_map = [&](CUtensorMap* tm, const void* U, long long head_stride, int R, const tc::Blocks& b) {
    const unsigned long long nh = head_stride ? (unsigned long long)layer->Hkv : 1ull;
    const unsigned long long dims[3] = {(unsigned long long)R, (unsigned long long)kD, nh};
    const unsigned long long strides[2] = {(unsigned long long)R * 2, (unsigned long long)(head_stride ? head_stride : (long long)kD * R) * 2};
    const unsigned box[3] = {(unsigned)b.bw, (unsigned)kD, 1u};
    return encode_bf16_map(tm, U, 3, dims, strides, box, swizzle_of(b.span));
  };
  if (!fold_k && !basis_map(&tmUk, layer->U_k, layer->uk_head_stride, RK, bk)) return STIEF_ERR_CUDA;
  if (!fold_v && !basis_map(&tmUv, layer->U_v, layer->uv_head_stride, RV, bv)) return STIEF_ERR_CUDA;
  auto pool_map = [&](CUtensorMap* tm, const void* pool, int R, const tc::Blocks& b) {
    const unsigned long long dims[2] = {(unsigned long long)R, (unsigned long long)layer->num_pages * layer->Hkv * kPage};
    const unsigned long long strides[1] = {(unsigned long long)R * 2};
    const unsigned box[2] = {(unsigned)b.bw, (unsigned)kPage};
    return encode_bf16_map(tm, pool, 2, dims, strides, box, swizzle_of(b.span));
  };
  if (!pool_map(&tmK, layer->k_pool, RK, bk) || !pool_map(&tmV, layer->v_pool, RV, bv)) return STIEF_ERR_CUDA;

  mq::Args& a = L.a;
  a.L.Hq = layer->Hq; a.L.Hkv = layer->Hkv; a.L.G = G; a.L.r_k = RK; a.L.r_v = RV; a.L.num_pages = layer->num_pages;
  a.L.U_k = reinterpret_cast<const __nv_bfloat16*>(layer->U_k); a.L.uk_stride = layer->uk_head_stride;
  a.L.U_v = reinterpret_cast<const __nv_bfloat16*>(layer->U_v); a.L.uv_stride = layer->uv_head_stride;
  a.L.k_pool = reinterpret_cast<__nv_bfloat16*>(layer->k_pool); a.L.v_pool = reinterpret_cast<__nv_bfloat16*>(layer->v_pool);
  a.Bt = host::to_dev(batch);
  a.q_lens = q_lens;
  a.n_q = n_q;
  a.out = reinterpret_cast<__nv_bfloat16*>(out);
  a.out_stride_b = out_stride_b;
  a.out_stride_t = out_stride_t;
  a.out_lse = out_lse;
  a.status = status;
  a.n_split = num_splits;
  a.dual = (num_splits > 1 && (long long)n_q * G <= mq::kRows) ? 1 : 0;       // the second tile would have no rows of its own
  a.n_parts = num_splits * (1 + a.dual);
  a.part_o = static_cast<float*>(workspace);
  a.part_ml = a.part_o ? a.part_o + (size_t)batch->B * n_q * layer->Hq * a.n_parts * RV : nullptr;
  a.qp_bytes = mq::kRows * 2 * (fold_v ? RK : (RK > RV ? RK : RV));
  const int fixed = 1024 + 2 * a.qp_bytes + mq::kCtrlBytes;
  a.nst = (mq::kSmemLimit - fixed) / mq::kStageBytes;
  if (a.nst > mq::kMaxStages) a.nst = mq::kMaxStages;
  if (a.nst < 3) return STIEF_ERR_UNSUPPORTED;       // two query tiles and U_k are in the ring together
  L.smem = fixed + a.nst * mq::kStageBytes;
  const long long n_units = (long long)((n_q + 2 * TT - 1) / (2 * TT)) * batch->B * layer->Hkv * num_splits;
  L.grid = (int)(n_units < host::sm_count() ? n_units : host::sm_count());
  cudaError_t e = cudaErrorInvalidValue;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  switch (RK) {
    case 32: e = launch_mq_rk32(L, st); break;
    case 48: e = launch_mq_rk48(L, st); break;
    case 64: e = launch_mq_rk64(L, st); break;
    case 96: e = launch_mq_rk96(L, st); break;
    case 128: e = launch_mq_rk128(L, st); break;
  }
  if (e == cudaSuccess && num_splits > 1) e = launch_mq_combine(a, st);
  return e == cudaSuccess ? STIEF_OK : STIEF_ERR_CUDA;
}
