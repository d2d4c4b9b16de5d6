// Internal interface between the C-ABI layer (stief_api.cu) and the kernel translation units.
#pragma once

#include "stief_common.cuh"

namespace stief {

struct PreArgs {
  LayerDev L;
  BatchDev Bt;
  const __nv_bfloat16* q;       // [B][Hq][128] or NULL (append only)
  const __nv_bfloat16* k_new;   // [B][Hkv][128] or NULL (query projection only)
  const __nv_bfloat16* v_new;
  float* q_proj;                // [B][Hq][r_k]
  int32_t* status;
};

struct CombineArgs {
  LayerDev L;
  BatchDev Bt;
  const float* partial_o;
  const float* partial_lse;
  int S, chunk_pages, len_add;
  __nv_bfloat16* out;           // [B][Hq][128]
  float* out_lse;               // [B][Hq] or NULL
};

struct PrefillArgs {
  LayerDev L;
  BatchDev Bt;
  const __nv_bfloat16* K;
  const __nv_bfloat16* V;
  long long stride_b, stride_t;
  int T_max;
  int32_t* status;
};

struct DecodeLaunch {
  LayerDev L;
  BatchDev Bt;
  const float* q_proj;
  float* partial_o;
  float* partial_lse;
  int S, chunk_pages, len_add;
  int32_t* status;
};

cudaError_t launch_pre(const PreArgs& a, cudaStream_t st);
cudaError_t launch_combine(const CombineArgs& a, cudaStream_t st);
cudaError_t launch_advance(int32_t* seq_lens, int B, int delta, cudaStream_t st);
cudaError_t launch_prefill(const PrefillArgs& a, cudaStream_t st);

// Returns cudaErrorInvalidValue for a rank pair that is not compiled in.
cudaError_t launch_decode(const DecodeLaunch& a, const CUtensorMap& tmK, const CUtensorMap& tmV, cudaStream_t st);
// Box width (elements) of the TMA tiles the decode kernel expects for rank r.
int decode_box_width(int r);

}  // namespace stief
