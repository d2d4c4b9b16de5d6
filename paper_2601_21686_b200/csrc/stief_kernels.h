// Internal interface between the C-ABI layer (stief_api.cu) and the kernel translation units.
#pragma once

#include "stief_decode_args.h"

namespace stief {

struct AppendArgs {
  LayerDev L;
  BatchDev Bt;
  const __nv_bfloat16* k_new;   // [B][Hkv][128]
  const __nv_bfloat16* v_new;
  int32_t* status;
};

struct AppendChunkArgs {
  LayerDev L;
  BatchDev Bt;
  const __nv_bfloat16* K;       // [B][T_chunk][Hkv][128 or r_k]
  const __nv_bfloat16* V;
  long long k_stride_b, k_stride_t, v_stride_b, v_stride_t;   // elements
  int T_chunk;
  const int32_t* chunk_lens;    // [B] or NULL = T_chunk
  int ends_at_len;              // 1: the chunk's last row is position seq_lens[b] - 1; 0: its first row is position seq_lens[b]
  int32_t* status;
};

struct CombineArgs {
  LayerDev L;
  BatchDev Bt;
  const float* partial_o;
  const float* partial_lse;
  int n_cta, QT, len_add;
  __nv_bfloat16* out;           // [B][Hq][128]
  float* out_lse;               // [B][Hq] or NULL
};

struct PrefillArgs {
  LayerDev L;
  BatchDev Bt;
  const __nv_bfloat16* K;
  const __nv_bfloat16* V;
  long long stride_b, stride_t;       // element strides of K between sequences / tokens
  long long v_stride_b, v_stride_t;   // the same for V
  int T_max;
  int32_t* status;
  bool overlap_previous;        // launch with programmatic stream serialization
};

struct DecodeLaunch {
  DecodeArgs args;
  int n_cta;
  bool overlap_previous;        // launch with programmatic stream serialization
};

cudaError_t launch_append(const AppendArgs& a, cudaStream_t st);
cudaError_t launch_append_chunk(const AppendChunkArgs& a, cudaStream_t st);
cudaError_t launch_combine(const CombineArgs& a, cudaStream_t st);
cudaError_t launch_advance(int32_t* seq_lens, int B, int delta, cudaStream_t st);
cudaError_t launch_prefill(const PrefillArgs& a, cudaStream_t st);
// The same projection with the quantising epilogue, 8-bit or 4-bit codes (both bases required; a.L's bf16 pools are unused).
cudaError_t launch_prefill_quant(const PrefillArgs& a, int bits, uint8_t* k_codes, uint8_t* v_codes, float* v_params,
                                 const float* k_params, cudaStream_t st);

// Returns cudaErrorInvalidValue for a rank pair that is not compiled in.
cudaError_t launch_decode(const DecodeLaunch& a, const CUtensorMap& tmK, const CUtensorMap& tmV, cudaStream_t st);
// Encodes a tiled bf16 tensor map (rank <= 5; dims/box in elements, strides in bytes for dims 1..rank-1) with the
// given swizzle.  Returns false when the driver entry point is missing or refuses the arguments.
bool encode_bf16_map(CUtensorMap* tm, const void* base, int rank, const unsigned long long* dims,
                     const unsigned long long* strides_bytes, const unsigned* box, CUtensorMapSwizzle swizzle);
// The same for a tensor of bytes.
bool encode_u8_map(CUtensorMap* tm, const void* base, int rank, const unsigned long long* dims,
                   const unsigned long long* strides_bytes, const unsigned* box, CUtensorMapSwizzle swizzle);
// Full-rank side of the prefill (no basis): the rows are copied to the pool unchanged.  side: 0 = keys, 1 = values.
cudaError_t launch_prefill_copy(const PrefillArgs& a, int side, cudaStream_t st);
// Shape of the TMA boxes the decode kernel expects for rank r (see Tile<R>).
int decode_swizzle_span(int r);
bool decode_tile_linear(int r);

}  // namespace stief
