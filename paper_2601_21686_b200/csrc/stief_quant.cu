// Integer-quantised compressed cache (paper Sec. 4.3), 8-bit and 4-bit codes, every rank: C-ABI entry points, the append
// kernel, and the dispatch to the quantised decode kernels (instantiated in stief_decode_q_inst.cu, one translation unit
// per key rank and code width).  The prefill projection with the quantising epilogue lives in stief_prefill_tc.cu.
#include "stief_decode_q.cuh"
#include "stief_host_util.h"

namespace stief {

// ---------------------------------------------------------------------------------------------
// append: project one new row per (sequence, KV head, side), quantise it, store codes (and value parameters)
// ---------------------------------------------------------------------------------------------
struct AppendQArgs {
  LayerDev L;
  BatchDev Bt;
  const __nv_bfloat16* k_new;   // [B][Hkv][128]
  const __nv_bfloat16* v_new;
  uint8_t* k_codes;
  uint8_t* v_codes;
  float* v_params;
  const float* k_params;
  int bits;
  int32_t* status;
};

constexpr int kAqThreads = 128;          // thread j owns output column j

__global__ void __launch_bounds__(kAqThreads)
append_q_kernel(const AppendQArgs a) {
  __shared__ float x[kD];
  __shared__ float gmin[2], gmax[2];
  __shared__ float wmin[4], wmax[4];
  __shared__ uint8_t codes[kD];
  const int h = blockIdx.x, b = blockIdx.y, side = blockIdx.z;       // side: 0 = key, 1 = value
  const int pos = a.Bt.seq_lens[b];
  const int pi = pos / kPage;
  int page = -1;
  if (pos >= 0 && pi < a.Bt.max_pages) page = a.Bt.block_table[(size_t)b * a.Bt.max_pages + pi];
  if (page < 0 || page >= a.L.num_pages) {
    if (threadIdx.x == 0) report(a.status, STIEF_ERR_BOUNDS);
    return;
  }
  const size_t row = ((size_t)page * a.L.Hkv + h) * kPage + (pos % kPage);
  const __nv_bfloat16* src = (side ? a.v_new : a.k_new) + ((size_t)b * a.L.Hkv + h) * kD;
  const __nv_bfloat16* U = (side ? a.L.U_v : a.L.U_k) + (size_t)h * (side ? a.L.uv_stride : a.L.uk_stride);
  const int R = side ? a.L.r_v : a.L.r_k, ng = (R + 63) >> 6;
  const int j = threadIdx.x;
  if (j < kD) x[j] = __bfloat162float(src[j]);
  __syncthreads();
  float acc = 0.f;
  if (j < R) {
#pragma unroll 8
    for (int d = 0; d < kD; ++d) acc = fmaf(x[d], __bfloat162float(U[(size_t)d * R + j]), acc);
  }
  const int g = j >> 6;
  const float levels = (float)((1 << a.bits) - 1);
  float sc, zp;
  if (side == 0) {
    sc = j < R ? a.k_params[((size_t)h * ng + g) * 2] : 1.f;
    zp = j < R ? a.k_params[((size_t)h * ng + g) * 2 + 1] : 0.f;
  } else {
    // token-wise group parameters: min and max over the group's columns (two warps per group of 64; columns at or
    // beyond the rank are neutral, so a short last group needs nothing special)
    float mn = j < R ? acc : INFINITY, mx = j < R ? acc : -INFINITY;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    if ((j & 31) == 0) {
      wmin[j >> 5] = mn;
      wmax[j >> 5] = mx;
    }
    __syncthreads();
    if (j < 2) {
      gmin[j] = fminf(wmin[2 * j], wmin[2 * j + 1]);
      gmax[j] = fmaxf(wmax[2 * j], wmax[2 * j + 1]);
    }
    __syncthreads();
    mn = gmin[g];
    mx = gmax[g];
    sc = mx > mn ? __fdiv_rn(mx - mn, levels) : 1.f;
    zp = mn;
    if (j < R && (j & 63) == 0) *reinterpret_cast<float2*>(a.v_params + (row * ng + g) * 2) = make_float2(sc, zp);
  }
  uint32_t code = 0;
  if (j < R) {
    const float y = __fmul_rn(__fsub_rn(acc, zp), __fdiv_rn(1.f, sc));
    code = (uint32_t)fminf(fmaxf(rintf(y), 0.f), levels);
  }
  const size_t tile = (size_t)page * a.L.Hkv + h;
  if (side == 0) {                                                     // [token][channel]
    const int krow = q_key_row_bytes(R, a.bits);
    if (j < kD) codes[j] = (uint8_t)code;
    __syncthreads();
    if (a.bits == 8) {
      if (j < R) a.k_codes[row * krow + j] = codes[j];
    } else if (j < krow) {
      const int lo = (j >> 4) * 32 + (j & 15), hi = lo + 16;
      a.k_codes[row * krow + j] = (uint8_t)((lo < R ? codes[lo] : 0) | ((hi < R ? codes[hi] : 0) << 4));
    }
  } else if (j < R) {                                                  // [channel][position]
    if (a.bits == 8) q_store_value_code<8>(a.v_codes + (tile * R + j) * 64, v_position(pos % kPage), code);
    else q_store_value_code<4>(a.v_codes + (tile * R + j) * 32, v_position(pos % kPage), code);
  }
}

// decode launchers, one per key rank and code width (stief_decode_q_inst.cu)
#define STIEF_DECL_Q(rk, bits) \
  cudaError_t launch_decode_q_rk##rk##_b##bits(const DecodeQArgs&, int n_cta, bool overlap_previous, cudaStream_t);
STIEF_DECL_Q(32, 8) STIEF_DECL_Q(48, 8) STIEF_DECL_Q(64, 8) STIEF_DECL_Q(96, 8) STIEF_DECL_Q(128, 8)
STIEF_DECL_Q(32, 4) STIEF_DECL_Q(48, 4) STIEF_DECL_Q(64, 4) STIEF_DECL_Q(96, 4) STIEF_DECL_Q(128, 4)
#undef STIEF_DECL_Q

static cudaError_t launch_decode_q(const DecodeQArgs& a, int bits, int n_cta, bool ov, cudaStream_t st) {
#define STIEF_CASE_Q(rk) \
  case rk: return bits == 8 ? launch_decode_q_rk##rk##_b8(a, n_cta, ov, st) : launch_decode_q_rk##rk##_b4(a, n_cta, ov, st);
  switch (a.L.r_k) {
    STIEF_CASE_Q(32) STIEF_CASE_Q(48) STIEF_CASE_Q(64) STIEF_CASE_Q(96) STIEF_CASE_Q(128)
    default: return cudaErrorInvalidValue;
  }
#undef STIEF_CASE_Q
}

namespace {

using namespace host;

bool q_rank_ok(int r) { return r == 32 || r == 48 || r == 64 || r == 96 || r == 128; }

int check_qlayer(const stief_qlayer* l) {
  if (!l) return STIEF_ERR_INVALID_ARG;
  if (l->Hq <= 0 || l->Hkv <= 0 || l->Hq % l->Hkv != 0 || l->num_pages <= 0) return STIEF_ERR_INVALID_ARG;
  if (l->d != kD) return STIEF_ERR_UNSUPPORTED;
  if (!q_rank_ok(l->r_k) || !q_rank_ok(l->r_v)) return STIEF_ERR_UNSUPPORTED;
  if (!l->U_k || !l->U_v) return STIEF_ERR_UNSUPPORTED;                  // folded sides are not taken by the quantised path
  if (!aligned(l->U_k, 128) || !aligned(l->U_v, 128)) return STIEF_ERR_INVALID_ARG;
  if (!l->k_codes || !l->v_codes || !l->v_params || !l->k_params) return STIEF_ERR_INVALID_ARG;
  if (!aligned(l->k_codes, 128) || !aligned(l->v_codes, 128) || !aligned(l->v_params, 128) || !aligned(l->k_params, 8))
    return STIEF_ERR_INVALID_ARG;
  if (l->uk_head_stride < 0 || l->uv_head_stride < 0 || (l->uk_head_stride % 64) != 0 || (l->uv_head_stride % 64) != 0)
    return STIEF_ERR_INVALID_ARG;
  if ((long long)l->num_pages * l->Hkv * 192 >= (1ll << 31)) return STIEF_ERR_INVALID_ARG;    // TMA row coordinates stay in int
  return STIEF_OK;
}

LayerDev qlayer_to_dev(const stief_qlayer* l) {
  LayerDev d;
  d.Hq = l->Hq; d.Hkv = l->Hkv; d.G = l->Hq / l->Hkv; d.r_k = l->r_k; d.r_v = l->r_v; d.num_pages = l->num_pages;
  d.U_k = reinterpret_cast<const __nv_bfloat16*>(l->U_k); d.uk_stride = l->uk_head_stride;
  d.U_v = reinterpret_cast<const __nv_bfloat16*>(l->U_v); d.uv_stride = l->uv_head_stride;
  d.k_pool = nullptr; d.v_pool = nullptr;
  return d;
}

int run_q_prefill(int bits, const stief_qlayer* layer, const stief_batch* batch, const uint16_t* K, const uint16_t* V,
                  int64_t stride_b, int64_t stride_t, int32_t T_max, uint32_t flags, int32_t* status, void* stream) {
  if (flags & ~STIEF_PREFILL_OVERLAP_PREVIOUS) return STIEF_ERR_INVALID_ARG;
  int rc = check_qlayer(layer);
  if (rc) return rc;
  rc = check_batch(batch);
  if (rc) return rc;
  if (!K || !V || !aligned(K, 16) || !aligned(V, 16)) return STIEF_ERR_INVALID_ARG;
  if (T_max <= 0 || stride_t < (int64_t)layer->Hkv * kD || stride_b < 0 || (stride_t % 8) != 0 || (stride_b % 8) != 0)
    return STIEF_ERR_INVALID_ARG;
  if (batch->B > 1 && stride_b == 0) return STIEF_ERR_INVALID_ARG;
  PrefillArgs a;
  a.L = qlayer_to_dev(layer);
  a.Bt = to_dev(batch);
  a.K = reinterpret_cast<const __nv_bfloat16*>(K);
  a.V = reinterpret_cast<const __nv_bfloat16*>(V);
  a.stride_b = stride_b; a.stride_t = stride_t; a.v_stride_b = stride_b; a.v_stride_t = stride_t;
  a.T_max = T_max; a.status = status;
  a.overlap_previous = (flags & STIEF_PREFILL_OVERLAP_PREVIOUS) != 0;
  return launch_prefill_quant(a, bits, layer->k_codes, layer->v_codes, layer->v_params, layer->k_params,
                              static_cast<cudaStream_t>(stream)) == cudaSuccess ? STIEF_OK : STIEF_ERR_CUDA;
}

int run_q_append(int bits, const stief_qlayer* layer, const stief_batch* batch, const uint16_t* k_new, const uint16_t* v_new,
                 int32_t* status, void* stream) {
  int rc = check_qlayer(layer);
  if (rc) return rc;
  rc = check_batch(batch);
  if (rc) return rc;
  if (!k_new || !v_new || !aligned(k_new, 16) || !aligned(v_new, 16)) return STIEF_ERR_INVALID_ARG;
  AppendQArgs a;
  a.L = qlayer_to_dev(layer);
  a.Bt = to_dev(batch);
  a.k_new = reinterpret_cast<const __nv_bfloat16*>(k_new);
  a.v_new = reinterpret_cast<const __nv_bfloat16*>(v_new);
  a.k_codes = layer->k_codes; a.v_codes = layer->v_codes; a.v_params = layer->v_params; a.k_params = layer->k_params;
  a.bits = bits;
  a.status = status;
  append_q_kernel<<<dim3(layer->Hkv, batch->B, 2), kAqThreads, 0, static_cast<cudaStream_t>(stream)>>>(a);
  return cudaGetLastError() == cudaSuccess ? STIEF_OK : STIEF_ERR_CUDA;
}

int run_q_decode(int bits, const stief_qlayer* layer, const stief_batch* batch, const uint16_t* q, const uint16_t* k_new,
                 const uint16_t* v_new, int32_t len_add, void* workspace, size_t workspace_bytes, int32_t num_parts,
                 uint16_t* out, float* out_lse, uint32_t flags, int32_t* status, void* stream) {
  if (flags & ~STIEF_DECODE_OVERLAP_PREVIOUS) return STIEF_ERR_INVALID_ARG;
  if (k_new && (!v_new || !aligned(k_new, 16) || !aligned(v_new, 16) || len_add != 1)) return STIEF_ERR_INVALID_ARG;
  int rc = check_qlayer(layer);
  if (rc) return rc;
  rc = check_batch(batch);
  if (rc) return rc;
  if (!q || !aligned(q, 16) || !workspace || !aligned(workspace, 128) || !out || !aligned(out, 16)) return STIEF_ERR_INVALID_ARG;
  if (len_add < 0 || len_add > 1 || num_parts < 0 || num_parts > 65535) return STIEF_ERR_INVALID_ARG;
  const int n_cta = resolve_parts(num_parts);
  const int QT = query_tiles(layer->Hq, layer->Hkv);
  if ((long long)batch->B * (batch->max_pages_per_seq + seg_pad_pages(layer->r_k, layer->r_v)) * layer->Hkv * QT >= (1ll << 31))
    return STIEF_ERR_INVALID_ARG;
  const Workspace w = carve(workspace, batch->B, layer->Hq, layer->Hkv, layer->r_v, n_cta, workspace_bytes);
  if (w.bytes > workspace_bytes) return STIEF_ERR_WORKSPACE;
  DecodeQArgs a;
  a.L = qlayer_to_dev(layer);
  a.Bt = to_dev(batch);
  a.k_codes = layer->k_codes; a.v_codes = layer->v_codes; a.v_params = layer->v_params; a.k_params = layer->k_params;
  a.q = reinterpret_cast<const __nv_bfloat16*>(q);
  a.k_new = reinterpret_cast<const __nv_bfloat16*>(k_new);
  a.v_new = reinterpret_cast<const __nv_bfloat16*>(v_new);
  const bool ov = (flags & STIEF_DECODE_OVERLAP_PREVIOUS) != 0 && n_cta >= sm_count();   // full grids only (see run_decode)
  const WorkspaceTurn turn = take_workspace_turn(workspace);
  a.partial_o = w.partial_o[turn.section]; a.partial_lse = w.partial_lse[turn.section]; a.counters = w.counters[turn.section];
  a.finished = w.control + turn.section;
  a.units_done = w.control + kWorkspaceSections + turn.section;
  a.epoch = turn.epoch;
  a.prev_epoch = ov ? turn.prev_epoch : 0u;
  a.out = reinterpret_cast<__nv_bfloat16*>(out);
  a.out_lse = out_lse;
  a.len_add = len_add;
  a.QT = QT;
  a.status = status;
  return launch_decode_q(a, bits, n_cta, ov, static_cast<cudaStream_t>(stream)) == cudaSuccess ? STIEF_OK : STIEF_ERR_CUDA;
}

}  // namespace
}  // namespace stief

using namespace stief;

extern "C" {

#define STIEF_Q_ENTRY_POINTS(bits)                                                                                              \
  int stief_q##bits##_prefill_compress(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* K, const uint16_t* V, \
                                       int64_t stride_b, int64_t stride_t, int32_t T_max, uint32_t flags, int32_t* status,        \
                                       void* stream) {                                                                            \
    return run_q_prefill(bits, layer, batch, K, V, stride_b, stride_t, T_max, flags, status, stream);                            \
  }                                                                                                                               \
  int stief_q##bits##_append(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* k_new, const uint16_t* v_new,   \
                             int32_t* status, void* stream) {                                                                     \
    return run_q_append(bits, layer, batch, k_new, v_new, status, stream);                                                       \
  }                                                                                                                               \
  int stief_q##bits##_decode_attention(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* q, int32_t len_add,   \
                                       void* workspace, size_t workspace_bytes, int32_t num_parts, uint16_t* out, float* out_lse, \
                                       uint32_t flags, int32_t* status, void* stream) {                                           \
    return run_q_decode(bits, layer, batch, q, nullptr, nullptr, len_add, workspace, workspace_bytes, num_parts, out, out_lse,   \
                        flags, status, stream);                                                                                   \
  }                                                                                                                               \
  int stief_q##bits##_decode_step(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* q, const uint16_t* k_new,  \
                                  const uint16_t* v_new, void* workspace, size_t workspace_bytes, int32_t num_parts,              \
                                  uint16_t* out, float* out_lse, uint32_t flags, int32_t* status, void* stream) {                 \
    if (!k_new || !v_new) return STIEF_ERR_INVALID_ARG;                                                                          \
    return run_q_decode(bits, layer, batch, q, k_new, v_new, 1, workspace, workspace_bytes, num_parts, out, out_lse, flags,      \
                        status, stream);                                                                                          \
  }

STIEF_Q_ENTRY_POINTS(8)
STIEF_Q_ENTRY_POINTS(4)
#undef STIEF_Q_ENTRY_POINTS

}  // extern "C"
