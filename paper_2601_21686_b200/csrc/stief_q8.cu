// 8-bit quantised compressed cache (paper Sec. 4.3): C-ABI entry points, the append kernel, and the launchers of
// the quantised decode kernel.  The prefill projection with the quantising epilogue lives in stief_prefill_tc.cu.
#include "stief_decode_q8.cuh"
#include "stief_host_util.h"

namespace stief {

// ---------------------------------------------------------------------------------------------
// append: project one new row per (sequence, KV head, side), quantise it, store codes (and value parameters)
// ---------------------------------------------------------------------------------------------
struct AppendQ8Args {
  LayerDev L;
  BatchDev Bt;
  const __nv_bfloat16* k_new;   // [B][Hkv][128]
  const __nv_bfloat16* v_new;
  uint8_t* k_codes;
  uint8_t* v_codes;
  float* v_params;
  const float* k_params;
  int32_t* status;
};

constexpr int kAq8Threads = 128;          // thread j owns output column j (ranks are 64 or 128)

__global__ void __launch_bounds__(kAq8Threads)
append_q8_kernel(const AppendQ8Args a) {
  __shared__ float x[kD];
  __shared__ float gmin[2], gmax[2];
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
  const int R = side ? a.L.r_v : a.L.r_k, ng = R >> 6;
  const int j = threadIdx.x;
  if (j < kD) x[j] = __bfloat162float(src[j]);
  __syncthreads();
  float acc = 0.f;
  if (j < R) {
#pragma unroll 8
    for (int d = 0; d < kD; ++d) acc = fmaf(x[d], __bfloat162float(U[(size_t)d * R + j]), acc);
  }
  const int g = j >> 6;
  float sc, zp;
  if (side == 0) {
    sc = j < R ? a.k_params[((size_t)h * ng + g) * 2] : 1.f;
    zp = j < R ? a.k_params[((size_t)h * ng + g) * 2 + 1] : 0.f;
  } else {
    // token-wise group parameters: min and max over the 64 columns of the group (two warps per group)
    float mn = j < R ? acc : INFINITY, mx = j < R ? acc : -INFINITY;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    __shared__ float wmin[4], wmax[4];
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
    sc = mx > mn ? __fdiv_rn(mx - mn, 255.f) : 1.f;
    zp = mn;
    if (j < R && (j & 63) == 0) *reinterpret_cast<float2*>(a.v_params + (row * ng + g) * 2) = make_float2(sc, zp);
  }
  if (j < R) {
    const float y = __fmul_rn(__fsub_rn(acc, zp), __fdiv_rn(1.f, sc));
    const uint8_t code = (uint8_t)fminf(fmaxf(rintf(y), 0.f), 255.f);
    const size_t tile = (size_t)page * a.L.Hkv + h;
    if (side == 0) a.k_codes[row * R + j] = code;                                             // [token][channel]
    else a.v_codes[(tile * R + j) * kPage + v_position(pos % kPage)] = code;                  // [channel][position]
  }
}

// ---------------------------------------------------------------------------------------------
// decode launchers
// ---------------------------------------------------------------------------------------------
template <int RK, int RV>
static cudaError_t launch_decode_q8(const DecodeQ8Args& a, int n_cta, bool overlap_previous, cudaStream_t st) {
  using C = DecodeQ8Cfg<RK, RV>;
  auto kern = decode_q8_kernel<RK, RV>;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
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
  // key codes: [tiles * 64 token rows][RK bytes], one box per tile; value codes: [tiles * RV channel rows][64 bytes]
  const unsigned long long tiles = (unsigned long long)a.L.num_pages * a.L.Hkv;
  CUtensorMap tmK, tmV;
  {
    const unsigned long long dims[2] = {(unsigned long long)RK, tiles * kPage}, strides[1] = {(unsigned long long)RK};
    const unsigned box[2] = {(unsigned)RK, (unsigned)kPage};
    if (!encode_u8_map(&tmK, a.k_codes, 2, dims, strides, box, RK == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B))
      return cudaErrorInvalidValue;
  }
  {
    const unsigned long long dims[2] = {(unsigned long long)kPage, tiles * RV}, strides[1] = {(unsigned long long)kPage};
    const unsigned box[2] = {(unsigned)kPage, (unsigned)RV};
    if (!encode_u8_map(&tmV, a.v_codes, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_64B)) return cudaErrorInvalidValue;
  }
  return cudaLaunchKernelEx(&cfg, kern, tmK, tmV, a);
}

namespace {

using namespace host;

int check_qlayer(const stief_qlayer* l) {
  if (!l) return STIEF_ERR_INVALID_ARG;
  if (l->Hq <= 0 || l->Hkv <= 0 || l->Hq % l->Hkv != 0 || l->num_pages <= 0) return STIEF_ERR_INVALID_ARG;
  if (l->d != kD) return STIEF_ERR_UNSUPPORTED;
  if ((l->r_k != 64 && l->r_k != 128) || (l->r_v != 64 && l->r_v != 128)) return STIEF_ERR_UNSUPPORTED;
  if (!l->U_k || !l->U_v || !aligned(l->U_k, 128) || !aligned(l->U_v, 128)) return STIEF_ERR_INVALID_ARG;
  if (!l->k_codes || !l->v_codes || !l->v_params || !l->k_params) return STIEF_ERR_INVALID_ARG;
  if (!aligned(l->k_codes, 128) || !aligned(l->v_codes, 128) || !aligned(l->v_params, 128) || !aligned(l->k_params, 8))
    return STIEF_ERR_INVALID_ARG;
  if (l->uk_head_stride < 0 || l->uv_head_stride < 0 || (l->uk_head_stride % 64) != 0 || (l->uv_head_stride % 64) != 0)
    return STIEF_ERR_INVALID_ARG;
  if ((long long)l->num_pages * l->Hkv * kPage >= (1ll << 31)) return STIEF_ERR_INVALID_ARG;
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

}  // namespace
}  // namespace stief

using namespace stief;

extern "C" {

int stief_q8_prefill_compress(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* K, const uint16_t* V,
                              int64_t stride_b, int64_t stride_t, int32_t T_max, uint32_t flags, int32_t* status, void* stream) {
  if (flags & ~STIEF_PREFILL_OVERLAP_PREVIOUS) return STIEF_ERR_INVALID_ARG;
  int rc = check_qlayer(layer);
  if (rc) return rc;
  rc = host::check_batch(batch);
  if (rc) return rc;
  if (!K || !V || !host::aligned(K, 16) || !host::aligned(V, 16)) return STIEF_ERR_INVALID_ARG;
  if (T_max <= 0 || stride_t < (int64_t)layer->Hkv * kD || stride_b < 0 || (stride_t % 8) != 0 || (stride_b % 8) != 0)
    return STIEF_ERR_INVALID_ARG;
  if (batch->B > 1 && stride_b == 0) return STIEF_ERR_INVALID_ARG;
  PrefillArgs a;
  a.L = qlayer_to_dev(layer);
  a.Bt = host::to_dev(batch);
  a.K = reinterpret_cast<const __nv_bfloat16*>(K);
  a.V = reinterpret_cast<const __nv_bfloat16*>(V);
  a.stride_b = stride_b; a.stride_t = stride_t; a.v_stride_b = stride_b; a.v_stride_t = stride_t;
  a.T_max = T_max; a.status = status;
  a.overlap_previous = (flags & STIEF_PREFILL_OVERLAP_PREVIOUS) != 0;
  return launch_prefill_q8(a, layer->k_codes, layer->v_codes, layer->v_params, layer->k_params, static_cast<cudaStream_t>(stream)) ==
                 cudaSuccess
             ? STIEF_OK
             : STIEF_ERR_CUDA;
}

int stief_q8_append(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* k_new, const uint16_t* v_new,
                    int32_t* status, void* stream) {
  int rc = check_qlayer(layer);
  if (rc) return rc;
  rc = host::check_batch(batch);
  if (rc) return rc;
  if (!k_new || !v_new || !host::aligned(k_new, 16) || !host::aligned(v_new, 16)) return STIEF_ERR_INVALID_ARG;
  AppendQ8Args a;
  a.L = qlayer_to_dev(layer);
  a.Bt = host::to_dev(batch);
  a.k_new = reinterpret_cast<const __nv_bfloat16*>(k_new);
  a.v_new = reinterpret_cast<const __nv_bfloat16*>(v_new);
  a.k_codes = layer->k_codes; a.v_codes = layer->v_codes; a.v_params = layer->v_params; a.k_params = layer->k_params;
  a.status = status;
  append_q8_kernel<<<dim3(layer->Hkv, batch->B, 2), kAq8Threads, 0, static_cast<cudaStream_t>(stream)>>>(a);
  return cudaGetLastError() == cudaSuccess ? STIEF_OK : STIEF_ERR_CUDA;
}

static int run_q8_decode(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* q, const uint16_t* k_new,
                         const uint16_t* v_new, int32_t len_add, void* workspace, size_t workspace_bytes, int32_t num_parts,
                         uint16_t* out, float* out_lse, uint32_t flags, int32_t* status, void* stream) {
  if (flags & ~STIEF_DECODE_OVERLAP_PREVIOUS) return STIEF_ERR_INVALID_ARG;
  if (k_new && (!v_new || !host::aligned(k_new, 16) || !host::aligned(v_new, 16) || len_add != 1)) return STIEF_ERR_INVALID_ARG;
  int rc = check_qlayer(layer);
  if (rc) return rc;
  rc = host::check_batch(batch);
  if (rc) return rc;
  if (!q || !host::aligned(q, 16) || !workspace || !host::aligned(workspace, 128) || !out || !host::aligned(out, 16))
    return STIEF_ERR_INVALID_ARG;
  if (len_add < 0 || len_add > 1 || num_parts < 0 || num_parts > 65535) return STIEF_ERR_INVALID_ARG;
  const int n_cta = host::resolve_parts(num_parts);
  const int QT = host::query_tiles(layer->Hq, layer->Hkv);
  if ((long long)batch->B * (batch->max_pages_per_seq + seg_pad_pages(layer->r_k, layer->r_v)) * layer->Hkv * QT >= (1ll << 31))
    return STIEF_ERR_INVALID_ARG;
  const host::Workspace w = host::carve(workspace, batch->B, layer->Hq, layer->Hkv, layer->r_v, n_cta);
  if (w.bytes > workspace_bytes) return STIEF_ERR_WORKSPACE;
  DecodeQ8Args a;
  a.L = qlayer_to_dev(layer);
  a.Bt = host::to_dev(batch);
  a.k_codes = layer->k_codes; a.v_codes = layer->v_codes; a.v_params = layer->v_params; a.k_params = layer->k_params;
  a.q = reinterpret_cast<const __nv_bfloat16*>(q);
  a.k_new = reinterpret_cast<const __nv_bfloat16*>(k_new);
  a.v_new = reinterpret_cast<const __nv_bfloat16*>(v_new);
  a.partial_o = w.partial_o; a.partial_lse = w.partial_lse; a.counters = w.counters;
  a.out = reinterpret_cast<__nv_bfloat16*>(out);
  a.out_lse = out_lse;
  a.len_add = len_add;
  a.QT = QT;
  a.status = status;
  const bool ov = (flags & STIEF_DECODE_OVERLAP_PREVIOUS) != 0 && n_cta >= host::sm_count();   // see run_decode: full grids only
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  if (layer->r_k == 64 && layer->r_v == 64) e = launch_decode_q8<64, 64>(a, n_cta, ov, st);
  else if (layer->r_k == 64) e = launch_decode_q8<64, 128>(a, n_cta, ov, st);
  else if (layer->r_v == 64) e = launch_decode_q8<128, 64>(a, n_cta, ov, st);
  else e = launch_decode_q8<128, 128>(a, n_cta, ov, st);
  return e == cudaSuccess ? STIEF_OK : STIEF_ERR_CUDA;
}

int stief_q8_decode_attention(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* q, int32_t len_add,
                              void* workspace, size_t workspace_bytes, int32_t num_parts, uint16_t* out, float* out_lse,
                              uint32_t flags, int32_t* status, void* stream) {
  return run_q8_decode(layer, batch, q, nullptr, nullptr, len_add, workspace, workspace_bytes, num_parts, out, out_lse, flags, status,
                       stream);
}

int stief_q8_decode_step(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* q, const uint16_t* k_new,
                         const uint16_t* v_new, void* workspace, size_t workspace_bytes, int32_t num_parts, uint16_t* out,
                         float* out_lse, uint32_t flags, int32_t* status, void* stream) {
  if (!k_new || !v_new) return STIEF_ERR_INVALID_ARG;
  return run_q8_decode(layer, batch, q, k_new, v_new, 1, workspace, workspace_bytes, num_parts, out, out_lse, flags, status, stream);
}

}  // extern "C"
