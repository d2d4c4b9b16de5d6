// Split-T decode attention in the compressed space (scores, online softmax, mix) for one GQA group.
//
// Work item = (sequence b, KV head h, chunk of pages).  One producer warp streams the chunk's
// compressed page tiles K_down[64 x RK], V_down[64 x RV] from HBM into a ring of shared-memory
// stages with TMA (hardware swizzle, completion on mbarriers); NW consumer warps each take every
// NW-th page, compute the scores S = q' K_down^T of the group's query heads against the 64 tokens on
// the tensor cores, keep an online softmax in registers, and accumulate P V_down.  Warps merge their
// running (max, sum, accumulator) at the end and write one chunk-normalised partial [G][RV] + lse.
//
// Every consumer warp owns SPW private stages of the ring and walks them in order, so each mbarrier
// is only ever waited on by one warp, phase after phase: a parity wait can tell two adjacent phases
// apart but not more, and a shared ring would let a fast warp wait on a phase that is two ahead of
// what a slot has completed.
//
// Precision: q' (already scaled by log2(e)/sqrt(128)) and P are each carried as a pair of bf16 words
// (value + remainder) occupying rows 0-7 and 8-15 of the 16-row MMA operand, so the products see
// ~16 significant bits of q' and P; accumulation is fp32.  Up to 8 query heads per KV head share one
// pass; larger groups are tiled over blockIdx.y.
#pragma once

#include "stief_common.cuh"

#ifndef STIEF_DECODE_NW
#define STIEF_DECODE_NW 4
#endif

namespace stief {

struct DecodeArgs {
  LayerDev L;
  BatchDev Bt;
  const float* q_proj;     // [B][Hq][RK]
  float* partial_o;        // [B][Hq][S][RV]
  float* partial_lse;      // [B][Hq][S]
  int S, chunk_pages, len_add;
  int32_t* status;
};

template <int RK, int RV>
struct DecodeCfg {
  using TK = Tile<RK>;
  using TV = Tile<RV>;
  static constexpr int NW = STIEF_DECODE_NW;            // consumer warps
  static constexpr int THREADS = (NW + 1) * 32;         // + 1 producer warp
  static constexpr int STAGE_BYTES = TK::BYTES + TV::BYTES;
  static constexpr int SPW_RAW = (98304 / STAGE_BYTES) / NW;
  static constexpr int SPW = SPW_RAW < 1 ? 1 : (SPW_RAW > 4 ? 4 : SPW_RAW);   // private stages per consumer warp
  static constexpr int NS = NW * SPW;
  static constexpr int RING_BYTES = NS * STAGE_BYTES;
  static constexpr int CTRL_BYTES = 512;                // full[NS], empty[NS], abort flag
  static constexpr int SMEM_BYTES = RING_BYTES + CTRL_BYTES + 1024;   // + slack to align the ring to 1 KiB
  static_assert(RK % 16 == 0 && RV % 16 == 0 && RK <= 128 && RV <= 128, "ranks are multiples of 16 up to 128");
  static_assert(NW * 8 * (RV + 2) * 4 <= RING_BYTES, "merge scratch must fit in the ring");
};

__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(STIEF_DECODE_NW * 32) : "memory"); }

template <int RK, int RV>
__global__ void __launch_bounds__(DecodeCfg<RK, RV>::THREADS, 2)
decode_split_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const DecodeArgs a) {
  using C = DecodeCfg<RK, RV>;
  using TK = typename C::TK;
  using TV = typename C::TV;
  constexpr int NW = C::NW, NS = C::NS, SPW = C::SPW;

  extern __shared__ uint8_t smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x;
  const int h = blockIdx.y % a.L.Hkv;
  const int qt = blockIdx.y / a.L.Hkv;
  const int b = blockIdx.z;

  int len = a.Bt.seq_lens[b] + a.len_add;
  if (len < 0) len = 0;
  int npages_seq = (len + kPage - 1) / kPage;
  if (npages_seq > a.Bt.max_pages) {
    if (tid == 0) report(a.status, STIEF_ERR_BOUNDS);
    npages_seq = a.Bt.max_pages;
    len = npages_seq * kPage;
  }
  const int p0 = split * a.chunk_pages;
  const int p1 = min(p0 + a.chunk_pages, npages_seq);
  if (p0 >= p1) return;                                  // chunk beyond this sequence: nothing to do
  const int npg = p1 - p0;

  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t ctrl = ring + C::RING_BYTES;
  uint8_t* ring_ptr = smem_raw + (ring - smem_u32(smem_raw));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ring_ptr + C::RING_BYTES + 2 * NS * 8);
  static_assert(2 * NS * 8 + 4 <= C::CTRL_BYTES, "control block too small");
  auto full_bar = [&](int s) { return ctrl + s * 8; };
  auto empty_bar = [&](int s) { return ctrl + (NS + s) * 8; };

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();

  // ------------------------------------------------------------------ producer warp
  if (warp == NW) {
    if (lane == 0) {
      tma_prefetch_desc(&tmK);
      tma_prefetch_desc(&tmV);
    }
    int tbl = 0;
    for (int i = 0; i < npg; ++i) {
      if ((i & 31) == 0) {
        const int idx = p0 + i + lane;
        tbl = (idx < p1) ? a.Bt.block_table[(size_t)b * a.Bt.max_pages + idx] : 0;
      }
      int page = __shfl_sync(0xffffffffu, tbl, i & 31);
      if (page < 0 || page >= a.L.num_pages) {
        if (lane == 0) report(a.status, STIEF_ERR_BOUNDS);
        page = 0;
      }
      const int slot = (i % NW) * SPW + (i / NW) % SPW;    // private stage of the page's consumer warp
      const int use = (i / NW) / SPW;                      // how often that stage has been filled before
      if (lane == 0) {
        if (use > 0) mbar_wait(empty_bar(slot), (use - 1) & 1, abort_flag, a.status);
        const uint32_t st = ring + slot * C::STAGE_BYTES;
        const int y = (page * a.L.Hkv + h) * kPage;
        mbar_arrive_expect_tx(full_bar(slot), C::STAGE_BYTES);
#pragma unroll
        for (int nb = 0; nb < TK::NB; ++nb) tma_load_2d(st + nb * TK::BOX_BYTES, &tmK, nb * TK::BW, y, full_bar(slot));
#pragma unroll
        for (int nb = 0; nb < TV::NB; ++nb)
          tma_load_2d(st + TK::BYTES + nb * TV::BOX_BYTES, &tmV, nb * TV::BW, y, full_bar(slot));
      }
      __syncwarp();
    }
    return;
  }

  // ------------------------------------------------------------------ consumer warps
  const int gid = lane >> 2, tid4 = lane & 3;
  const int G = a.L.G;
  const int g = qt * 8 + gid;                            // query head inside the group (row of the MMA)
  const bool row_ok = g < G;

  // A operand of the score MMA: rows 0-7 = bf16(q'), rows 8-15 = bf16(q' - bf16(q'))
  uint32_t qa[RK / 16][4];
  {
    const float* qp = a.q_proj + ((size_t)b * a.L.Hq + (size_t)h * G + (row_ok ? g : 0)) * RK;
#pragma unroll
    for (int ks = 0; ks < RK / 16; ++ks) {
      float2 x = make_float2(0.f, 0.f), y = make_float2(0.f, 0.f);
      if (row_ok) {
        x = *reinterpret_cast<const float2*>(qp + 16 * ks + 2 * tid4);
        y = *reinterpret_cast<const float2*>(qp + 16 * ks + 8 + 2 * tid4);
      }
      split_bf16(x.x, x.y, qa[ks][0], qa[ks][1]);
      split_bf16(y.x, y.y, qa[ks][2], qa[ks][3]);
    }
  }

  float m = -INFINITY, l = 0.f;
  float o[RV / 8][4];
#pragma unroll
  for (int n = 0; n < RV / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;

  const int last_valid = len - (npages_seq - 1) * kPage;   // tokens in the sequence's last page (1..64)

  for (int i = warp; i < npg; i += NW) {
    const int slot = warp * SPW + (i / NW) % SPW;
    mbar_wait(full_bar(slot), ((i / NW) / SPW) & 1, abort_flag, a.status);
    const uint32_t kt = ring + slot * C::STAGE_BYTES;
    const uint32_t vt = kt + TK::BYTES;
    const bool tail = (p0 + i == npages_seq - 1) && (last_valid < kPage);

    // ---- scores of the page: s[j] covers tokens 8j..8j+7; c0,c1 from bf16(q'), c2,c3 from the remainder
    float sc[16];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float s[4] = {0.f, 0.f, 0.f, 0.f};
      constexpr int NCH = RK / 8;
#pragma unroll
      for (int kc = 0; kc + 4 <= NCH; kc += 4) {
        uint32_t r0, r1, r2, r3;
        ldsm_x4(kt + TK::chunk(8 * j + (lane & 7), kc + (lane >> 3)), r0, r1, r2, r3);
        mma_bf16(s, qa[kc / 2], r0, r1);
        mma_bf16(s, qa[kc / 2 + 1], r2, r3);
      }
      if constexpr (NCH % 4 == 2) {
        uint32_t r0, r1;
        ldsm_x2(kt + TK::chunk(8 * j + (lane & 7), NCH - 2 + ((lane >> 3) & 1)), r0, r1);
        mma_bf16(s, qa[NCH / 2 - 1], r0, r1);
      }
      sc[2 * j] = s[0] + s[2];
      sc[2 * j + 1] = s[1] + s[3];
    }
    if (tail) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int t = 8 * j + 2 * tid4;
        if (t >= last_valid) sc[2 * j] = -INFINITY;
        if (t + 1 >= last_valid) sc[2 * j + 1] = -INFINITY;
      }
      // rows past the end hold unspecified bits: zero them in V so that 0 * garbage cannot make a NaN
      constexpr int NCV = RV / 8;
      for (int idx = lane; idx < (kPage - last_valid) * NCV; idx += 32) {
        const int t = last_valid + idx / NCV, c = idx % NCV;
        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(vt + TV::chunk(t, c)), "r"(0u) : "memory");
      }
      __syncwarp();
    }

    // ---- online softmax (base 2; the scale is folded into q')
    float mx = sc[0];
#pragma unroll
    for (int e = 1; e < 16; ++e) mx = fmaxf(mx, sc[e]);
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(m, mx);
    const float alpha = fast_exp2(m - m_new);
    m = m_new;
    uint32_t pa[4][4];
    float ps = 0.f;
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      const float p0_ = fast_exp2(sc[4 * kk + 0] - m), p1_ = fast_exp2(sc[4 * kk + 1] - m);
      const float p2_ = fast_exp2(sc[4 * kk + 2] - m), p3_ = fast_exp2(sc[4 * kk + 3] - m);
      ps += (p0_ + p1_) + (p2_ + p3_);
      split_bf16(p0_, p1_, pa[kk][0], pa[kk][1]);
      split_bf16(p2_, p3_, pa[kk][2], pa[kk][3]);
    }
    l = l * alpha + ps;
#pragma unroll
    for (int n = 0; n < RV / 8; ++n) {
      o[n][0] *= alpha; o[n][1] *= alpha; o[n][2] *= alpha; o[n][3] *= alpha;
    }

    // ---- mix: o += P V_down (tokens are the contraction index; V tile read transposed)
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
      for (int np = 0; np < RV / 16; ++np) {
        uint32_t r0, r1, r2, r3;
        ldsm_x4_t(vt + TV::chunk(16 * kk + (lane & 7) + ((lane >> 3) & 1) * 8, 2 * np + (lane >> 4)), r0, r1, r2, r3);
        mma_bf16(o[2 * np], pa[kk], r0, r1);
        mma_bf16(o[2 * np + 1], pa[kk], r2, r3);
      }
    }

    if (tail) fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) mbar_arrive(empty_bar(slot));
  }

  // ------------------------------------------------------------------ merge the four warps
  l += __shfl_xor_sync(0xffffffffu, l, 1);
  l += __shfl_xor_sync(0xffffffffu, l, 2);
  consumer_bar();                                        // every tile has been consumed: the ring is free
  float* wo = reinterpret_cast<float*>(ring_ptr);        // [NW][8][RV]
  float* wm = wo + NW * 8 * RV;                          // [NW][8]
  float* wl = wm + NW * 8;                               // [NW][8]
#pragma unroll
  for (int n = 0; n < RV / 8; ++n) {
    *reinterpret_cast<float2*>(wo + (warp * 8 + gid) * RV + 8 * n + 2 * tid4) =
        make_float2(o[n][0] + o[n][2], o[n][1] + o[n][3]);
  }
  if (tid4 == 0) {
    wm[warp * 8 + gid] = m;
    wl[warp * 8 + gid] = l;
  }
  consumer_bar();
  for (int idx = tid; idx < 8 * RV; idx += NW * 32) {
    const int gg = idx / RV, j = idx % RV;
    const int gq = qt * 8 + gg;
    if (gq >= G) break;
    float M = wm[gg];
#pragma unroll
    for (int w = 1; w < NW; ++w) M = fmaxf(M, wm[w * 8 + gg]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float e = exp2f(wm[w * 8 + gg] - M);
      num += e * wo[(w * 8 + gg) * RV + j];
      den += e * wl[w * 8 + gg];
    }
    const size_t row = ((size_t)b * a.L.Hq + (size_t)h * G + gq) * a.S + split;
    a.partial_o[row * RV + j] = num / den;
    if (j == 0) a.partial_lse[row] = (M + log2f(den)) * kLn2;
  }
}

}  // namespace stief
