// Decode attention over the 8-bit quantised compressed cache (paper Sec. 4.3): the persistent split-T kernel of
// stief_decode.cuh with a different way of getting a page's operands into shared memory.  The cache holds
// K codes [64 x RK] and V codes [64 x RV] (uint8) per (page, head) plus the value rows' (scale, zero) pairs; the
// three contiguous blocks of a page are fetched with 1-D bulk async copies into the lane's ring stage.  The
// consuming warp then expands them once into bf16 operand tiles in a private scratch area (swizzled like the bf16
// kernel's TMA tiles) -- key codes as they are (integers up to 255 are exact in bf16; the key scale is folded into
// the projected query and the key zero-point only shifts a row's scores by a constant, so it enters out_lse alone),
// value codes dequantised as code * scale + zero -- frees the stage at once, and runs the same tensor-core score /
// online-softmax / mix code as the bf16 kernel on the scratch tiles.  Partition, prologue (query projection, no
// fused append here), segment merge and last-arriver combine are the bf16 kernel's.
//
// This first version spends more issue slots on the expansion than the bf16 kernel spends on a whole page, so it
// is bound by that, not by HBM: what it buys is cache capacity (136 instead of 256 bytes per token and head at rank
// 64/64).  The faster route (integer tensor-core MMAs on the raw codes with value pages stored channel-major) is
// described in the design notes.
#pragma once

#include "stief_decode.cuh"
#include "stief_partition.cuh"

namespace stief {

struct DecodeQ8Args {
  LayerDev L;                    // bases and shape (the bf16 pool pointers are unused)
  BatchDev Bt;
  const uint8_t* k_codes;        // [pages][Hkv][64][RK]
  const uint8_t* v_codes;        // [pages][Hkv][64][RV]
  const float* v_params;         // [pages][Hkv][64][RV/64][2] (scale, zero)
  const float* k_params;         // [Hkv][RK/64][2] (scale, zero)
  const __nv_bfloat16* q;        // [B][Hq][128]
  float* partial_o;
  float* partial_lse;
  int* counters;
  __nv_bfloat16* out;
  float* out_lse;
  int len_add;
  int QT;
  int32_t* status;
};

template <int RK, int RV>
struct DecodeQ8Cfg {
  using TK = Tile<RK>;
  using TV = Tile<RV>;
  static constexpr int NGV = RV / 64;
  static constexpr int K_BYTES = kPage * RK, V_BYTES = kPage * RV, P_BYTES = kPage * NGV * 8;
  static constexpr int STAGE_BYTES = K_BYTES + V_BYTES + P_BYTES;        // all multiples of 16
  static constexpr int SCRATCH_BYTES = TK::BYTES + TV::BYTES;            // one lane's bf16 operand tiles
  static constexpr int HALF = 1;
  static constexpr int CTRL_BYTES = 512;
  static constexpr int PREF_BYTES = ((kMaxBatch + 1) * 4 + 127) / 128 * 128;
  static constexpr int QP_BYTES = kGroupTile * kD * 4;
  static constexpr int ROWS_BYTES = 10 * kD * 4;
  static constexpr int MISC4 = CTRL_BYTES + PREF_BYTES + QP_BYTES + ROWS_BYTES + 4 * 9 * kD * 4;
  // four page lanes when their scratch tiles leave room for at least two stages each, else two
  static constexpr int NP = (232448 - 1024 - MISC4 - 4 * SCRATCH_BYTES >= 4 * 2 * STAGE_BYTES) ? 4 : 2;
  static constexpr int NW = NP * HALF;
  static constexpr int NT = NW * 32;
  static constexpr int THREADS = NT + NP * 32;
  static constexpr int RED_BYTES = NW * 9 * kD * 4;
  static constexpr int UNION_BYTES = (ROWS_BYTES + RED_BYTES) > 24576 ? (ROWS_BYTES + RED_BYTES) : 24576;
  static constexpr int MISC = CTRL_BYTES + PREF_BYTES + QP_BYTES + UNION_BYTES;
  static constexpr int RING_BUDGET = 232448 - 1024 - MISC - NP * SCRATCH_BYTES;
  static constexpr int SPW = (RING_BUDGET / (NP * STAGE_BYTES)) > 4 ? 4 : (RING_BUDGET / (NP * STAGE_BYTES));
  static constexpr int NS = NP * SPW;
  static constexpr int RING_BYTES = NS * STAGE_BYTES;
  static constexpr int SMEM_BYTES = 1024 + RING_BYTES + NP * SCRATCH_BYTES + MISC;
  static_assert(RK % 64 == 0 && RV % 64 == 0 && RK <= 128 && RV <= 128, "quantisation groups are 64 channels");
  static_assert(SPW >= 2 && NS <= 16, "ring shape");
  static_assert((NW * 8 * RV + 2 * NW * 8) * 4 <= UNION_BYTES, "merge scratch must fit");
  static_assert(kCombineScratchFloats * 4 <= UNION_BYTES, "combine scratch must fit");
  static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KiB shared memory of an SM");
};

// 1-D bulk async copy global -> shared (both 16-byte aligned, size a multiple of 16), completion in bytes on an mbarrier
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}


template <int RK, int RV>
__global__ void __launch_bounds__(DecodeQ8Cfg<RK, RV>::THREADS, 1)
decode_q8_kernel(const DecodeQ8Args a) {
  using C = DecodeQ8Cfg<RK, RV>;
  using TK = typename C::TK;
  using TV = typename C::TV;
  constexpr int NW = C::NW, NS = C::NS, SPW = C::SPW, NT = C::NT, NP = C::NP, HALF = C::HALF;
  constexpr int NJ = 8 / HALF;                           // 8-token score tiles per consumer warp and page
  constexpr int KK = 4 / HALF;                           // 16-token contraction steps of the mix per warp and page

  extern __shared__ uint8_t smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c = blockIdx.x, n_cta = gridDim.x;

  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* ring_ptr = smem_raw + (ring - smem_u32(smem_raw));
  const uint32_t scratch = ring + C::RING_BYTES;                        // NP lanes x (K tile, V tile) in bf16
  uint8_t* ctrl_ptr = ring_ptr + C::RING_BYTES + NP * C::SCRATCH_BYTES;
  const uint32_t ctrl = scratch + NP * C::SCRATCH_BYTES;
  auto full_bar = [&](int s) { return ctrl + s * 8; };
  auto empty_bar = [&](int s) { return ctrl + (16 + s) * 8; };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl_ptr + 33 * 8);
  volatile int* last_flag = reinterpret_cast<volatile int*>(ctrl_ptr + 33 * 8 + 4);
  float* lse_shift = reinterpret_cast<float*>(ctrl_ptr + 34 * 8);      // [8]: q' . key zero-point / sqrt(128) of the unit's rows
  int* pref = reinterpret_cast<int*>(ctrl_ptr + C::CTRL_BYTES);
  float* qp = reinterpret_cast<float*>(ctrl_ptr + C::CTRL_BYTES + C::PREF_BYTES);
  float* un = reinterpret_cast<float*>(ctrl_ptr + C::CTRL_BYTES + C::PREF_BYTES + C::QP_BYTES);

  // The next kernel on the stream may take over each SM as soon as this grid's CTA leaves it.
  launch_dependents();
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), HALF);
    }
    *abort_flag = 0;
    *last_flag = 0;
    mbar_fence_init();
  }
  const int pad = seg_pad_pages(RK, RV);
  build_page_prefix(pref, a.Bt, a.len_add, pad, c == 0 ? a.status : nullptr);   // ends with __syncthreads

  const int B = a.Bt.B, Hkv = a.L.Hkv, QT = a.QT, G = a.L.G;
  const int upb = Hkv * QT;
  const int total = pref[B] * upb;
  const int P = pages_per_cta(total, n_cta);

  SegmentWalker walk;
  walk.init(pref, B, upb, pad, c, P, total);
  Segment seg;

  // ------------------------------------------------------------------ producer warps
  // Producer warp pw feeds page lane pw: it issues the TMA loads of every NP-th page into that lane's private
  // stages.  One issuing thread per CTA could not keep up with small page tiles (a page costs it a few hundred
  // cycles of waits and descriptor traffic whatever its size), so the issue work is split the way the pages are.
  if (warp >= NW) {
    const int pw = warp - NW;
    int i_base = 0;            // pages of this CTA before the current segment
    while (walk.next(seg)) {
      const int h = seg.j / QT;
      const int npg = seg.p1 - seg.p0;
      int tbl = 0, win = -1;
      for (int k = (pw - i_base % NP + NP) % NP; k < npg; k += NP) {
        if ((k >> 5) != win) {                             // block-table entries of a window of 32 pages, one per lane
          win = k >> 5;
          const int idx = seg.p0 + (win << 5) + lane;
          tbl = (idx < seg.p1) ? a.Bt.block_table[(size_t)seg.b * a.Bt.max_pages + idx] : 0;
        }
        int page = __shfl_sync(0xffffffffu, tbl, k & 31);
        if (page < 0 || page >= a.L.num_pages) {
          if (lane == 0) report(a.status, STIEF_ERR_BOUNDS);
          page = 0;
        }
        const int kw = (i_base + k) / NP;                  // the lane's kw-th page
        const int slot = pw * SPW + kw % SPW;
        const int use = kw / SPW;
        if (lane == 0) {
          if (use > 0) mbar_wait(empty_bar(slot), (use - 1) & 1, abort_flag, a.status);
          const uint32_t st = ring + slot * C::STAGE_BYTES;
          const size_t tile = (size_t)page * Hkv + h;
          mbar_arrive_expect_tx(full_bar(slot), C::STAGE_BYTES);
          bulk_load_1d(st, a.k_codes + tile * C::K_BYTES, C::K_BYTES, full_bar(slot));
          bulk_load_1d(st + C::K_BYTES, a.v_codes + tile * C::V_BYTES, C::V_BYTES, full_bar(slot));
          bulk_load_1d(st + C::K_BYTES + C::V_BYTES, a.v_params + tile * (C::P_BYTES / 4), C::P_BYTES, full_bar(slot));
        }
        __syncwarp();
      }
      i_base += npg;
    }
    return;
  }

  // ------------------------------------------------------------------ consumer warps
  const int gid = lane >> 2, tid4 = lane & 3, l7 = lane & 7;
  const float qscale = kLog2e * 0.08838834764831845f;     // log2(e) / sqrt(128)

  // per-lane pieces of the ldmatrix addresses (the swizzle term depends on the lane only)
  constexpr int NCH = RK / 8;
  uint32_t koff[(NCH + 3) / 4];
#pragma unroll
  for (int q4 = 0; q4 < (NCH + 3) / 4; ++q4) {
    const int cc = (4 * q4 + 4 <= NCH) ? 4 * q4 + (lane >> 3) : 4 * q4 + ((lane >> 3) & 1);
    koff[q4] = TK::chunk(l7, cc);
  }
  uint32_t voff[RV / 16];
#pragma unroll
  for (int np = 0; np < RV / 16; ++np) voff[np] = TV::chunk(l7 + ((lane >> 3) & 1) * 8, 2 * np + (lane >> 4));

  int i_base = 0;              // pages of this CTA before the current segment

  while (walk.next(seg)) {
    const int b = seg.b, h = seg.j / QT, qt = seg.j % QT;
    const int npg = seg.p1 - seg.p0;
    const int ng = min(kGroupTile, G - qt * kGroupTile);
    const size_t head0 = (size_t)b * a.L.Hq + (size_t)h * G + (size_t)qt * kGroupTile;
    const int len_raw = a.Bt.seq_lens[b] + a.len_add;
    const int len = min(max(len_raw, 0), seg.npages * kPage);
    const int last_valid = len - (seg.npages - 1) * kPage;          // tokens in the sequence's last page (1..64)
    // ---- prologue: q' = q U_k for the unit's queries.  The key scale of each 64-channel group is folded into
    // q' (scores are then taken against the raw codes); the key zero-point shifts all scores of a row by
    // q' . zero, which cancels in the softmax and across segments and is added to out_lse at the very end.
    float* rows = un;                    // [9][128] fp32 (row 8 unused here)
    float* red = un + 10 * kD;           // [NW][9][128]
    const __nv_bfloat16* Uk = a.L.U_k + (size_t)h * a.L.uk_stride;
    const uint32_t row_mask = (1u << ng) - 1u;
    {
      BasisSlice<NW, RK> sk;
      sk.load(Uk, warp, lane);
      constexpr int NPC = (8 * 16 + NT - 1) / NT;
      uint4 pc[NPC];
#pragma unroll
      for (int i = 0; i < NPC; ++i) {
        const int idx = tid + i * NT, r = idx / 16, c = idx % 16;
        pc[i] = make_uint4(0u, 0u, 0u, 0u);
        if (r < ng) pc[i] = __ldg(reinterpret_cast<const uint4*>(a.q + (head0 + r) * kD) + c);
      }
#pragma unroll
      for (int i = 0; i < NPC; ++i) {
        const int idx = tid + i * NT;
        if (idx < 8 * 16) {
          const uint32_t w[4] = {pc[i].x, pc[i].y, pc[i].z, pc[i].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) *reinterpret_cast<float2*>(rows + idx * 8 + 2 * e) = make_float2(bf16_lo(w[e]), bf16_hi(w[e]));
        }
      }
      bar1(NT);
      sk.contract(rows, row_mask, red, warp, lane);
    }
    bar1(NT);
    const float* kpar = a.k_params + (size_t)h * (RK / 64) * 2;
    for (int idx = tid; idx < 8 * RK; idx += NT) {
      const int r = idx / RK, j = idx % RK;
      const float x = ((row_mask >> r) & 1u) ? warp_shares<NW>(red, r, j) : 0.f;
      qp[r * RK + j] = x * qscale * __ldg(kpar + 2 * (j >> 6));
    }
    if (tid < 8) {
      float sh = 0.f;
      if ((row_mask >> tid) & 1u)
        for (int j = 0; j < RK; ++j) sh = fmaf(warp_shares<NW>(red, tid, j), __ldg(kpar + 2 * (j >> 6) + 1), sh);
      lse_shift[tid] = sh * 0.08838834764831845f;          // / sqrt(128)
    }
    bar1(NT);

    // A operand of the score MMA: rows 0-7 = bf16(q'), rows 8-15 = bf16(q' - bf16(q'))
    uint32_t qa[RK / 16][4];
#pragma unroll
    for (int ks = 0; ks < RK / 16; ++ks) {
      const float2 x = *reinterpret_cast<const float2*>(qp + gid * RK + 16 * ks + 2 * tid4);
      const float2 y = *reinterpret_cast<const float2*>(qp + gid * RK + 16 * ks + 8 + 2 * tid4);
      split_bf16(x.x, x.y, qa[ks][0], qa[ks][1]);
      split_bf16(y.x, y.y, qa[ks][2], qa[ks][3]);
    }

    float m = -INFINITY, l = 0.f;
    float o[RV / 8][4];
#pragma unroll
    for (int n = 0; n < RV / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;

    // first page of this segment that belongs to this warp's lane: global index i = i_base + k, i % NP == pl
    const int pl = warp % NP, hf = warp / NP;
    const int tb = hf * (kPage / HALF);                    // first token of the page this warp handles
    int k0 = (pl - i_base % NP + NP) % NP;
    for (int k = k0; k < npg; k += NP) {
      const int kw = (i_base + k) / NP;
      const int slot = pl * SPW + kw % SPW;
      mbar_wait(full_bar(slot), (kw / SPW) & 1, abort_flag, a.status);
      const bool tail = (seg.p0 + k == seg.npages - 1) && (last_valid < kPage);
      // ---- expand the page's codes into this lane's bf16 operand tiles, then give the stage back
      const uint32_t st = ring + slot * C::STAGE_BYTES;
      const uint32_t kt = scratch + pl * C::SCRATCH_BYTES;
      const uint32_t vt = kt + TK::BYTES;
      __syncwarp();                                        // the previous page's ldmatrix reads of the tiles are done
      {
        constexpr int KP = RK / 16;                        // 16-byte pieces (16 codes) per key row
#pragma unroll 4
        for (int idx = lane; idx < kPage * KP; idx += 32) {
          const int t = idx / KP, pc = idx % KP;
          uint32_t w0, w1, w2, w3;
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3) : "r"(st + idx * 16));
          const uint32_t w[4] = {w0, w1, w2, w3};
          uint32_t o[8];
#pragma unroll
          for (int e = 0; e < 4; ++e) {                    // integers up to 255 are exact in bf16
            o[2 * e] = pack_bf16((float)(w[e] & 0xffu), (float)((w[e] >> 8) & 0xffu));
            o[2 * e + 1] = pack_bf16((float)((w[e] >> 16) & 0xffu), (float)(w[e] >> 24));
          }
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(kt + TK::chunk(t, 2 * pc)), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(kt + TK::chunk(t, 2 * pc + 1)), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
        }
        constexpr int VP = RV / 16;
        const uint32_t vs = st + C::K_BYTES, ps = vs + C::V_BYTES;
#pragma unroll 4
        for (int idx = lane; idx < kPage * VP; idx += 32) {
          const int t = idx / VP, pc = idx % VP;
          uint32_t w0, w1, w2, w3;
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3) : "r"(vs + idx * 16));
          float sc, zp;                                    // the row's parameters of the group this piece lies in
          asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(sc), "=f"(zp) : "r"(ps + (t * C::NGV + (pc >> 2)) * 8));
          const uint32_t w[4] = {w0, w1, w2, w3};
          uint32_t o[8];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            o[2 * e] = pack_bf16(fmaf((float)(w[e] & 0xffu), sc, zp), fmaf((float)((w[e] >> 8) & 0xffu), sc, zp));
            o[2 * e + 1] = pack_bf16(fmaf((float)((w[e] >> 16) & 0xffu), sc, zp), fmaf((float)(w[e] >> 24), sc, zp));
          }
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(vt + TV::chunk(t, 2 * pc)), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(vt + TV::chunk(t, 2 * pc + 1)), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar(slot));         // the stage's bytes have been read: it may be refilled

      // ---- scores of the page: n-tile j covers tokens 8j..8j+7; c0,c1 from bf16(q'), c2,c3 from the remainder
      float sc[2 * NJ];
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int q4 = 0; 4 * q4 + 4 <= NCH; ++q4) {
          uint32_t r0, r1, r2, r3;
          ldsm_x4(kt + koff[q4] + (hf * NJ + j) * 8 * TK::RB, r0, r1, r2, r3);
          mma_bf16(s, qa[2 * q4], r0, r1);
          mma_bf16(s, qa[2 * q4 + 1], r2, r3);
        }
        if constexpr (NCH % 4 == 2) {
          uint32_t r0, r1;
          ldsm_x2(kt + koff[NCH / 4] + (hf * NJ + j) * 8 * TK::RB, r0, r1);
          mma_bf16(s, qa[NCH / 2 - 1], r0, r1);
        }
        sc[2 * j] = s[0] + s[2];
        sc[2 * j + 1] = s[1] + s[3];
      }
      if (tail) {
#pragma unroll
        for (int j = 0; j < NJ; ++j) {
          const int t = tb + 8 * j + 2 * tid4;
          if (t >= last_valid) sc[2 * j] = -INFINITY;
          if (t + 1 >= last_valid) sc[2 * j + 1] = -INFINITY;
        }
        // rows past the end hold unspecified bits: zero them in V so that 0 * garbage cannot make a NaN
        constexpr int NCV = RV / 8;
        const int z0 = max(last_valid, tb);                // this warp's rows past the end
        for (int idx = lane; idx < (tb + kPage / HALF - z0) * NCV; idx += 32) {
          const int t = z0 + idx / NCV, cc = idx % NCV;
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(vt + TV::chunk(t, cc)), "r"(0u) : "memory");
        }
        __syncwarp();
      }

      // ---- online softmax (base 2; the scale is folded into q')
      float mx = sc[0];
#pragma unroll
      for (int e = 1; e < 2 * NJ; ++e) mx = fmaxf(mx, sc[e]);
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m, mx);
      const float alpha = fast_exp2(m - m_new);
      m = m_new;
      uint32_t pa[KK][4];
      float ps = 0.f;
#pragma unroll
      for (int kk = 0; kk < KK; ++kk) {
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
      for (int kk = 0; kk < KK; ++kk) {
#pragma unroll
        for (int np = 0; np < RV / 16; ++np) {
          uint32_t r0, r1, r2, r3;
          ldsm_x4_t(vt + voff[np] + (hf * KK + kk) * 16 * TV::RB, r0, r1, r2, r3);
          mma_bf16(o[2 * np], pa[kk], r0, r1);
          mma_bf16(o[2 * np + 1], pa[kk], r2, r3);
        }
      }

    }
    i_base += npg;

    // ------------------------------------------------------------------ merge the warps of this segment
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    float* wo = un;                      // [NW][8][RV]
    float* wm = wo + NW * 8 * RV;        // [NW][8]
    float* wl = wm + NW * 8;             // [NW][8]
#pragma unroll
    for (int n = 0; n < RV / 8; ++n) {
      *reinterpret_cast<float2*>(wo + (warp * 8 + gid) * RV + 8 * n + 2 * tid4) = make_float2(o[n][0] + o[n][2], o[n][1] + o[n][3]);
    }
    if (tid4 == 0) {
      wm[warp * 8 + gid] = m;
      wl[warp * 8 + gid] = l;
    }
    bar1(NT);
    const int u = b * upb + seg.j;
    const int slot_id = c + u;
    // Everything up to here only read inputs (and appended this step's rows); the workspace and the
    // outputs may still be in use by the kernel before this one when the launch overlaps it.
    grid_dependency_wait();
    for (int idx = tid; idx < ng * RV; idx += NT) {
      const int gg = idx / RV, j = idx % RV;
      float M = wm[gg];
#pragma unroll
      for (int w = 1; w < NW; ++w) M = fmaxf(M, wm[w * 8 + gg]);
      float num = 0.f, den = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const float e = fast_exp2(wm[w * 8 + gg] - M);
        num += e * wo[(w * 8 + gg) * RV + j];
        den += e * wl[w * 8 + gg];
      }
      __stcg(a.partial_o + ((size_t)slot_id * kGroupTile + gg) * RV + j, num / den);
      if (j == 0) __stcg(a.partial_lse + (size_t)slot_id * kGroupTile + gg, (M + log2f(den)) * kLn2);
    }

    // ------------------------------------------------------------------ the unit's last partial triggers the combine
    if (a.out != nullptr) {
      int first, last;
      unit_cta_span(pref, upb, pad, P, b, seg.j, &first, &last);
      const int nseg = last - first + 1;
      __threadfence();
      bar1(NT);
      if (tid == 0) {
        int is_last = 1;
        if (nseg > 1) {
          const int prev = atomicAdd(a.counters + u, 1);
          is_last = (prev == nseg - 1);
          if (is_last) a.counters[u] = 0;                  // leave the counter clean for the next call
        }
        *last_flag = is_last;
      }
      bar1(NT);
      if (*last_flag) {
        __threadfence();
        combine_unit<RV>(a.L, b, h, qt, first + u, nseg, a.partial_o, a.partial_lse, a.out, a.out_lse, un, un + kGroupTile * kD, tid, NT, lse_shift);
      }
    }
    bar1(NT);
  }

  // units of empty sequences get their zero rows from CTA (u mod n_cta)
  if (a.out != nullptr) {
    grid_dependency_wait();
    for (int u = c; u < B * upb; u += n_cta) {
      const int b = u / upb, j = u % upb;
      if (pref[b + 1] != pref[b]) continue;
      const int h = j / QT, qt = j % QT;
      const int ng = min(kGroupTile, G - qt * kGroupTile);
      const size_t head0 = (size_t)b * a.L.Hq + (size_t)h * G + (size_t)qt * kGroupTile;
      for (int idx = tid; idx < ng * kD; idx += NT) a.out[head0 * kD + idx] = __float2bfloat16_rn(0.f);
      if (a.out_lse && tid < ng) a.out_lse[head0 + tid] = -INFINITY;
    }
  }
  grid_dependency_wait();    // never finish before the kernel this one was allowed to overlap (keeps stream order transitive)
}

}  // namespace stief
