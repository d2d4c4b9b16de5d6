// Attention of SEVERAL causal query rows per head over the compressed cache (chunked prefill, speculative
// decode): App. A.1 of the paper (during prefilling Q has one row per prefix token; Eq. 18 per row), evaluated in
// the compressed space like the decode path:  out_i = softmax(q_i' K_down[0..p_i]^T / sqrt(d_h)) V_down[0..p_i] U_v^T,
// q_i' = q_i U_k, p_i = position of query row i.  With many rows per cache page this is a dense contraction, so it
// runs on the 5th-generation tensor cores: four tcgen05.mma GEMMs per work unit, accumulators in TMEM.
//
// A work unit is (sequence b, KV head h, 256 query rows): two row tiles of 128 rows, a row being (token i, query
// head g of the group of h), token-major.  Both tiles use every cache page once it is in shared memory.
// One persistent CTA per SM, 352 threads, warp-specialised:
//   warp 0      producer.  Items go through a ring of 32 KiB stages, in the order the MMA warp consumes them: the
//               raw query tiles and U_k (unless the key side is folded), the cache pages (K page | V page), U_v
//               (unless the value side is folded).  Everything arrives by tiled TMA loads, in the swizzled blocks
//               that tcgen05.mma reads (see Blocks); block-table entries are fetched 32 at a time, a batch ahead.
//   warps 1,10  MMA issue, one thread per tile (warp 1 also allocates TMEM).  Per unit: Q' = Q U_k  (A = raw q rows, B = U_k as an
//               MN-major operand) into the tile's accumulator columns; per page j and tile: S = Q' K_j^T (N = 64
//               positions) into one of two score buffers, then O += P_j V_j (A = P_j read from TMEM, B = the V page,
//               MN-major) once the softmax warps have published P_j; finally OUT = O_down U_v^T (B = U_v, K-major).  QK of page j+1 is
//               issued before PV of page j, so the tensor pipe works on the next scores while P_j is being made.
//   warps 2-5   softmax / epilogue of tile 0, warps 6-9 of tile 1; thread = row (TMEM lane).  Round Q' to bf16 into
//               the A operand; per page: tcgen05.ld the scores, causal mask on the boundary pages, running
//               reference maximum, p = 2^(c s - c m) as bf16 pairs back into the score buffer (TMEM), row sum.  The accumulator in TMEM
//               is rescaled only when a row's maximum has grown by more than 2^8 since the reference was set
//               (p <= 256 stays exact enough in bf16/fp32); that is decided per warp and done with tcgen05.ld/st
//               after the previous PV has completed.  Epilogue: O / l as two bf16 terms (value and residual), the A
//               operands of two accumulating back-projection passes, then the 128 output columns to global memory,
//               256 contiguous bytes per row.
// TMEM (512 columns): per tile two score buffers of 64 columns (which also take OUT at the end of a unit) and
// 128 columns for Q' / O.
// Units are taken round-robin (unit u -> CTA u mod grid), heaviest (latest query tokens) first.
// With few query rows and a long cache (speculative decode) the units are too few to fill the GPU: the host then cuts
// every unit's page range into n_split parts, which run as units of their own and leave partial results (unnormalised
// mix, reference maximum, row sum) that mq_combine_kernel merges, normalises and back-projects.
//
// Precision: q' and P pass through bf16 (as the cache itself does); scores, sums and O_down keep fp32 accuracy.
// Every wait is bounded (see mbar_wait): on a timeout the status word says so, later waits return at once, every
// role walks to the end of its loops and TMEM is released.
#pragma once

#include <type_traits>

#include "stief_kernels.h"
#include "stief_tc.cuh"

#ifndef STIEF_MQ_POLY_EVERY
#define STIEF_MQ_POLY_EVERY 4
#endif

namespace stief {
namespace mq {

using namespace tc;

constexpr int kThreads = 352;
constexpr int kRows = 128;                      // rows per tile
constexpr int kStageBytes = 32768;              // one ring stage
constexpr int kCtrlBytes = 1024;
constexpr int kSmemLimit = 232448;              // 227 KiB per CTA
constexpr int kTmemCols = 512;
constexpr int kMaxStages = 6;
constexpr int kPolyEvery = STIEF_MQ_POLY_EVERY;   // every kPolyEvery-th pair of exponentials runs as a polynomial on the FMA pipe
constexpr float kRescaleLog2 = 8.0f;            // rescale the accumulator when a maximum grew by more than 2^8

struct Args {
  LayerDev L;
  BatchDev Bt;
  const int32_t* q_lens;         // [B] query rows (tokens) per sequence, or NULL = n_q for all
  int n_q;                       // query tokens per sequence in the q / out tensors
  __nv_bfloat16* out;            // [B][n_q][Hq][d_out], d_out = 128, or r_v when the value side is folded
  long long out_stride_b, out_stride_t;    // elements
  float* out_lse;                // [B][n_q][Hq] or NULL
  int32_t* status;
  int nst;                       // ring stages
  int qp_bytes;                  // bytes of one tile's Q' / O_down operand region
  // Split-T (few query rows, long cache): every unit's page range is cut into n_split parts that run as separate
  // units and leave partial results; mq_combine_kernel merges them.  n_split = 1: results are final.
  int n_split;
  // With at most 128 query rows per (sequence, KV head) the second tile of a unit would idle.  dual = 1 gives it the
  // SAME rows and lets the two tiles take alternate pages of the unit's range (two independent softmax streams per
  // CTA, each with its own partial result): a single stream is bound by the latency of its score -> softmax -> P V
  // chain, two overlap.  Parts per row in the workspace: n_parts = n_split * (1 + dual).
  int dual;
  int n_parts;
  float* part_o;                 // [B * n_q * Hq][n_parts][r_v]  unnormalised mix, relative to the part's own reference
  float* part_ml;                // [B * n_q * Hq][n_parts][2]    that reference in base-2 units, and the row sum
};

// A unit as every role derives it (same loads, same arithmetic)
struct Unit {
  int b, h;
  int tok0[2];                   // first query token of each tile
  int np[2];                     // cache pages each tile reads in this unit (0 = none)
  int cnt;                       // pages of the unit that go through the ring (dual: the tiles take alternate ones)
  int p_lo;                      // first of those pages (0 unless the sequence's pages are split over several units)
  int split;                     // which part of the page range this unit is
  int q_len, q_start;            // query tokens of the sequence; absolute position of its query token 0
  int seq_len;                   // cached tokens of the sequence
  bool valid;
};

__device__ __forceinline__ Unit decode_unit(const Args& a, int u, int TT) {
  Unit w;
  const int bh = a.Bt.B * a.L.Hkv;
  const int n_t2 = (a.n_q + 2 * TT - 1) / (2 * TT);
  const int ub = u / a.n_split;
  w.split = u - ub * a.n_split;
  w.p_lo = 0;
  const int t2 = n_t2 - 1 - ub / bh;             // heaviest tiles first
  const int r = ub % bh;
  w.b = r / a.L.Hkv;
  w.h = r - w.b * a.L.Hkv;
  int ql = a.q_lens ? a.q_lens[w.b] : a.n_q;
  ql = min(max(ql, 0), a.n_q);
  const int sl = a.Bt.seq_lens[w.b];
  w.q_len = ql;
  w.q_start = sl - ql;
  w.seq_len = sl;
  w.valid = false;
  w.np[0] = w.np[1] = 0;
  w.cnt = 0;
  w.tok0[0] = t2 * 2 * TT;
  w.tok0[1] = a.dual ? w.tok0[0] : w.tok0[0] + TT;
  if (w.tok0[0] >= ql) return w;
  if (w.q_start < 0 || (sl + kPage - 1) / kPage > a.Bt.max_pages) {   // fewer cached tokens than query rows, or a table too short
    report(a.status, STIEF_ERR_BOUNDS);
    return w;
  }
  int full[2] = {0, 0};                          // pages each tile attends in all
#pragma unroll
  for (int t = 0; t < 2; ++t)
    if (w.tok0[t] < ql) full[t] = (w.q_start + min(w.tok0[t] + TT, ql) - 1) / kPage + 1;
  const int all = max(full[0], full[1]);
  const int lo = (int)((long long)w.split * all / a.n_split), hi = (int)((long long)(w.split + 1) * all / a.n_split);
  w.p_lo = lo;
  if (a.dual) {                                  // page lo + j goes to tile j & 1
    w.cnt = max(0, min(hi, all) - lo);
    w.np[0] = (w.cnt + 1) >> 1;
    w.np[1] = w.cnt >> 1;
  } else {
#pragma unroll
    for (int t = 0; t < 2; ++t) w.np[t] = max(0, min(hi, full[t]) - lo);
    w.cnt = max(w.np[0], w.np[1]);
  }
  w.valid = w.cnt != 0;                          // a part may be empty when there are fewer pages than parts
  return w;
}

// packed fp32 pairs (sm_100): one instruction for two lanes of arithmetic
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// 2^x for a pair of x in [-125, 16] on the FMA pipe: x = n + f with n = rint(x) (the 1.5 * 2^23 trick leaves n in the low
// mantissa bits of t), 2^f by a cubic fitted to [-0.5, 0.5] (relative error 7.5e-5, far below the bf16 rounding of
// the probabilities), 2^n by adding n to the exponent field.  The special-function pipe does 16 ex2 per clock and SM,
// which at 64 of them per score row and page is this kernel's tightest unit; a quarter of the exponentials go here.
__device__ __forceinline__ void exp2_pair_fma(uint64_t x2, float& e0, float& e1) {
  const uint64_t magic = pack2(12582912.f, 12582912.f), neg_magic = pack2(-12582912.f, -12582912.f);
  const uint64_t t = add2(x2, magic);
  const uint64_t n = add2(t, neg_magic);
  const uint64_t f = fma2(n, pack2(-1.f, -1.f), x2);
  uint64_t q = fma2(f, pack2(0.05517145f, 0.05517145f), pack2(0.24261084f, 0.24261084f));
  q = fma2(q, f, pack2(0.69326097f, 0.69326097f));
  q = fma2(q, f, pack2(0.99992812f, 0.99992812f));
  float t0, t1, q0, q1;
  unpack2(t, t0, t1);
  unpack2(q, q0, q1);
  e0 = __int_as_float(__float_as_int(q0) + (__float_as_int(t0) << 23));
  e1 = __int_as_float(__float_as_int(q1) + (__float_as_int(t1) << 23));
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// 16 fp32 values of a row -> 8 packed bf16 words
__device__ __forceinline__ void pack16(const uint32_t (&v)[16], float scale, uint32_t (&w)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) w[i] = pack_bf16(__uint_as_float(v[2 * i]) * scale, __uint_as_float(v[2 * i + 1]) * scale);
}

// The ranks are template parameters: the descriptor offsets and K-step counts of the MMA role are then constants,
// which matters because every scalar instruction of that role sits between two tensor-core instructions.
template <int RK, int RV>
__global__ void __launch_bounds__(kThreads, 1)
mq_attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmUk,
                    const __grid_constant__ CUtensorMap tmUv, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const Args a) {
  extern __shared__ uint8_t smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int nst = a.nst;
  const uint32_t ring = base;
  const uint32_t qp = ring + nst * kStageBytes;                 // Q' / O_down operands, one region per tile
  uint8_t* qp_ptr = base_ptr + nst * kStageBytes;
  const uint32_t ctrl = qp + 2 * a.qp_bytes;
  uint8_t* ctrl_ptr = qp_ptr + 2 * a.qp_bytes;
  auto full_bar = [&](int s) { return ctrl + s * 8; };
  auto empty_bar = [&](int s) { return ctrl + (6 + s) * 8; };
  auto s_full = [&](int t, int i) { return ctrl + (12 + t * 2 + i) * 8; };
  auto p_full = [&](int t, int i) { return ctrl + (20 + t * 2 + i) * 8; };
  auto p_free = [&](int t, int i) { return ctrl + (24 + t * 2 + i) * 8; };
  auto qacc_full = [&](int t) { return ctrl + (28 + t) * 8; };
  auto qp_ready = [&](int t) { return ctrl + (30 + t) * 8; };
  auto o_full = [&](int t) { return ctrl + (32 + t) * 8; };
  auto od_ready = [&](int t) { return ctrl + (34 + t) * 8; };
  auto out_full = [&](int t) { return ctrl + (36 + t) * 8; };
  auto unit_done = [&](int t) { return ctrl + (38 + t) * 8; };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl_ptr + 40 * 8);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl_ptr + 40 * 8 + 4);

  const int G = a.L.G, Hkv = a.L.Hkv;
  const bool fold_k = a.L.U_k == nullptr, fold_v = a.L.U_v == nullptr;
  const int TT = kRows / G;                                     // query tokens per tile
  const Blocks bk = blocks_of(RK), bv = blocks_of(RV);
  const int n_units = ((a.n_q + 2 * TT - 1) / (2 * TT)) * a.Bt.B * Hkv * a.n_split;
  const bool backproj = !fold_v && a.n_split == 1;               // else the compressed (partial) result leaves the kernel
  int32_t* status = a.status;

  if (tid == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 2);        // one arrival from each tile's MMA thread
    }
    for (int t = 0; t < 2; ++t) {
      for (int i = 0; i < 2; ++i) {
        mbar_init(s_full(t, i), 1);
        mbar_init(p_full(t, i), 4);       // one arrival per softmax warp of the tile
        mbar_init(p_free(t, i), 1);
      }
      mbar_init(qacc_full(t), 1);
      mbar_init(qp_ready(t), fold_k ? 1 : 4);   // folded keys: the producer's TMA load completes it
      mbar_init(o_full(t), 1);
      mbar_init(od_ready(t), 4);
      mbar_init(out_full(t), 1);
      mbar_init(unit_done(t), 4);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------------------------------ producer
    if (lane == 0) {
      tma_prefetch_desc(&tmK);
      tma_prefetch_desc(&tmV);
      if (!fold_k) tma_prefetch_desc(&tmUk);
      if (backproj) tma_prefetch_desc(&tmUv);
      tma_prefetch_desc(&tmQ);
    }
    int st = 0, use = 0;                                        // ring stage of the next item, times it has been used
    int kt[2] = {0, 0};
    auto acquire = [&]() -> uint32_t {                          // lane 0 only: next stage, free to be filled
      if (use > 0) mbar_wait(empty_bar(st), (use - 1) & 1, abort_flag, status);
      return ring + st * kStageBytes;
    };
    auto advance = [&]() {
      if (++st == nst) {
        st = 0;
        ++use;
      }
    };
    for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
      const Unit w = decode_unit(a, u, TT);
      if (!w.valid) continue;
      const int npmax = w.cnt;
      const int* bt = a.Bt.block_table + (size_t)w.b * a.Bt.max_pages;
      int ids = lane < npmax ? bt[w.p_lo + lane] : 0;                    // first batch of page ids, in flight during the q loads
      if (lane == 0) {
        if (fold_k) {
          for (int t = 0; t < 2; ++t) {
            if (w.np[t] == 0) continue;
            if (kt[t] > 0) mbar_wait(unit_done(t), (kt[t] - 1) & 1, abort_flag, status);   // the tile's Q' region is free
            mbar_arrive_expect_tx(qp_ready(t), kRows * RK * 2);
            for (int i = 0; i < bk.nb; ++i)
              tma_load_4d(qp + t * a.qp_bytes + i * kRows * bk.span, &tmQ, i * bk.bw, w.h * G, w.tok0[t], w.b, qp_ready(t));
          }
        } else {
          for (int t = 0; t < 2; ++t) {
            if (w.np[t] == 0) continue;
            const uint32_t dst = acquire();
            mbar_arrive_expect_tx(full_bar(st), kStageBytes);
            tma_load_4d(dst, &tmQ, 0, w.h * G, w.tok0[t], w.b, full_bar(st));
            tma_load_4d(dst + kStageBytes / 2, &tmQ, 64, w.h * G, w.tok0[t], w.b, full_bar(st));
            advance();
          }
          const uint32_t dst = acquire();
          mbar_arrive_expect_tx(full_bar(st), kD * RK * 2);
          for (int i = 0; i < bk.nb; ++i)
            tma_load_3d(dst + i * kD * bk.span, &tmUk, i * bk.bw, 0, a.L.uk_stride ? w.h : 0, full_bar(st));
          advance();
        }
      }
      for (int j0 = 0; j0 < npmax; j0 += 32) {
        const int nxt = j0 + 32 + lane < npmax ? bt[w.p_lo + j0 + 32 + lane] : 0;    // the next batch, a batch ahead
        const int cnt = min(32, npmax - j0);
        for (int jj = 0; jj < cnt; ++jj) {
          int pg = __shfl_sync(0xffffffffu, ids, jj);
          if (lane == 0) {
            if (pg < 0 || pg >= a.L.num_pages) {
              report(status, STIEF_ERR_BOUNDS);
              pg = 0;
            }
            const uint32_t dst = acquire();
            const int row = (pg * Hkv + w.h) * kPage;
            mbar_arrive_expect_tx(full_bar(st), kPage * (RK + RV) * 2);
            for (int i = 0; i < bk.nb; ++i) tma_load_2d(dst + i * kPage * bk.span, &tmK, i * bk.bw, row, full_bar(st));
            const uint32_t vdst = dst + kPage * RK * 2;
            for (int i = 0; i < bv.nb; ++i) tma_load_2d(vdst + i * kPage * bv.span, &tmV, i * bv.bw, row, full_bar(st));
            advance();
          }
        }
        ids = nxt;
      }
      if (lane == 0 && backproj) {
        const uint32_t dst = acquire();
        mbar_arrive_expect_tx(full_bar(st), kD * RV * 2);
        for (int i = 0; i < bv.nb; ++i)
          tma_load_3d(dst + i * kD * bv.span, &tmUv, i * bv.bw, 0, a.L.uv_stride ? w.h : 0, full_bar(st));
        advance();
      }
      for (int t = 0; t < 2; ++t) kt[t] += w.np[t] > 0;
    }
  } else if (warp == 1 || warp == 10) {
    // ------------------------------------------------------------------------------------------ MMA issue
    // One thread per tile feeds the tensor core (warp 1 for tile 0, warp 10 for tile 1): issuing a tcgen05.mma costs
    // the issuing thread some tens of cycles, more than these small MMAs (N = 64, K = 16) occupy the tensor pipe, so
    // two issuers keep it busier than one.  Every instruction between two MMAs is on the critical path: descriptors
    // are a per-buffer base plus an offset that is a shift and a mask, and the K loops are unrolled.
    // Both threads walk ALL ring items in order; an item a thread has no use for is released with a plain arrive
    // once it has landed, so each stage always collects two arrivals.
    // The whole warp runs the role's control flow and address arithmetic (so the compiler can keep the descriptors in
    // uniform registers, which is where tcgen05.mma takes them from); only the MMA, commit and arrive instructions
    // themselves are predicated on the leader lane.
    {
      const bool leader = lane == 0;
      const int mt = __shfl_sync(0xffffffffu, warp, 0) == 1 ? 0 : 1;
      const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
      const uint32_t id_qk = idesc_bf16_f32(kRows, kPage);
      const uint32_t id_pv = idesc_bf16_f32_bmn(kRows, RV);
      const uint32_t id_pj = idesc_bf16_f32_bmn(kRows, RK);
      const uint32_t id_bp = idesc_bf16_f32(kRows, kD);
      const uint64_t d_kmaj_k = desc_template(bk.layout, 16, 8 * bk.span);          // Q' rows / K page rows, K = rank
      const uint64_t d_kmaj_v = desc_template(bv.layout, 16, 8 * bv.span);          // O_down rows / U_v rows
      const uint64_t d_sw128 = desc_template(2, 16, 1024);                          // raw q rows, P rows
      const uint64_t d_vpage = desc_template(bv.layout, kPage * bv.span, 8 * bv.span);   // V page, MN-major
      const uint64_t d_uk = desc_template(bk.layout, kD * bk.span, 8 * bk.span);    // U_k, MN-major
      const int nk = RK / 16, nv = RV / 16;
      // descriptor offset (in 16-byte units) of K step k of a K-major operand: inside a block 2 units (32 bytes) per
      // step, then the next block.  Steps per block are 4, 2 or 1: a shift and a mask.
      const int lgk = bk.bw == 64 ? 2 : bk.bw == 32 ? 1 : 0, lgv = bv.bw == 64 ? 2 : bv.bw == 32 ? 1 : 0;
      const uint32_t qblk = (uint32_t)(kRows * bk.span) >> 4, kblk = (uint32_t)(kPage * bk.span) >> 4;
      const uint32_t oblk = (uint32_t)(kRows * bv.span) >> 4;
      auto koff = [](int k, int lg, uint32_t blk) { return (uint32_t)(k >> lg) * blk + (uint32_t)(k & ((1 << lg) - 1)) * 2u; };
      const uint32_t pv_b = (uint32_t)(16 * bv.span) >> 4;                          // V page: 16 rows per K step
      const uint64_t dq = desc_at(d_kmaj_k, qp + mt * a.qp_bytes);                  // this tile's Q' operand
      const uint64_t dod = desc_at(d_kmaj_v, qp + mt * a.qp_bytes);                 // and its O_down operand (same region)
      const uint32_t t_s = tmem_u + mt * 256, t_o = t_s + 128;                   // score buffers; Q' / O accumulator
      int st = 0, use = 0;
      int kt = 0, pn = 0;
      auto consume = [&](uint32_t& addr, int& stage) {          // next item of the ring, once it has landed
        mbar_wait(full_bar(st), use & 1, abort_flag, status);
        addr = ring + st * kStageBytes;
        stage = st;
        if (++st == nst) {
          st = 0;
          ++use;
        }
      };
      auto release = [&](int stage, bool used) {                // after the MMAs that read it, or at once when unused
        if (leader) {
          if (used) umma_commit(empty_bar(stage));
          else mbar_arrive(empty_bar(stage));
        }
      };
      for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
        const Unit w = decode_unit(a, u, TT);
        // the unit's shape comes from global loads; broadcasting it from lane 0 tells the compiler that the control
        // flow and the addresses below are the same in every lane
        if (!__shfl_sync(0xffffffffu, (int)w.valid, 0)) continue;
        const int wnp0 = __shfl_sync(0xffffffffu, w.np[0], 0), wnp1 = __shfl_sync(0xffffffffu, w.np[1], 0);
        const int np = mt ? wnp1 : wnp0;
        const int npmax = __shfl_sync(0xffffffffu, w.cnt, 0);
        const bool active = np > 0;
        const bool dual = a.dual != 0;
        if (!fold_k) {
          uint32_t qa = 0, ua, tmp;
          int qs = -1, us, ts;
          if (wnp0 > 0) {                                       // tile 0's raw queries
            if (mt == 0) consume(qa, qs);
            else { consume(tmp, ts); release(ts, false); }
          }
          if (wnp1 > 0) {                                       // tile 1's
            if (mt == 1) consume(qa, qs);
            else { consume(tmp, ts); release(ts, false); }
          }
          consume(ua, us);
          if (active) {
            if (kt > 0) mbar_wait(unit_done(mt), (kt - 1) & 1, abort_flag, status);   // the tile's accumulator columns are free
            tc_fence_after();
            const uint64_t da = desc_at(d_sw128, qa), db = desc_at(d_uk, ua);
#pragma unroll
            for (int k = 0; k < kD / 16; ++k)
              if (leader) umma_bf16(t_o, da + (uint32_t)(((k >> 2) * (kStageBytes / 2) + (k & 3) * 32) >> 4), db + (uint32_t)(k * bk.span),
                        id_pj, k > 0 ? 1u : 0u);
            if (leader) umma_commit(qacc_full(mt));
            release(qs, true);
          }
          release(us, active);
        }
        if (active) mbar_wait(qp_ready(mt), kt & 1, abort_flag, status);
        tc_fence_after();

        // jo counts this tile's own pages within the unit (every page it shares with the other tile, or every second
        // page of the range when the tiles run as two streams over the same rows)
        auto issue_pv = [&](int jo, uint32_t vaddr, int stage) {
          const int n = pn + jo;
          mbar_wait(p_full(mt, n & 1), (n >> 1) & 1, abort_flag, status);
          tc_fence_after();
          const uint32_t pa = t_s + (n & 1) * 64;                       // P_n: packed bf16 pairs in the score buffer's first 32 columns
          const uint64_t db = desc_at(d_vpage, vaddr);
#pragma unroll
          for (int k = 0; k < kPage / 16; ++k)
            if (leader) umma_bf16_ts(t_o, pa + 8 * k, db + (uint32_t)k * pv_b, id_pv, (jo > 0 || k > 0) ? 1u : 0u);
          if (leader) umma_commit(p_free(mt, n & 1));
          release(stage, true);                                 // K and V of this page are no longer needed by this tile
        };
        uint32_t prev_v = 0;
        int prev_stage = -1, jo = 0;                            // the page whose P V is still to be issued; own pages so far
        for (int j = 0; j < npmax; ++j) {
          uint32_t kaddr;
          int stage;
          consume(kaddr, stage);
          const bool mine = dual ? (j & 1) == mt : j < np;
          if (!mine) {
            release(stage, false);
            continue;
          }
          const int n = pn + jo;
          if (n >= 2) mbar_wait(p_free(mt, n & 1), ((n >> 1) - 1) & 1, abort_flag, status);   // P_(n-2), which sat in this buffer, has been consumed
          tc_fence_after();
          const uint32_t d_tmem = t_s + (n & 1) * 64;
          const uint64_t db = desc_at(d_kmaj_k, kaddr);
#pragma unroll
          for (int k = 0; k < 8; ++k)
            if (k < nk && leader) umma_bf16(d_tmem, dq + koff(k, lgk, qblk), db + koff(k, lgk, kblk), id_qk, k > 0 ? 1u : 0u);
          if (leader) umma_commit(s_full(mt, n & 1));
          if (jo > 0) issue_pv(jo - 1, prev_v, prev_stage);
          prev_v = kaddr + kPage * RK * 2;
          prev_stage = stage;
          ++jo;
        }
        if (jo > 0) issue_pv(jo - 1, prev_v, prev_stage);
        if (active && leader) umma_commit(o_full(mt));
        if (backproj) {
          // OUT = O_down U_v^T with O_down handed over as two bf16 terms (value, then residual): two accumulating
          // passes into the tile's score columns, which are idle by now
          uint32_t ua;
          int us;
          consume(ua, us);
          if (active) {
            const uint64_t db = desc_at(d_kmaj_v, ua);
            for (int pass = 0; pass < 2; ++pass) {
              mbar_wait(od_ready(mt), pass, abort_flag, status);
              tc_fence_after();
#pragma unroll
              for (int k = 0; k < 8; ++k)
                if (k < nv && leader) umma_bf16(t_s, dod + koff(k, lgv, oblk), db + koff(k, lgv, oblk), id_bp, (pass > 0 || k > 0) ? 1u : 0u);
              if (leader) umma_commit(out_full(mt));
            }
          }
          release(us, active);
        }
        pn += np;
        kt += active;
      }
    }
  } else {
    // ------------------------------------------------------------------------------------------ softmax / epilogue
    const int t = (warp - 2) >> 2;                              // the tile this warp works for
    const int q4 = warp & 3;                                    // TMEM lane quarter this warp may access
    const int row = 32 * q4 + lane;                             // row of the tile = TMEM lane
    const uint32_t t_lane = tmem_base + ((uint32_t)(32 * q4) << 16) + t * 256;
    const uint32_t t_out = t_lane + 128;                        // Q' / O columns
    uint8_t* my_qp = qp_ptr + t * a.qp_bytes;
    const float c = kLog2e * rsqrtf((float)kD);                 // scores are scaled by 1/sqrt(d_h); exponent in base 2
    const int d_out = fold_v ? RV : kD;
    int kt = 0, pn = 0;
    int item = 0;                                               // ring items issued before the current unit
    auto arrive_warp = [&](uint32_t bar) {                      // after every lane's shared/TMEM accesses are ordered
      __syncwarp();
      if (lane == 0) mbar_arrive(bar);
    };
    for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
      const Unit w = decode_unit(a, u, TT);
      if (!w.valid) continue;
      const int lead = fold_k ? 0 : (w.np[0] > 0) + (w.np[1] > 0) + 1;      // items ahead of the unit's first page
      const int item0 = item + lead;
      item += lead + w.cnt + (backproj ? 1 : 0);
      if (w.np[t] == 0) continue;
      const int np = w.np[t];
      const int tok = w.tok0[t] + row / G, g = row - (row / G) * G;
      const bool row_valid = tok < w.q_len;
      const int q_pos = w.q_start + min(tok, w.q_len - 1);      // rows past the end behave like the last valid token

      if (!fold_k) {                                            // Q' = bf16(q U_k) into the A operand of the score GEMM
        mbar_wait(qacc_full(t), kt & 1, abort_flag, status);
        tc_fence_after();
        for (int c0 = 0; c0 < RK; c0 += 16) {
          uint32_t v[16], pk[8];
          tmem_ld16(t_out + c0, v);
          tmem_ld_wait();
          pack16(v, 1.0f, pk);
          *reinterpret_cast<uint4*>(my_qp + block_offset(bk, kRows, row, c0)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          *reinterpret_cast<uint4*>(my_qp + block_offset(bk, kRows, row, c0 + 8)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
        }
        fence_proxy_async_smem();
        tc_fence_before();
        arrive_warp(qp_ready(t));
      }

      float m_ref = 0.f, l = 0.f;
      for (int jo = 0; jo < np; ++jo) {
        const int j = a.dual ? 2 * jo + t : jo;                 // the page within the unit's range
        const int n = pn + jo, sb = n & 1;
        mbar_wait(s_full(t, sb), (n >> 1) & 1, abort_flag, status);
        tc_fence_after();
        uint32_t sv[64];
#pragma unroll
        for (int i = 0; i < 4; ++i) tmem_ld16(t_lane + sb * 64 + i * 16, *reinterpret_cast<uint32_t(*)[16]>(&sv[16 * i]));
        tmem_ld_wait();
        float* s = reinterpret_cast<float*>(sv);
        const int p0 = (w.p_lo + j) * kPage;
        if (p0 + kPage - 1 > q_pos) {                           // a boundary page: positions after the row's own are masked
#pragma unroll
          for (int i = 0; i < 64; ++i)
            if (p0 + i > q_pos) s[i] = -INFINITY;
        }
        float mx0 = max3(s[0], s[1], s[2]), mx1 = max3(s[3], s[4], s[5]);     // two chains of three-input maxima
#pragma unroll
        for (int i = 6; i < 62; i += 4) {
          mx0 = max3(mx0, s[i], s[i + 1]);
          mx1 = max3(mx1, s[i + 2], s[i + 3]);
        }
        const float mx = fmaxf(max3(mx0, s[62], s[63]), mx1);
        if (jo == 0) {
          // The reference is the first page's maximum: finite when position 0 is in it.  A later part of a split range
          // can be masked entirely for a row; a finite stand-in then gives p = 0 and an empty partial (l = 0).
          m_ref = fmaxf(mx, -1e30f);
          l = 0.f;
        } else if (__any_sync(0xffffffffu, (mx - m_ref) * c > kRescaleLog2)) {
          mbar_wait(p_free(t, (n - 1) & 1), ((n - 1) >> 1) & 1, abort_flag, status);   // every earlier update of O is complete
          tc_fence_after();
          const float m_new = fmaxf(m_ref, mx);
          const float f = fast_exp2((m_ref - m_new) * c);
          l *= f;
          m_ref = m_new;
          for (int c0 = 0; c0 < RV; c0 += 16) {
            uint32_t v[16];
            tmem_ld16(t_out + c0, v);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * f);
            tmem_st16(t_out + c0, v);
          }
          tmem_st_wait();
        }
        if (p0 + kPage > w.seq_len) {
          // The page holds rows past the end of the sequence: whatever bits they have (NaN included) must not reach
          // the accumulator through 0 * x.  Zero those V rows in the stage (both tiles do; the values are the same).
          const int idx = item0 + j, stg = idx % nst;
          mbar_wait(full_bar(stg), (idx / nst) & 1, abort_flag, status);
          uint8_t* vrows = base_ptr + stg * kStageBytes + kPage * RK * 2;
          const int lo = w.seq_len - p0, cpr = bv.span / 16, per_row = RV / 8;        // first dead row; 16-byte pieces
          for (int e = row; e < (kPage - lo) * per_row; e += kRows) {
            const int r = lo + e / per_row, ch = e % per_row;
            *reinterpret_cast<uint4*>(vrows + (ch / cpr) * kPage * bv.span + r * bv.span + (ch % cpr) * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async_smem();                              // generic writes -> visible to the tensor core's reads
        }
        const uint64_t c2 = pack2(c, c), neg2 = pack2(-m_ref * c, -m_ref * c);
        uint64_t sum2 = pack2(0.f, 0.f);
        uint32_t pk[32];
        // Part of the pairs go to the FMA pipe as a polynomial, where the exponentials and not the MMAs set the pace
        // (small ranks).  The polynomial needs x >= -125 and cannot return an exact zero, so a page on which some row of
        // the warp has masked positions (-inf) takes the special-function unit for all of them: two copies of the loop.
        auto exponentials = [&](auto poly_tag) {
          constexpr bool kPoly = decltype(poly_tag)::value;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            float x0, x1, e0, e1;
            unpack2(fma2(pack2(s[2 * i], s[2 * i + 1]), c2, neg2), x0, x1);
            if (kPoly && (i % kPolyEvery) == 0) {
              exp2_pair_fma(pack2(fmaxf(x0, -125.f), fmaxf(x1, -125.f)), e0, e1);
            } else {
              e0 = fast_exp2(x0);
              e1 = fast_exp2(x1);
            }
            sum2 = add2(sum2, pack2(e0, e1));
            pk[i] = pack_bf16(e0, e1);
          }
        };
        if ((RK + RV <= 160) && !__any_sync(0xffffffffu, p0 + kPage - 1 > q_pos)) exponentials(std::true_type{});
        else exponentials(std::false_type{});
        {
          float a0, a1;
          unpack2(sum2, a0, a1);
          l += a0 + a1;
        }
        // P_n replaces the scores in TMEM: bf16 pairs in the first 32 columns of the buffer, where the P V MMA reads
        // its A operand (no trip through shared memory, no proxy fence)
        tmem_st16(t_lane + sb * 64, *reinterpret_cast<uint32_t(*)[16]>(&pk[0]));
        tmem_st16(t_lane + sb * 64 + 16, *reinterpret_cast<uint32_t(*)[16]>(&pk[16]));
        tmem_st_wait();
        tc_fence_before();
        arrive_warp(p_full(t, sb));
      }

      // ---- epilogue of the unit
      mbar_wait(o_full(t), kt & 1, abort_flag, status);
      tc_fence_after();
      const float inv = 1.0f / l;
      __nv_bfloat16* orow = a.out + (size_t)w.b * a.out_stride_b + (size_t)tok * a.out_stride_t + (size_t)(w.h * G + g) * d_out;
      if (a.n_split > 1) {
        // partial result of this part of the page range: unnormalised mix, reference (base-2 units) and row sum
        const size_t prow = (((size_t)w.b * a.n_q + tok) * a.L.Hq + w.h * G + g) * a.n_parts + (a.dual ? 2 * w.split + t : w.split);
        for (int c0 = 0; c0 < RV; c0 += 16) {
          uint32_t v[16];
          tmem_ld16(t_out + c0, v);
          tmem_ld_wait();
          if (row_valid) {
            float4* dst = reinterpret_cast<float4*>(a.part_o + prow * RV + c0);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              dst[i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]), __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
          }
        }
        if (row_valid) *reinterpret_cast<float2*>(a.part_ml + prow * 2) = make_float2(m_ref * c, l);
      } else if (fold_v) {
        for (int c0 = 0; c0 < RV; c0 += 16) {
          uint32_t v[16], pk[8];
          tmem_ld16(t_out + c0, v);
          tmem_ld_wait();
          pack16(v, inv, pk);
          if (row_valid) {
            *reinterpret_cast<uint4*>(orow + c0) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            *reinterpret_cast<uint4*>(orow + c0 + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
          }
        }
      } else {
        // O_down = O / l goes to the back-projection as bf16(x) and then bf16(x - bf16(x)): two accumulating passes
        // keep about 16 significant bits, so the result is rounded once, at the output
        for (int pass = 0; pass < 2; ++pass) {
          for (int c0 = 0; c0 < RV; c0 += 16) {
            uint32_t v[16], pk[8];
            tmem_ld16(t_out + c0, v);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float x0 = __uint_as_float(v[2 * i]) * inv, x1 = __uint_as_float(v[2 * i + 1]) * inv;
              uint32_t hi, lo;
              split_bf16(x0, x1, hi, lo);
              pk[i] = pass ? lo : hi;
            }
            *reinterpret_cast<uint4*>(my_qp + block_offset(bv, kRows, row, c0)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            *reinterpret_cast<uint4*>(my_qp + block_offset(bv, kRows, row, c0 + 8)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
          }
          fence_proxy_async_smem();
          tc_fence_before();
          arrive_warp(od_ready(t));
          mbar_wait(out_full(t), pass, abort_flag, status);     // the pass has read the operand (after the second: OUT is complete)
          tc_fence_after();
        }
        for (int c0 = 0; c0 < kD; c0 += 16) {
          uint32_t v[16], pk[8];
          tmem_ld16(t_lane + c0, v);
          tmem_ld_wait();
          pack16(v, 1.0f, pk);
          if (row_valid) {
            *reinterpret_cast<uint4*>(orow + c0) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            *reinterpret_cast<uint4*>(orow + c0 + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
          }
        }
      }
      if (row_valid && a.out_lse && a.n_split == 1)
        a.out_lse[((size_t)w.b * a.n_q + tok) * a.L.Hq + w.h * G + g] = kLn2 * (m_ref * c + log2f(l));
      tc_fence_before();
      arrive_warp(unit_done(t));                                // the tile's TMEM columns and operand region are free
      pn += np;
      ++kt;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// Merges the parts of a split page range (log-sum-exp over the parts' references), normalises, back-projects and
// writes the rows.  One block per (token, KV head, sequence): its G query rows share U_v.  A part that had no page
// for the row's tile was never written and is skipped by redoing the range arithmetic of decode_unit.
constexpr int kCombineThreads = 128;
template <int kInstance>                                         // a template only so that the header can be included by several units
__global__ void __launch_bounds__(kCombineThreads)
mq_combine_kernel(const Args a) {
  __shared__ float od[16][kD];                                   // up to 16 query rows of the group at a time
  __shared__ float lse_s[16];
  const int tok = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int G = a.L.G, RV = a.L.r_v, TT = kRows / G;
  int ql = a.q_lens ? a.q_lens[b] : a.n_q;
  ql = min(max(ql, 0), a.n_q);
  const int sl = a.Bt.seq_lens[b], q_start = sl - ql;
  if (tok >= ql || q_start < 0 || (sl + kPage - 1) / kPage > a.Bt.max_pages) return;
  // pages of the row's tile and of the unit (both tiles), as decode_unit derives them
  const int t2 = tok / (2 * TT), first = t2 * 2 * TT;
  int full[2] = {0, 0};
  for (int t = 0; t < 2; ++t)
    if (first + t * TT < ql) full[t] = (q_start + min(first + (t + 1) * TT, ql) - 1) / kPage + 1;
  const int all = max(full[0], full[1]), mine = full[(tok - first) / TT];
  const bool fold_v = a.L.U_v == nullptr;
  const int d_out = fold_v ? RV : kD;
  const __nv_bfloat16* Uv = fold_v ? nullptr : a.L.U_v + (size_t)h * a.L.uv_stride;
  for (int g0 = 0; g0 < G; g0 += 16) {
    const int ng = min(16, G - g0);
    __syncthreads();
    for (int e = threadIdx.x; e < ng * RV; e += kCombineThreads) {
      const int g = e / RV, cidx = e - g * RV;
      const size_t prow = (((size_t)b * a.n_q + tok) * a.L.Hq + h * G + g0 + g) * a.n_parts;
      // part i exists for this row if its share of the page range reaches into the pages of the row's tile
      auto exists = [&](int i) {
        const int sp = a.dual ? i >> 1 : i, off = a.dual ? i & 1 : 0;
        return (int)((long long)sp * all / a.n_split) + off < min((int)((long long)(sp + 1) * all / a.n_split), mine);
      };
      float M = -INFINITY;
      for (int i = 0; i < a.n_parts; ++i)
        if (exists(i)) M = fmaxf(M, a.part_ml[(prow + i) * 2]);
      float num = 0.f, den = 0.f;
      for (int i = 0; i < a.n_parts; ++i)
        if (exists(i)) {
          const float2 ml = *reinterpret_cast<const float2*>(a.part_ml + (prow + i) * 2);
          const float wgt = fast_exp2(ml.x - M);
          den += ml.y * wgt;
          num += a.part_o[(prow + i) * RV + cidx] * wgt;
        }
      od[g][cidx] = num / den;
      if (cidx == 0) lse_s[g] = kLn2 * (M + log2f(den));
    }
    __syncthreads();
    for (int g = 0; g < ng; ++g) {
      const int hq = h * G + g0 + g;
      __nv_bfloat16* orow = a.out + (size_t)b * a.out_stride_b + (size_t)tok * a.out_stride_t + (size_t)hq * d_out;
      if (fold_v) {
        for (int cidx = threadIdx.x; cidx < RV; cidx += kCombineThreads) orow[cidx] = __float2bfloat16_rn(od[g][cidx]);
      } else {
        const int d = threadIdx.x;                               // one output element per thread: row d of U_v
        const uint4* urow = reinterpret_cast<const uint4*>(Uv + (size_t)d * RV);
        float acc = 0.f;
        for (int c8 = 0; c8 < RV / 8; ++c8) {
          const uint4 u = urow[c8];
          const uint32_t wv[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            acc = fmaf(od[g][c8 * 8 + 2 * i], bf16_lo(wv[i]), acc);
            acc = fmaf(od[g][c8 * 8 + 2 * i + 1], bf16_hi(wv[i]), acc);
          }
        }
        orow[d] = __float2bfloat16_rn(acc);
      }
      if (threadIdx.x == 0 && a.out_lse) a.out_lse[((size_t)b * a.n_q + tok) * a.L.Hq + hq] = lse_s[g];
    }
  }
}

// What the host hands to a launcher: the argument block, the five tensor maps, the launch shape.
struct Launch {
  Args a;
  CUtensorMap tmQ, tmUk, tmUv, tmK, tmV;
  int grid, smem;
};

}  // namespace mq

// One launcher per key rank (each its own translation unit); cudaErrorInvalidValue for a value rank that is not compiled in.
cudaError_t launch_mq_rk32(const mq::Launch& l, cudaStream_t st);
cudaError_t launch_mq_rk48(const mq::Launch& l, cudaStream_t st);
cudaError_t launch_mq_rk64(const mq::Launch& l, cudaStream_t st);
cudaError_t launch_mq_rk96(const mq::Launch& l, cudaStream_t st);
cudaError_t launch_mq_rk128(const mq::Launch& l, cudaStream_t st);
cudaError_t launch_mq_combine(const mq::Args& a, cudaStream_t st);


}  // namespace stief
