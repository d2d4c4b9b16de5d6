// Persistent split-T decode attention in the compressed space: one launch does the whole decode step
// of a layer -- (optional) projection + append of the new token's k, v (Eq. 1), query projection
// q' = q U_k, scores q' K_down^T, online softmax, mix P V_down, and (optional) the log-sum-exp merge
// over chunks with the back-projection by U_v^T (Eq. 7, Eq. 18).
//
// One CTA per SM.  The batch's page tiles are split evenly over the CTAs (stief_partition.cuh); a CTA
// walks the segments of its range.  Pages are dealt round-robin to NP page lanes.  Each lane has its own
// producer warp, which streams the lane's page tiles K_down[64 x RK], V_down[64 x RV] from HBM into the
// lane's private stages of a shared-memory ring with TMA (hardware swizzle, completion on mbarriers) and
// never stops at segment borders, so the next segment's tiles are already in flight while the consumers
// finish the current one.  A lane's pages are consumed by one warp (small tiles) or by two warps that take
// 32 tokens each (large tiles): scores of the group's query heads against the tokens on the tensor cores,
// online softmax in registers, P V_down accumulated in registers; every consumer warp is an independent
// online-softmax stream.  At a segment's end the warps merge their running (max, sum, accumulator) and
// write one chunk-normalised partial; the CTA that delivers a unit's last partial merges all of them and
// back-projects.
//
// A lane's stages are walked in order and each full-barrier is only waited on by the lane's own consumer
// warps, phase after phase (a parity wait can tell two adjacent phases apart but not more); the empty-
// barrier of a stage collects one arrival per consumer warp of the lane before the producer refills it.
//
// Precision: q' (already scaled by log2(e)/sqrt(128)) and P are each carried as a pair of bf16 words
// (value + remainder) occupying rows 0-7 and 8-15 of the 16-row MMA operand, so the products see
// ~16 significant bits of q' and P; accumulation is fp32.  Up to 8 query heads of a KV head form one
// unit; larger groups become several units.
#pragma once

#include "stief_decode_args.h"
#include "stief_partition.cuh"

namespace stief {

template <int RK, int RV>
struct DecodeCfg {
  using TK = Tile<RK>;
  using TV = Tile<RV>;
  static constexpr int STAGE_BYTES = TK::BYTES + TV::BYTES;
  static constexpr int RING_BUDGET = 192 * 1024;
  static constexpr int NSTAGE_MAX = RING_BUDGET / STAGE_BYTES;
  // Pages are dealt round-robin to NP "page lanes"; a lane owns SPW private ring stages, is fed by its own
  // producer warp and consumed by HALF warps that each take 64 / HALF of the page's tokens (an independent
  // online-softmax stream each).  Small tiles: 4 lanes x 1 warp.  Tiles above 24 KiB leave room for 6 stages
  // only, and one warp per page could not keep up with their MMA work: 2 lanes x 2 warps.
  static constexpr int HALF = NSTAGE_MAX >= 8 ? 1 : 2;
  static constexpr int NP = NSTAGE_MAX >= 8 ? 4 : 2;
  static constexpr int NW = NP * HALF;                   // consumer warps
  static constexpr int SPW = (NSTAGE_MAX / NP) > 4 ? 4 : (NSTAGE_MAX / NP);        // private stages per page lane
  static constexpr int NS = NP * SPW;
  static constexpr int NT = NW * 32;                     // consumer threads
  static constexpr int THREADS = NT + NP * 32;           // + one producer warp per page lane
  static constexpr int RING_BYTES = NS * STAGE_BYTES;
  // scratch after the ring
  static constexpr int CTRL_BYTES = 384;                 // full[16], empty[16], flags
  static constexpr int PREF_BYTES = ((kMaxBatch + 1) * 4 + 15) / 16 * 16;
  static constexpr int QP_BYTES = kGroupTile * kD * 4;   // q' fp32 [8][RK]
  static constexpr int ROWS_BYTES = 10 * kD * 4;         // vectors to project: 8 queries, the new key, the new value
  static constexpr int RED_BYTES = NW * 10 * kD * 4;     // per-warp partial projections: 9 rows of the key side, 1 of the value side
  static constexpr int NEW_BYTES = 2 * kD * 2;           // the appended key and value rows as stored (bf16)
  static constexpr int UNION_BYTES = ROWS_BYTES + RED_BYTES + NEW_BYTES;   // front part also: merge scratch [NW][8][RV]+[2][NW][8]; combine scratch
  static constexpr int SMEM_BYTES = 1024 + RING_BYTES + CTRL_BYTES + PREF_BYTES + QP_BYTES + UNION_BYTES;
  static_assert(RK % 16 == 0 && RV % 16 == 0 && RK <= 128 && RV <= 128, "ranks are multiples of 16 up to 128");
  static_assert(SPW >= 1 && NS <= 16, "ring shape");
  static_assert((NW * 8 * RV + 2 * NW * 8) * 4 <= ROWS_BYTES + RED_BYTES, "merge scratch must fit in front of the appended rows");
  static_assert(kCombineScratchFloats * 4 <= UNION_BYTES && NT >= 128, "combine scratch must fit; combine_unit wants >= 128 threads");
  static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KiB shared memory of an SM");
};

// Projection of a few rows onto a basis, X U with X fp32 [rows][128] in shared memory and U bf16
// [128][R] in global memory, by NW warps.  Warp w contracts the d-range [w*DPW, (w+1)*DPW); lane l owns
// the column pairs l and l+32.  The kernel runs while the whole GPU streams the cache, so a dependent
// global load costs microseconds: a thread therefore fetches its whole slice of U into registers with
// independent loads (one round trip) before any arithmetic.
template <int NW, int R>
struct BasisSlice {
  static constexpr int DPW = ((kD + NW - 1) / NW + 3) / 4 * 4;   // d values per warp (multiple of 4)
  static constexpr int NP = (R / 2 + 31) / 32;                   // column-pair passes per lane
  uint32_t u[NP][DPW];

  __device__ __forceinline__ void load(const __nv_bfloat16* __restrict__ U, int warp, int lane) {
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const int cp = lane + 32 * p;
#pragma unroll
      for (int i = 0; i < DPW; ++i) {
        const int d = warp * DPW + i;
        u[p][i] = (cp < R / 2 && d < kD) ? __ldg(reinterpret_cast<const uint32_t*>(U + (size_t)d * R + 2 * cp)) : 0u;
      }
    }
  }

  // red[(warp*rpw + r)*128 + j] = this warp's share of sum_d rows[r][d] U[d][j], for the rows whose bit is
  // set in row_mask (bit r <-> row r, r < 9); rpw = rows each warp keeps in `red`
  __device__ __forceinline__ void contract(const float* rows, uint32_t row_mask, float* red, int warp, int lane, int rpw = 9) const {
#pragma unroll
    for (int r = 0; r < 9; ++r) {
      if (!((row_mask >> r) & 1u)) continue;               // uniform over the CTA
      float acc[NP][2];
#pragma unroll
      for (int p = 0; p < NP; ++p) acc[p][0] = acc[p][1] = 0.f;
#pragma unroll
      for (int i = 0; i < DPW; i += 4) {
        const int d = warp * DPW + i;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (d < kD) x = *reinterpret_cast<const float4*>(rows + r * kD + d);
        const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
#pragma unroll
          for (int p = 0; p < NP; ++p) {
            acc[p][0] = fmaf(xs[e], bf16_lo(u[p][i + e]), acc[p][0]);
            acc[p][1] = fmaf(xs[e], bf16_hi(u[p][i + e]), acc[p][1]);
          }
      }
#pragma unroll
      for (int p = 0; p < NP; ++p) {
        const int cp = lane + 32 * p;
        if (cp < R / 2) *reinterpret_cast<float2*>(red + (warp * rpw + r) * kD + 2 * cp) = make_float2(acc[p][0], acc[p][1]);
      }
    }
  }
};

// sum over the warps' shares of (row r, column j)
template <int NW>
__device__ __forceinline__ float warp_shares(const float* red, int r, int j, int rpw = 9) {
  float s = 0.f;
#pragma unroll
  for (int w = 0; w < NW; ++w) s += red[(w * rpw + r) * kD + j];
  return s;
}

template <int RK, int RV>
__global__ void __launch_bounds__(DecodeCfg<RK, RV>::THREADS, 1)
decode_persistent_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const DecodeArgs a) {
  using C = DecodeCfg<RK, RV>;
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
  uint8_t* ctrl_ptr = ring_ptr + C::RING_BYTES;
  const uint32_t ctrl = ring + C::RING_BYTES;
  auto full_bar = [&](int s) { return ctrl + s * 8; };
  auto empty_bar = [&](int s) { return ctrl + (16 + s) * 8; };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl_ptr + 33 * 8);
  volatile int* n_pending = reinterpret_cast<volatile int*>(ctrl_ptr + 33 * 8 + 4);   // segments whose arrival is not yet counted
  constexpr int kMaxPending = 4;
  int* pending = reinterpret_cast<int*>(ctrl_ptr + 34 * 8);                           // [kMaxPending][4]: b, j, first CTA or -1, segments
  volatile int* section_free = reinterpret_cast<volatile int*>(ctrl_ptr + 34 * 8 + kMaxPending * 16);   // see the producer
  volatile int* gate = section_free + 1;                   // thread 0's verdict for the segment at hand (see the merge)
  int* pref = reinterpret_cast<int*>(ctrl_ptr + C::CTRL_BYTES);
  float* qp = reinterpret_cast<float*>(ctrl_ptr + C::CTRL_BYTES + C::PREF_BYTES);
  float* un = reinterpret_cast<float*>(ctrl_ptr + C::CTRL_BYTES + C::PREF_BYTES + C::QP_BYTES);

  // The next kernel on the stream may take over each SM as soon as this grid's CTA leaves it.
  launch_dependents();
  unsigned long long* const trc = a.trace ? a.trace + (size_t)c * kTraceSlots : nullptr;
  if (tid == 0) stamp(trc, kTrEntry);
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), HALF);
    }
    *abort_flag = 0;
    *n_pending = 0;
    *section_free = 0;
    mbar_fence_init();
  }
  const int pad = seg_pad_pages(RK, RV);
  build_page_prefix(pref, a.Bt, a.len_add, pad, c == 0 ? a.status : nullptr);   // ends with __syncthreads

  if (tid == 0) stamp(trc, kTrPrefix);
  const int B = a.Bt.B, Hkv = a.L.Hkv, QT = a.QT, G = a.L.G;
  const int upb = Hkv * QT;
  const int total = pref[B] * upb;
  const int P = pages_per_cta(total, n_cta);
  const bool appending = a.k_new != nullptr;

  SegmentWalker walk;
  walk.init(pref, B, upb, pad, c, P, total);
  Segment seg;

  // ------------------------------------------------------------------ producer warps
  // Producer warp pw feeds page lane pw: it issues the TMA loads of every NP-th page into that lane's private
  // stages.  One issuing thread per CTA could not keep up with small page tiles (a page costs it a few hundred
  // cycles of waits and descriptor traffic whatever its size), so the issue work is split the way the pages are.
  if (warp >= NW) {
    const int pw = warp - NW;
    if (lane == 0) {
      tma_prefetch_desc(&tmK);
      tma_prefetch_desc(&tmV);
    }
    // This kernel may overlap its predecessors, which work in other sections of the workspace.  What must be over
    // before the consumers write into this section is the section's previous user, a few launches back; it normally
    // is by the time this CTA starts.  Producer 0 looks (here, and again after each segment while the answer is no)
    // and leaves the answer in shared memory.
    auto look_at_section = [&]() {
      if (pw == 0 && lane == 0 && a.prev_epoch != 0u && *section_free == 0) {
        int seen;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(a.finished) : "memory");
        if ((unsigned)seen == a.prev_epoch) *section_free = 1;
      }
    };
    look_at_section();
    int i_base = 0;            // pages of this CTA before the current segment
    bool issued = false;
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
          const int tile = page * Hkv + h;
          mbar_arrive_expect_tx(full_bar(slot), C::STAGE_BYTES);
          if constexpr (TK::BULK) {
            bulk_load_1d(st, a.L.k_pool + (size_t)tile * kPage * RK, TK::BYTES, full_bar(slot));
          } else {
#pragma unroll
            for (int nb = 0; nb < TK::NB; ++nb)
              tma_load_2d(st + nb * TK::BOX_BYTES, &tmK, TK::tma_x(nb), TK::tma_y(tile), full_bar(slot));
          }
          if constexpr (TV::BULK) {
            bulk_load_1d(st + TK::BYTES, a.L.v_pool + (size_t)tile * kPage * RV, TV::BYTES, full_bar(slot));
          } else {
#pragma unroll
            for (int nb = 0; nb < TV::NB; ++nb)
              tma_load_2d(st + TK::BYTES + nb * TV::BOX_BYTES, &tmV, TV::tma_x(nb), TV::tma_y(tile), full_bar(slot));
          }
          if (pw == 0) {
            if (!issued) stamp(trc, kTrFirstIssue);
            issued = true;
          }
        }
        __syncwarp();
      }
      i_base += npg;
      look_at_section();
    }
    if (pw == 0 && lane == 0) stamp(trc, kTrLastIssue);
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
  int n_seg = 0, n_comb = 0;

  // Counts the arrivals of the noted segments at their units and merges the units this CTA completed (see below).
  auto settle = [&]() -> int {
    const int np_ = *n_pending;
    __threadfence();                                       // this thread's partial stores are visible GPU-wide
    bar1(NT);
    if (tid < np_) {
      const int pb = pending[4 * tid], pj = pending[4 * tid + 1];
      int first, last;
      unit_cta_span(pref, upb, pad, P, pb, pj, &first, &last);
      const int nseg = last - first + 1, u = pb * upb + pj;
      int is_last = 1;
      if (nseg > 1) {
        const int prev = atomicAdd(a.counters + u, 1);
        is_last = (prev == nseg - 1);
        if (is_last) a.counters[u] = 0;                    // leave the counter clean for the next call
      }
      pending[4 * tid + 2] = is_last ? first : -1;
      pending[4 * tid + 3] = nseg;
    }
    bar1(NT);
    if (tid == 0) stamp(trc, kTrArrived);
    int done = 0;
    for (int e = 0; e < np_; ++e) {
      const int first = pending[4 * e + 2];
      if (first < 0) continue;                             // uniform over the CTA
      const int pb = pending[4 * e], pj = pending[4 * e + 1], nseg = pending[4 * e + 3];
      __threadfence();
      combine_unit<RV>(a.L, pb, pj / QT, pj % QT, first + pb * upb + pj, nseg, a.partial_o, a.partial_lse, a.out, a.out_lse, un, tid, NT);
      ++done;
    }
    bar1(NT);
    if (tid == 0) *n_pending = 0;
    bar1(NT);
    return done;
  };

  while (walk.next(seg)) {
    ++n_seg;
    const int b = seg.b, h = seg.j / QT, qt = seg.j % QT;
    const int npg = seg.p1 - seg.p0;
    const int ng = min(kGroupTile, G - qt * kGroupTile);
    const size_t head0 = (size_t)b * a.L.Hq + (size_t)h * G + (size_t)qt * kGroupTile;
    const int pos_raw = a.Bt.seq_lens[b];                            // first use is well below: the load runs meanwhile
    const bool has_final = seg.p1 == seg.npages;
    // This step's token is appended by the CTA whose segment holds the sequence's last page.  Its projected rows go to
    // the pool for later steps; THIS step reads them from shared memory: the page tile arrives with whatever the pool
    // held at that row and the consumer that owns the row overwrites it in the stage before use.  Nothing therefore
    // waits for the stores to land, and the producers never wait for the consumers.
    const bool may_append = appending && has_final;
    // The page that will take the new rows: when a token is appended the sequence's last page is the one at index
    // npages - 1 of its block table, which is known without waiting for seq_lens.  Every global load of the prologue
    // is issued up front: one issued a microsecond later queues behind the page requests of the whole GPU.
    int new_page = -1;
    if (may_append) new_page = a.Bt.block_table[(size_t)b * a.Bt.max_pages + seg.npages - 1];

    // ---- prologue: q' = q U_k for the unit's queries (rows 0..7), the new key's row k U_k (row 8) and the
    // new value's row v U_v.  All global loads are issued before the first use of any of them.
    float* rows = un;                    // [9][128] fp32
    float* vrow = un + 9 * kD;           // [128]
    float* red = un + 10 * kD;           // [NW][9][128]
    float* redv = red + NW * 9 * kD;     // [NW][128]
    __nv_bfloat16* newk = reinterpret_cast<__nv_bfloat16*>(redv + NW * kD);   // [128] the appended key row as stored
    __nv_bfloat16* newv = newk + kD;                                          // [128] the appended value row
    const __nv_bfloat16* Uk = a.L.U_k ? a.L.U_k + (size_t)h * a.L.uk_stride : nullptr;
    const __nv_bfloat16* Uv = a.L.U_v ? a.L.U_v + (size_t)h * a.L.uv_stride : nullptr;
    const uint32_t row_mask = ((1u << ng) - 1u) | (may_append ? 0x100u : 0u);
    // a side without a basis is handled in its own dimension: its q / k (or v) rows arrive with r elements
    const int dk = Uk ? kD : RK, dv = Uv ? kD : RV;
    bool do_append = false;
    size_t new_row = ~(size_t)0;
    {
      BasisSlice<NW, RK> sk;
      BasisSlice<NW, RV> sv;
      if (Uk) sk.load(Uk, warp, lane);
      if (may_append && Uv) sv.load(Uv, warp, lane);
      // rows as 16-byte pieces: piece idx -> row idx / 16, elements 8 * (idx % 16) ..
      constexpr int NPC = (9 * 16 + NT - 1) / NT;
      uint4 pc[NPC];
#pragma unroll
      for (int i = 0; i < NPC; ++i) {
        const int idx = tid + i * NT, r = idx / 16, c = idx % 16;
        pc[i] = make_uint4(0u, 0u, 0u, 0u);
        if (8 * c < dk) {
          if (r < ng) pc[i] = __ldg(reinterpret_cast<const uint4*>(a.q + (head0 + r) * dk) + c);
          else if (r == 8 && may_append) pc[i] = __ldg(reinterpret_cast<const uint4*>(a.k_new + ((size_t)b * Hkv + h) * dk) + c);
        }
      }
      uint4 pv = make_uint4(0u, 0u, 0u, 0u);
      if (may_append && tid < 16 && 8 * tid < dv) pv = __ldg(reinterpret_cast<const uint4*>(a.v_new + ((size_t)b * Hkv + h) * dv) + tid);
#pragma unroll
      for (int i = 0; i < NPC; ++i) {
        const int idx = tid + i * NT;
        if (idx < 9 * 16) {
          const uint32_t w[4] = {pc[i].x, pc[i].y, pc[i].z, pc[i].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) *reinterpret_cast<float2*>(rows + idx * 8 + 2 * e) = make_float2(bf16_lo(w[e]), bf16_hi(w[e]));
        }
      }
      if (may_append && tid < 16) {
        const uint32_t w[4] = {pv.x, pv.y, pv.z, pv.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) *reinterpret_cast<float2*>(vrow + tid * 8 + 2 * e) = make_float2(bf16_lo(w[e]), bf16_hi(w[e]));
      }
      // where the new rows go (pos_raw / 64 == npages - 1 unless the sequence outgrew its block table: then nothing is appended)
      if (may_append && pos_raw >= 0 && pos_raw / kPage < a.Bt.max_pages && pos_raw / kPage == seg.npages - 1) {
        do_append = true;
        if (new_page >= 0 && new_page < a.L.num_pages) new_row = ((size_t)new_page * Hkv + h) * kPage + (pos_raw % kPage);
      }
      bar1(NT);
      if (Uk) sk.contract(rows, row_mask, red, warp, lane);
      if (may_append && Uv) sv.contract(vrow, 1u, redv, warp, lane, 1);      // the value row sits where row 0 is expected
    }
    bar1(NT);
    for (int idx = tid; idx < 9 * RK; idx += NT) {
      const int r = idx / RK, j = idx % RK;
      if (!((row_mask >> r) & 1u)) {
        if (r < 8) qp[r * RK + j] = 0.f;
        continue;
      }
      const float x = Uk ? warp_shares<NW>(red, r, j) : rows[r * kD + j];
      if (r < 8) {
        qp[r * RK + j] = x * qscale;
      } else {
        const __nv_bfloat16 xb = __float2bfloat16_rn(x);
        newk[j] = xb;
        if (new_row != ~(size_t)0) a.L.k_pool[new_row * RK + j] = xb;
      }
    }
    if (may_append) {
      for (int j = tid; j < RV; j += NT) {
        const __nv_bfloat16 xb = __float2bfloat16_rn(Uv ? warp_shares<NW>(redv, 0, j, 1) : vrow[j]);
        newv[j] = xb;
        if (new_row != ~(size_t)0) a.L.v_pool[new_row * RV + j] = xb;
      }
      if (do_append && new_row == ~(size_t)0 && tid == 0) report(a.status, STIEF_ERR_BOUNDS);
    }
    bar1(NT);
    const int len = min(max(pos_raw + a.len_add, 0), seg.npages * kPage);
    const int last_valid = len - (seg.npages - 1) * kPage;          // tokens in the sequence's last page (1..64)

    // A operand of the score MMA: rows 0-7 = bf16(q'), rows 8-15 = bf16(q' - bf16(q'))
    uint32_t qa[RK / 16][4];
#pragma unroll
    for (int ks = 0; ks < RK / 16; ++ks) {
      const float2 x = *reinterpret_cast<const float2*>(qp + gid * RK + 16 * ks + 2 * tid4);
      const float2 y = *reinterpret_cast<const float2*>(qp + gid * RK + 16 * ks + 8 + 2 * tid4);
      split_bf16(x.x, x.y, qa[ks][0], qa[ks][1]);
      split_bf16(y.x, y.y, qa[ks][2], qa[ks][3]);
    }

    if (tid == 0 && n_seg == 1) stamp(trc, kTrPrologue);
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
      if (tid == 0 && i_base + k == 0) stamp(trc, kTrFirstPage);
      const uint32_t kt = ring + slot * C::STAGE_BYTES;
      const uint32_t vt = kt + TK::BYTES;
      const bool final_page = seg.p0 + k == seg.npages - 1;
      const bool tail = final_page && (last_valid < kPage);
      if (HALF > 1 && tail && last_valid <= tb) {          // none of this warp's tokens exists: nothing to add
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar(slot));
        continue;
      }

      // this step's own token is the sequence's last one: its rows are put into the tile here (see the prologue)
      const int tn = last_valid - 1;
      const bool patch = do_append && final_page && tn >= tb && tn < tb + kPage / HALF;
      if (patch) {
        if (lane < RK / 8) {
          const uint4 w = *reinterpret_cast<const uint4*>(newk + 8 * lane);
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(kt + TK::chunk(tn, lane)), "r"(w.x), "r"(w.y), "r"(w.z), "r"(w.w) : "memory");
        }
        if (lane < RV / 8) {
          const uint4 w = *reinterpret_cast<const uint4*>(newv + 8 * lane);
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(vt + TV::chunk(tn, lane)), "r"(w.x), "r"(w.y), "r"(w.z), "r"(w.w) : "memory");
        }
        __syncwarp();
      }

      // ---- scores of the page: n-tile j covers tokens 8j..8j+7; c0,c1 from bf16(q'), c2,c3 from the remainder
      float sc[2 * NJ];
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int q4 = 0; 4 * q4 + 4 <= NCH; ++q4) {
          uint32_t r0, r1, r2, r3;
          ldsm_x4(kt + (koff[q4] ^ ((j & 1) * TK::K8X)) + (hf * NJ + j) * 8 * TK::RB, r0, r1, r2, r3);
          mma_bf16(s, qa[2 * q4], r0, r1);
          mma_bf16(s, qa[2 * q4 + 1], r2, r3);
        }
        if constexpr (NCH % 4 == 2) {
          uint32_t r0, r1;
          ldsm_x2(kt + (koff[NCH / 4] ^ ((j & 1) * TK::K8X)) + (hf * NJ + j) * 8 * TK::RB, r0, r1);
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

      if (tail || patch) fence_proxy_async_smem();          // generic-proxy writes to the stage before TMA refills it
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar(slot));
    }
    i_base += npg;
    if (tid == 0) stamp(trc, kTrLastPage);                 // overwritten by every segment: the last one stays

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
    // Everything up to here only read inputs (and appended this step's rows).  This section of the workspace may
    // still be in use by its previous user when the launch overlaps earlier kernels.  Thread 0 settles the question
    // for the CTA before the barrier: yes if producer 0 saw that user's epoch in the control word, else it looks once
    // more itself; without a yes everyone waits for the predecessor grid (which completes only after all before it).
    if (tid == 0) {
      int go = *section_free;
      if (go == 0 && a.prev_epoch != 0u) {
        int seen;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(a.finished) : "memory");
        go = (unsigned)seen == a.prev_epoch;
        if (go) *section_free = 1;
      }
      *gate = go;
    }
    bar1(NT);
    const int u = b * upb + seg.j;
    const int slot_id = c + u;
    if (*gate == 0) grid_dependency_wait();
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

    if (tid == 0) stamp(trc, kTrPartial);
    // ------------------------------------------------------------------ the unit's last partial triggers the combine
    // Counting the arrival means a fence and an atomic whose answer must come back: two trips through a memory system
    // that is busy streaming pages.  Between segments that would stall the consumers while the ring fills up, so the
    // segment is only noted here; the arrivals of all noted segments are counted together once the CTA has no pages left
    // (or the list is full), one thread per segment, and whichever of them turn out to be last are merged then.
    if (a.out != nullptr) {
      if (tid == 0) {
        int* e = pending + 4 * *n_pending;
        e[0] = b; e[1] = seg.j;
        *n_pending = *n_pending + 1;
      }
      bar1(NT);
      if (*n_pending == kMaxPending) n_comb += settle();
    } else {
      bar1(NT);
    }
  }
  if (a.out != nullptr) {
    if (*n_pending > 0) n_comb += settle();
    if (tid == 0) stamp(trc, kTrCombined);
  }

  // units of empty sequences get their zero rows from CTA (u mod n_cta)
  int n_zero = 0;
  if (a.out != nullptr) {
    for (int u = c; u < B * upb; u += n_cta) {
      const int b = u / upb, j = u % upb;
      if (pref[b + 1] != pref[b]) continue;
      const int h = j / QT, qt = j % QT;
      const int ng = min(kGroupTile, G - qt * kGroupTile);
      const size_t head0 = (size_t)b * a.L.Hq + (size_t)h * G + (size_t)qt * kGroupTile;
      const int d_out = a.L.U_v ? kD : RV;
      for (int idx = tid; idx < ng * d_out; idx += NT) a.out[head0 * d_out + idx] = __float2bfloat16_rn(0.f);
      if (a.out_lse && tid < ng) a.out_lse[head0 + tid] = -INFINITY;
      ++n_zero;
    }
  }
  // Every unit is finalised by exactly one CTA (merged, or zero-filled).  The CTA that finalises the kernel's last unit
  // publishes the kernel's epoch: from then on this section of the workspace is free for its next user.  That CTA also
  // waits for the predecessor grid before it leaves, so that this grid never completes before an earlier one (stream
  // order stays transitive); the others leave at once and hand their SMs to the next kernel.
  if (a.out == nullptr) {
    grid_dependency_wait();
  } else if (n_comb + n_zero > 0) {
    bar1(NT);                                              // all of the CTA's reads of partials and writes of outputs are issued
    if (tid == 0) {
      __threadfence();
      const int before = atomicAdd(a.units_done, n_comb + n_zero);
      if (before + n_comb + n_zero == B * upb) {
        *a.units_done = 0;
        __threadfence();
        asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(a.finished), "r"((int)a.epoch) : "memory");
        grid_dependency_wait();
      }
    }
  }
  if (tid == 0 && trc) {
    stamp(trc, kTrExit);
    trc[kTrSegments] = (unsigned long long)n_seg;
    trc[kTrCombines] = (unsigned long long)n_comb;
    unsigned smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    trc[kTrSm] = smid;
  }
}

}  // namespace stief
