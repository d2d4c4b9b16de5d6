// Prefill compression on the 5th-generation tensor cores (Eq. 1 for a whole prompt):
//     X_down[t, :] = rnd_bf16( X[t, :] U ),   X = K or V rows of one KV head, U = that head's basis.
// A streaming GEMM with tokens as M (tiles of 128), the rank as N and d_h = 128 as the whole K extent.
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      producer: one TMA tiled load per half tile (128 tokens x 64 elements, 128-byte swizzle)
//               of the caller's [B][T][Hkv][128] tensor into a ring of NST stages, completion on mbarriers.
//   warp 1      MMA: allocates TMEM, and one lane issues tcgen05.mma (kind::f16, bf16 x bf16 -> fp32,
//               M = 128, N = r, 8 instructions of K = 16 per tile) from shared-memory descriptors into one of
//               two TMEM accumulators; tcgen05.commit frees the ring stage and publishes the accumulator.
//   warps 2..9  epilogue, two groups of four warps that take alternate tiles (group g owns accumulator g):
//               tcgen05.ld the accumulator (lane = token row), round to bf16 into a swizzled staging box, TMA
//               store to the paged pool.  The first group also brings the basis into shared memory, transposed
//               to the K-major swizzled layout the MMA wants, one buffer ahead of the MMA warp.
// Work is the list of valid tiles ordered (side, head, sequence, tile) and cut into equal contiguous ranges,
// so a CTA changes basis at most a couple of times.  The projection is HBM-bound (about 43-64 flop per byte
// against a ridge near 250): the tensor pipe idles most of the time by construction, and what matters is that
// no issue slot stands between HBM and the MMA.
//
// Every wait is bounded: when one runs out the status word says STIEF_ERR_TIMEOUT, later waits of the CTA
// return at once, every role walks to the end of its loop, and the TMEM allocation is released.
#include "stief_kernels.h"
#include "stief_partition.cuh"
#include "stief_tc.cuh"

namespace stief {

namespace tc {

constexpr int kTileM = 128;                       // tokens per tile
constexpr int kMaxNST = 4;                        // ring stages (3 when rank 128 and a large batch leave no room)
constexpr int kStageBytes = kTileM * kD * 2;      // 32 KiB: two halves of 128 rows x 128 bytes
constexpr int kHalfBytes = kStageBytes / 2;
constexpr int kThreads = 320;                     // producer warp, MMA warp, two epilogue groups of four warps
constexpr int kTmemCols = 256;                    // two accumulators of up to 128 fp32 columns
constexpr int kCtrlBytes = 256;
constexpr int kSmemLimit = 232448;                // 227 KiB per CTA

// Shared memory, from a 1024-byte aligned base: ring [nst][32 KiB] | two basis buffers [rmax * 256] |
// output staging [8 warps][32 rows][rmax * 2] | barriers and flags | tile prefix sums [B + 1].

struct Args {
  PrefillArgs p;
  int n_side;                // sides that have a basis (1 or 2)
  int side0;                 // which side comes first: 0 = keys, 1 = values
  int n_chunks;              // chunks per unit's tile list (see TileWalker)
  int nst;                   // ring stages
  int rmax;                  // larger of the ranks that are projected
  // quantised cache (QBITS = 8 or 4 only): code pools, value parameters [pages][Hkv][64][groups][2] fp32 (scale, zero),
  // static key parameters [Hkv][groups][2] fp32; groups of 64 channels, the last one shorter for ranks 32, 48, 96
  uint8_t* k_codes;
  uint8_t* v_codes;
  float* v_params;
  const float* k_params;
};

// position of token t (0..63) inside a quantised value page's channel rows (see stief_decode_q.cuh)
__device__ __forceinline__ int q_v_position(int t) {
  const int u = t & 15;
  return (t & ~15) + 4 * ((u & 7) >> 1) + (u & 1) + 2 * (u >> 3);
}

// A tile of the work list
struct WorkTile {
  int side;     // 0 = keys, 1 = values
  int h, b, t0; // head, sequence, first token
  int len;      // tokens of the sequence if this is its last tile, else any value >= t0 + 128
  int unit;     // side slot * Hkv + h: tiles of one unit share a basis
};

// Work list.  A unit is (side, head): its tiles share a basis.  pref[b] = tiles of the sequences before b within
// one unit, tiles_all = pref[B].  Every unit's tile list is cut into n_chunks contiguous chunks of (almost) equal
// size; item j is chunk j / n_units of unit j % n_units, and CTA c works through items c, c + n_cta, ...
// Units vary fastest, so the CTAs that run side by side read the SAME tokens' rows for different heads at about
// the same time: the 256-byte slices of one 2 KiB token row are then fetched together instead of minutes of DRAM
// time apart.  The host picks n_chunks so that the items fill whole waves of CTAs.
// Each role runs a walker on a single thread, so a step is a few adds; divisions happen once per item.
struct TileWalker {
  const int* pref;
  int B, Hkv, side0, tiles_all, n_units, n_chunks, n_cta;
  int j;                           // current item (>= n_units * n_chunks: past the end)
  int left;                        // tiles left in the current item
  int unit, side, h, b, k, nb;     // current unit (its side and head), sequence, tile within it, tiles of the sequence

  __device__ __forceinline__ void load_item() {
    left = 0;
    while (j < n_units * n_chunks) {
      const int u = j % n_units, chunk = j / n_units;
      const int c0 = (int)((long long)chunk * tiles_all / n_chunks), c1 = (int)((long long)(chunk + 1) * tiles_all / n_chunks);
      if (c1 > c0) {
        unit = u;
        const int slot = u / Hkv;
        side = slot == 0 ? side0 : 1 - side0;
        h = u - slot * Hkv;
        int lo = 0, hi = B;                               // largest b with pref[b] <= c0
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (pref[mid] <= c0) lo = mid; else hi = mid;
        }
        b = lo;
        k = c0 - pref[lo];
        nb = pref[lo + 1] - pref[lo];
        left = c1 - c0;
        return;
      }
      j += n_cta;
    }
  }
  __device__ void init(const int* pref_, int B_, int Hkv_, int side0_, int n_side, int n_chunks_, int cta, int n_cta_) {
    pref = pref_; B = B_; Hkv = Hkv_; side0 = side0_; n_cta = n_cta_;
    tiles_all = pref_[B_];
    n_units = n_side * Hkv_;
    n_chunks = max(1, min(n_chunks_, tiles_all));
    unit = side = h = b = k = 0; nb = 1;
    j = tiles_all > 0 ? cta : n_units * n_chunks;
    load_item();
  }
  __device__ __forceinline__ bool valid() const { return left > 0; }
  __device__ __forceinline__ WorkTile cur(const int* seq_lens, int T_max) const {
    WorkTile t;
    t.side = side; t.h = h; t.b = b; t.unit = unit;
    t.t0 = k * kTileM;
    // only a sequence's last tile can be partial; the others never touch global memory here (a dependent
    // global load per tile would serialise the role on memory latency)
    t.len = (k + 1 == nb) ? min(max(seq_lens[b], 0), T_max) : t.t0 + kTileM;
    return t;
  }
  __device__ __forceinline__ void advance() {
    if (--left <= 0) {
      j += n_cta;
      load_item();
      return;
    }
    if (++k < nb) return;
    k = 0;
    do {                                                  // left > 0: a sequence with tiles lies ahead, inside the unit
      ++b;
      nb = pref[b + 1] - pref[b];
    } while (nb == 0);
  }
  // unit of the tile after the current one, or -1 when the CTA has no further tile
  __device__ __forceinline__ int next_unit() const {
    if (left > 1) return unit;
    for (int jj = j + n_cta; jj < n_units * n_chunks; jj += n_cta) {
      const int chunk = jj / n_units;
      if ((int)((long long)(chunk + 1) * tiles_all / n_chunks) > (int)((long long)chunk * tiles_all / n_chunks)) return jj % n_units;
    }
    return -1;
  }
};

}  // namespace tc

using namespace tc;

// Brings one basis U [128][Rn] (bf16, row-major) into shared memory as the K-major operand the MMA reads:
// element (d, j) of U goes to row j, 64-element half d / 64, 16-byte piece ((d % 64) / 8) ^ (j % 8) of the
// 128-byte row.  Called by the 128 threads of the first epilogue group (et = 0..127); each warp's lane 0 then
// arrives on `ready_bar`.
__device__ __forceinline__ void stage_basis(const __nv_bfloat16* __restrict__ U, int Rn, uint8_t* dst, uint32_t ready_bar, int et, int lane) {
  // 16-byte pieces (8 columns of one row d of U), at most 16 per thread, fetched in one or two rounds of
  // independent loads
  const int ppr = Rn / 8, total = kD * ppr;            // pieces per row, pieces in all
#pragma unroll 1
  for (int n0 = 0; n0 < 16 && n0 * 128 < total; n0 += 8) {
  uint4 v[8];
#pragma unroll
  for (int n = 0; n < 8; ++n) {
    const int qi = et + (n0 + n) * 128;
    v[n] = qi < total ? __ldg(reinterpret_cast<const uint4*>(U) + qi) : make_uint4(0u, 0u, 0u, 0u);
  }
#pragma unroll
  for (int n = 0; n < 8; ++n) {
    const int qi = et + (n0 + n) * 128;
    if (qi < total) {
      const int d = qi / ppr, j0 = 8 * (qi - d * ppr);
      const int half = d >> 6, piece = (d & 63) >> 3, e = d & 7;
      const uint32_t w[4] = {v[n].x, v[n].y, v[n].z, v[n].w};
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) {
        const int row = j0 + jj;                       // rows j0 .. j0+7 share row >> 3 (j0 is a multiple of 8)
        const uint32_t off = half * (Rn * 128) + (row >> 3) * 1024 + (row & 7) * 128 + ((piece ^ (row & 7)) << 4) + e * 2;
        *reinterpret_cast<uint16_t*>(dst + off) = (uint16_t)((jj & 1) ? (w[jj >> 1] >> 16) : (w[jj >> 1] & 0xffffu));
      }
    }
  }
  }
  fence_proxy_async_smem();                                // generic-proxy writes -> visible to the tensor core's reads
  __syncwarp();
  if (lane == 0) mbar_arrive(ready_bar);
}

// QBITS = 0: bf16 cache.  QBITS = 8 or 4: the epilogue quantises each group of up to 64 channels of a row to integer
// codes of that width (asymmetric; static key parameters, token-wise value parameters) instead of rounding it to bf16.
template <int QBITS>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                  const __grid_constant__ CUtensorMap tmPK, const __grid_constant__ CUtensorMap tmPV, const Args a) {
  extern __shared__ uint8_t smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int kNST = a.nst;
  const int kUBytes = a.rmax * 256;                             // one basis, K-major: rmax rows of 256 bytes
  const int kOutBytes = 32 * a.rmax * 2;                        // one warp's 32 output rows
  const uint32_t ring = base;                                   // nst stages, each 1024-byte aligned
  const uint32_t ubuf = base + kNST * kStageBytes;              // two basis buffers
  uint8_t* ubuf_ptr = base_ptr + kNST * kStageBytes;
  const uint32_t obuf = ubuf + 2 * kUBytes;                     // output staging, one region per epilogue warp
  uint8_t* obuf_ptr = ubuf_ptr + 2 * kUBytes;
  const uint32_t ctrl = obuf + 8 * kOutBytes;
  uint8_t* ctrl_ptr = obuf_ptr + 8 * kOutBytes;
  auto full_bar = [&](int s) { return ctrl + s * 8; };
  auto empty_bar = [&](int s) { return ctrl + (8 + s) * 8; };
  auto acc_full = [&](int i) { return ctrl + (16 + i) * 8; };
  auto acc_empty = [&](int i) { return ctrl + (18 + i) * 8; };
  auto u_ready = [&](int i) { return ctrl + (20 + i) * 8; };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl_ptr + 22 * 8);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl_ptr + 22 * 8 + 4);
  int* pref = reinterpret_cast<int*>(ctrl_ptr + kCtrlBytes);

  const PrefillArgs& p = a.p;
  const int B = p.Bt.B, Hkv = p.L.Hkv;
  launch_dependents();       // the next kernel on the stream may take over each SM as this grid's CTA leaves it

  if (tid == 0) {
    for (int s = 0; s < kNST; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(acc_full(i), 1);
      mbar_init(acc_empty(i), 4);          // one arrival per epilogue warp
      mbar_init(u_ready(i), 4);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  // tiles per sequence (one head, one side), exclusive prefix sums
  if (warp == 0) {
    int carry = 0;
    for (int b0 = 0; b0 < B; b0 += 32) {
      const int b = b0 + lane;
      int v = 0;
      if (b < B) v = (min(max(p.Bt.seq_lens[b], 0), p.T_max) + kTileM - 1) / kTileM;
      int s = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, s, o);
        if (lane >= o) s += t;
      }
      if (b < B) pref[b + 1] = carry + s;
      carry += __shfl_sync(0xffffffffu, s, 31);
    }
    if (lane == 0) pref[0] = 0;
  }
  if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;


  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      tma_prefetch_desc(&tmK);
      tma_prefetch_desc(&tmV);
      tma_prefetch_desc(&tmPK);
      tma_prefetch_desc(&tmPV);
      TileWalker wk;
      wk.init(pref, B, Hkv, a.side0, a.n_side, a.n_chunks, blockIdx.x, gridDim.x);
      int s = 0, use = 0;                                  // ring stage and how often it has been used
      for (; wk.valid(); wk.advance()) {
        const int t_side = wk.side, t_h = wk.h, t_b = wk.b, t_t0 = wk.k * kTileM;
        if (use > 0) mbar_wait(empty_bar(s), (use - 1) & 1, abort_flag, p.status);
        const uint32_t dst = ring + s * kStageBytes;
        const CUtensorMap* tm = t_side ? &tmV : &tmK;
        mbar_arrive_expect_tx(full_bar(s), kStageBytes);
        tma_load_4d(dst, tm, 0, t_h, t_t0, t_b, full_bar(s));
        tma_load_4d(dst + kHalfBytes, tm, 64, t_h, t_t0, t_b, full_bar(s));
        if (++s == kNST) {
          s = 0;
          ++use;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      int cur_unit = -1, gen = -1;
      uint32_t idesc = 0;
      int R = 0;
      TileWalker wk;
      wk.init(pref, B, Hkv, a.side0, a.n_side, a.n_chunks, blockIdx.x, gridDim.x);
      int s = 0, use = 0;
      for (int i = 0; wk.valid(); wk.advance(), ++i) {
        if (wk.unit != cur_unit) {                         // a new basis: wait until the epilogue warps have staged it
          cur_unit = wk.unit;
          ++gen;
          R = wk.side ? p.L.r_v : p.L.r_k;
          idesc = idesc_bf16_f32(kTileM, R);
          mbar_wait(u_ready(gen & 1), (gen >> 1) & 1, abort_flag, p.status);
        }
        const int acc = i & 1;
        if (i >= 2) mbar_wait(acc_empty(acc), ((i >> 1) - 1) & 1, abort_flag, p.status);
        mbar_wait(full_bar(s), use & 1, abort_flag, p.status);
        tc_fence_after();
        const uint32_t a_base = ring + s * kStageBytes;
        const uint32_t b_base = ubuf + (gen & 1) * kUBytes;
        const uint32_t d_tmem = tmem_base + acc * 128;
#pragma unroll
        for (int k = 0; k < kD / 16; ++k) {
          const uint32_t koff = (k & 3) * 32;              // 16 bf16 = 32 bytes inside the 128-byte swizzled row
          const uint64_t da = kmajor_sw128_desc(a_base + (k >> 2) * kHalfBytes + koff);
          const uint64_t db = kmajor_sw128_desc(b_base + (k >> 2) * (R * 128) + koff);
          umma_bf16(d_tmem, da, db, idesc, k > 0 ? 1u : 0u);
        }
        umma_commit(empty_bar(s));                         // the stage may be refilled once these MMAs have read it
        umma_commit(acc_full(acc));                        // and the accumulator is complete
        if (++s == kNST) {
          s = 0;
          ++use;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (2..9)
    const int q = warp & 3;                                // TMEM lane quarter this warp may read
    const int grp = (warp - 2) >> 2;                       // group 0 takes the even tiles of the CTA, group 1 the odd ones
    const int et = tid - 64;                               // 0..127 inside group 0, which stages the bases
    int cur_unit = -1, gen = -1;
    int R = 0;

    auto stage_basis_of = [&](int side, int h, int g) {
      const __nv_bfloat16* Ub = side ? p.L.U_v : p.L.U_k;
      stage_basis(Ub + (size_t)h * (side ? p.L.uv_stride : p.L.uk_stride), side ? p.L.r_v : p.L.r_k,
                  ubuf_ptr + (g & 1) * kUBytes, u_ready(g & 1), et, lane);
    };

    TileWalker wk;
    wk.init(pref, B, Hkv, a.side0, a.n_side, a.n_chunks, blockIdx.x, gridDim.x);
    if (grp == 0 && wk.valid()) stage_basis_of(wk.side, wk.h, ++gen);      // the basis of the CTA's first tile
    for (int i = 0; wk.valid(); wk.advance(), ++i) {
      const bool mine = (i & 1) == grp;
      if (wk.unit != cur_unit) {
        cur_unit = wk.unit;
        R = wk.side ? p.L.r_v : p.L.r_k;
      }
      // Group 0 stages the next basis one buffer ahead.  That buffer was last read by the MMAs of the unit before
      // the current one, which ended at a tile <= i - 1; they are known to be complete once this group has seen
      // the accumulator of a tile >= that one: its own tile i (then stage after the wait below), else tile i - 1.
      const int nu = grp == 0 ? wk.next_unit() : -1;
      const bool stage_next = nu >= 0 && nu != cur_unit;
      const WorkTile t = wk.cur(p.Bt.seq_lens, p.T_max);
      // the page of this warp's 32 tokens: fetched before the wait so its latency hides behind the accumulator's
      const int tok0 = t.t0 + 32 * q;                      // the warp's first token; its 32 tokens share a page
      int page = -1;
      if (mine && lane == 0 && tok0 < t.len && tok0 / kPage < p.Bt.max_pages)
        page = p.Bt.block_table[(size_t)t.b * p.Bt.max_pages + tok0 / kPage];

      const int acc = i & 1;
      if (mine) {
        mbar_wait(acc_full(acc), (i >> 1) & 1, abort_flag, p.status);
        tc_fence_after();
        // where the warp's 32 rows go
        bool valid = tok0 < t.len;
        page = __shfl_sync(0xffffffffu, page, 0);
        if (valid && (page < 0 || page >= p.L.num_pages)) {
          if (lane == 0) report(p.status, STIEF_ERR_BOUNDS);
          valid = false;
        }
        const bool full = QBITS == 0 && valid && tok0 + 32 <= t.len;   // else the sequence ends inside these rows (or codes are stored)
        const int row0 = (max(page, 0) * Hkv + t.h) * kPage + (tok0 % kPage);  // pool row of the warp's first token
        // full case: rows are rounded to bf16 into swizzled staging boxes and leave by TMA stores.  A box is 32
        // rows x BW elements (BW = 64, 32 or 16: the largest that divides R), swizzle span = box row.
        const int lbw = (R % 64 == 0) ? 6 : (R % 32 == 0) ? 5 : 4;             // log2 of the box width
        const int BW = 1 << lbw, RB = BW * 2, CPB = BW / 8;
        const uint32_t wbase = obuf + (warp - 2) * kOutBytes;
        uint8_t* wptr = obuf_ptr + (warp - 2) * kOutBytes;
        __nv_bfloat16* pool = t.side ? p.L.v_pool : p.L.k_pool;
        uint4* dst = reinterpret_cast<uint4*>(pool + ((size_t)row0 + lane) * R);   // partial case: direct stores
        const bool row_ok = valid && tok0 + lane < t.len;
        if (full) {
          if (lane == 0) bulk_wait_read_all();             // the previous tile's stores have left the staging region
          __syncwarp();
        }
        const uint32_t taddr = tmem_base + ((uint32_t)(32 * q) << 16) + acc * 128;
#pragma unroll
        for (int c0 = 0; c0 < 8; c0 += 4) {                // two batches of up to 64 columns keep the live registers down
          if (c0 * 16 < R) {
            uint32_t v[4][16];
#pragma unroll
            for (int c = 0; c < 4; ++c)
              if ((c0 + c) * 16 < R) tmem_ld16(taddr + (c0 + c) * 16, v[c]);
            tmem_ld_wait();
            if constexpr (QBITS != 0) {
              // columns 16 c0 .. are one quantisation group of this thread's row: 64 of them, or the 32 / 48 that a
              // short last group has (nc chunks of 16).  Codes are decided in fp32 from the fp32 accumulator.
              const int g = c0 >> 2, ng = (R + 63) >> 6, nc = min(4, R / 16 - c0);
              constexpr float kLevels = (float)((1 << QBITS) - 1);
              float sc = 1.f, zp = 0.f;
              if (t.side == 0) {
                const float2 kp = *reinterpret_cast<const float2*>(a.k_params + ((size_t)t.h * ng + g) * 2);
                sc = kp.x;
                zp = kp.y;
              } else {
                float mn = __uint_as_float(v[0][0]), mx = mn;
#pragma unroll
                for (int c = 0; c < 4; ++c)
                  if (c < nc) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                      mn = fminf(mn, __uint_as_float(v[c][e]));
                      mx = fmaxf(mx, __uint_as_float(v[c][e]));
                    }
                  }
                sc = mx > mn ? __fdiv_rn(mx - mn, kLevels) : 1.f;
                zp = mn;
                if (row_ok) *reinterpret_cast<float2*>(a.v_params + (((size_t)row0 + lane) * ng + g) * 2) = make_float2(sc, zp);
              }
              const float inv = __fdiv_rn(1.f, sc);
              // clamp(rint(y), 0, levels) = rint(clamp(y, 0, levels)); adding 1.5 * 2^23 rounds to the nearest integer, ties
              // to even, and leaves it in the low mantissa bits: no float-to-int conversion on this busy path
              auto code = [&](int c, int e) -> uint32_t {
                const float y = __fmul_rn(__fsub_rn(__uint_as_float(v[c][e]), zp), inv);
                return __float_as_uint(__fadd_rn(fminf(fmaxf(y, 0.f), kLevels), 12582912.f)) & 0xFFu;
              };
              const int tp = (row0 % kPage) + lane;                                   // token within its page
              if (t.side) {
                // value codes are stored channel-major with the page's 64 positions permuted (q_v_position)
                if constexpr (QBITS == 8) {
                  // the 32 lanes of the warp write 32 bytes of one channel row
                  if (row_ok) {
                    uint8_t* vrow = a.v_codes + ((size_t)(row0 / kPage) * R + 64 * g) * kPage + q_v_position(tp);
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                      if (c < nc) {
#pragma unroll
                        for (int e = 0; e < 16; ++e) vrow[(size_t)(16 * c + e) * kPage] = (uint8_t)code(c, e);
                      }
                  }
                } else {
                  // 4-bit: a channel row has 32 bytes; the byte of position p also holds position p + 16, which is the
                  // token 16 rows on (lane + 16).  Lanes exchange their codes eight at a time; the lower lane stores.
                  const int pos = q_v_position(tp);
                  uint8_t* vrow = a.v_codes + ((size_t)(row0 / kPage) * R + 64 * g) * 32 + (pos >> 5) * 16 + (pos & 15);
#pragma unroll
                  for (int c = 0; c < 4; ++c)
                    if (c < nc) {                                                     // uniform over the warp
#pragma unroll
                      for (int e8 = 0; e8 < 2; ++e8) {
                        uint32_t mine = 0;
#pragma unroll
                        for (int e = 0; e < 8; ++e) mine |= (row_ok ? code(c, 8 * e8 + e) : 0u) << (4 * e);
                        const uint32_t other = __shfl_xor_sync(0xffffffffu, mine, 16);
                        if (lane < 16 && row_ok) {
#pragma unroll
                          for (int e = 0; e < 8; ++e)
                            vrow[(size_t)(16 * c + 8 * e8 + e) * 32] = (uint8_t)(((mine >> (4 * e)) & 0xFu) | (((other >> (4 * e)) & 0xFu) << 4));
                        }
                      }
                    }
                }
              } else if (row_ok) {
                if constexpr (QBITS == 8) {
                  uint8_t* qdst = a.k_codes + ((size_t)row0 + lane) * R + 64 * g;
#pragma unroll
                  for (int c = 0; c < 4; ++c)
                    if (c < nc) {
                      uint32_t w[4];
#pragma unroll
                      for (int e4 = 0; e4 < 4; ++e4) w[e4] = code(c, 4 * e4) | (code(c, 4 * e4 + 1) << 8) | (code(c, 4 * e4 + 2) << 16) | (code(c, 4 * e4 + 3) << 24);
                      *reinterpret_cast<uint4*>(qdst + 16 * c) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                } else {
                  // 4-bit key rows: per 32 channels, byte i holds channel i (low nibble) and i + 16 (high nibble);
                  // a lone block of 16 channels (rank 48) keeps its high nibbles zero (row padded to 32 bytes)
                  const int krow = R == 48 ? 32 : R / 2;
                  uint8_t* qdst = a.k_codes + ((size_t)row0 + lane) * krow + 32 * g;
#pragma unroll
                  for (int c = 0; c < 4; c += 2)
                    if (c < nc) {
                      const bool has_hi = c + 1 < nc;
                      uint32_t w[4];
#pragma unroll
                      for (int e4 = 0; e4 < 4; ++e4) {
                        uint32_t word = 0;
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                          word |= (code(c, 4 * e4 + e) | ((has_hi ? code(c + 1, 4 * e4 + e) : 0u) << 4)) << (8 * e);
                        w[e4] = word;
                      }
                      *reinterpret_cast<uint4*>(qdst + 8 * c) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
              }
            } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              if ((c0 + c) * 16 < R) {
                uint4 o[2];
                o[0].x = pack_bf16(__uint_as_float(v[c][0]), __uint_as_float(v[c][1]));
                o[0].y = pack_bf16(__uint_as_float(v[c][2]), __uint_as_float(v[c][3]));
                o[0].z = pack_bf16(__uint_as_float(v[c][4]), __uint_as_float(v[c][5]));
                o[0].w = pack_bf16(__uint_as_float(v[c][6]), __uint_as_float(v[c][7]));
                o[1].x = pack_bf16(__uint_as_float(v[c][8]), __uint_as_float(v[c][9]));
                o[1].y = pack_bf16(__uint_as_float(v[c][10]), __uint_as_float(v[c][11]));
                o[1].z = pack_bf16(__uint_as_float(v[c][12]), __uint_as_float(v[c][13]));
                o[1].w = pack_bf16(__uint_as_float(v[c][14]), __uint_as_float(v[c][15]));
                if (full) {
#pragma unroll
                  for (int e = 0; e < 2; ++e) {
                    const int col = 16 * (c0 + c) + 8 * e; // first of the 8 columns in this 16-byte piece
                    const int nb = col >> lbw, cc = (col & (BW - 1)) >> 3;
                    uint32_t off = (uint32_t)(lane * RB + cc * 16);
                    off ^= ((off >> 7) & (uint32_t)(CPB - 1)) << 4;
                    *reinterpret_cast<uint4*>(wptr + ((nb * 32) << (lbw + 1)) + off) = o[e];
                  }
                } else if (row_ok) {                       // rows at or beyond the sequence length stay untouched
                  dst[2 * (c0 + c)] = o[0];
                  dst[2 * (c0 + c) + 1] = o[1];
                }
              }
            }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty(acc));        // this warp has read its quarter of the accumulator
        if (full) {
          fence_proxy_async_smem();                        // generic-proxy writes -> visible to the TMA store
          __syncwarp();
          if (lane == 0) {
            const CUtensorMap* tmP = t.side ? &tmPV : &tmPK;
            for (int nb = 0; nb < (R >> lbw); ++nb) tma_store_2d(tmP, nb * BW, row0, wbase + nb * 32 * RB);
            bulk_commit_group();
          }
        }
      }
      if (stage_next) {
        const int slot = nu / Hkv;
        stage_basis_of(slot == 0 ? a.side0 : 1 - a.side0, nu - slot * Hkv, ++gen);
      }
    }
  }

  if (warp >= 2 && lane == 0) bulk_wait_all();            // this lane's TMA stores are complete
  // Never complete before the kernel this one was allowed to overlap (stream order stays transitive).  One CTA that
  // waits is enough for that; the others leave and hand their SMs to the next kernel, also when the kernel before
  // this one is a longer one that is still at work.
  if (blockIdx.x == 0) grid_dependency_wait();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

namespace {

int sm_count_of_current_device() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    return 148;
  }
  return n;
}

// [B][T_max][Hkv][128] bf16 with element strides (stride_b, stride_t, 128, 1), boxes of 128 tokens x 64 elements
bool make_input_map(CUtensorMap* tm, const void* X, const PrefillArgs& a, bool value_side) {
  const long long stride_b = value_side ? a.v_stride_b : a.stride_b, stride_t = value_side ? a.v_stride_t : a.stride_t;
  const unsigned long long sb = stride_b > 0 ? (unsigned long long)stride_b : (unsigned long long)stride_t * a.T_max;
  const unsigned long long dims[4] = {(unsigned long long)kD, (unsigned long long)a.L.Hkv, (unsigned long long)a.T_max,
                                      (unsigned long long)a.Bt.B};
  const unsigned long long strides[3] = {(unsigned long long)kD * 2, (unsigned long long)stride_t * 2, sb * 2};
  const unsigned box[4] = {64, 1, (unsigned)kTileM, 1};
  return encode_bf16_map(tm, X, 4, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

// pool [num_pages * Hkv * 64 rows][r] bf16, stored in boxes of 32 rows x BW elements, swizzle span = box row
bool make_pool_store_map(CUtensorMap* tm, const void* pool, int r, const PrefillArgs& a) {
  const int bw = (r % 64 == 0) ? 64 : (r % 32 == 0) ? 32 : 16;
  const unsigned long long dims[2] = {(unsigned long long)r, (unsigned long long)a.L.num_pages * a.L.Hkv * kPage};
  const unsigned long long strides[1] = {(unsigned long long)r * 2};
  const unsigned box[2] = {(unsigned)bw, 32};
  const CUtensorMapSwizzle sw = bw == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : bw == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
  return encode_bf16_map(tm, pool, 2, dims, strides, box, sw);
}

int smem_bytes(int nst, int rmax, int B) {
  return 1024 + nst * kStageBytes + 2 * rmax * 256 + 8 * 32 * rmax * 2 + kCtrlBytes + ((B + 1) * 4 + 127) / 128 * 128;
}

}  // namespace

namespace {

template <int QBITS>
cudaError_t launch_prefill_tc(const PrefillArgs& a, const Args* q8, cudaStream_t st) {
  const bool proj_k = a.L.U_k != nullptr, proj_v = a.L.U_v != nullptr;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(prefill_tc_kernel<QBITS>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  CUtensorMap tmK, tmV;
  if (!make_input_map(&tmK, proj_k ? a.K : a.V, a, !proj_k) || !make_input_map(&tmV, proj_v ? a.V : a.K, a, proj_v))
    return cudaErrorInvalidValue;
  CUtensorMap tmPK = tmK, tmPV = tmV;                     // the quantising kernel stores without TMA: placeholders
  if (QBITS == 0 && (!make_pool_store_map(&tmPK, a.L.k_pool, a.L.r_k, a) || !make_pool_store_map(&tmPV, a.L.v_pool, a.L.r_v, a)))
    return cudaErrorInvalidValue;
  Args args = {};
  if (q8) args = *q8;
  args.p = a;
  args.n_side = (proj_k ? 1 : 0) + (proj_v ? 1 : 0);
  args.side0 = proj_k ? 0 : 1;
  args.rmax = 0;
  if (proj_k) args.rmax = a.L.r_k;
  if (proj_v && a.L.r_v > args.rmax) args.rmax = a.L.r_v;
  {
    // items = units x chunks should fill whole waves of CTAs: the fewest waves whose fill is >= 95 %, else the best seen
    const int n_units = args.n_side * a.L.Hkv, n_cta = sm_count_of_current_device();
    int best_chunks = 1;
    double best_fill = 0.0;
    for (int waves = 1; waves <= 8; ++waves) {
      const int chunks = waves * n_cta / n_units;
      if (chunks < 1) continue;
      const int items = chunks * n_units;
      const double fill = (double)items / ((double)((items + n_cta - 1) / n_cta) * n_cta);
      if (fill > best_fill + 1e-9) {
        best_fill = fill;
        best_chunks = chunks;
      }
      if (fill >= 0.95) break;
    }
    args.n_chunks = best_chunks;
  }
  args.nst = kMaxNST;
  while (args.nst > 2 && smem_bytes(args.nst, args.rmax, a.Bt.B) > kSmemLimit) --args.nst;
  const int smem = smem_bytes(args.nst, args.rmax, a.Bt.B);
  if (smem > kSmemLimit) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(sm_count_of_current_device());
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.overlap_previous ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, prefill_tc_kernel<QBITS>, tmK, tmV, tmPK, tmPV, args);
}

}  // namespace

cudaError_t launch_prefill(const PrefillArgs& a, cudaStream_t st) {
  const bool proj_k = a.L.U_k != nullptr, proj_v = a.L.U_v != nullptr;
  if (!proj_k) {
    cudaError_t e = launch_prefill_copy(a, 0, st);
    if (e != cudaSuccess) return e;
  }
  if (!proj_v) {
    cudaError_t e = launch_prefill_copy(a, 1, st);
    if (e != cudaSuccess) return e;
  }
  if (!proj_k && !proj_v) return cudaSuccess;
  return launch_prefill_tc<0>(a, nullptr, st);
}

cudaError_t launch_prefill_quant(const PrefillArgs& a, int bits, uint8_t* k_codes, uint8_t* v_codes, float* v_params,
                                 const float* k_params, cudaStream_t st) {
  Args q = {};
  q.k_codes = k_codes;
  q.v_codes = v_codes;
  q.v_params = v_params;
  q.k_params = k_params;
  return bits == 8 ? launch_prefill_tc<8>(a, &q, st) : bits == 4 ? launch_prefill_tc<4>(a, &q, st) : cudaErrorInvalidValue;
}

}  // namespace stief
