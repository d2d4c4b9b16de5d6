// Decode attention over the integer-quantised compressed cache (paper Sec. 4.3; 8-bit and 4-bit codes, every rank):
// the persistent split-T kernel of stief_decode.cuh with the page operands kept as integer codes all the way into
// the tensor cores.
//
// The cache holds, per (page, head): K codes [64 tokens][key row bytes] (token-major), V codes [RV channels][64
// positions] (channel-major, see below) and the value rows' (scale, zero) pairs, one pair per group of 64 channels
// (the last group of ranks 32, 48, 96 is shorter).  K and V tiles are fetched by TMA box loads, with a hardware swizzle
// where ldmatrix would otherwise meet bank conflicts, the parameters by a 1-D bulk copy.  Both contractions run on
// mma.sync s8 x u8 -> s32 (k = 32; one k = 16 step for the 16-channel remainder of rank 48) with the raw codes as B operand:
//   scores: A = q' (key scale folded in) as a per-row 16-bit fixed point split into two signed 8-bit digits, which
//           occupy rows 0-7 and 8-15 of the 16-row operand; the integer sums are recombined as 256 hi + lo and
//           scaled back per row.  The key zero-point shifts all scores of a row equally: it only enters out_lse.
//   mix:    A = p_t * scale_t,g per value group g, again as two digits of a per-row, per-page fixed point; the value
//           zero-points add sum_t p_t zero_t,g to every channel of the group (kept as a running scalar per group).
// No code is ever expanded to floating point in shared memory.
//
// 4-bit codes are stored two to a byte in the order the tensor cores will want them after a shift and a mask: within
// 32 consecutive contraction indices (channels of a key row, token positions of a value row) byte i holds index i in
// its low and index i + 16 in its high nibble.  A 32-bit word of ldmatrix output then unpacks with (w & 0x0f0f0f0f) and
// ((w >> 4) & 0x0f0f0f0f) into exactly the two B registers of one k = 32 step.  Key rows of rank 48 are padded to 64
// nibbles (32 bytes), the unused ones zero.
//
// Why value pages are channel-major and their 64 token positions permuted: the B fragment of the mix needs four
// consecutive TOKENS of one channel in a register, which is what ldmatrix delivers from channel-major rows; and the
// A fragment wants, for the thread (gid, tid4), the probabilities of k-slots 4 tid4 .. 4 tid4 + 3 of each 16-slot
// chunk, while the score accumulators leave that thread with tokens 2 tid4, 2 tid4 + 1 of each 8-token tile.  So
// within every 16 tokens, token u sits at position 4 (u mod 8 / 2) + (u mod 2) + 2 (u / 8): the thread's own
// probabilities are then exactly its A fragment and no lane ever exchanges data (v_position() below).
//
// Four page lanes, each with its own producer warp and two consumer warps that take 32 tokens of a page each.
#pragma once

#include "stief_decode.cuh"
#include "stief_partition.cuh"

namespace stief {

struct DecodeQArgs {
  LayerDev L;                    // bases and shape (the bf16 pool pointers are unused)
  BatchDev Bt;
  uint8_t* k_codes;              // [pages][Hkv][64][key row bytes]
  uint8_t* v_codes;              // [pages][Hkv][RV][64 positions, 8 or 4 bits each]
  float* v_params;               // [pages][Hkv][64][groups of RV][2] (scale, zero)
  const float* k_params;         // [Hkv][groups of RK][2] (scale, zero)
  const __nv_bfloat16* q;        // [B][Hq][128]
  const __nv_bfloat16* k_new;    // [B][Hkv][128] or NULL: project, quantise and store at position seq_lens[b] first
  const __nv_bfloat16* v_new;
  float* partial_o;
  float* partial_lse;
  int* counters;
  // one section of the workspace, its control words and the epochs: as in DecodeArgs
  int* finished;
  int* units_done;
  unsigned epoch, prev_epoch;
  __nv_bfloat16* out;
  float* out_lse;
  int len_add;
  int QT;
  int32_t* status;
};

// position of token t (0..63) inside a value page's channel rows
__host__ __device__ __forceinline__ int v_position(int t) {
  const int u = t & 15;
  return (t & ~15) + 4 * ((u & 7) >> 1) + (u & 1) + 2 * (u >> 3);
}

// bytes of one key row: RK codes of BITS bits (rank 48 at 4 bits is padded to 32 bytes)
__host__ __device__ constexpr int q_key_row_bytes(int rk, int bits) { return bits == 8 ? rk : (rk == 48 ? 32 : rk / 2); }
__host__ __device__ constexpr int q_groups(int r) { return (r + 63) / 64; }

// Byte offset of 16-byte chunk c of row t in a shared-memory tile of 64 rows of ROWB bytes, as TMA leaves it:
//   16, 48: dense rows (ldmatrix on 8 consecutive rows is conflict-free as it is)
//   32, 64, 128: boxes of 64 rows with the swizzle span of the row (32-, 64-, 128-byte swizzle)
//   96:     the tile viewed as 192 lines of 32 bytes, 32-byte swizzle on the linear offset
// A step of 8 rows leaves the swizzle term unchanged in every form.
template <int ROWB>
__device__ __forceinline__ uint32_t qtile_chunk(int t, int c) {
  uint32_t off = static_cast<uint32_t>(t * ROWB + c * 16);
  if constexpr (ROWB == 32 || ROWB == 96) off ^= ((off >> 7) & 1u) << 4;
  if constexpr (ROWB == 64) off ^= ((off >> 7) & 3u) << 4;
  if constexpr (ROWB == 128) off ^= ((off >> 7) & 7u) << 4;
  return off;
}

// ---- where a code goes ------------------------------------------------------------------------------------------
// Byte (and, for 4-bit codes, nibble) that holds contraction index i of a row: 8-bit: byte i; 4-bit: within every 32
// indices, byte i % 16 of the block holds index i (low nibble) and i + 16 (high nibble).
template <int BITS>
__host__ __device__ __forceinline__ int q_code_byte(int i) { return BITS == 8 ? i : (i >> 5) * 16 + (i & 15); }
template <int BITS>
__host__ __device__ __forceinline__ int q_code_shift(int i) { return BITS == 8 ? 0 : 4 * ((i >> 4) & 1); }

// The quantiser's decision (fp32, round to nearest even, clamp): code = clamp(rint((x - zero) * (1 / scale)))
template <int BITS>
__device__ __forceinline__ uint32_t q_encode(float x, float scale, float zero) {
  const float y = __fmul_rn(__fsub_rn(x, zero), __fdiv_rn(1.f, scale));
  return (uint32_t)fminf(fmaxf(rintf(y), 0.f), (float)((1 << BITS) - 1));
}

// Writes one key row from per-channel codes in shared memory (codes[j], j < RK): byte b of the row is assembled by one thread.
template <int RK, int BITS>
__device__ __forceinline__ void q_store_key_row(uint8_t* row, const uint8_t* codes, int tid, int nt) {
  constexpr int KROW = q_key_row_bytes(RK, BITS);
  for (int bi = tid; bi < KROW; bi += nt) {
    if constexpr (BITS == 8) {
      row[bi] = codes[bi];
    } else {
      const int lo = (bi >> 4) * 32 + (bi & 15), hi = lo + 16;
      row[bi] = (uint8_t)((lo < RK ? codes[lo] : 0) | ((hi < RK ? codes[hi] : 0) << 4));
    }
  }
}

// Writes the code of one (channel row, position) of a value page.  4-bit: the byte is shared with the token 16 positions
// away, which is written at another time: the nibble is replaced with two atomic bit operations on the enclosing word.
template <int BITS>
__device__ __forceinline__ void q_store_value_code(uint8_t* channel_row, int pos, uint32_t code) {
  if constexpr (BITS == 8) {
    channel_row[pos] = (uint8_t)code;
  } else {
    uint8_t* bp = channel_row + q_code_byte<4>(pos);
    unsigned* w = reinterpret_cast<unsigned*>(reinterpret_cast<uintptr_t>(bp) & ~(uintptr_t)3);
    const int sh = 8 * (int)(reinterpret_cast<uintptr_t>(bp) & 3) + q_code_shift<4>(pos);
    atomicAnd(w, ~(0xFu << sh));
    atomicOr(w, code << sh);
  }
}

template <int RK, int RV, int BITS>
struct DecodeQCfg {
  static_assert(BITS == 8 || BITS == 4, "8-bit or 4-bit codes");
  static constexpr int KROW = q_key_row_bytes(RK, BITS); // bytes of a key row
  static constexpr int VROW = BITS == 8 ? 64 : 32;       // bytes of a value channel row (64 positions)
  static constexpr int NGK = q_groups(RK), NGV = q_groups(RV);
  static constexpr int K_BYTES = kPage * KROW, V_BYTES = RV * VROW, P_BYTES = kPage * NGV * 8;
  static constexpr int TX_BYTES = K_BYTES + V_BYTES + P_BYTES;           // bytes one page brings into a stage
  static constexpr int STAGE_BYTES = (TX_BYTES + 1023) / 1024 * 1024;    // stages keep the key tile's swizzle alignment
  static constexpr int HALF = 2;
  static constexpr int NP = 4;
  static constexpr int NW = NP * HALF;
  static constexpr int NT = NW * 32;
  static constexpr int THREADS = NT + NP * 32;
  static constexpr int CTRL_BYTES = 512;
  static constexpr int PREF_BYTES = ((kMaxBatch + 1) * 4 + 127) / 128 * 128;
  static constexpr int QP_BYTES = kGroupTile * kD * 4;
  static constexpr int ROWS_BYTES = 10 * kD * 4;
  static constexpr int RED_BYTES = NW * 9 * kD * 4;
  static constexpr int UNION_BYTES = ROWS_BYTES + RED_BYTES;
  static constexpr int MISC = CTRL_BYTES + PREF_BYTES + QP_BYTES + UNION_BYTES;
  static constexpr int RING_BUDGET = 232448 - 1024 - MISC;
  static constexpr int SPW = (RING_BUDGET / (NP * STAGE_BYTES)) > 4 ? 4 : (RING_BUDGET / (NP * STAGE_BYTES));
  static constexpr int NS = NP * SPW;
  static constexpr int RING_BYTES = NS * STAGE_BYTES;
  static constexpr int SMEM_BYTES = 1024 + RING_BYTES + MISC;
  static_assert(RK % 16 == 0 && RV % 16 == 0 && RK >= 32 && RV >= 32 && RK <= 128 && RV <= 128, "ranks are multiples of 16 in 32..128");
  static_assert(K_BYTES % 1024 == 0 && V_BYTES % 16 == 0, "the value tile and the parameters keep their alignment behind the key tile");
  static_assert(SPW >= 2 && NS <= 16, "ring shape");
  static_assert((NW * 8 * RV + 2 * NW * 8) * 4 <= UNION_BYTES, "merge scratch must fit");
  static_assert(kCombineScratchFloats * 4 <= UNION_BYTES, "combine scratch must fit");
  static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KiB shared memory of an SM");
};

// D += A(16x32, row, s8) * B(32x8, col, u8), s32 accumulate
__device__ __forceinline__ void mma_s8u8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// D += A(16x16, row, s8) * B(16x8, col, u8), s32 accumulate
__device__ __forceinline__ void mma_s8u8_k16(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(b0));
}
__device__ __forceinline__ void ldsm_x1(uint32_t addr, uint32_t& r0) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x1.shared.b16 {%0}, [%1];" : "=r"(r0) : "r"(addr));
}

// Two signed 8-bit digits of a 16-bit fixed-point value a in [-32640, 32639]: a = 256 hi + lo, both in [-128, 127]
__device__ __forceinline__ void digits(float x, float inv_delta, int& hi, int& lo) {
  int v = __float2int_rn(x * inv_delta);
  v = max(-32640, min(32639, v));
  hi = (v + 128) >> 8;
  lo = v - (hi << 8);
}
__device__ __forceinline__ uint32_t pack4(int b0, int b1, int b2, int b3) {
  return (uint32_t)(b0 & 0xff) | ((uint32_t)(b1 & 0xff) << 8) | ((uint32_t)(b2 & 0xff) << 16) | ((uint32_t)(b3 & 0xff) << 24);
}
constexpr float kFixedMax = 32639.f;

// The same digits for four values at once, already packed as the two A-operand words (high digits, low digits), without
// a float-to-int conversion: adding 1.5 * 2^23 leaves round(x * inv_delta) in the low mantissa bits; with 128 added the
// 16-bit pattern's high byte is the high digit and its low byte the low digit + 128 (flip the top bit of each byte).
// Needs |x * inv_delta| <= 32639, which holds when inv_delta = 32639 / max |x|.
__device__ __forceinline__ void digits4(float x0, float x1, float x2, float x3, float inv_delta, uint32_t& hi, uint32_t& lo) {
  constexpr float kMagic = 12582912.f;                     // 0x4B400000
  constexpr int kBias = 128 - 0x4B400000;
  const uint32_t u0 = (uint32_t)(__float_as_int(fmaf(x0, inv_delta, kMagic)) + kBias);
  const uint32_t u1 = (uint32_t)(__float_as_int(fmaf(x1, inv_delta, kMagic)) + kBias);
  const uint32_t u2 = (uint32_t)(__float_as_int(fmaf(x2, inv_delta, kMagic)) + kBias);
  const uint32_t u3 = (uint32_t)(__float_as_int(fmaf(x3, inv_delta, kMagic)) + kBias);
  const uint32_t w01 = __byte_perm(u0, u1, 0x5410), w23 = __byte_perm(u2, u3, 0x5410);
  hi = __byte_perm(w01, w23, 0x7531);
  lo = __byte_perm(w01, w23, 0x6420) ^ 0x80808080u;
}


template <int RK, int RV, int BITS>
__global__ void __launch_bounds__(DecodeQCfg<RK, RV, BITS>::THREADS, 1)
decode_q_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const DecodeQArgs a) {
  using C = DecodeQCfg<RK, RV, BITS>;
  constexpr int NW = C::NW, NS = C::NS, SPW = C::SPW, NT = C::NT, NP = C::NP, HALF = C::HALF;
  constexpr int NJ = 4;                                  // 8-token score tiles per consumer warp and page (32 tokens)
  constexpr int NGV = C::NGV, NGK = C::NGK, KROW = C::KROW, VROW = C::VROW;
  constexpr int QMAX = (1 << BITS) - 1;                  // largest code
  // contraction steps of the scores: blocks of 32 channels, and (8-bit rank 48 only) one step of 16
  constexpr int KB32 = BITS == 8 ? RK / 32 : KROW / 16;
  constexpr int KREM = (BITS == 8 && RK % 32 != 0) ? 1 : 0;

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
  volatile int* last_flag = reinterpret_cast<volatile int*>(ctrl_ptr + 33 * 8 + 4);
  float* lse_shift = reinterpret_cast<float*>(ctrl_ptr + 34 * 8);      // [8]: q' . key zero-point / sqrt(128) of the unit's rows
  float* q_delta = reinterpret_cast<float*>(ctrl_ptr + 38 * 8);        // [8]: fixed-point step of the unit's scaled query rows
  volatile int* append_done = reinterpret_cast<volatile int*>(ctrl_ptr + 32 * 8);   // appending segments whose rows are stored
  volatile int* section_free = reinterpret_cast<volatile int*>(ctrl_ptr + 42 * 8);  // the workspace section's previous user is done
  volatile int* gate = section_free + 1;                                            // thread 0's verdict for the segment at hand
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
    *section_free = 0;
    *last_flag = 0;
    *append_done = 0;
    mbar_fence_init();
  }
  const int pad = seg_pad_pages(RK, RV);
  build_page_prefix(pref, a.Bt, a.len_add, pad, c == 0 ? a.status : nullptr);   // ends with __syncthreads

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
    // Consecutive launches take the workspace sections in turn; before the consumers write into this one its previous
    // user must be done, which the section's control word tells (decode_persistent_kernel does the same).
    auto look_at_section = [&]() {
      if (pw == 0 && lane == 0 && a.prev_epoch != 0u && *section_free == 0) {
        int seen;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(a.finished) : "memory");
        if ((unsigned)seen == a.prev_epoch) *section_free = 1;
      }
    };
    look_at_section();
    int i_base = 0;            // pages of this CTA before the current segment
    int n_append = 0;          // appending segments of this CTA so far
    while (walk.next(seg)) {
      const int h = seg.j / QT;
      const int npg = seg.p1 - seg.p0;
      bool wait_append = false;
      if (appending && seg.p1 == seg.npages) {
        const int pos = a.Bt.seq_lens[seg.b];
        wait_append = pos >= 0 && pos / kPage < a.Bt.max_pages;
      }
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
          if (wait_append && k == npg - 1) {
            // the sequence's last page receives the new token's codes from this CTA's consumers first
            wait_count(append_done, n_append + 1, abort_flag, a.status);
            __threadfence();
            asm volatile("fence.proxy.async.global;" ::: "memory");
          }
          const uint32_t st = ring + slot * C::STAGE_BYTES;
          const size_t tile = (size_t)page * Hkv + h;
          mbar_arrive_expect_tx(full_bar(slot), C::TX_BYTES);
          // 64 token rows of KROW bytes (96-byte rows: the tile as 192 lines of 32 bytes); RV channel rows of VROW bytes
          tma_load_2d(st, &tmK, 0, (int)tile * (KROW == 96 ? 192 : kPage), full_bar(slot));
          tma_load_2d(st + C::K_BYTES, &tmV, 0, (int)tile * RV, full_bar(slot));
          bulk_load_1d(st + C::K_BYTES + C::V_BYTES, a.v_params + tile * (C::P_BYTES / 4), C::P_BYTES, full_bar(slot));
        }
        __syncwarp();
      }
      i_base += npg;
      if (wait_append) ++n_append;
      look_at_section();
    }
    return;
  }

  // ------------------------------------------------------------------ consumer warps
  const int gid = lane >> 2, tid4 = lane & 3, l7 = lane & 7;
  const float qscale = kLog2e * 0.08838834764831845f;     // log2(e) / sqrt(128)

  // per-lane pieces of the ldmatrix addresses (the swizzle term depends on the lane only).  A key ldmatrix.x4
  // covers 8 tokens x 64 channels (four 16-byte chunks); a value ldmatrix.x4 covers two 8-channel tiles x the
  // warp's 32 positions (two chunks each).
  const int pl = warp % NP, hf = warp / NP;               // page lane; which 32 tokens of a page this warp takes
  constexpr int NKC = KROW / 16;                           // 16-byte chunks of a key row
  uint32_t koff[(NKC + 3) / 4];                            // chunk 4 q + (lane / 8) of row l7 (wrapped inside the row for short tails)
#pragma unroll
  for (int q4 = 0; q4 < (NKC + 3) / 4; ++q4) {
    const int rest = NKC - 4 * q4;                         // chunks this ldmatrix really covers: 4, 2 or 1
    const int m = lane >> 3;
    koff[q4] = qtile_chunk<KROW>(l7, 4 * q4 + min(m, rest - 1));     // matrices beyond the row's end repeat its last chunk
  }
  // value rows: 8-bit: two 8-channel tiles x the warp's two 16-position chunks per ldmatrix.x4;
  //             4-bit: four 8-channel tiles x the warp's one chunk of 32 positions
  const uint32_t voff = BITS == 8 ? qtile_chunk<64>(l7 + 8 * (lane >> 4), 2 * hf + ((lane >> 3) & 1))
                                  : qtile_chunk<32>(l7 + 8 * (lane >> 3), hf);
  int i_base = 0;              // pages of this CTA before the current segment
  int n_final = 0;             // units this CTA finalised (merged or zero-filled)

  while (walk.next(seg)) {
    const int b = seg.b, h = seg.j / QT, qt = seg.j % QT;
    const int npg = seg.p1 - seg.p0;
    const int ng = min(kGroupTile, G - qt * kGroupTile);
    const size_t head0 = (size_t)b * a.L.Hq + (size_t)h * G + (size_t)qt * kGroupTile;
    const int len_raw = a.Bt.seq_lens[b] + a.len_add;
    const int len = min(max(len_raw, 0), seg.npages * kPage);
    const int last_valid = len - (seg.npages - 1) * kPage;          // tokens in the sequence's last page (1..64)
    const bool has_final = seg.p1 == seg.npages;
    bool do_append = false;
    int new_page = -1, new_pos = 0;
    if (appending && has_final) {
      const int pos = a.Bt.seq_lens[b];
      if (pos >= 0 && pos / kPage < a.Bt.max_pages) {
        do_append = true;                                            // the producer waits for our signal
        new_pos = pos % kPage;
        new_page = a.Bt.block_table[(size_t)b * a.Bt.max_pages + pos / kPage];
        if (new_page < 0 || new_page >= a.L.num_pages) new_page = -1;     // bad page: signal, but store nothing
      }
    }
    // ---- prologue: q' = q U_k for the unit's queries.  The key scale of each 64-channel group is folded into
    // q' (scores are then taken against the raw codes); the key zero-point shifts all scores of a row by
    // q' . zero, which cancels in the softmax and across segments and is added to out_lse at the very end.
    float* rows = un;                    // [9][128] fp32: the queries, row 8 = the new key
    float* vrow = un + 9 * kD;           // [128]: the new value, later its projection
    uint8_t* kcode_s = reinterpret_cast<uint8_t*>(rows + 8 * kD);    // the new key's codes, once its input row is used up
    float* red = un + 10 * kD;           // [NW][9][128]
    const __nv_bfloat16* Uk = a.L.U_k + (size_t)h * a.L.uk_stride;
    const __nv_bfloat16* Uv = a.L.U_v + (size_t)h * a.L.uv_stride;
    const uint32_t row_mask = ((1u << ng) - 1u) | (do_append ? 0x100u : 0u);
    {
      BasisSlice<NW, RK> sk;
      sk.load(Uk, warp, lane);
      constexpr int NPC = (9 * 16 + NT - 1) / NT;
      uint4 pc[NPC];
#pragma unroll
      for (int i = 0; i < NPC; ++i) {
        const int idx = tid + i * NT, r = idx / 16, c = idx % 16;
        pc[i] = make_uint4(0u, 0u, 0u, 0u);
        if (r < ng) pc[i] = __ldg(reinterpret_cast<const uint4*>(a.q + (head0 + r) * kD) + c);
        else if (r == 8 && do_append) pc[i] = __ldg(reinterpret_cast<const uint4*>(a.k_new + ((size_t)b * Hkv + h) * kD) + c);
      }
      uint4 pv = make_uint4(0u, 0u, 0u, 0u);
      if (do_append && tid < 16) pv = __ldg(reinterpret_cast<const uint4*>(a.v_new + ((size_t)b * Hkv + h) * kD) + tid);
      if (do_append && tid < 16) {
        const uint32_t w[4] = {pv.x, pv.y, pv.z, pv.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) *reinterpret_cast<float2*>(vrow + tid * 8 + 2 * e) = make_float2(bf16_lo(w[e]), bf16_hi(w[e]));
      }
#pragma unroll
      for (int i = 0; i < NPC; ++i) {
        const int idx = tid + i * NT;
        if (idx < 9 * 16) {
          const uint32_t w[4] = {pc[i].x, pc[i].y, pc[i].z, pc[i].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) *reinterpret_cast<float2*>(rows + idx * 8 + 2 * e) = make_float2(bf16_lo(w[e]), bf16_hi(w[e]));
        }
      }
      bar1(NT);
      sk.contract(rows, row_mask, red, warp, lane);
    }
    BasisSlice<NW, RV> sv;
    if (do_append) sv.load(Uv, warp, lane);                // in flight while the key side is reduced
    bar1(NT);
    const float* kpar = a.k_params + (size_t)h * NGK * 2;
    for (int idx = tid; idx < 9 * RK; idx += NT) {
      const int r = idx / RK, j = idx % RK;
      const float x = ((row_mask >> r) & 1u) ? warp_shares<NW>(red, r, j) : 0.f;
      if (r < 8) {
        qp[r * RK + j] = x * qscale * __ldg(kpar + 2 * (j >> 6));
      } else if (do_append) {                              // the new key's code under the head's static parameters
        kcode_s[j] = (uint8_t)q_encode<BITS>(x, __ldg(kpar + 2 * (j >> 6)), __ldg(kpar + 2 * (j >> 6) + 1));
      }
    }
    if (tid < 8) {
      float sh = 0.f;
      if ((row_mask >> tid) & 1u)
        for (int j = 0; j < RK; ++j) sh = fmaf(warp_shares<NW>(red, tid, j), __ldg(kpar + 2 * (j >> 6) + 1), sh);
      lse_shift[tid] = sh * 0.08838834764831845f;          // / sqrt(128)
    }
    bar1(NT);
    if (tid < 8) {                                         // fixed-point step of each scaled query row
      float mx = 0.f;
      for (int j = 0; j < RK; ++j) mx = fmaxf(mx, fabsf(qp[tid * RK + j]));
      q_delta[tid] = mx > 0.f ? mx / kFixedMax : 1.f;
    }
    bar1(NT);
    if (do_append) {
      if (new_page >= 0)
        q_store_key_row<RK, BITS>(a.k_codes + (((size_t)new_page * Hkv + h) * kPage + new_pos) * KROW, kcode_s, tid, NT);
      // the new value row: project (the row sits where row 0 is expected), then token-wise group parameters and codes
      sv.contract(vrow, 1u, red, warp, lane);
      bar1(NT);
      for (int j = tid; j < RV; j += NT) vrow[j] = warp_shares<NW>(red, 0, j);
      bar1(NT);
      if (new_page >= 0) {
        for (int j = tid; j < RV; j += NT) {
          const int g = j >> 6, g1 = min(64 * g + 64, RV);
          float mn = vrow[64 * g], mxv = mn;
          for (int e = 64 * g + 1; e < g1; ++e) {
            mn = fminf(mn, vrow[e]);
            mxv = fmaxf(mxv, vrow[e]);
          }
          const float sc = mxv > mn ? __fdiv_rn(mxv - mn, (float)QMAX) : 1.f;
          const size_t tile = (size_t)new_page * Hkv + h;
          q_store_value_code<BITS>(a.v_codes + (tile * RV + j) * VROW, v_position(new_pos), q_encode<BITS>(vrow[j], sc, mn));
          if ((j & 63) == 0) *reinterpret_cast<float2*>(a.v_params + ((tile * kPage + new_pos) * NGV + g) * 2) = make_float2(sc, mn);
        }
      } else if (tid == 0) {
        report(a.status, STIEF_ERR_BOUNDS);
      }
      __threadfence();
      asm volatile("fence.proxy.async.global;" ::: "memory");
      bar1(NT);
      if (tid == 0) *append_done = *append_done + 1;       // codes are in the pools: the last page may be fetched
    }

    // A operand of the score MMA: rows 0-7 = high digits of the scaled query rows, rows 8-15 = low digits
    const float dq = q_delta[gid];
    uint32_t qa[KB32][4];
    uint32_t qrem[2] = {0u, 0u};                           // the 16-channel remainder (8-bit codes, rank 48)
    {
      const float inv = 1.f / dq;
      auto qv = [&](int ch) { return ch < RK ? qp[gid * RK + ch] : 0.f; };   // channels of a padded key row contribute nothing
#pragma unroll
      for (int ks = 0; ks < KB32; ++ks) {
        int hi[8], lo[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          digits(qv(32 * ks + 4 * tid4 + e), inv, hi[e], lo[e]);
          digits(qv(32 * ks + 16 + 4 * tid4 + e), inv, hi[4 + e], lo[4 + e]);
        }
        qa[ks][0] = pack4(hi[0], hi[1], hi[2], hi[3]);
        qa[ks][1] = pack4(lo[0], lo[1], lo[2], lo[3]);
        qa[ks][2] = pack4(hi[4], hi[5], hi[6], hi[7]);
        qa[ks][3] = pack4(lo[4], lo[5], lo[6], lo[7]);
      }
      if constexpr (KREM != 0) {
        int hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) digits(qv(32 * KB32 + 4 * tid4 + e), inv, hi[e], lo[e]);
        qrem[0] = pack4(hi[0], hi[1], hi[2], hi[3]);
        qrem[1] = pack4(lo[0], lo[1], lo[2], lo[3]);
      }
    }

    float m = -INFINITY, l = 0.f;
    float o[RV / 8][2];                                    // row gid, channels 8 n + 2 tid4, + 1
    float zc[NGV];                                         // sum_t p_t zero_t,g over this thread's tokens
#pragma unroll
    for (int n = 0; n < RV / 8; ++n) o[n][0] = o[n][1] = 0.f;
#pragma unroll
    for (int g = 0; g < NGV; ++g) zc[g] = 0.f;

    // first page of this segment that belongs to this warp's lane: global index i = i_base + k, i % NP == pl
    const int tb = 32 * hf;                                // first token of the page this warp handles
    int k0 = (pl - i_base % NP + NP) % NP;
    for (int k = k0; k < npg; k += NP) {
      const int kw = (i_base + k) / NP;
      const int slot = pl * SPW + kw % SPW;
      mbar_wait(full_bar(slot), (kw / SPW) & 1, abort_flag, a.status);
      const uint32_t kt = ring + slot * C::STAGE_BYTES;
      const uint32_t vt = kt + C::K_BYTES;
      const uint32_t pt = vt + C::V_BYTES;
      const bool tail = (seg.p0 + k == seg.npages - 1) && (last_valid < kPage);
      if (tail && last_valid <= tb) {                      // none of this warp's tokens exists: nothing to add
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar(slot));
        continue;
      }

      // ---- scores of the warp's 32 tokens: tile j covers tokens tb + 8j .. + 7; integer sums of both digits
      float sc[2 * NJ];
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        int s4[4] = {0, 0, 0, 0};
#pragma unroll
        for (int q4 = 0; q4 < (NKC + 3) / 4; ++q4) {
          const int rest = NKC - 4 * q4;                   // chunks left in the row: a compile-time value once unrolled
          uint32_t r[4] = {0u, 0u, 0u, 0u};
          const uint32_t addr = kt + koff[q4] + (tb + 8 * j) * KROW;
          if (rest >= 3) ldsm_x4(addr, r[0], r[1], r[2], r[3]);
          else if (rest == 2) ldsm_x2(addr, r[0], r[1]);
          else ldsm_x1(addr, r[0]);
          if constexpr (BITS == 8) {                       // two chunks of 16 codes per step of 32 channels
            mma_s8u8(s4, qa[2 * q4], r[0], r[1]);
            if (rest >= 4) mma_s8u8(s4, qa[2 * q4 + 1], r[2], r[3]);
            else if (rest == 3) mma_s8u8_k16(s4, qrem[0], qrem[1], r[2]);
          } else {                                         // one chunk of 32 nibbles per step of 32 channels
#pragma unroll
            for (int mm = 0; mm < 4; ++mm)
              if (mm < rest) mma_s8u8(s4, qa[4 * q4 + mm], r[mm] & 0x0f0f0f0fu, (r[mm] >> 4) & 0x0f0f0f0fu);
          }
        }
        sc[2 * j] = dq * (float)(256 * s4[0] + s4[2]);
        sc[2 * j + 1] = dq * (float)(256 * s4[1] + s4[3]);
      }
      // value parameters of this thread's 8 tokens (token of tile j, element e: tb + 8j + 2 tid4 + e)
      float vs[NGV][2 * NJ], vz[NGV][2 * NJ];
#pragma unroll
      for (int j = 0; j < NJ; ++j)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int t = tb + 8 * j + 2 * tid4 + e;
          const bool ok = !tail || t < last_valid;
          if (!ok) sc[2 * j + e] = -INFINITY;
#pragma unroll
          for (int g = 0; g < NGV; ++g) {
            float x, y;
            asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(x), "=f"(y) : "r"(pt + (t * NGV + g) * 8));
            vs[g][2 * j + e] = ok ? x : 0.f;               // rows past the end hold unspecified bits
            vz[g][2 * j + e] = ok ? y : 0.f;
          }
        }

      // ---- online softmax (base 2; the scale is folded into q')
      float mx = fmaxf(fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3])), fmaxf(fmaxf(sc[4], sc[5]), fmaxf(sc[6], sc[7])));   // a tree: this sits on the page's critical chain
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m, mx);
      // the running maximum seldom grows after a sequence's first pages: rescale only when some row's did
      const bool grew = __any_sync(0xffffffffu, m_new > m);
      if (grew) {
        const float alpha = fast_exp2(m - m_new);
        l *= alpha;
#pragma unroll
        for (int n = 0; n < RV / 8; ++n) {
          o[n][0] *= alpha;
          o[n][1] *= alpha;
        }
#pragma unroll
        for (int g = 0; g < NGV; ++g) zc[g] *= alpha;
      }
      m = m_new;
      float pr[2 * NJ];
      float ps = 0.f;
#pragma unroll
      for (int e = 0; e < 2 * NJ; ++e) {
        pr[e] = fast_exp2(sc[e] - m);
        ps += pr[e];
      }
      l += ps;

      // ---- mix: per value group, p_t * scale_t,g as two digits of a per-row fixed point against the raw codes
#pragma unroll
      for (int g = 0; g < NGV; ++g) {
        float w[2 * NJ], zsum = 0.f;
#pragma unroll
        for (int e = 0; e < 2 * NJ; ++e) {
          w[e] = pr[e] * vs[g][e];
          zsum = fmaf(pr[e], vz[g][e], zsum);
        }
        float wmax = fmaxf(fmaxf(fmaxf(w[0], w[1]), fmaxf(w[2], w[3])), fmaxf(fmaxf(w[4], w[5]), fmaxf(w[6], w[7])));
        zc[g] += zsum;
        wmax = fmaxf(wmax, __shfl_xor_sync(0xffffffffu, wmax, 1));
        wmax = fmaxf(wmax, __shfl_xor_sync(0xffffffffu, wmax, 2));
        // fixed-point step of this page's weights and its reciprocal: an approximate reciprocal is enough (the digits
        // stand for w * inv * dp, and inv * dp = 1 to 2 ulp), and two IEEE divisions would sit on every page's critical chain
        // (weights all below 1e-30 add nothing that fp32 accumulators holding O(1) sums could register: digits 0)
        const bool live = wmax > 1e-30f;
        const float dp = live ? wmax * (1.f / kFixedMax) : 1.f;
        float inv;
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(dp));
        inv = live ? inv : 0.f;
        // k-slots 4 tid4 .. + 3 of the first 16 positions hold tiles 0 and 1, of the second 16 tiles 2 and 3
        uint32_t pa[4];
        digits4(w[0], w[1], w[2], w[3], inv, pa[0], pa[1]);
        digits4(w[4], w[5], w[6], w[7], inv, pa[2], pa[3]);
        const int GT = (min(64 * g + 64, RV) - 64 * g) / 8;       // 8-channel tiles of the group: 8, or 4 / 6 in a short last group
        if constexpr (BITS == 8) {
#pragma unroll
          for (int n2 = 0; n2 < 4; ++n2) {                 // two 8-channel tiles x two chunks of 16 positions per ldmatrix
            if (2 * n2 < GT) {
              const int n = 8 * g + 2 * n2;
              uint32_t r0, r1, r2, r3;
              ldsm_x4(vt + voff + n * 8 * VROW, r0, r1, r2, r3);
              int c0[4] = {0, 0, 0, 0}, c1[4] = {0, 0, 0, 0};
              mma_s8u8(c0, pa, r0, r1);
              mma_s8u8(c1, pa, r2, r3);
              o[n][0] = fmaf(dp, (float)(256 * c0[0] + c0[2]), o[n][0]);
              o[n][1] = fmaf(dp, (float)(256 * c0[1] + c0[3]), o[n][1]);
              o[n + 1][0] = fmaf(dp, (float)(256 * c1[0] + c1[2]), o[n + 1][0]);
              o[n + 1][1] = fmaf(dp, (float)(256 * c1[1] + c1[3]), o[n + 1][1]);
            }
          }
        } else {
#pragma unroll
          for (int n4 = 0; n4 < 2; ++n4) {                 // four 8-channel tiles x one chunk of 32 positions per ldmatrix
            const int left = GT - 4 * n4;                  // tiles left in the group: 4 or more, 2, or none
            if (left > 0) {
              const int n = 8 * g + 4 * n4;
              uint32_t r[4] = {0u, 0u, 0u, 0u};
              if (left >= 4) ldsm_x4(vt + voff + n * 8 * VROW, r[0], r[1], r[2], r[3]);
              else ldsm_x2(vt + voff + n * 8 * VROW, r[0], r[1]);
#pragma unroll
              for (int mm = 0; mm < 4; ++mm) {
                if (mm < left) {
                  int c0[4] = {0, 0, 0, 0};
                  mma_s8u8(c0, pa, r[mm] & 0x0f0f0f0fu, (r[mm] >> 4) & 0x0f0f0f0fu);
                  o[n + mm][0] = fmaf(dp, (float)(256 * c0[0] + c0[2]), o[n + mm][0]);
                  o[n + mm][1] = fmaf(dp, (float)(256 * c0[1] + c0[3]), o[n + mm][1]);
                }
              }
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar(slot));
    }
    i_base += npg;

    // ------------------------------------------------------------------ merge the warps of this segment
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    float* wo = un;                      // [NW][8][RV]
    float* wm = wo + NW * 8 * RV;        // [NW][8]
    float* wl = wm + NW * 8;             // [NW][8]
#pragma unroll
    for (int g = 0; g < NGV; ++g) {                        // the group's zero-point term, summed over the row's four threads
      zc[g] += __shfl_xor_sync(0xffffffffu, zc[g], 1);
      zc[g] += __shfl_xor_sync(0xffffffffu, zc[g], 2);
    }
#pragma unroll
    for (int n = 0; n < RV / 8; ++n) {
      *reinterpret_cast<float2*>(wo + (warp * 8 + gid) * RV + 8 * n + 2 * tid4) = make_float2(o[n][0] + zc[n / 8], o[n][1] + zc[n / 8]);
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
        combine_unit<RV>(a.L, b, h, qt, first + u, nseg, a.partial_o, a.partial_lse, a.out, a.out_lse, un, tid, NT, lse_shift);
        ++n_final;
      }
    }
    bar1(NT);
  }

  // units of empty sequences get their zero rows from CTA (u mod n_cta)
  if (a.out != nullptr) {
    for (int u = c; u < B * upb; u += n_cta) {
      const int b = u / upb, j = u % upb;
      if (pref[b + 1] != pref[b]) continue;
      const int h = j / QT, qt = j % QT;
      const int ng = min(kGroupTile, G - qt * kGroupTile);
      const size_t head0 = (size_t)b * a.L.Hq + (size_t)h * G + (size_t)qt * kGroupTile;
      for (int idx = tid; idx < ng * kD; idx += NT) a.out[head0 * kD + idx] = __float2bfloat16_rn(0.f);
      if (a.out_lse && tid < ng) a.out_lse[head0 + tid] = -INFINITY;
      ++n_final;
    }
  }
  // Every unit is finalised by exactly one CTA (merged, or zero-filled).  The CTA that finalises the kernel's last unit
  // publishes the kernel's epoch: from then on this section of the workspace is free for its next user.  That CTA also
  // waits for the predecessor grid before it leaves, so that this grid never completes before an earlier one (stream
  // order stays transitive); the others leave at once and hand their SMs to the next kernel.
  if (a.out == nullptr) {
    grid_dependency_wait();
  } else if (n_final > 0) {
    bar1(NT);                                              // all of the CTA's reads of partials and writes of outputs are issued
    if (tid == 0) {
      __threadfence();
      const int before = atomicAdd(a.units_done, n_final);
      if (before + n_final == B * upb) {
        *a.units_done = 0;
        __threadfence();
        asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(a.finished), "r"((int)a.epoch) : "memory");
        grid_dependency_wait();
      }
    }
  }
}

}  // namespace stief
