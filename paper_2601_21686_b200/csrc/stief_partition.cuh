// Even split of a batch's cache pages over CTAs, and the merge that undoes it.
//
// Work is measured in page tiles.  A "unit" is (sequence b, KV head h, query tile qt) and owns the
// pages_b pages of its sequence; units are laid end to end on one global page axis (b slowest) and
// CTA c takes the contiguous range [c*P, (c+1)*P), P = ceil(total / n_cta) (at least kMinPagesPerCta).
// A CTA's range cuts out one "segment" of every unit it overlaps; each segment yields one
// chunk-normalised partial result.  Because both the CTA index and the unit index grow along the
// axis, segment (c, u) is stored in slot c + u, and the segments of unit u occupy the consecutive
// slots first_cta(u)+u .. last_cta(u)+u.
//
// Starting a segment is not free (the unit's queries are projected, and the previous segment's partial
// is merged and written), and a CTA that pauses cannot make the time up later because the memory system
// is saturated.  The axis therefore charges every unit `pad` virtual pages in front of its real ones: a
// CTA whose range crosses into a new unit gets that many fewer pages to stream, so all CTAs finish
// together.  `pad` depends on the ranks only (seg_pad_pages).
//
// Everything here is a pure function of (seq_lens, len_add, max_pages, n_cta, ranks), recomputed
// identically by the split-T kernel and by the combine.
#pragma once

#include "stief_common.cuh"

namespace stief {

constexpr int kMaxBatch = 1024;          // sequences per call (prefix sums live in shared memory)
constexpr int kMinPagesPerCta = 2;
constexpr int kGroupTile = 8;            // query heads per unit (rows of the MMA operand)
constexpr int kSegOverheadBytes = 288 * 1024;   // cache bytes one CTA streams in the time a segment start costs

__host__ __device__ __forceinline__ int seg_pad_pages(int r_k, int r_v) { return kSegOverheadBytes / ((r_k + r_v) * kPage * 2); }

__device__ __forceinline__ int clamped_pages(const BatchDev& Bt, int b, int len_add, bool* clamped = nullptr) {
  int len = Bt.seq_lens[b] + len_add;
  if (len < 0) len = 0;
  int n = (len + kPage - 1) / kPage;
  if (n > Bt.max_pages) {
    n = Bt.max_pages;
    if (clamped) *clamped = true;
  }
  return n;
}

// pref[0..B]: exclusive prefix sums of the axis length of one unit of each sequence: pages + pad for a
// sequence that has tokens, 0 for an empty one.  Called by all threads of the CTA; the first warp
// computes.  Ends with a __syncthreads.
__device__ __forceinline__ void build_page_prefix(int* pref, const BatchDev& Bt, int len_add, int pad, int32_t* status) {
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    int carry = 0;
    bool clamped = false;
    for (int base = 0; base < Bt.B; base += 32) {
      const int b = base + lane;
      int v = (b < Bt.B) ? clamped_pages(Bt, b, len_add, &clamped) : 0;
      if (v > 0) v += pad;
      int s = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, s, o);
        if (lane >= o) s += t;
      }
      if (b < Bt.B) pref[b + 1] = carry + s;
      carry += __shfl_sync(0xffffffffu, s, 31);
    }
    if (lane == 0) pref[0] = 0;
    if (clamped) report(status, STIEF_ERR_BOUNDS);      // a sequence longer than its block table
  }
  __syncthreads();
}

__device__ __forceinline__ int pages_per_cta(int total, int n_cta) {
  const int p = (total + n_cta - 1) / n_cta;
  return p < kMinPagesPerCta ? kMinPagesPerCta : p;
}

struct Segment {
  int b, j;          // sequence, unit within the sequence (j = h * QT + qt)
  int p0, p1;        // page range inside the sequence
  int npages;        // pages of the sequence
};

// Walks the segments of CTA c in order.  Every thread that walks gets the same sequence.
struct SegmentWalker {
  const int* pref;
  int B, upb, pad, g, g_end, b, j, p;      // p: position inside the current unit's axis span (pad included)
  __device__ void init(const int* pref_, int B_, int upb_, int pad_, int c, int P, int total) {
    pref = pref_; B = B_; upb = upb_; pad = pad_;
    const long long g0 = (long long)c * P;
    if (g0 >= total) { g = g_end = 0; b = B; j = p = 0; return; }
    g = (int)g0;
    g_end = (int)min((long long)total, g0 + P);
    int lo = 0, hi = B;                                   // largest b with pref[b]*upb <= g
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if ((long long)pref[mid] * upb <= g) lo = mid; else hi = mid;
    }
    b = lo;
    while (b < B && pref[b + 1] == pref[b]) ++b;          // skip empty sequences that share the offset
    const int lb = pref[b + 1] - pref[b];
    const int rem = g - pref[b] * upb;
    j = rem / lb;
    p = rem % lb;
  }
  __device__ bool next(Segment& s) {
    while (g < g_end) {
      const int lb = pref[b + 1] - pref[b];               // pad + pages
      const int take = min(lb - p, g_end - g);
      const int q0 = max(p, pad) - pad, q1 = max(p + take, pad) - pad;   // the real pages inside the piece
      s.b = b; s.j = j; s.p0 = q0; s.p1 = q1; s.npages = lb - pad;
      g += take;
      p += take;
      if (p == lb) {
        p = 0;
        if (++j == upb) {
          j = 0;
          ++b;
          while (b < B && pref[b + 1] == pref[b]) ++b;
        }
      }
      if (q1 > q0) return true;                           // a piece that is all padding holds no work
    }
    return false;
  }
};

// CTAs whose ranges overlap the real pages of unit (b, j)
__device__ __forceinline__ void unit_cta_span(const int* pref, int upb, int pad, int P, int b, int j, int* first, int* last) {
  const int lb = pref[b + 1] - pref[b];
  const int start = pref[b] * upb + j * lb;
  *first = (start + pad) / P;
  *last = (start + lb - 1) / P;
}

// ---------------------------------------------------------------------------------------------
// merge of a unit's segments + back-projection (Eq. 18 re-associated over chunks; Eq. 7 applied to
// the mixed values).  Called by nt threads that share barrier 1; `od` is shared scratch
// [kGroupTile][128] floats.  Partials: partial_o [slot][8][RV], partial_lse [slot][8].
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void bar1(int nt) { asm volatile("bar.sync 1, %0;" ::"r"(nt) : "memory"); }

// The merge may run while other CTAs still stream the cache, when a dependent global load costs microseconds, so a
// thread issues everything it needs at once: the log-sum-exps of up to kSegBatch segments of its row and those
// segments' partials of the output elements it owns are all in flight together (one round trip for a unit of up to
// kSegBatch segments; longer units loop with a running maximum).  Every thread of a row derives the row's weights by
// itself from the same values in the same order, so there is nothing to exchange and the result does not depend on
// the number of threads.  The back-projection o_down U_v^T runs on the tensor cores: the eight merged rows, split into
// bf16 value + remainder (rows 0-7 / 8-15 of the A operand, ~16 significant bits), against U_v read from global memory
// in the order the B fragments want it; warp w of the first four produces output columns 32 w .. 32 w + 31.
// Called by nt >= 128 threads (a multiple of 32) that share barrier 1; `od` is shared scratch of kCombineScratchFloats.
constexpr int kSegBatch = 8;       // segments whose partials a thread holds in registers at once
constexpr int kCombineScratchFloats = kGroupTile * (kD + 4);

template <int RV>
__device__ __forceinline__ void combine_unit(const LayerDev& L, int b, int h, int qt, int slot0, int nseg, const float* partial_o,
                                             const float* partial_lse, __nv_bfloat16* out, float* out_lse, float* od,
                                             int tid, int nt, const float* lse_shift = nullptr) {
  constexpr int NV = RV / 4;                               // float4 pieces per row
  constexpr int IPT = 2;                                   // pieces per thread: 8 * NV <= 256 = 2 * 128
  constexpr int S = RV + 4;                                // row stride of od: keeps the 16-byte reads of phase 2 conflict-free
  const int G = L.G;
  const int ng = min(kGroupTile, G - qt * kGroupTile);
  const int n_items = ng * NV;
  const size_t head0 = (size_t)b * L.Hq + (size_t)h * G + (size_t)qt * kGroupTile;
  const __nv_bfloat16* Uv = L.U_v ? L.U_v + (size_t)h * L.uv_stride : nullptr;
  const int warp = tid >> 5, lane = tid & 31, gid = lane >> 2, tid4 = lane & 3;

  // ---- phase 2's operand from global memory, requested first: warp w, n-tile t covers output columns 32 w + 8 t + gid;
  // per 32 contraction indices a thread holds the 8 consecutive elements 32 q + 8 tid4 .. + 7 of its column's row of U_v
  constexpr int QF = RV / 32, REM = RV % 32;               // full groups of 32, and a remainder of 16 (ranks 48)
  uint4 ub[4][QF > 0 ? QF : 1];
  uint32_t ur[4][2];
  if (Uv && warp < 4) {
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const __nv_bfloat16* row = Uv + (size_t)(32 * warp + 8 * t + gid) * RV;
#pragma unroll
      for (int q = 0; q < QF; ++q) ub[t][q] = __ldg(reinterpret_cast<const uint4*>(row + 32 * q + 8 * tid4));
      if constexpr (REM != 0) {
        ur[t][0] = __ldg(reinterpret_cast<const uint32_t*>(row + 32 * QF + 2 * tid4));
        ur[t][1] = __ldg(reinterpret_cast<const uint32_t*>(row + 32 * QF + 8 + 2 * tid4));
      }
    }
  }

  // ---- phase 1: merge the segments (Eq. 18 re-associated over chunks of the token axis)
  float4 num[IPT];
  float m_run[IPT], d_run[IPT];
#pragma unroll
  for (int i = 0; i < IPT; ++i) {
    num[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    m_run[i] = -INFINITY;
    d_run[i] = 0.f;
  }
  for (int k0 = 0; k0 < nseg; k0 += kSegBatch) {
    float lv[IPT][kSegBatch];
    float4 ov[IPT][kSegBatch];
#pragma unroll
    for (int i = 0; i < IPT; ++i) {
      const int item = tid + i * nt;                       // item = r * NV + j4
      const int r = item / NV;
#pragma unroll
      for (int k = 0; k < kSegBatch; ++k) {
        lv[i][k] = -INFINITY;
        ov[i][k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (item < n_items && k0 + k < nseg) {
          lv[i][k] = __ldcg(partial_lse + (size_t)(slot0 + k0 + k) * kGroupTile + r);
          ov[i][k] = __ldcg(reinterpret_cast<const float4*>(partial_o + (size_t)(slot0 + k0 + k) * kGroupTile * RV) + item);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < IPT; ++i) {
      float m = m_run[i];
#pragma unroll
      for (int k = 0; k < kSegBatch; ++k) m = fmaxf(m, lv[i][k]);
      if (m > -INFINITY) {                                 // else: nothing but empty segments so far
        const float sc = __expf(m_run[i] - m);             // 0 when nothing was accumulated before
        num[i].x *= sc; num[i].y *= sc; num[i].z *= sc; num[i].w *= sc;
        float d = d_run[i] * sc;
#pragma unroll
        for (int k = 0; k < kSegBatch; ++k) {
          const float w = __expf(lv[i][k] - m);            // an empty segment (lse = -inf) weighs nothing
          d += w;
          num[i].x = fmaf(w, ov[i][k].x, num[i].x);
          num[i].y = fmaf(w, ov[i][k].y, num[i].y);
          num[i].z = fmaf(w, ov[i][k].z, num[i].z);
          num[i].w = fmaf(w, ov[i][k].w, num[i].w);
        }
        d_run[i] = d;
        m_run[i] = m;
      }
    }
  }
#pragma unroll
  for (int i = 0; i < IPT; ++i) {
    const int item = tid + i * nt;
    if (item < n_items) {
      const int r = item / NV, j4 = item % NV;
      const float inv = d_run[i] > 0.f ? 1.f / d_run[i] : 0.f;
      *reinterpret_cast<float4*>(od + r * S + 4 * j4) = make_float4(num[i].x * inv, num[i].y * inv, num[i].z * inv, num[i].w * inv);
      // lse_shift: a per-row constant that was left out of every score of the unit (it cancels in the softmax)
      if (j4 == 0 && out_lse)
        out_lse[head0 + r] = d_run[i] > 0.f ? m_run[i] + __logf(d_run[i]) + (lse_shift ? lse_shift[r] : 0.f) : -INFINITY;
    }
  }
  for (int idx = tid; idx < (kGroupTile - ng) * RV; idx += nt) od[(ng + idx / RV) * S + idx % RV] = 0.f;   // rows without a query head
  bar1(nt);

  // ---- phase 2: back-projection (Eq. 7 applied to the mixed values), or the compressed rows as they are
  if (Uv) {
    if (warp < 4) {
      float acc[4][4];
#pragma unroll
      for (int t = 0; t < 4; ++t) acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
      const float* orow = od + gid * S;
#pragma unroll
      for (int q = 0; q < QF; ++q) {
        const float4 x0 = *reinterpret_cast<const float4*>(orow + 32 * q + 8 * tid4);
        const float4 x1 = *reinterpret_cast<const float4*>(orow + 32 * q + 8 * tid4 + 4);
        uint32_t a0[4], a1[4];                             // rows 0-7: value, rows 8-15: remainder
        split_bf16(x0.x, x0.y, a0[0], a0[1]);
        split_bf16(x0.z, x0.w, a0[2], a0[3]);
        split_bf16(x1.x, x1.y, a1[0], a1[1]);
        split_bf16(x1.z, x1.w, a1[2], a1[3]);
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          mma_bf16(acc[t], a0, ub[t][q].x, ub[t][q].y);
          mma_bf16(acc[t], a1, ub[t][q].z, ub[t][q].w);
        }
      }
      if constexpr (REM != 0) {
        const float2 x0 = *reinterpret_cast<const float2*>(orow + 32 * QF + 2 * tid4);
        const float2 x1 = *reinterpret_cast<const float2*>(orow + 32 * QF + 8 + 2 * tid4);
        uint32_t a0[4];
        split_bf16(x0.x, x0.y, a0[0], a0[1]);
        split_bf16(x1.x, x1.y, a0[2], a0[3]);
#pragma unroll
        for (int t = 0; t < 4; ++t) mma_bf16(acc[t], a0, ur[t][0], ur[t][1]);
      }
      if (gid < ng) {
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const int dd = 32 * warp + 8 * t + 2 * tid4;     // accumulator columns 2 tid4, 2 tid4 + 1 of row gid (value) and gid + 8 (remainder)
          *reinterpret_cast<uint32_t*>(out + (head0 + gid) * kD + dd) = pack_bf16(acc[t][0] + acc[t][2], acc[t][1] + acc[t][3]);
        }
      }
    }
  } else {
    for (int idx = tid; idx < ng * RV; idx += nt) out[(head0 + idx / RV) * RV + idx % RV] = __float2bfloat16_rn(od[(idx / RV) * S + idx % RV]);
  }
  bar1(nt);
}

}  // namespace stief
