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
// Everything here is a pure function of (seq_lens, len_add, max_pages, n_cta), recomputed identically
// by the split-T kernel and by the combine.
#pragma once

#include "stief_common.cuh"

namespace stief {

constexpr int kMaxBatch = 1024;          // sequences per call (prefix sums live in shared memory)
constexpr int kMinPagesPerCta = 2;
constexpr int kGroupTile = 8;            // query heads per unit (rows of the MMA operand)

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

// pref[0..B]: exclusive prefix sums of pages per sequence.  Called by all threads of the CTA; the
// first warp computes.  Ends with a __syncthreads.
__device__ __forceinline__ void build_page_prefix(int* pref, const BatchDev& Bt, int len_add, int32_t* status) {
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    int carry = 0;
    bool clamped = false;
    for (int base = 0; base < Bt.B; base += 32) {
      const int b = base + lane;
      int v = (b < Bt.B) ? clamped_pages(Bt, b, len_add, &clamped) : 0;
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
  int B, upb, g, g_end, b, j, p;
  __device__ void init(const int* pref_, int B_, int upb_, int c, int P, int total) {
    pref = pref_; B = B_; upb = upb_;
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
    const int pb = pref[b + 1] - pref[b];
    const int rem = g - pref[b] * upb;
    j = rem / pb;
    p = rem % pb;
  }
  __device__ bool next(Segment& s) {
    if (g >= g_end) return false;
    const int pb = pref[b + 1] - pref[b];
    const int take = min(pb - p, g_end - g);
    s.b = b; s.j = j; s.p0 = p; s.p1 = p + take; s.npages = pb;
    g += take;
    p += take;
    if (p == pb) {
      p = 0;
      if (++j == upb) {
        j = 0;
        ++b;
        while (b < B && pref[b + 1] == pref[b]) ++b;
      }
    }
    return true;
  }
};

// CTAs whose ranges overlap unit (b, j)
__device__ __forceinline__ void unit_cta_span(const int* pref, int upb, int P, int b, int j, int* first, int* last) {
  const int pb = pref[b + 1] - pref[b];
  const int start = pref[b] * upb + j * pb;
  *first = start / P;
  *last = (start + pb - 1) / P;
}

// ---------------------------------------------------------------------------------------------
// merge of a unit's segments + back-projection (Eq. 18 re-associated over chunks; Eq. 7 applied to
// the mixed values).  Called by nt threads that share barrier 1; `od` is shared scratch
// [kGroupTile][128] floats.  Partials: partial_o [slot][8][RV], partial_lse [slot][8].
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void bar1(int nt) { asm volatile("bar.sync 1, %0;" ::"r"(nt) : "memory"); }

__device__ __forceinline__ void combine_unit(const LayerDev& L, int b, int h, int qt, int slot0, int nseg, const float* partial_o,
                                             const float* partial_lse, __nv_bfloat16* out, float* out_lse, float* od, int tid, int nt) {
  const int RV = L.r_v;
  const int G = L.G;
  const int ng = min(kGroupTile, G - qt * kGroupTile);
  const size_t head0 = (size_t)b * L.Hq + (size_t)h * G + (size_t)qt * kGroupTile;
  for (int idx = tid; idx < ng * RV; idx += nt) {
    const int r = idx / RV, jj = idx % RV;
    float M = -INFINITY;
    for (int s = 0; s < nseg; ++s) M = fmaxf(M, __ldcg(partial_lse + (size_t)(slot0 + s) * kGroupTile + r));
    float num = 0.f, den = 0.f;
    for (int s = 0; s < nseg; ++s) {
      const float w = __expf(__ldcg(partial_lse + (size_t)(slot0 + s) * kGroupTile + r) - M);
      num = fmaf(w, __ldcg(partial_o + ((size_t)(slot0 + s) * kGroupTile + r) * RV + jj), num);
      den += w;
    }
    od[r * kD + jj] = nseg > 0 ? num / den : 0.f;
    if (jj == 0 && out_lse) out_lse[head0 + r] = nseg > 0 ? M + __logf(den) : -INFINITY;
  }
  bar1(nt);
  const __nv_bfloat16* Uv = L.U_v ? L.U_v + (size_t)h * L.uv_stride : nullptr;
  for (int dd = tid; dd < kD; dd += nt) {
    float acc[kGroupTile];
#pragma unroll
    for (int r = 0; r < kGroupTile; ++r) acc[r] = 0.f;
    if (Uv) {
      const uint4* urow = reinterpret_cast<const uint4*>(Uv + (size_t)dd * RV);
      for (int c = 0; c < RV / 8; ++c) {
        const uint4 u = __ldg(urow + c);
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float u0 = bf16_lo(w[e]), u1 = bf16_hi(w[e]);
#pragma unroll
          for (int r = 0; r < kGroupTile; ++r) {
            acc[r] = fmaf(od[r * kD + 8 * c + 2 * e], u0, acc[r]);
            acc[r] = fmaf(od[r * kD + 8 * c + 2 * e + 1], u1, acc[r]);
          }
        }
      }
    } else {
#pragma unroll
      for (int r = 0; r < kGroupTile; ++r) acc[r] = od[r * kD + dd];
    }
#pragma unroll
    for (int r = 0; r < kGroupTile; ++r)
      if (r < ng) out[(head0 + r) * kD + dd] = __float2bfloat16_rn(acc[r]);
  }
  bar1(nt);
}

}  // namespace stief
