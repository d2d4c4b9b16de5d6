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

// The merge runs while other CTAs still stream the cache, so a dependent global load costs
// microseconds.  Loads are therefore issued in bulk before anything waits on them: a thread's row of
// U_v, the segments' log-sum-exps and the first kSegBatch segments' partials of every output element the
// thread owns are all in flight together; a unit of up to kSegBatch segments costs one round trip.
// `od` is shared scratch [8][128] floats, `wsm` shared scratch [kSegChunk][8] + 24 floats; nt >= 96.
constexpr int kSegBatch = 8;       // segments whose partials a thread holds in registers at once
constexpr int kSegChunk = 32;      // segments whose weights sit in shared memory at once
constexpr int kCombineScratchFloats = kGroupTile * kD + kSegChunk * kGroupTile + 24;

template <int RV>
__device__ __forceinline__ void combine_unit(const LayerDev& L, int b, int h, int qt, int slot0, int nseg, const float* partial_o,
                                             const float* partial_lse, __nv_bfloat16* out, float* out_lse, float* od, float* wsm,
                                             int tid, int nt, const float* lse_shift = nullptr) {
  constexpr int NV = RV / 4;                               // float4 pieces per row
  constexpr int IPT = 3;                                   // pieces per thread: 8 * NV <= 256 <= 3 * 96
  const int G = L.G;
  const int ng = min(kGroupTile, G - qt * kGroupTile);
  const int n_items = ng * NV;
  const size_t head0 = (size_t)b * L.Hq + (size_t)h * G + (size_t)qt * kGroupTile;
  const __nv_bfloat16* Uv = L.U_v ? L.U_v + (size_t)h * L.uv_stride : nullptr;
  float* Mrow = wsm + kSegChunk * kGroupTile;              // running max per row
  float* Drow = Mrow + 8;                                  // running denominator per row
  float* Srow = Drow + 8;                                  // rescale of what was accumulated before this chunk

  // this thread's row of U_v for the back-projection (output column dd = tid)
  uint4 urow[RV / 8];
  if (Uv && tid < kD) {
#pragma unroll
    for (int c = 0; c < RV / 8; ++c) urow[c] = __ldg(reinterpret_cast<const uint4*>(Uv + (size_t)tid * RV) + c);
  }
  if (tid < 8) {
    Mrow[tid] = -INFINITY;
    Drow[tid] = 0.f;
  }
  float4 num[IPT];
#pragma unroll
  for (int i = 0; i < IPT; ++i) num[i] = make_float4(0.f, 0.f, 0.f, 0.f);

  for (int c0 = 0; c0 < nseg; c0 += kSegChunk) {
    const int n = min(kSegChunk, nseg - c0);
    const float* lse0 = partial_lse + (size_t)(slot0 + c0) * kGroupTile;       // n * 8 contiguous floats
    const float4* po0 = reinterpret_cast<const float4*>(partial_o + (size_t)(slot0 + c0) * kGroupTile * RV);
    float lv[IPT];
#pragma unroll
    for (int i = 0; i < IPT; ++i) {
      const int idx = tid + i * nt;
      lv[i] = idx < n * kGroupTile ? __ldcg(lse0 + idx) : 0.f;
    }
    float4 ov[IPT][kSegBatch];
    auto fetch = [&](int k0) {
#pragma unroll
      for (int i = 0; i < IPT; ++i) {
        const int item = tid + i * nt;
#pragma unroll
        for (int k = 0; k < kSegBatch; ++k) {
          ov[i][k] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (item < n_items && k0 + k < n) ov[i][k] = __ldcg(po0 + (size_t)(k0 + k) * kGroupTile * NV + item);   // item = r * NV + j4
        }
      }
    };
    fetch(0);
#pragma unroll
    for (int i = 0; i < IPT; ++i) {
      const int idx = tid + i * nt;
      if (idx < n * kGroupTile) wsm[idx] = lv[i];
    }
    bar1(nt);
    if (tid < 8) {
      const float m_old = Mrow[tid];
      float m = m_old;
      for (int s = 0; s < n; ++s) m = fmaxf(m, wsm[s * kGroupTile + tid]);
      float sc = 1.f, d = Drow[tid];
      if (m > -INFINITY) {
        sc = __expf(m_old - m);                            // 0 when nothing was accumulated before
        d *= sc;
        for (int s = 0; s < n; ++s) d += __expf(wsm[s * kGroupTile + tid] - m);
      }
      Mrow[tid] = m;
      Drow[tid] = d;
      Srow[tid] = sc;
    }
    bar1(nt);
    for (int idx = tid; idx < n * kGroupTile; idx += nt) {
      const float m = Mrow[idx % kGroupTile];
      wsm[idx] = m > -INFINITY ? __expf(wsm[idx] - m) : 0.f;      // an empty segment (lse = -inf) weighs nothing
    }
    bar1(nt);
    for (int k0 = 0; k0 < n; k0 += kSegBatch) {
      if (k0 > 0) fetch(k0);
#pragma unroll
      for (int i = 0; i < IPT; ++i) {
        const int item = tid + i * nt;
        if (item >= n_items) continue;
        const int r = item / NV;
        if (k0 == 0) {
          const float sc = Srow[r];
          num[i].x *= sc; num[i].y *= sc; num[i].z *= sc; num[i].w *= sc;
        }
#pragma unroll
        for (int k = 0; k < kSegBatch; ++k) {
          if (k0 + k < n) {
            const float w = wsm[(k0 + k) * kGroupTile + r];
            num[i].x = fmaf(w, ov[i][k].x, num[i].x);
            num[i].y = fmaf(w, ov[i][k].y, num[i].y);
            num[i].z = fmaf(w, ov[i][k].z, num[i].z);
            num[i].w = fmaf(w, ov[i][k].w, num[i].w);
          }
        }
      }
    }
    bar1(nt);                                              // the next chunk overwrites wsm
  }
  if (nseg <= 0) bar1(nt);                                 // Mrow/Drow initialised above must be visible
#pragma unroll
  for (int i = 0; i < IPT; ++i) {
    const int item = tid + i * nt;
    if (item < n_items) {
      const int r = item / NV, j4 = item % NV;
      const float den = Drow[r];
      const float inv = den > 0.f ? 1.f / den : 0.f;
      *reinterpret_cast<float4*>(od + r * kD + 4 * j4) = make_float4(num[i].x * inv, num[i].y * inv, num[i].z * inv, num[i].w * inv);
    }
  }
  // lse_shift: a per-row constant that was left out of every score of the unit (it cancels in the softmax)
  if (tid < ng && out_lse)
    out_lse[head0 + tid] = Drow[tid] > 0.f ? Mrow[tid] + __logf(Drow[tid]) + (lse_shift ? lse_shift[tid] : 0.f) : -INFINITY;
  bar1(nt);
  const int d_out = Uv ? kD : RV;                           // without a value basis the output stays in the compressed space
  for (int dd = tid; dd < d_out; dd += nt) {
    float acc[kGroupTile];
#pragma unroll
    for (int r = 0; r < kGroupTile; ++r) acc[r] = 0.f;
    if (Uv) {
      if (dd != tid) {                                      // second pass of a CTA with fewer than 128 threads
#pragma unroll
        for (int c = 0; c < RV / 8; ++c) urow[c] = __ldg(reinterpret_cast<const uint4*>(Uv + (size_t)dd * RV) + c);
      }
#pragma unroll
      for (int c = 0; c < RV / 8; ++c) {
        const uint32_t w[4] = {urow[c].x, urow[c].y, urow[c].z, urow[c].w};
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
      if (r < ng) out[(head0 + r) * d_out + dd] = __float2bfloat16_rn(acc[r]);
  }
  bar1(nt);
}

}  // namespace stief
