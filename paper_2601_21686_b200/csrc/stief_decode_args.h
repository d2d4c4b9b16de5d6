// Kernel argument block of the persistent decode kernel (shared by the kernel and its launchers).
#pragma once

#include "stief_common.cuh"

namespace stief {

struct DecodeArgs {
  LayerDev L;
  BatchDev Bt;
  const __nv_bfloat16* q;        // [B][Hq][128]
  const __nv_bfloat16* k_new;    // [B][Hkv][128] or NULL: project and store at position seq_lens[b] first
  const __nv_bfloat16* v_new;
  float* partial_o;              // [n_cta + n_units][8][RV]
  float* partial_lse;            // [n_cta + n_units][8]
  int* counters;                 // [n_units], zero on entry, zero again on exit (fused combine only)
  // The three arrays above are one section of the workspace.  *finished holds the epoch of the last kernel that
  // finished with this section, *units_done counts the units this kernel has finalised.  A kernel whose launch
  // overlaps its predecessors may write its section as soon as *finished == prev_epoch (the section's previous user
  // is done); prev_epoch == 0: not known, wait for the predecessor grid instead.
  int* finished;
  int* units_done;
  unsigned epoch, prev_epoch;
  __nv_bfloat16* out;            // [B][Hq][128] or NULL (partials only)
  float* out_lse;                // [B][Hq] or NULL
  int len_add;                   // tokens attended beyond seq_lens (1 when appending)
  int QT;                        // query tiles per KV head = ceil(G / 8)
  int32_t* status;
  unsigned long long* trace;     // NULL, or [n_cta][kTraceSlots] time stamps (measurement aid, see stamp())
};

// Slots of the per-CTA time-stamp record (nanoseconds of the GPU's global timer; 0 = never reached).
enum TraceSlot {
  kTrEntry = 0,        // first instruction of the CTA
  kTrPrefix = 1,       // page prefix sums built, partition known
  kTrFirstIssue = 2,   // producer lane 0: first TMA request issued
  kTrPrologue = 3,     // consumers: first segment's projections done, about to wait for pages
  kTrFirstPage = 4,    // consumers (warp 0): first page tile landed
  kTrLastIssue = 5,    // producer lane 0: last TMA request issued
  kTrLastPage = 6,     // consumers (warp 0): last page of the last segment consumed
  kTrPartial = 7,      // last segment's partial stored
  kTrCombined = 8,     // after the (possible) combine of the last segment's unit
  kTrExit = 9,         // after the final dependency wait
  kTrSegments = 10,    // number of segments this CTA worked on (a count, not a time)
  kTrCombines = 11,    // number of unit combines this CTA performed (a count)
  kTrArrived = 12,     // last segment: arrival at the unit's counter known (a time)
  kTrSm = 13,          // the SM the CTA ran on
  kTraceSlots = 16
};

}  // namespace stief
