// Host-side helpers shared by the translation units that implement C-ABI entry points: pointer checks, the
// batch descriptor, the SM count, and the carving of the decode workspace.
#pragma once

#include "stief_kernels.h"
#include "stief_partition.cuh"

namespace stief {
namespace host {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline int check_batch(const stief_batch* b) {
  if (!b || b->B <= 0 || b->max_pages_per_seq <= 0 || !b->block_table || !b->seq_lens) return STIEF_ERR_INVALID_ARG;
  if (b->B > kMaxBatch) return STIEF_ERR_INVALID_ARG;
  return STIEF_OK;
}

inline BatchDev to_dev(const stief_batch* b) {
  BatchDev d;
  d.B = b->B; d.max_pages = b->max_pages_per_seq; d.block_table = b->block_table; d.seq_lens = b->seq_lens;
  return d;
}

inline int sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return 148;
  }
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      n = 148;
    }
    cached[dev] = n;
  }
  return cached[dev];
}

inline int resolve_parts(int num_parts) { return num_parts > 0 ? num_parts : sm_count(); }
inline int query_tiles(int Hq, int Hkv) { return (Hq / Hkv + kGroupTile - 1) / kGroupTile; }

// The decode workspace.  Two kernels of an overlapped chain may be at work at the same time, so everything a kernel
// writes exists twice ("halves") and consecutive launches on a workspace alternate between them; a kernel then only has
// to know that the LAST user of its own half has finished, which the control words tell it:
//   control[0..1]  finished[h]:   epoch of the last kernel that finished all its work on half h
//   control[2..3]  units_done[h]: units finalised so far by the kernel now using half h (zero between kernels)
// followed by the arrival counters and the partials of half 0 and of half 1.
struct Workspace {
  int* control;
  int* counters[2];
  float* partial_o[2];
  float* partial_lse[2];
  size_t control_bytes;      // control words and both halves' counters: what must be zero before the first use
  size_t bytes;
};
// Layers of different r_v may share a workspace (the layers of one decode step do), and two of them may be at work in
// the two halves at once, so where a half lies must not depend on r_v: half 0 follows the counters, half 1 begins in the
// middle of what is left of the caller's buffer (`total_bytes`, the size every call on this buffer is given; 0: the
// size just computed, for planning).  `bytes` is what this shape needs; a caller's buffer below that is refused.
inline Workspace carve(void* base, int B, int Hq, int Hkv, int r_v, int n_cta, size_t total_bytes = 0) {
  Workspace w;
  const size_t n_units = (size_t)B * Hkv * query_tiles(Hq, Hkv);
  const size_t slots = n_units + (size_t)n_cta;
  size_t off = 0;
  uint8_t* p = static_cast<uint8_t*>(base);
  w.control = reinterpret_cast<int*>(p + off);
  off += 128;
  for (int h = 0; h < 2; ++h) {
    w.counters[h] = reinterpret_cast<int*>(p + off);
    off += align_up(n_units * 4, 128);
  }
  w.control_bytes = off;
  const size_t po = align_up(slots * kGroupTile * r_v * 4, 128), pl = align_up(slots * kGroupTile * 4, 128);
  w.bytes = off + 2 * (po + pl);
  const size_t half1 = total_bytes > w.bytes ? (total_bytes - off) / 2 / 128 * 128 : po + pl;
  for (int h = 0; h < 2; ++h) {
    const size_t at = off + (h ? half1 : 0);
    w.partial_o[h] = reinterpret_cast<float*>(p + at);
    w.partial_lse[h] = reinterpret_cast<float*>(p + at + po);
  }
  return w;
}

// Which half a launch takes, its epoch, and the epoch of the previous user of that half (0 = not known: the kernel
// then waits for its predecessor on the stream to complete, which is always safe).  Epochs are unique within the
// process and never 0.  The record is per host thread and per workspace address; a thread that has not seen a
// workspace before simply starts with "not known".
struct WorkspaceTurn {
  int half;
  unsigned epoch, prev_epoch;
};
struct WorkspaceRecord {
  const void* ws;
  unsigned last_epoch[2];
  int last_half;
};
inline WorkspaceRecord* workspace_record(const void* ws) {
  constexpr int kRecords = 16;
  static thread_local WorkspaceRecord recs[kRecords] = {};
  static thread_local int next = 0;
  for (int i = 0; i < kRecords; ++i)
    if (recs[i].ws == ws) return &recs[i];
  WorkspaceRecord* r = &recs[next];
  next = (next + 1) % kRecords;
  r->ws = ws; r->last_epoch[0] = r->last_epoch[1] = 0u; r->last_half = 1;
  return r;
}
unsigned next_workspace_epoch();     // stief_api.cu: one counter for the whole process
// A launch that merges its units itself (the fused kernels): alternates the halves and publishes its epoch.
inline WorkspaceTurn take_workspace_turn(const void* ws) {
  WorkspaceRecord* r = workspace_record(ws);
  WorkspaceTurn t;
  t.half = 1 - r->last_half;
  t.epoch = next_workspace_epoch();
  t.prev_epoch = r->last_epoch[t.half];
  r->last_epoch[t.half] = t.epoch;
  r->last_half = t.half;
  return t;
}
// A launch that uses half 0 without publishing an epoch (partials for stief_split_combine, kernels that keep to the
// plain dependency wait): whoever takes half 0 next must not trust the record.
inline WorkspaceTurn take_workspace_half0(const void* ws) {
  WorkspaceRecord* r = workspace_record(ws);
  r->last_epoch[0] = 0u;
  r->last_half = 0;
  return WorkspaceTurn{0, 0u, 0u};
}
inline void forget_workspace(const void* ws) {
  WorkspaceRecord* r = workspace_record(ws);
  r->last_epoch[0] = r->last_epoch[1] = 0u;
  r->last_half = 1;
}

}  // namespace host
}  // namespace stief
