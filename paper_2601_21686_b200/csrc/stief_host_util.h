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

// The decode workspace.  Several kernels of an overlapped chain may be at work at the same time, so everything a kernel
// writes exists kWorkspaceSections times and consecutive launches on a workspace take the sections in turn; a kernel
// then only has to know that the LAST user of its own section has finished, which the control words tell it:
//   control[s]                       finished:   epoch of the last kernel that finished all its work on section s
//   control[kWorkspaceSections + s]  units_done: units finalised so far by the kernel now using section s (zero between kernels)
// followed by the arrival counters of every section, then the sections' partials.
constexpr int kWorkspaceSections = 4;
struct Workspace {
  int* control;
  int* counters[kWorkspaceSections];
  float* partial_o[kWorkspaceSections];
  float* partial_lse[kWorkspaceSections];
  size_t control_bytes;      // control words and all counters: what must be zero before the first use
  size_t bytes;
};
// Layers of different r_v may share a workspace (the layers of one decode step do), and several of them may be at work
// in different sections at once, so where a section lies must not depend on r_v: section 0 follows the counters, the
// others divide what is left of the caller's buffer evenly (`total_bytes`, the size every call on this buffer is given;
// 0: the size just computed, for planning).  `bytes` is what this shape needs; a caller's buffer below that is refused.
inline Workspace carve(void* base, int B, int Hq, int Hkv, int r_v, int n_cta, size_t total_bytes = 0) {
  Workspace w;
  const size_t n_units = (size_t)B * Hkv * query_tiles(Hq, Hkv);
  const size_t slots = n_units + (size_t)n_cta;
  size_t off = 0;
  uint8_t* p = static_cast<uint8_t*>(base);
  w.control = reinterpret_cast<int*>(p + off);
  off += 128;
  for (int h = 0; h < kWorkspaceSections; ++h) {
    w.counters[h] = reinterpret_cast<int*>(p + off);
    off += align_up(n_units * 4, 128);
  }
  w.control_bytes = off;
  const size_t po = align_up(slots * kGroupTile * r_v * 4, 128), pl = align_up(slots * kGroupTile * 4, 128);
  w.bytes = off + kWorkspaceSections * (po + pl);
  const size_t pitch = total_bytes > w.bytes ? (total_bytes - off) / kWorkspaceSections / 128 * 128 : po + pl;
  for (int h = 0; h < kWorkspaceSections; ++h) {
    w.partial_o[h] = reinterpret_cast<float*>(p + off + h * pitch);
    w.partial_lse[h] = reinterpret_cast<float*>(p + off + h * pitch + po);
  }
  return w;
}

// Which section a launch takes, its epoch, and the epoch of the previous user of that section (0 = not known: the
// kernel then waits for its predecessor on the stream to complete, which is always safe).  Epochs are unique within
// the process and never 0.  The record is per host thread and per workspace address; a thread that has not seen a
// workspace before simply starts with "not known".
struct WorkspaceTurn {
  int section;
  unsigned epoch, prev_epoch;
};
struct WorkspaceRecord {
  const void* ws;
  unsigned last_epoch[kWorkspaceSections];
  int last_section;
};
inline void reset_record(WorkspaceRecord* r, const void* ws) {
  r->ws = ws;
  for (int h = 0; h < kWorkspaceSections; ++h) r->last_epoch[h] = 0u;
  r->last_section = kWorkspaceSections - 1;
}
inline WorkspaceRecord* workspace_record(const void* ws) {
  constexpr int kRecords = 16;
  static thread_local WorkspaceRecord recs[kRecords] = {};
  static thread_local int next = 0;
  for (int i = 0; i < kRecords; ++i)
    if (recs[i].ws == ws) return &recs[i];
  WorkspaceRecord* r = &recs[next];
  next = (next + 1) % kRecords;
  reset_record(r, ws);
  return r;
}
unsigned next_workspace_epoch();     // stief_api.cu: one counter for the whole process
// A launch that merges its units itself (the fused kernels): takes the next section and publishes its epoch there.
inline WorkspaceTurn take_workspace_turn(const void* ws) {
  WorkspaceRecord* r = workspace_record(ws);
  WorkspaceTurn t;
  t.section = (r->last_section + 1) % kWorkspaceSections;
  t.epoch = next_workspace_epoch();
  t.prev_epoch = r->last_epoch[t.section];
  r->last_epoch[t.section] = t.epoch;
  r->last_section = t.section;
  return t;
}
// A launch that uses section 0 without publishing an epoch (partials for stief_split_combine, kernels that keep to the
// plain dependency wait): whoever takes section 0 next must not trust the record.
inline WorkspaceTurn take_workspace_section0(const void* ws) {
  WorkspaceRecord* r = workspace_record(ws);
  r->last_epoch[0] = 0u;
  r->last_section = 0;
  return WorkspaceTurn{0, 0u, 0u};
}
inline void forget_workspace(const void* ws) { reset_record(workspace_record(ws), ws); }

}  // namespace host
}  // namespace stief
