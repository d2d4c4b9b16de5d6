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

struct Workspace {
  int* counters;
  float* partial_o;
  float* partial_lse;
  size_t bytes;
};
inline Workspace carve(void* base, int B, int Hq, int Hkv, int r_v, int n_cta) {
  Workspace w;
  const size_t n_units = (size_t)B * Hkv * query_tiles(Hq, Hkv);
  const size_t slots = n_units + (size_t)n_cta;
  size_t off = 0;
  uint8_t* p = static_cast<uint8_t*>(base);
  w.counters = reinterpret_cast<int*>(p + off);
  off += align_up(n_units * 4, 128);
  w.partial_o = reinterpret_cast<float*>(p + off);
  off += align_up(slots * kGroupTile * r_v * 4, 128);
  w.partial_lse = reinterpret_cast<float*>(p + off);
  off += align_up(slots * kGroupTile * 4, 128);
  w.bytes = off;
  return w;
}

}  // namespace host
}  // namespace stief
