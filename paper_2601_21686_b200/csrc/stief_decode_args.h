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
  __nv_bfloat16* out;            // [B][Hq][128] or NULL (partials only)
  float* out_lse;                // [B][Hq] or NULL
  int len_add;                   // tokens attended beyond seq_lens (1 when appending)
  int QT;                        // query tiles per KV head = ceil(G / 8)
  int32_t* status;
};

}  // namespace stief
