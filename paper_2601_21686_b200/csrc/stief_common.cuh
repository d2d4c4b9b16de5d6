// Shared device-side helpers for the sm_100a kernels: PTX wrappers (mbarrier, TMA, ldmatrix, mma),
// bf16 packing, the status word, and launch descriptors passed from the host API to the kernels.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "stief.h"

namespace stief {

constexpr int kPage = STIEF_PAGE;       // tokens per cache page
constexpr int kD = STIEF_D_HEAD;        // head dimension
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// ---------------------------------------------------------------------------------------------
// status word: first error wins
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void report(int32_t* status, int code) {
  if (status != nullptr) atomicCAS(status, 0, code);
}

// ---------------------------------------------------------------------------------------------
// shared-memory addresses, mbarriers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  `abort_flag` (shared memory) short-circuits every later wait of the CTA once one
// wait has run out, so a lost copy can never hang the kernel: results are then garbage, the status
// word says STIEF_ERR_TIMEOUT, and control flow continues to the normal exit.
// `limit` is the number of polls after which the wait gives up (the kernels use the default; the wait-limit
// self-test passes a small one).  Returns true when the barrier phase completed, false when the wait gave up.
constexpr uint32_t kWaitSpins = 1u << 24;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          uint32_t limit = kWaitSpins) {
  if (mbar_try_wait(bar, parity)) return true;
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  report(status, STIEF_ERR_TIMEOUT);
  return false;
}

// The same bounded wait on the non-blocking form.  mbarrier.try_wait may park the thread for a while before it looks
// again; where a short wait sits on a latency-critical chain between a few warps, polling test_wait reacts at once.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_poll(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                               uint32_t limit = kWaitSpins << 2) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_test_wait(bar, parity)) return true;
    if ((i & 4095u) == 4095u && *abort_flag) return false;
  }
  *abort_flag = 1;
  report(status, STIEF_ERR_TIMEOUT);
  return false;
}

// Programmatic dependent launch.  launch_dependents lets the next kernel on the stream (if it was
// launched with programmatic stream serialization) start as soon as every CTA of this grid has passed
// this point or exited; grid_dependency_wait blocks until the grids this one depends on have completed
// and their writes are visible (a no-op for a normally launched kernel).
__device__ __forceinline__ void launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Bounded wait until a shared-memory counter (written by other warps of the CTA after a fence) reaches `target`
__device__ __forceinline__ bool wait_count(volatile int* counter, int target, volatile int* abort_flag, int32_t* status,
                                           uint32_t limit = kWaitSpins) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (*counter >= target) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  report(status, STIEF_ERR_TIMEOUT);
  return false;
}

// Measurement aid: one time stamp of the GPU-wide nanosecond timer into slot k of a per-CTA record (when tracing is on)
__device__ __forceinline__ void stamp(unsigned long long* rec, int k) {
  if (rec != nullptr) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    rec[k] = t;
  }
}

__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------
// TMA (tensor maps live in kernel parameter space as __grid_constant__)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tm)) : "memory");
}
// 2-D tiled load global -> shared, completion counted in bytes on an mbarrier.  x is the inner
// (element) coordinate: x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// one contiguous piece of global memory (16-byte aligned, a multiple of 16 bytes) into shared memory
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}

// ---------------------------------------------------------------------------------------------
// warp-level matrix ops
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t addr, uint32_t& r0, uint32_t& r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D += A(16x16, row) * B(16x8, col), bf16 inputs, fp32 accumulate
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float fast_exp2(float x) {   // 2^x, ex2.approx: exp2(-inf) = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---------------------------------------------------------------------------------------------
// bf16 helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {   // lo -> bits [0,16)
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
// x = hi + lo with hi = bf16(x), lo = bf16(x - hi): two bf16 words carrying ~16 significant bits
__device__ __forceinline__ void split_bf16(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  hi = pack_bf16(x0, x1);
  lo = pack_bf16(x0 - bf16_lo(hi), x1 - bf16_hi(hi));
}

// ---------------------------------------------------------------------------------------------
// swizzled page tiles in shared memory
// ---------------------------------------------------------------------------------------------
// A page tile holds 64 cache rows of R bf16 and is one contiguous block of 128 R bytes in the pool.  The TMA unit
// works through a box line by line, and at about one line per 1.3 cycles the line count, not the byte count,
// bounds what an SM can request: narrow lines waste it.  So every tile is fetched with the widest lines its
// ldmatrix access pattern allows:
//   R = 64, 128 ("boxed"):  boxes of 64 rows x 64 elements with the 128-byte swizzle (R = 128 takes two boxes);
//                           the eight 16-byte row pieces of an 8x8 ldmatrix tile fall in distinct banks.
//   R = 32 ("linear"):      the block is viewed as 32 lines of 128 bytes (two cache rows per line) with the 128-byte
//                           swizzle applied to the linear offset: conflict-free, half the lines of a 64-byte box.
//   R = 96 ("linear"):      192 lines of 64 bytes with the 64-byte swizzle (conflict-free; wider lines would cost a
//                           two-way conflict).
//   R = 48 ("bulk"):        one 1-D bulk copy of the 6144 contiguous bytes, no swizzle: rows back to back at 96 bytes,
//                           a two-way bank conflict on every ldmatrix, which is cheap beside the 192 lines of 32 bytes
//                           that a conflict-free swizzled fetch needs (rank 48/48 decode: 37.1 -> 32.0 us).
// A step of 16 rows leaves the swizzle term of an address unchanged in every form; a step of 8 rows does too except
// for R = 32, where it flips the term's bit 6 for odd 8-row groups: K8X is that bit, to be XORed into a lane's base
// offset (which addresses rows 0-7) before the plain multiple of 8 * RB is added.
template <int R>
struct Tile {
  static constexpr bool LINEAR = (R == 32 || R == 48 || R == 96);
  static constexpr bool BULK = (R == 48);                                  // fetched as one contiguous piece, unswizzled
  static constexpr int SW = (R == 48) ? 32 : (R == 96) ? 64 : 128;          // swizzle span = line width, bytes (unused for BULK)
  static constexpr uint32_t K8X = (R == 32) ? 64u : 0u;                     // see above
  static constexpr int BW = SW / 2;                                         // box width, elements
  static constexpr int NB = LINEAR ? 1 : (2 * R) / SW;                      // boxes per tile
  static constexpr int RB = LINEAR ? 2 * R : SW;                            // bytes from one token row to the next
  static constexpr int CPB = SW / 16;                                       // 16-byte chunks per swizzle span
  static constexpr int BOX_ROWS = LINEAR ? (128 * R) / SW : kPage;          // rows of the TMA box
  static constexpr int BOX_BYTES = BOX_ROWS * SW;
  static constexpr int BYTES = kPage * R * 2;
  // byte offset inside the tile of 16-byte chunk c (0 .. R/8-1) of row t
  __device__ static __forceinline__ uint32_t chunk(int t, int c) {
    if constexpr (BULK) {
      return static_cast<uint32_t>(t * RB + c * 16);
    } else if constexpr (LINEAR) {
      uint32_t off = static_cast<uint32_t>(t * RB + c * 16);
      off ^= ((off >> 7) & (CPB - 1)) << 4;
      return off;
    } else {
      const int sub = c / CPB, cc = c % CPB;
      uint32_t off = static_cast<uint32_t>(t * RB + cc * 16);
      off ^= ((off >> 7) & (CPB - 1)) << 4;
      return static_cast<uint32_t>(sub * BOX_BYTES) + off;
    }
  }
  // TMA coordinates of box nb of the tile with index `tile` (= page * Hkv + head)
  __device__ static __forceinline__ int tma_x(int nb) { return LINEAR ? 0 : nb * BW; }
  __device__ static __forceinline__ int tma_y(int tile) { return tile * BOX_ROWS; }
};

// ---------------------------------------------------------------------------------------------
// plain-old-data launch descriptors (host API -> kernels)
// ---------------------------------------------------------------------------------------------
struct LayerDev {
  int Hq, Hkv, G, r_k, r_v, num_pages;
  const __nv_bfloat16* U_k;
  long long uk_stride;
  const __nv_bfloat16* U_v;
  long long uv_stride;
  __nv_bfloat16* k_pool;
  __nv_bfloat16* v_pool;
};
struct BatchDev {
  int B, max_pages;
  const int* block_table;
  const int* seq_lens;
};

}  // namespace stief
