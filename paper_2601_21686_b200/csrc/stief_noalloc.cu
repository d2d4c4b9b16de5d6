// stief_decode_attention_static: decode attention whose split-T scratch lives inside the library.
//
// The ordinary entry point takes a caller-allocated workspace.  Some callers have no way to get one:
// a plug-in running inside a host engine that has already handed every byte of device memory to its
// own pool and exposes no allocator, or a latency-critical loop in which cudaMalloc (which
// synchronises the device) is forbidden.  For them the scratch is the file-scope device array below.
// It is part of the loaded module, so every GPU that loads the library carries it until the process
// exits, which is why it is kept small.
//
// The array's name means different things on the two sides of the compiler: in device code it is the
// array; in host code it is only a handle for the runtime's symbol lookup and must never be given to a
// kernel as a pointer.  The device address is looked up once per device with cudaGetSymbolAddress and
// that address is what the decode kernel receives.
#include <cuda_runtime.h>

#include <mutex>

#include "stief.h"

static __device__ __align__(256) unsigned char g_static_workspace[STIEF_STATIC_WORKSPACE_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_addr[kMaxDevices] = {};

// Device address of g_static_workspace on the current device (looked up on the first call per device).
int static_workspace(void** addr) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return STIEF_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || p == nullptr) return STIEF_ERR_CUDA;
    g_addr[dev] = p;
  }
  *addr = g_addr[dev];
  return STIEF_OK;
}

}  // namespace

extern "C" int stief_decode_attention_static(const stief_layer* layer, const stief_batch* batch, const uint16_t* q,
                                             int32_t len_add, int32_t num_parts, uint16_t* out, float* out_lse,
                                             int32_t* status, void* stream) {
  if (!layer || !batch || !out) return STIEF_ERR_INVALID_ARG;
  const size_t need = stief_decode_workspace_bytes(batch->B, layer->Hq, layer->Hkv, layer->r_v, num_parts);
  if (need == 0) return STIEF_ERR_INVALID_ARG;
  if (need > (size_t)STIEF_STATIC_WORKSPACE_BYTES) return STIEF_ERR_WORKSPACE;   // shape too large for the built-in scratch
  void* ws = nullptr;
  const int rc = static_workspace(&ws);
  if (rc != STIEF_OK) return rc;
  // The array keeps whatever the previous call left.  Only the control words and the arrival counters of its four
  // sections, which sit at its start, must be zero on entry (a call that ended with a device-side error may have left
  // them non-zero): 128 bytes, then four times the counters rounded up to 128 bytes.
  const size_t groups = (size_t)(layer->Hq / layer->Hkv + 7) / 8;
  const size_t counter_bytes = 128 + 4 * (((size_t)batch->B * layer->Hkv * groups * 4 + 127) / 128 * 128);
  if (cudaMemsetAsync(ws, 0, counter_bytes, static_cast<cudaStream_t>(stream)) != cudaSuccess) return STIEF_ERR_CUDA;
  return stief_decode_attention(layer, batch, q, len_add, ws, (size_t)STIEF_STATIC_WORKSPACE_BYTES, num_parts, out, out_lse,
                                0u, status, stream);
}
