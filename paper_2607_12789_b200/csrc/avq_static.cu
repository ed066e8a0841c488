// avq_forward_static: the forward pass for callers that cannot provide device scratch.
//
// Some hosts of this library may not call cudaMalloc at the point where they need attention:
// code running inside a framework's memory-planned region, a real-time loop that forbids
// allocator calls after start-up, or a plugin whose only device memory is what the host
// application hands it for inputs and outputs.  avq_forward needs a workspace for the key
// indices and the per-codeword aggregates between its stages; here that workspace is a
// fixed array that lives in the library's device image.
//
// Host code must not treat the array's name as a device address: on the host the symbol is
// only a handle.  The address the kernels need comes from cudaGetSymbolAddress, queried once
// per device with that device current.
#include <mutex>

#include "avq_internal.h"

namespace {

constexpr size_t kStaticBytes = (size_t)AVQ_STATIC_WORKSPACE_BYTES;
constexpr int kMaxDevices = 64;

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_workspace[kStaticBytes];

std::mutex g_mu;
void* g_dev_ptr[kMaxDevices] = {};

// Device address of the array on the current device, resolved on first use.
avq_status static_workspace_ptr(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return AVQ_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return AVQ_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_dev_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) return AVQ_ERR_CUDA;
    g_dev_ptr[dev] = p;
  }
  *out = g_dev_ptr[dev];
  return AVQ_OK;
}

}  // namespace

extern "C" {

size_t avq_static_workspace_bytes(void) { return kStaticBytes; }

avq_status avq_forward_static(const avq_problem* prob, const void* Q, const void* K, const void* V,
                              const void* Cp, const void* Cc, int32_t P, int32_t block_q, void* Y,
                              int32_t* topp_out, float* importance_out, void* stream) {
  const size_t need = avq_workspace_bytes(prob, P, block_q);
  if (need == 0) {
    // Invalid or unsupported problem: let the regular entry point name the reason.  It
    // rejects before it touches the (absent) workspace.
    return avq_forward(prob, Q, K, V, Cp, Cc, P, block_q, Y, topp_out, importance_out, nullptr, 0, stream);
  }
  if (need > kStaticBytes) return AVQ_ERR_WORKSPACE;
  void* ws = nullptr;
  avq_status s = static_workspace_ptr(&ws);
  if (s != AVQ_OK) return s;
  // avq_forward clears the status header and zeroes the aggregates it accumulates into on
  // every call, so the previous call's contents never leak into this one.
  return avq_forward(prob, Q, K, V, Cp, Cc, P, block_q, Y, topp_out, importance_out, ws, kStaticBytes, stream);
}

avq_status avq_check_static(void* stream) {
  void* ws = nullptr;
  avq_status s = static_workspace_ptr(&ws);
  if (s != AVQ_OK) return s;
  return avq_check(ws, stream);
}

}  // extern "C"
