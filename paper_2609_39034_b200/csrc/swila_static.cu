// Prefill from host buffers for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is not an option: inside a host
// application whose memory budget is fixed at start-up, or in a plug-in that is handed a
// stream but no allocator.  swila_forward_host needs a device workspace from its caller;
// this variant brings its own, a fixed array that is part of the library image.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/swila.h"

namespace {

// The workspace.  It lives in the device's global memory for as long as the library is
// loaded, on every GPU that loads it.  In host code the identifier below is only a handle for
// the runtime's symbol table, not an address a kernel or a copy may use: the device address is
// looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_workspace[SWILA_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
void *g_workspace_addr[kMaxDevices] = {};
std::mutex g_setup_mutex;

// Device address of the workspace on the current device (set-up on first use), or nullptr.
void *workspace_on_current_device(cudaError_t *err) {
  int dev = -1;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= kMaxDevices) {
    *err = cudaErrorInvalidDevice;
    return nullptr;
  }
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_workspace_addr[dev] == nullptr) {
    void *p = nullptr;
    *err = cudaGetSymbolAddress(&p, g_static_workspace);  // resolves against the CURRENT device
    if (*err != cudaSuccess) return nullptr;
    g_workspace_addr[dev] = p;
  }
  return g_workspace_addr[dev];
}

}  // namespace

extern "C" {

size_t swila_forward_host_static_capacity(void) { return (size_t)SWILA_STATIC_WORKSPACE_BYTES; }

int swila_forward_host_static(const swila_shape_t *shape, const void *q, const void *k, const void *v,
                              const swila_gates_t *gates, const swila_state_t *state_in, swila_state_t *state_out,
                              void *o, void *stream) {
  const size_t need = swila_forward_host_workspace_bytes(shape);
  if (need == 0)  // invalid shape: let the general entry point name the reason (it checks the shape first)
    return swila_forward_host(shape, q, k, v, gates, state_in, state_out, o, nullptr, 0, stream);
  if (need > (size_t)SWILA_STATIC_WORKSPACE_BYTES) return SWILA_ERR_SIZE;
  cudaError_t err = cudaSuccess;
  void *ws = workspace_on_current_device(&err);
  if (ws == nullptr) return SWILA_ERR_CUDA;
  // Nothing in the workspace has to start at zero: every byte the kernel reads is written by
  // this call's own host-to-device copies first, so the previous call's contents are inert.
  return swila_forward_host(shape, q, k, v, gates, state_in, state_out, o, ws, (size_t)SWILA_STATIC_WORKSPACE_BYTES,
                            stream);
}

}  // extern "C"
