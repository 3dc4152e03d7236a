// tkphi_build_summaries_static: the prefill summary build for callers that cannot
// allocate device memory.  Its scratch lives in a fixed array inside this library's
// device image instead of a caller-provided workspace.
#include "../../include/tkphi.h"

#include <cuda_runtime.h>
#include <cstdio>
#include <mutex>

namespace {

// Scratch shared by every call on a device.  Each GPU context that loads the library
// holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[TKPHI_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

thread_local char g_static_err[256] = "";

// In host code `g_static_scratch` is only a handle for the runtime, not an address a
// kernel can use: the device address is looked up once per device, with that device
// current, and cached.
cudaError_t scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" {

const char* tkphi_static_last_error(void) { return g_static_err; }

tkphi_status tkphi_build_summaries_static(const tkphi_kv_desc* kv, const tkphi_phi_desc* phi, float* S, float* u,
                                          void* cuda_stream) {
  g_static_err[0] = 0;
  const size_t need = tkphi_workspace_bytes(kv, nullptr, 0, TKPHI_WS_BUILD);
  if (need == 0) {
    snprintf(g_static_err, sizeof(g_static_err), "%s", tkphi_last_error());
    return TKPHI_ERR_INVALID_ARG;
  }
  if (need > (size_t)TKPHI_STATIC_SCRATCH_BYTES) {
    snprintf(g_static_err, sizeof(g_static_err),
             "this problem needs %zu bytes of scratch; the built-in scratch holds %zu: use tkphi_build_summaries "
             "with a caller-allocated workspace",
             need, (size_t)TKPHI_STATIC_SCRATCH_BYTES);
    return TKPHI_ERR_WORKSPACE;
  }
  void* scratch = nullptr;
  cudaError_t e = scratch_address(&scratch);
  if (e != cudaSuccess) {
    snprintf(g_static_err, sizeof(g_static_err), "looking up the built-in scratch: %s", cudaGetErrorString(e));
    return TKPHI_ERR_CUDA;
  }
  // The build clears the counters it needs at the head of the scratch on the stream
  // before its kernel runs, so whatever the previous call left there does not matter.
  tkphi_status st = tkphi_build_summaries(kv, phi, S, u, scratch, (size_t)TKPHI_STATIC_SCRATCH_BYTES, cuda_stream);
  if (st != TKPHI_OK) snprintf(g_static_err, sizeof(g_static_err), "%s", tkphi_last_error());
  return st;
}

}  // extern "C"
