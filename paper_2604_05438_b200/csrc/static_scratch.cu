// tkphi_build_summaries_static: the prefill summary build for callers that cannot
// allocate device memory.  Its scratch lives in a fixed array inside this library's
// device image instead of a caller-provided workspace.
#include "../../include/tkphi.h"

#include <cuda_runtime.h>
#include <cstdio>
#include <mutex>

namespace {

// Scratch shared by every call on a device.  The array is part of this library's device
// code: each GPU on which the CUDA runtime loads that code (at the latest on the first
// call of the entry point below on that GPU) holds these bytes until the process exits.
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
  // Nothing in the scratch has to be cleared between calls: the build kernel sets the
  // status word at its head itself and overwrites every partial sum before one is read.
  tkphi_status st = tkphi_build_summaries(kv, phi, S, u, scratch, (size_t)TKPHI_STATIC_SCRATCH_BYTES, cuda_stream);
  if (st != TKPHI_OK) snprintf(g_static_err, sizeof(g_static_err), "%s", tkphi_last_error());
  return st;
}

tkphi_status tkphi_static_device_status(void* cuda_stream, int32_t* status_out) {
  g_static_err[0] = 0;
  if (!status_out) {
    snprintf(g_static_err, sizeof(g_static_err), "status_out is NULL");
    return TKPHI_ERR_INVALID_ARG;
  }
  int dev = -1;
  void* scratch = nullptr;
  if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) {
    std::lock_guard<std::mutex> lock(g_mu);
    scratch = g_scratch_addr[dev];
  }
  if (!scratch) {
    snprintf(g_static_err, sizeof(g_static_err), "no tkphi_build_summaries_static call has been made on this device");
    return TKPHI_ERR_INVALID_ARG;
  }
  // the status word is the first word of the scratch, as in a caller-provided workspace
  tkphi_status st = tkphi_device_status(scratch, cuda_stream, status_out);
  if (st != TKPHI_OK) snprintf(g_static_err, sizeof(g_static_err), "%s", tkphi_last_error());
  return st;
}

}  // extern "C"
