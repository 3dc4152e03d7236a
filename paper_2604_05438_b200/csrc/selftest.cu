// tkphi_selftest_timeout: drives the error path of the bounded device-side waits.
// Every wait in the library's kernels gives up after a fixed number of polls, raises the
// CTA's abort flag (which makes the other warps of the CTA leave their own waits), and the
// CTA stores kStatusTimeout in the workspace's status word before it returns.  No ordinary
// input makes a wait run out, so this one-CTA kernel stages the situation: warp 0 waits on
// an mbarrier that nothing arrives on, with a limit of 4096 polls; warp 1 waits, with the
// library's ordinary limit, on a barrier that warp 0 would have signalled after its wait,
// and must be released early by the abort flag.  The kernel ends by itself in microseconds.
#include "../../include/tkphi.h"
#include "common.cuh"
#include "sm100.cuh"

namespace tkphi {

constexpr uint32_t kSelftestPolls = 1u << 12;

__global__ void __launch_bounds__(64) selftest_timeout_kernel(int* status) {
  __shared__ uint64_t bars[2];       // [0]: never signalled; [1]: warp 0 -> warp 1 hand-off
  __shared__ int s_abort;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    mbar_init(&bars[0], 1);
    mbar_init(&bars[1], 1);
    mbar_fence_init();
    s_abort = 0;
  }
  __syncthreads();
  bool ok;
  if (warp == 0) {
    ok = mbar_wait_limit(&bars[0], 0, &s_abort, kSelftestPolls);      // runs out
    __syncwarp();
    if (ok && lane == 0) mbar_arrive(&bars[1]);
  } else {
    ok = mbar_wait(&bars[1], 0, &s_abort);                            // released by the abort flag
  }
  // teardown as in the library's kernels: all roles meet, one thread reports
  __syncthreads();
  if (s_abort && tid == 0) atomicExch(status, kStatusTimeout);
}

}  // namespace tkphi

extern "C" tkphi_status tkphi_selftest_timeout(void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < 256) return TKPHI_ERR_WORKSPACE;
  tkphi::selftest_timeout_kernel<<<1, 64, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<int*>(workspace));
  return cudaGetLastError() == cudaSuccess ? TKPHI_OK : TKPHI_ERR_CUDA;
}
