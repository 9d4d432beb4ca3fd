// Forward entry point for callers that cannot hand the library any scratch memory of their own.
//
// Some callers of this library run where device allocation is off the table: an inference plug-in whose host
// framework gives it nothing but the input and output buffers of one layer and forbids allocation inside the
// enqueue call (a device allocation synchronises the whole GPU and would stall every other stream of the process), or a
// control loop with a fixed memory budget decided at start-up.  For them the scratch memory of the time-split forward
// path lives in a fixed array inside the library's own device image instead of in a caller-provided workspace.
//
// The array is a file-scope __device__ object, so every GPU that loads the library carries it until the process
// exits.  In host code its name is only a host-side handle of the symbol, not a device address: the address is looked up
// once per device with cudaGetSymbolAddress while that device is current, and that pointer is what the kernels get.
#include <cuda_runtime.h>

#include <mutex>

#include "ssm_scan.h"

namespace {

static __device__ __align__(256) unsigned char g_static_scratch[SSM_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};
bool g_scratch_ready[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up on the first call per device).
cudaError_t static_scratch_on_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ready[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = ptr;
    g_scratch_ready[dev] = true;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" ssm_status_t ssm_scan_fwd_static(const ssm_problem_t* p, const void* x, const void* delta, const float* A,
                                            const void* B, const void* C, const float* D_skip, const void* z, void* out,
                                            void* saved_states, void* stream) {
  // Size check first: a problem whose scratch does not fit the fixed array is refused before anything else happens.
  // (An invalid problem reports 0 bytes here and is then rejected by the regular argument checks below.)
  const size_t need = ssm_scan_fwd_workspace_bytes(p);
  if (need > (size_t)SSM_STATIC_SCRATCH_BYTES) return SSM_ERR_WORKSPACE;
  void* scratch = nullptr;
  if (static_scratch_on_current_device(&scratch) != cudaSuccess) return SSM_ERR_CUDA;
  // The scratch needs no preparation here: ssm_scan_fwd clears the status word and the hand-off flags at its head on
  // the caller's stream (memsets, no allocation), the summary pass writes every segment end state and step-size sum,
  // and the carry pass writes every segment start state, before any of them is read.
  return ssm_scan_fwd(p, x, delta, A, B, C, D_skip, z, out, saved_states, scratch, (size_t)SSM_STATIC_SCRATCH_BYTES,
                      stream);
}
