// rt_layer_decode_step_static: the single-layer decode step for callers that cannot allocate.
//
// Some hosts of this library have no way to get device memory for a workspace at the moment
// they need a decode step: a serving loop that runs inside a region where the allocator is
// off limits (a latency-critical section that forbids cudaMalloc because it synchronises the
// device), a plug-in that is handed input and output buffers by its framework and nothing
// else, or a process whose memory pool is already fully committed to K/V caches.  For them the
// scratch the decode step needs lives here, in a fixed array in device memory that is part of
// the library image: every GPU that loads the library holds these bytes until the process
// exits, whether or not this entry point is ever called.
//
// The entry point obtains the array's device address once per device and then simply calls
// rt_layer_decode_step with it, so the arithmetic is that of the existing entry point.
#include <mutex>

#include "../../include/rt.h"
#include <cuda_runtime.h>

namespace {

constexpr size_t kStaticScratchBytes = RT_STATIC_SCRATCH_BYTES;

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device pointer.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device (looked up on first use).
rt_status scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RT_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return RT_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return RT_OK;
}

}  // namespace

extern "C" rt_status rt_layer_decode_step_static(const rt_config* cfg, const rt_layer_weights* w, const void* x,
                                                 int32_t B, int32_t pos, void* z, void* k_cache, void* v_cache,
                                                 int32_t N_max, void* cuda_stream) {
  const size_t need = rt_workspace_bytes(cfg, B, 1, 1);
  if (need == 0) return RT_ERR_INVALID_ARG;
  if (need > kStaticScratchBytes) return RT_ERR_WORKSPACE;      // shape too large for the built-in scratch
  void* scratch = nullptr;
  const rt_status st = scratch_for_current_device(&scratch);
  if (st != RT_OK) return st;
  return rt_layer_decode_step(cfg, w, x, B, pos, z, k_cache, v_cache, N_max, scratch, kStaticScratchBytes, cuda_stream);
}

extern "C" rt_status rt_static_get_status(void) {
  void* scratch = nullptr;
  const rt_status st = scratch_for_current_device(&scratch);
  if (st != RT_OK) return st;
  return rt_get_status(scratch);      // the status word is the first word of the scratch, as in any workspace
}
