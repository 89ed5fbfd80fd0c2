// laser_route_static: one-layer routing whose scratch lives inside the library image.
//
// Some callers cannot allocate device memory at all: a plugin running inside another
// program's fixed memory pool, a service whose allocator was frozen after start-up, a loop
// that must not call cudaMalloc because an allocation stalls every stream of the process.
// For them the scratch that laser_route() takes from the caller is a fixed array in this
// translation unit.  The array is part of the loaded module, so every GPU that loads the
// library holds LASER_STATIC_SCRATCH_BYTES of it until the process exits.
//
// Host code cannot use the array's name as a pointer (on the host the name is only a handle
// for the runtime), so the device address is looked up once per device with
// cudaGetSymbolAddress and cached.
#include "../../include/laser.h"

#include <cuda_runtime.h>

#include <mutex>

namespace {

static __device__ __align__(256) unsigned char g_static_scratch[LASER_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device

// Device address of the scratch array on the current device; nullptr if the lookup fails.
void* static_scratch_for_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) {
      (void)cudaGetLastError();
      return nullptr;
    }
    g_scratch_addr[dev] = ptr;
  }
  return g_scratch_addr[dev];
}

}  // namespace

extern "C" int laser_route_static(const void* hidden, const void* w_g, const float* bias,
                                  int32_t* loads, const int32_t* expert_to_bin,
                                  int32_t* bin_loads, const laser_params* p,
                                  int32_t* expert_ids, float* weights, int32_t* offsets,
                                  int32_t* perm, float* logits_out, int32_t* status_word,
                                  void* cuda_stream) {
  size_t need = 0;
  const int rc = laser_workspace_bytes(p, &need);
  if (rc != LASER_OK) return rc;
  if (need > (size_t)LASER_STATIC_SCRATCH_BYTES) return LASER_ERR_STATIC_SCRATCH;
  void* scratch = static_scratch_for_current_device();
  if (!scratch) return LASER_ERR_CUDA;
  // The routing kernels clear the one part of the scratch that must start at zero (the
  // router's ready flags) on the stream themselves; everything else is written before it is
  // read, so the previous call's contents do no harm.
  return laser_route(hidden, w_g, bias, loads, expert_to_bin, bin_loads, p, expert_ids, weights,
                     offsets, perm, logits_out, status_word, scratch,
                     (size_t)LASER_STATIC_SCRATCH_BYTES, cuda_stream);
}
