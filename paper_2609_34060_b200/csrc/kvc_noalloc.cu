// kvc_state_update_noalloc: the state update for callers that cannot allocate device
// memory.  Its scratch (Gram matrices and eigenvalues of FIT mode) is a fixed array that is
// part of the loaded library image on every GPU, so no cudaMalloc is ever needed.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/kvc.h"

namespace {

// Built-in scratch: room for 128 Gram problems of 128 x 128 float32 (two partial sums each)
// plus their 128 eigenvalues each.
// Every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[KVC_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static void* g_scratch_addr[kMaxDevices];   // device address of the array, per device
static std::mutex g_setup_mutex;

// In host code `g_static_scratch` is only a handle for the runtime, not a device address:
// the address has to be asked for, once per device, with that device current.
static int scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return KVC_E_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return KVC_E_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return KVC_OK;
}

}  // namespace

extern "C" int kvc_state_update_noalloc(const kvc_cache* src, const kvc_cache* tgt, int32_t shift,
                                        const kvc_rope* rope, kvc_state* st, int32_t mode, void* stream) {
  if (!tgt || !st) return KVC_E_INVALID_ARG;
  const size_t need = kvc_workspace_bytes(tgt, st, mode);
  if (need > (size_t)KVC_STATIC_SCRATCH_BYTES) return KVC_E_TOO_LARGE;
  if (need == 0) return kvc_state_update(src, tgt, shift, rope, st, mode, nullptr, 0, stream);
  void* scratch = nullptr;
  const int rc = scratch_for_current_device(&scratch);
  if (rc != KVC_OK) return rc;
  // The array still holds whatever the previous call left there: start from zeros.
  if (cudaMemsetAsync(scratch, 0, need, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return KVC_E_CUDA;
  return kvc_state_update(src, tgt, shift, rope, st, mode, scratch, (size_t)KVC_STATIC_SCRATCH_BYTES, stream);
}
