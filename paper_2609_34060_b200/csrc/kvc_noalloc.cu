// kvc_state_update_noalloc: the state update for callers that cannot allocate device
// memory.  Its scratch (Gram matrices and eigenvalues of FIT mode) is a fixed array that is
// part of the loaded library image on every GPU, so no cudaMalloc is ever needed.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/kvc.h"

namespace {

// Built-in scratch: room for 128 Gram problems of 128 x 128 float32 (two partial sums each)
// plus their 128 eigenvalues each, and 1 KiB for KVC_FIT_FAST's one solver code per problem.
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
  // the argument checks of kvc_state_update come first: a bad call gets its own error, launches nothing
  int rc = kvc_state_update_check(src, tgt, shift, rope, st, mode);
  if (rc != KVC_OK) return rc;
  // every first call on a device, whatever its mode, resolves the array (and makes the driver load it)
  void* scratch = nullptr;
  if ((rc = scratch_for_current_device(&scratch)) != KVC_OK) return rc;
  if (st->r == 0 || st->n_cov == 0) return KVC_OK;
  const size_t need = kvc_workspace_bytes(tgt, st, mode);
  if (need > (size_t)KVC_STATIC_SCRATCH_BYTES) return KVC_E_TOO_LARGE;
  if (need == 0) return kvc_state_update(src, tgt, shift, rope, st, mode, nullptr, 0, stream);
  // The array still holds what the previous call left there; no clearing is needed, the Gram kernels
  // write every partial sum and the eigensolvers every eigenvalue before anything reads them.
  return kvc_state_update(src, tgt, shift, rope, st, mode, scratch, (size_t)KVC_STATIC_SCRATCH_BYTES, stream);
}
