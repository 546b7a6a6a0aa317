// Host-side launch interface between the C ABI and the kernel translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "kvc_dev.cuh"

namespace kvc {

// A kernel's attributes (the opt-in to more than 48 KB of dynamic shared memory) belong to the device
// they were set on, and the device current at a call is the one that call uses: each launch site
// keeps one of these and sets the attribute once per device, not once per process.
class DeviceOnce {
 public:
  // true until mark() has been called for the current device; *dev is that device (-1 if unknown)
  bool pending(int* dev) {
    int d = -1;
    if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= 64) {
      *dev = -1;
      return true;
    }
    *dev = d;
    return !((mask_.load(std::memory_order_acquire) >> d) & 1ull);
  }
  void mark(int dev) {
    if (dev >= 0) mask_.fetch_or(1ull << dev, std::memory_order_release);
  }

 private:
  std::atomic<uint64_t> mask_{0};
};

// SM count of the current device (cached per device).
inline int device_sm_count() {
  static std::atomic<int> cache[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  const bool cacheable = dev >= 0 && dev < 64;
  int n = cacheable ? cache[dev].load(std::memory_order_relaxed) : 0;
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  if (cacheable) cache[dev].store(n, std::memory_order_relaxed);
  return n;
}

// device address of the current device's status word (kvc_api.cu); nullptr on failure
uint32_t* status_word_ptr();

// CUDA-core family (kvc_generic.cu)
cudaError_t launch_apply_generic(const ApplyLaunch& L, int d, cudaStream_t s);
int generic_apply_tile(int d);                     // tokens per tile of the generic apply kernel
constexpr int kGenericProjectTile = 64;
cudaError_t launch_project_generic(const UpdateLaunch& U, const SegTable* seg, int d, int64_t tiles, cudaStream_t s);
cudaError_t launch_gram_generic(const FitLaunch& F, const SegTable* seg, int d, cudaStream_t s);
// full eigensolver; solver != nullptr: matrices with solver[m] == 0 are skipped (already served)
cudaError_t launch_eig(const FitLaunch& F, int d, const int32_t* solver, cudaStream_t s);
// top-r subspace solver (kvc_eig_subspace.cu): sums and symmetrises the partial Grams, serves the
// matrices whose spectrum has a gap behind the r-th eigenvalue, writes 0 or a reason per matrix
constexpr int kSubspaceMaxRank = 32;
cudaError_t launch_eig_subspace(const FitLaunch& F, int d, int32_t* solver, cudaStream_t s);

// FIT of layer-grouped states (kvc_group_fit.cu)
constexpr int kGroupFitParts = 4;   // token ranges whose back-projections are summed in a fixed order (CUDA-core pass; the tensor-core pass uses 2)
constexpr int kGroupFitTraceParts = 32;   // room for the partial sums of the trace (tensor-core pass: half x team warp)
cudaError_t launch_group_backproject(const GroupFitLaunch& G, const SegTable* seg, cudaStream_t s);
cudaError_t launch_group_small(const GroupFitLaunch& G, int op, cudaStream_t s);
cudaError_t launch_group_coeff_transform(const GroupFitLaunch& G, cudaStream_t s);
cudaError_t launch_zero_if(float* ptr, int64_t n, const int32_t* run_if, cudaStream_t s);

// reliability gate (kvc_gate.cu)
cudaError_t launch_gate_generic(const GateLaunch& g, int d, cudaStream_t s);
cudaError_t launch_effective_rank(const float* evals, int n_mat, int d, float energy, int32_t* out, cudaStream_t s);
cudaError_t launch_realign_basis(const RealignLaunch& q, cudaStream_t s);
cudaError_t launch_token_weights(const float* scores, const TokenWeightsLaunch& q, cudaStream_t s);
cudaError_t launch_gate_weights(const double* dist_sq, int n, double temperature, double* gw, double* entropy, cudaStream_t s);

}  // namespace kvc
