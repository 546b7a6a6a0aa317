// Host-side launch interface between the C ABI and the kernel translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvc_dev.cuh"

namespace kvc {

// CUDA-core family (kvc_generic.cu)
cudaError_t launch_apply_generic(const ApplyLaunch& L, int d, cudaStream_t s);
int generic_apply_tile(int d);                     // tokens per tile of the generic apply kernel
constexpr int kGenericProjectTile = 64;
cudaError_t launch_project_generic(const UpdateLaunch& U, int d, int64_t tiles, cudaStream_t s);
cudaError_t launch_gram_generic(const FitLaunch& F, int d, cudaStream_t s);
// full eigensolver; solver != nullptr: matrices with solver[m] == 0 are skipped (already served)
cudaError_t launch_eig(const FitLaunch& F, int d, const int32_t* solver, cudaStream_t s);
// top-r subspace solver (kvc_eig_subspace.cu): sums and symmetrises the partial Grams, serves the
// matrices whose spectrum has a gap behind the r-th eigenvalue, writes 0 or a reason per matrix
constexpr int kSubspaceMaxRank = 32;
cudaError_t launch_eig_subspace(const FitLaunch& F, int d, int32_t* solver, cudaStream_t s);

// reliability gate (kvc_gate.cu)
cudaError_t launch_gate_generic(const GateLaunch& g, int d, cudaStream_t s);
cudaError_t launch_effective_rank(const float* evals, int n_mat, int d, float energy, int32_t* out, cudaStream_t s);
cudaError_t launch_realign_basis(const RealignLaunch& q, cudaStream_t s);
cudaError_t launch_token_weights(const float* scores, const TokenWeightsLaunch& q, cudaStream_t s);
cudaError_t launch_gate_weights(const double* dist_sq, int n, double temperature, double* gw, double* entropy, cudaStream_t s);

}  // namespace kvc
