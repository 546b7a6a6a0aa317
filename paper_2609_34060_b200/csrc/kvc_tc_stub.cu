// Tensor-core variants of the state-update kernels that are not built yet: the C ABI
// falls back to the CUDA-core kernels when these answer KVC_E_UNSUPPORTED.
#include "../../include/kvc.h"
#include "kvc_tc.h"
namespace kvc {
int tc_project(const UpdateLaunch&, int, cudaStream_t) { return KVC_E_UNSUPPORTED; }
int tc_gram(const FitLaunch&, int, cudaStream_t) { return KVC_E_UNSUPPORTED; }
}  // namespace kvc
