#include "../../include/kvc.h"
#include "kvc_tc.h"
namespace kvc {
int tc_apply_single(const DevItem&, int, int, uint32_t*, cudaStream_t) { return KVC_E_UNSUPPORTED; }
int tc_apply_batch(DevItem*, int64_t*, int, int, int, uint32_t*, void*, void*, size_t, cudaStream_t) { return KVC_E_UNSUPPORTED; }
size_t tc_batch_extra_bytes(int) { return 0; }
int tc_project(const UpdateLaunch&, int, cudaStream_t) { return KVC_E_UNSUPPORTED; }
int tc_gram(const FitLaunch&, int, cudaStream_t) { return KVC_E_UNSUPPORTED; }
}
