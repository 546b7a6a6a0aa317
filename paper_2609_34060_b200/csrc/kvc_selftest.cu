// kvc_selftest_wait_expiry: the give-up branch of the bounded waits, taken on purpose and safely.
//
// Every asynchronous-copy wait of the tensor-core kernels is mbar_wait(): it polls an mbarrier and,
// once a cycle limit has passed, raises the CTA's abort flag and returns false; the kernel then
// drains, ORs KVC_FLAG_WAIT_EXPIRED into the status word and returns.  In normal operation that
// branch never runs.  This entry point runs it: one CTA waits, with a limit of about a millisecond,
// on an mbarrier that nothing ever arrives on.  No trap, no bad address, no endless loop: the wait
// is the library's own bounded wait with a shorter limit, so the context stays usable.
#include <cuda_runtime.h>

#include "../../include/kvc.h"
#include "kvc_launch.h"
#include "kvc_tc_ptx.cuh"

namespace kvc {
namespace {

// out[0] = threads whose wait returned true (must be 0), out[1] = the abort flag, out[2] = cycles waited by thread 0
__global__ void wait_expiry_kernel(long long limit_cycles, uint32_t* status, int* out) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  __shared__ int n_ok;
  if (threadIdx.x == 0) {
    tc::mbar_init(tc::smem_u32(&bar), 1);   // one arrival expected; nobody arrives
    tc::fence_barrier_init();
    abort_flag = 0;
    n_ok = 0;
  }
  __syncthreads();
  const long long t0 = clock64();
  const bool ok = tc::mbar_wait_for(tc::smem_u32(&bar), 0, &abort_flag, limit_cycles);
  const long long waited = clock64() - t0;
  if (ok) atomicAdd(&n_ok, 1);
  __syncthreads();
  if (threadIdx.x == 0) {
    if (abort_flag) atomicOr(status, KVC_FLAG_WAIT_EXPIRED);
    out[0] = n_ok;
    out[1] = abort_flag;
    out[2] = (int)(waited > 2147483647LL ? 2147483647LL : waited);
  }
}

}  // namespace
}  // namespace kvc

extern "C" int kvc_selftest_wait_expiry(double limit_ms, int32_t* result, void* stream) {
  if (!result || !(limit_ms > 0.0) || limit_ms > 100.0) return KVC_E_INVALID_ARG;
  int dev = 0, khz = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return KVC_E_CUDA;
  if (cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev) != cudaSuccess || khz <= 0) return KVC_E_CUDA;
  const long long limit_cycles = (long long)(limit_ms * (double)khz);
  uint32_t* status = kvc::status_word_ptr();
  if (!status) return KVC_E_CUDA;
  int* out = nullptr;
  if (cudaMalloc(&out, 3 * sizeof(int)) != cudaSuccess) return KVC_E_CUDA;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int rc = KVC_OK;
  kvc::wait_expiry_kernel<<<1, 128, 0, s>>>(limit_cycles, status, out);
  int host[3] = {-1, -1, -1};
  if (cudaGetLastError() != cudaSuccess || cudaMemcpyAsync(host, out, sizeof(host), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    rc = KVC_E_CUDA;
  cudaFree(out);
  result[0] = host[0];
  result[1] = host[1];
  result[2] = host[2];
  return rc;
}
