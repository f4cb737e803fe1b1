// Diagnostic for the bounded waits: every mbarrier wait of the pass kernels goes through
// mbar_wait(), which gives up after a fixed time, raises the CTA's abort flag and lets the
// kernel return with MIXKV_ERR_TIMEOUT in the caller's status word instead of hanging.  This
// kernel makes such a wait run out on purpose (a barrier nothing ever arrives on), with the same
// helper and the same error path, so that a test can check the mechanism without any fault: the
// kernel ends by itself and the context stays usable.
#include "common.cuh"
#include "tc_common.cuh"

namespace mixkv {
namespace {

__global__ void k_wait_runs_out(int* status, unsigned long long* waited_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    mbar_init_fence();
  }
  __syncthreads();
  const unsigned long long t0 = global_ns();
  const bool ok = mbar_wait(&bar, 0, &abort_flag);   // phase 0 never completes
  __syncthreads();
  if (threadIdx.x == 0) {
    if (waited_ns) *waited_ns = global_ns() - t0;
    if (!ok && abort_flag && status) atomicExch(status, MIXKV_ERR_TIMEOUT);
  }
}

}  // namespace
}  // namespace mixkv

extern "C" int mixkv_selftest_bounded_wait(int32_t* status_dev, unsigned long long* waited_ns_dev,
                                           void* stream) {
  if (!status_dev) return MIXKV_ERR_INVALID_ARG;
  mixkv::k_wait_runs_out<<<1, 64, 0, (cudaStream_t)stream>>>(status_dev, waited_ns_dev);
  return cudaGetLastError() == cudaSuccess ? MIXKV_OK : MIXKV_ERR_CUDA;
}
