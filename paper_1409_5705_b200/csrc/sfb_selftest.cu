// Self-test of the bounded device-side wait.  Every pipeline wait of the tensor-core kernels goes through
// ptx::mbar_wait, which gives up after a cycle limit, raises the CTA's abort flag and lets the kernel set
// SFB_STATUS_TIMEOUT and return.  This file drives that same path on purpose, in its harmless form: one CTA, one
// mbarrier that nothing ever arrives at, a short limit, no copy in flight and no tensor memory held.
#include "sfb_internal.h"
#include "sfb_ptx.cuh"

namespace sfb {
namespace {

__global__ void __launch_bounds__(32) wait_timeout_kernel(long long max_cycles, uint32_t* status, long long* waited_cycles) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_word;
  volatile uint32_t* abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_word = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const long long t0 = clock64();
    ptx::mbar_wait(&bar, 0, abort_flag, max_cycles);            // phase 0 never completes: nobody arrives
    if (waited_cycles) *waited_cycles = clock64() - t0;
  }
  __syncthreads();
  // the same read-out as the product kernels: a wait that ran out is reported through the status word
  if (*abort_flag && threadIdx.x == 0) atomicOr(status, SFB_STATUS_TIMEOUT);
}

}  // namespace
}  // namespace sfb

extern "C" int sfb_selftest_wait_timeout(sfb_ctx* ctx, int64_t max_cycles) {
  if (!ctx) return SFB_ERR_ARG;
  if (max_cycles < 1 || max_cycles > 2000000000ll) return SFB_ERR_ARG;      // at most about a second
  sfb::wait_timeout_kernel<<<1, 32, 0, ctx->stream>>>(max_cycles, ctx->at<uint32_t>(ctx->lay.status), nullptr);
  sfb::count_launch();
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    ctx->last_cuda = static_cast<int>(e);
    return SFB_ERR_CUDA;
  }
  return SFB_OK;
}
