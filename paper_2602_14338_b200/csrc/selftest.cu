// Self-test of the bounded waits: every pipeline wait of the tensor-core kernels goes through
// tc::mbar_wait, which gives up after a time limit and reports it.  This file holds a kernel of
// its own (one warp, no product kernel is involved) that waits on a barrier nobody ever arrives
// at, so that the give-up path -- return false, raise AERO_ST_TIMEOUT, leave normally -- can be
// seen to work without anything hanging.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace {

__global__ void __launch_bounds__(32) wait_timeout_kernel(uint32_t* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);
    abort_flag = 0;
    tc::fence_barrier_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    // phase 0 of a fresh barrier completes only when someone arrives; no one will
    const bool completed = tc::mbar_wait(&bar, 0u, &abort_flag, limit_ns);
    if (!completed) aero_raise(status, AERO_ST_TIMEOUT);
  }
}

}  // namespace

extern "C" int aero_selftest_bounded_wait(aero_ctx* ctx, uint32_t limit_us) {
  if (!ctx || limit_us == 0 || limit_us > 1000000u) return AERO_ERR_INVALID;
  if (cudaSetDevice(ctx->device) != cudaSuccess) return AERO_ERR_CUDA;
  wait_timeout_kernel<<<1, 32, 0, ctx->stream>>>(ctx->d_status, (unsigned long long)limit_us * 1000ull);
  ctx->launches += 1;
  AERO_CUDA_TRY(cudaGetLastError());
  return AERO_OK;
}
