// Self-test of the bounded waits: a one-CTA kernel that waits, with the library's own wait routine, on a barrier
// that nothing ever arrives on, and then takes the same way out as the tensor-core kernels do after a wait has run
// out (abort flag, status word, TMEM released, normal exit).  No copy and no MMA is ever in flight, so the exit is
// safe by construction; what it shows is that a wait that cannot end costs `limit_ns`, not a hung GPU, and that
// the context works afterwards.
#include "common.cuh"
#include "ptx.cuh"

namespace {

__global__ void __launch_bounds__(128, 1) wait_timeout_kernel(int* dev_status, unsigned long long limit_ns) {
  __shared__ uint64_t never;           // a barrier with one pending arrival that no thread makes
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  grid_dependency_enter();
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&never, 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 0) { ptx::tmem_alloc(&tmem_slot, 32); ptx::tmem_relinquish(); }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  // every thread waits, as the consumer warps of the real kernels do; the first one whose limit passes raises the
  // flag and writes the status word, the others see the flag at their next check
  (void)ptx::mbar_wait_limit(&never, 0, &abort_flag, dev_status, limit_ns);
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) ptx::tmem_dealloc(tmem, 32);
}

}  // namespace

int launch_wait_timeout_selftest(d3tom_ctx* ctx, long long limit_ns, cudaStream_t s) {
  D3TOM_CUDA_TRY(ctx, launch_serialized(wait_timeout_kernel, 1, 128, 0, s, ctx->dev_status, (unsigned long long)limit_ns));
  D3TOM_LAUNCH_CHECK(ctx);
  return D3TOM_OK;
}
