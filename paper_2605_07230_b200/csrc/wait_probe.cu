// A self-test of the library's failure path: one CTA waits, with the context's wait limit, on an mbarrier that
// nothing ever arrives on and that no copy is in flight for.  The wait gives up, the error word is set, and the
// CTA leaves through the same teardown the tensor-core kernels use (abort flag, pause, TMEM freed), so the
// context stays usable.  cascade_check then reports CASCADE_ERR_TIMEOUT.
#include "cascade_internal.h"
#include "ptx.cuh"

namespace {

__global__ void __launch_bounds__(64, 1) k_wait_probe(int* err, unsigned long long wait_ns, unsigned int* waited_ns) {
  __shared__ __align__(8) uint64_t never;
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&never, 1);
    s_abort = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(&s_tmem_base, 32);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  volatile int* abort_flag = &s_abort;
  if (threadIdx.x == 0) {
    const uint64_t t0 = ptx::global_timer_ns();
    const bool arrived = ptx::mbar_wait(&never, 0, abort_flag, err, wait_ns);
    if (waited_ns != nullptr) *waited_ns = arrived ? 0u : (unsigned int)min(ptx::global_timer_ns() - t0, (uint64_t)0xffffffffu);
  } else if (threadIdx.x == 32) {
    // a second role polling the same barrier sees the first one's abort flag or its own limit, whichever is first
    (void)ptx::mbar_wait(&never, 0, abort_flag, err, wait_ns);
  }
  __syncwarp();
  __syncthreads();
  if (*abort_flag) __nanosleep(1000);
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(s_tmem_base, 32);
  }
}

}  // namespace

extern "C" int cascade_wait_probe(cascade_ctx* ctx, uint32_t* waited_ns, void* stream) {
  if (ctx == nullptr) return CASCADE_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  ctx->launches = 0;
  {
    KernelScope ks(ctx, K_WAIT_PROBE, s);
    k_wait_probe<<<1, 64, 0, s>>>(ctx->dev_error, ctx->wait_limit_ns, waited_ns);
  }
  CASCADE_CUDA_TRY(cudaGetLastError());
  return CASCADE_OK;
}
