// Self-test of the bounded wait: a barrier on which nobody arrives.  The kernels of this library never wait without
// a limit; this entry point lets a test watch the limit work -- the wait gives up after the requested time, the
// kernel records LA_ERR_TIMEOUT in the context's status word and returns normally, and the context stays usable.
#include "la_common.cuh"

namespace la {

__global__ void __launch_bounds__(64) wait_timeout_kernel(int* status, unsigned long long limit_ns, long long* waited_ns) {
  __shared__ unsigned long long barrier;
  __shared__ int abort_flag;
  const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&barrier);
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
    abort_flag = 0;
  }
  __syncthreads();
  const unsigned long long t0 = global_ns();
  const bool ok = mbar_wait(bar, 0, &abort_flag, limit_ns);      // phase 0 never completes
  if (!ok && threadIdx.x == 0) {
    report(status, LA_ERR_TIMEOUT);
    if (waited_ns) *waited_ns = (long long)(global_ns() - t0);
  }
}

}  // namespace la

extern "C" la_status la_selftest_wait_timeout(la_ctx* ctx, uint32_t limit_us, int64_t* waited_ns, void* stream) {
  if (!ctx || limit_us == 0 || limit_us > 1000000u) return LA_ERR_INVALID_ARG;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return LA_ERR_CUDA;
  if (prev != ctx->device && cudaSetDevice(ctx->device) != cudaSuccess) return LA_ERR_CUDA;
  la::wait_timeout_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(ctx->d_status, 1000ull * limit_us,
                                                                          reinterpret_cast<long long*>(waited_ns));
  const cudaError_t e = cudaGetLastError();
  ctx->launches += 1;
  if (prev != ctx->device) cudaSetDevice(prev);
  return e == cudaSuccess ? LA_OK : LA_ERR_CUDA;
}
