// Shared device helpers: io-type loads and stores, the feature map, the sticky status word.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "la.h"

namespace la {

// ---- io type ---------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// ---- feature map (Sec. 3: Sim(Q,K) ~ phi(Q) phi(K)^T) ------------------------------------
template <int PHI> __device__ __forceinline__ float phi(float x) {
  if (PHI == LA_PHI_ELU1) return x > 0.f ? x + 1.f : expf(x);
  return fmaxf(x, 0.f);
}

// ---- bounded waits on shared-memory barriers -------------------------------------------------
// Every wait of a kernel on an mbarrier goes through mbar_wait: it returns false once `limit_ns` nanoseconds of
// %globaltimer have passed (and raises the CTA's abort flag, so that every other waiter of the CTA gives up at its
// next check), never spins without bound and never traps.  The kernel then records LA_ERR_TIMEOUT and leaves.
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // one second per wait
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort,
                                          unsigned long long limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
#pragma unroll 1
    for (int it = 0; it < 64; ++it)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort) return false;
    if (global_ns() - t0 > limit_ns) {
      *abort = 1;
      return false;
    }
  }
}

// ---- programmatic dependent launch ----------------------------------------------------------
// A kernel launched with launch_pdl() may start while its predecessor in the stream is still running (as SMs
// become free), so that its launch latency and its set-up overlap the predecessor's tail.  Every thread calls
// pdl_wait() before it touches global memory: it returns once the predecessor has completed and its writes are
// visible.  pdl_trigger() then lets the successor start in the same way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- sticky device status ---------------------------------------------------------------
__device__ __forceinline__ void report(int* status, int code) { atomicCAS(status, 0, code); }

// Block-wide sum of one float per thread; result valid in every thread.  `scratch` holds
// at least 33 floats.
__device__ __forceinline__ float block_sum(float x, float* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  if (lane == 0) scratch[warp] = x;
  __syncthreads();
  if (warp == 0) {
    float y = lane < nwarp ? scratch[lane] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) y += __shfl_xor_sync(0xffffffffu, y, o);
    if (lane == 0) scratch[32] = y;
  }
  __syncthreads();
  float r = scratch[32];
  __syncthreads();
  return r;
}

}  // namespace la

// ---- host side --------------------------------------------------------------------------
struct la_ctx {
  la_config cfg;
  int device;
  int* d_status;          // device status word
  int prefill_kernel;     // 0 auto, 1 CUDA-core kernel
  int64_t launches;
  int sm_count;
  void* ws;               // caller-provided device workspace (may be null)
  size_t ws_bytes;
};

// Launch with programmatic stream serialization allowed (see pdl_wait above).
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Kernel launchers (one per translation unit).  All return the cudaError_t of the launch.
namespace la {
cudaError_t launch_decode(la_ctx* ctx, int B, const void* q, const void* k, const void* v, const float* w,
                          const la_state& st, void* o, cudaStream_t s);
cudaError_t launch_prefill_simt(la_ctx* ctx, int B, int T, const void* q, const void* k, const void* v,
                                const float* w, int init_state, const la_state& st, void* o, cudaStream_t s);
cudaError_t launch_verify(la_ctx* ctx, int B, int N, const void* q, const void* k, const void* v,
                          const int32_t* parent, const float* w, const la_state& st, void* o, cudaStream_t s);
cudaError_t launch_commit(la_ctx* ctx, int B, int N, const void* k, const void* v, const int32_t* parent,
                          const int32_t* accept, const la_state& st, int32_t* path_out, int32_t* commit_len,
                          cudaStream_t s);
// Tensor-core prefill (bf16, d = 128).  Sets *handled to false when the shape is not covered.
cudaError_t launch_prefill_tc(la_ctx* ctx, int B, int T, const void* q, const void* k, const void* v,
                              const float* w, int init_state, const la_state& st, void* o, cudaStream_t s,
                              bool* handled);
// Tensor-core tree verification (bf16, d = 128).  Sets *handled to false when the shape is not covered.
cudaError_t launch_verify_tc(la_ctx* ctx, int B, int N, const void* q, const void* k, const void* v,
                             const int32_t* parent, const float* w, const la_state& st, void* o, cudaStream_t s,
                             bool* handled);
cudaError_t launch_accept(la_ctx* ctx, int B, int N, const int32_t* parent, const int32_t* draft, const int32_t* pred_root,
                          const int32_t* pred, int32_t* accept_node, int32_t* accept_len, int32_t* next_token,
                          cudaStream_t s);
cudaError_t launch_accept_threshold(la_ctx* ctx, int B, int N, const int32_t* parent, const float* score, const float* thresh,
                                    int32_t* accept_node, int32_t* accept_len, cudaStream_t s);
// The three-branch block (group-exclusive linear attention, softmax inside a group, convolution) on the CUDA cores.
cudaError_t launch_prefill_grouped(la_ctx* ctx, int B, int T, const void* q, const void* k, const void* v, const float* w,
                                   int group, float alpha, float scale, int init_state, const la_state& st, void* o,
                                   cudaStream_t s);
cudaError_t launch_prefill_grouped_tc(la_ctx* ctx, int B, int T, const void* q, const void* k, const void* v, const float* w,
                                      int group, float alpha, float scale, int init_state, const la_state& st, void* o,
                                      cudaStream_t s, bool* handled);
int prefill_grouped_max_group(const la_config& c);   // largest group size the kernel's shared memory holds
// Sums of one segment of the sequence (dS = sum phi(k) v^T, dz = sum phi(k)), and sums of such parts.
cudaError_t launch_segment_state(la_ctx* ctx, int B, int T, const void* k, const void* v, float* dS, float* dz, cudaStream_t s);
cudaError_t launch_segment_state_tc(la_ctx* ctx, int B, int T, const void* k, const void* v, float* dS, float* dz,
                                    cudaStream_t s, bool* handled);
cudaError_t launch_state_prefix(la_ctx* ctx, const float* parts, const float* base, float* out, size_t n, int count,
                                cudaStream_t s);
// Workspace la_prefill can use for a launch of B sequences of T tokens (0: none needed).
size_t prefill_workspace_bytes(const la_ctx* ctx, int B, int T);
}  // namespace la
