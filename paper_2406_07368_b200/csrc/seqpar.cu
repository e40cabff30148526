// Pieces of a prefill that is cut along the sequence (Sec. 4.1: between groups only the cumulative sums of
// phi(k) v^T and phi(k) are carried, so a segment of the sequence needs from everything before it just those sums
// and the last W-1 values of v).  A segment first computes its own sums (la_segment_state), the sums of the
// segments before it are added up (la_state_prefix), and la_prefill then continues from that state.  Several GPUs
// each take one segment and exchange the sums with one all-gather.
#include "la_common.cuh"

namespace la {
namespace sp {

constexpr int kThreads = 256, kStage = 32;    // tokens staged in shared memory at a time

// fp32 CUDA-core version: one CTA per (batch, head), every thread owns a square block of dS in registers.
template <typename T, int D, int PHI>
__global__ void __launch_bounds__(kThreads)
segment_state_simt_kernel(const T* __restrict__ k, const T* __restrict__ v, float* __restrict__ dS,
                          float* __restrict__ dz, int Tlen) {
  constexpr int SB = D / 16;
  __shared__ __align__(16) float fk[kStage][D];
  __shared__ __align__(16) float vv[kStage][D];
  const int bh = blockIdx.x, tid = threadIdx.x;
  const int sa = (tid / 16) * SB, sc = (tid % 16) * SB;
  const size_t base = (size_t)bh * Tlen * D;
  float s[SB][SB];
  float zacc = 0.f;
#pragma unroll
  for (int a = 0; a < SB; ++a)
#pragma unroll
    for (int c = 0; c < SB; ++c) s[a][c] = 0.f;
  for (int t0 = 0; t0 < Tlen; t0 += kStage) {
    const int nt = min(kStage, Tlen - t0);
    __syncthreads();
    for (int idx = tid; idx < nt * D; idx += kThreads) {
      fk[idx / D][idx % D] = phi<PHI>(to_f32(k[base + (size_t)t0 * D + idx]));
      vv[idx / D][idx % D] = to_f32(v[base + (size_t)t0 * D + idx]);
    }
    __syncthreads();
    for (int j = 0; j < nt; ++j) {
#pragma unroll
      for (int a = 0; a < SB; ++a) {
        const float f = fk[j][sa + a];
#pragma unroll
        for (int c = 0; c < SB; ++c) s[a][c] = fmaf(f, vv[j][sc + c], s[a][c]);
      }
    }
    if (tid < D)
      for (int j = 0; j < nt; ++j) zacc += fk[j][tid];
  }
#pragma unroll
  for (int a = 0; a < SB; ++a)
#pragma unroll
    for (int c = 0; c < SB; ++c) dS[(size_t)bh * D * D + (size_t)(sa + a) * D + sc + c] = s[a][c];
  if (tid < D) dz[(size_t)bh * D + tid] = zacc;
}

// out = (base or 0) + sum of the first `count` of `nseg` equally sized parts, elementwise (four floats per thread).
__global__ void __launch_bounds__(256)
state_prefix_kernel(const float* __restrict__ parts, const float* __restrict__ base, float* __restrict__ out, size_t n4,
                    int count) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  float4 acc = base ? reinterpret_cast<const float4*>(base)[i] : make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s = 0; s < count; ++s) {
    const float4 x = reinterpret_cast<const float4*>(parts)[(size_t)s * n4 + i];
    acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
  }
  reinterpret_cast<float4*>(out)[i] = acc;
}

template <typename T, int D>
static cudaError_t launch_simt(la_ctx* ctx, int B, int Tlen, const void* k, const void* v, float* dS, float* dz,
                               cudaStream_t s) {
  const la_config& c = ctx->cfg;
  if (c.phi == LA_PHI_ELU1)
    segment_state_simt_kernel<T, D, LA_PHI_ELU1><<<dim3(B * c.H), dim3(kThreads), 0, s>>>((const T*)k, (const T*)v, dS, dz, Tlen);
  else
    segment_state_simt_kernel<T, D, LA_PHI_RELU><<<dim3(B * c.H), dim3(kThreads), 0, s>>>((const T*)k, (const T*)v, dS, dz, Tlen);
  ctx->launches += 1;
  return cudaGetLastError();
}

}  // namespace sp

cudaError_t launch_segment_state(la_ctx* ctx, int B, int Tlen, const void* k, const void* v, float* dS, float* dz,
                                 cudaStream_t s) {
  const la_config& c = ctx->cfg;
  if (ctx->prefill_kernel == 0) {
    bool handled = false;
    cudaError_t e = launch_segment_state_tc(ctx, B, Tlen, k, v, dS, dz, s, &handled);
    if (e != cudaSuccess || handled) return e;
  }
  if (c.io_dtype == LA_F32)
    return c.d == 64 ? sp::launch_simt<float, 64>(ctx, B, Tlen, k, v, dS, dz, s)
                     : sp::launch_simt<float, 128>(ctx, B, Tlen, k, v, dS, dz, s);
  return c.d == 64 ? sp::launch_simt<__nv_bfloat16, 64>(ctx, B, Tlen, k, v, dS, dz, s)
                   : sp::launch_simt<__nv_bfloat16, 128>(ctx, B, Tlen, k, v, dS, dz, s);
}

cudaError_t launch_state_prefix(la_ctx* ctx, const float* parts, const float* base, float* out, size_t n, int count,
                                cudaStream_t s) {
  const size_t n4 = n / 4;
  sp::state_prefix_kernel<<<dim3((unsigned)((n4 + 255) / 256)), dim3(256), 0, s>>>(parts, base, out, n4, count);
  ctx->launches += 1;
  return cudaGetLastError();
}

}  // namespace la
