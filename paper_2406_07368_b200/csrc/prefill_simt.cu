// Prefill on the CUDA cores in fp32: serves fp32 inputs, head dimension 64, and any shape
// the tensor-core kernel does not take.  One CTA per (batch, head) keeps the d x d state in
// registers and walks the tokens in order -- the cumulative sum of Sec. 4.1 taken literally
// -- staging 32 tokens at a time in shared memory.  Every product is a plain fp32 FMA, so
// the result meets the fp32 tolerance that a single-pass tf32/bf16 contraction would not.
#include "la_common.cuh"

namespace la {

constexpr int kTB = 32;                      // tokens staged per block
constexpr int kHalo = LA_MAX_TAPS - 1;       // rows kept in front of the staged v block

template <int D> struct SimtSmem {
  float fq[kTB][D];
  float fk[kTB][D];
  float v[kHalo + kTB][D];                   // rows [kHalo - (W-1), kHalo) hold the carried window
  float red[2][256 / (D / 4)][D];
  float redden[2][256 / (D / 4)];
  float w[LA_MAX_TAPS][D];
};

template <typename T, int D, int PHI>
__global__ void __launch_bounds__(256)
prefill_simt_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                    const float* __restrict__ w, float* __restrict__ S, float* __restrict__ z, T* __restrict__ win,
                    int64_t* __restrict__ pos, T* __restrict__ o, int H, int Tlen, int W, float eps, int init) {
  constexpr int TPR = D / 4, RPP = 256 / TPR, PASSES = D / RPP;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SimtSmem<D>& sm = *reinterpret_cast<SimtSmem<D>*>(smem_raw);

  const int bh = blockIdx.x, h = bh % H, t = threadIdx.x;
  const int c4 = (t % TPR) * 4, rg = t / TPR;
  const bool lead = (t % TPR) == 0;
  const size_t base = (size_t)bh * Tlen * D;
  float* Sb = S + (size_t)bh * D * D;
  float* zb = z + (size_t)bh * D;
  T* wb = win + (size_t)bh * (W - 1) * D;

  float4 s[PASSES];
  float zr[PASSES];
#pragma unroll
  for (int m = 0; m < PASSES; ++m) {
    const int r = rg + RPP * m;
    s[m] = init ? *reinterpret_cast<const float4*>(Sb + (size_t)r * D + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
    zr[m] = init ? zb[r] : 0.f;
  }
  for (int idx = t; idx < W * D; idx += 256) {
    const int tap = idx / D, c = idx % D;
    sm.w[tap][c] = w[((size_t)h * D + c) * W + tap];
  }
  for (int idx = t; idx < (W - 1) * D; idx += 256) {
    const int i = idx / D, c = idx % D;                       // window entry i, oldest first
    sm.v[kHalo - (W - 1) + i][c] = init ? to_f32(wb[(size_t)i * D + c]) : 0.f;
  }

  for (int i0 = 0; i0 < Tlen; i0 += kTB) {
    const int nb = min(kTB, Tlen - i0);
    __syncthreads();
    for (int idx = t; idx < nb * D; idx += 256) {
      const int j = idx / D, e = idx % D;
      const size_t g = base + (size_t)(i0 + j) * D + e;
      sm.fq[j][e] = phi<PHI>(to_f32(q[g]));
      sm.fk[j][e] = phi<PHI>(to_f32(k[g]));
      sm.v[kHalo + j][e] = to_f32(v[g]);
    }
    __syncthreads();
    for (int j = 0; j < nb; ++j) {
      const int par = j & 1;
      const float4 v4 = *reinterpret_cast<const float4*>(&sm.v[kHalo + j][c4]);
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float denp = 0.f;
#pragma unroll
      for (int m = 0; m < PASSES; ++m) {
        const int r = rg + RPP * m;
        const float a = sm.fk[j][r], b = sm.fq[j][r];
        s[m].x = fmaf(a, v4.x, s[m].x);
        s[m].y = fmaf(a, v4.y, s[m].y);
        s[m].z = fmaf(a, v4.z, s[m].z);
        s[m].w = fmaf(a, v4.w, s[m].w);
        acc.x = fmaf(b, s[m].x, acc.x);
        acc.y = fmaf(b, s[m].y, acc.y);
        acc.z = fmaf(b, s[m].z, acc.z);
        acc.w = fmaf(b, s[m].w, acc.w);
        zr[m] += a;
        denp = fmaf(b, zr[m], denp);
      }
      *reinterpret_cast<float4*>(&sm.red[par][rg][c4]) = acc;
      if (lead) sm.redden[par][rg] = denp;
      __syncthreads();
      if (t < D) {
        float num = 0.f, den = 0.f;
#pragma unroll
        for (int g = 0; g < RPP; ++g) {
          num += sm.red[par][g][t];
          den += sm.redden[par][g];
        }
        float conv = 0.f;
        for (int tap = 0; tap < W; ++tap) conv = fmaf(sm.w[tap][t], sm.v[kHalo + j - tap][t], conv);
        o[base + (size_t)(i0 + j) * D + t] = from_f32<T>(num / (den + eps) + conv);
      }
    }
    __syncthreads();
    // carry the last W-1 values of v in front of the next block (ascending copy, source above target)
    if (t < D)
      for (int i = 0; i < W - 1; ++i) sm.v[kHalo - (W - 1) + i][t] = sm.v[kHalo - (W - 1) + i + nb][t];
  }
  __syncthreads();

#pragma unroll
  for (int m = 0; m < PASSES; ++m) {
    const int r = rg + RPP * m;
    *reinterpret_cast<float4*>(Sb + (size_t)r * D + c4) = s[m];
    if (lead) zb[r] = zr[m];
  }
  for (int idx = t; idx < (W - 1) * D; idx += 256) {
    const int i = idx / D, c = idx % D;
    wb[(size_t)i * D + c] = from_f32<T>(sm.v[kHalo - (W - 1) + i][c]);
  }
  if (h == 0 && t == 0) pos[bh / H] = (init ? pos[bh / H] : 0) + Tlen;
}

template <typename T, int D, int PHI>
static cudaError_t launch_t(la_ctx* ctx, int B, int Tlen, const void* q, const void* k, const void* v, const float* w,
                            int init, const la_state& st, void* o, cudaStream_t s) {
  const la_config& c = ctx->cfg;
  auto kern = prefill_simt_kernel<T, D, PHI>;
  const size_t smem = sizeof(SimtSmem<D>);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<dim3(B * c.H), dim3(256), smem, s>>>((const T*)q, (const T*)k, (const T*)v, w, st.S, st.z, (T*)st.win, st.pos,
                                               (T*)o, c.H, Tlen, c.conv_taps, c.eps, init);
  ctx->launches += 1;
  return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t launch_phi(la_ctx* ctx, int B, int Tlen, const void* q, const void* k, const void* v, const float* w,
                              int init, const la_state& st, void* o, cudaStream_t s) {
  return ctx->cfg.phi == LA_PHI_ELU1 ? launch_t<T, D, LA_PHI_ELU1>(ctx, B, Tlen, q, k, v, w, init, st, o, s)
                                     : launch_t<T, D, LA_PHI_RELU>(ctx, B, Tlen, q, k, v, w, init, st, o, s);
}

cudaError_t launch_prefill_simt(la_ctx* ctx, int B, int Tlen, const void* q, const void* k, const void* v,
                                const float* w, int init, const la_state& st, void* o, cudaStream_t s) {
  const la_config& c = ctx->cfg;
  if (c.io_dtype == LA_F32)
    return c.d == 64 ? launch_phi<float, 64>(ctx, B, Tlen, q, k, v, w, init, st, o, s)
                     : launch_phi<float, 128>(ctx, B, Tlen, q, k, v, w, init, st, o, s);
  return c.d == 64 ? launch_phi<__nv_bfloat16, 64>(ctx, B, Tlen, q, k, v, w, init, st, o, s)
                   : launch_phi<__nv_bfloat16, 128>(ctx, B, Tlen, q, k, v, w, init, st, o, s);
}

}  // namespace la
