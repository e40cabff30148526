// Single-token decode: the recurrence behind the cumulative sum of Sec. 4.1.
//   S += phi(k) v^T,  z += phi(k),  o = phi(q)^T S / (phi(q).z + eps) + conv(window, v)
// One CTA per (sequence, head).  The d x d fp32 state is streamed through registers exactly
// once (128-bit loads, all of a thread's loads in flight before the first use), updated,
// read out against phi(q) in the same pass and written back; the convolution over the
// carried window and the window shift are done by the same CTA.
#include "la_common.cuh"

namespace la {

template <typename T, int D, int PHI, int WCAP>
__global__ void __launch_bounds__(256)
decode_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
              const float* __restrict__ w, float* __restrict__ S, float* __restrict__ z, T* __restrict__ win,
              int64_t* __restrict__ pos, T* __restrict__ o, int H, int W, float eps) {
  constexpr int TPR = D / 4;       // threads covering one row of S with float4
  constexpr int RPP = 256 / TPR;   // rows per pass of the whole CTA
  constexpr int PASSES = D / RPP;
  __shared__ __align__(16) float fq[D], fk[D], vv[D];
  __shared__ __align__(16) float red[RPP][D];
  __shared__ float scratch[33];

  const int bh = blockIdx.x, h = bh % H, t = threadIdx.x;
  const size_t vec = (size_t)bh * D;
  pdl_wait();                      // the kernel before this one in the stream may still be running until here
  pdl_trigger();
  const int c4 = (t % TPR) * 4, rg = t / TPR;
  float* Sb = S + (size_t)bh * D * D;

  // Issue the state loads first: they do not depend on q, k, v.
  float4 s[PASSES];
#pragma unroll
  for (int m = 0; m < PASSES; ++m) s[m] = __ldcs(reinterpret_cast<const float4*>(Sb + (size_t)(rg + RPP * m) * D + c4));

  // ... and, for short tap windows (W <= WCAP; WCAP = 0: any W, handled at the end), so are the window and the taps
  // of this channel: in registers before they are needed, so that the shift at the end is stores only
  constexpr int NW = WCAP > 0 ? WCAP - 1 : 1;
  T wr[NW];
  float wc[NW], w0 = 0.f;                        // wc[i]: the tap that meets window row i (W-1-i steps back)
  T* wb = win + (size_t)bh * (W - 1) * D;
  if (WCAP > 0 && t < D) {
#pragma unroll
    for (int i = 0; i < WCAP - 1; ++i)
      if (i < W - 1) wr[i] = wb[(size_t)i * D + t];
    w0 = w[((size_t)h * D + t) * W];
#pragma unroll
    for (int i = 0; i < WCAP - 1; ++i)
      if (i < W - 1) wc[i] = w[((size_t)h * D + t) * W + (W - 1 - i)];
  }

  float den_part = 0.f;
  if (t < D) {
    const float fqv = phi<PHI>(to_f32(q[vec + t])), fkv = phi<PHI>(to_f32(k[vec + t]));
    fq[t] = fqv;
    fk[t] = fkv;
    vv[t] = to_f32(v[vec + t]);
    const float zn = z[vec + t] + fkv;   // update first, then read (inclusive sum)
    z[vec + t] = zn;
    den_part = fqv * zn;
  }
  const float den = block_sum(den_part, scratch);   // also publishes fq, fk, vv

  const float4 v4 = *reinterpret_cast<const float4*>(&vv[c4]);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int m = 0; m < PASSES; ++m) {
    const int r = rg + RPP * m;
    const float a = fk[r], b = fq[r];
    s[m].x = fmaf(a, v4.x, s[m].x);
    s[m].y = fmaf(a, v4.y, s[m].y);
    s[m].z = fmaf(a, v4.z, s[m].z);
    s[m].w = fmaf(a, v4.w, s[m].w);
    acc.x = fmaf(b, s[m].x, acc.x);
    acc.y = fmaf(b, s[m].y, acc.y);
    acc.z = fmaf(b, s[m].z, acc.z);
    acc.w = fmaf(b, s[m].w, acc.w);
    __stcs(reinterpret_cast<float4*>(Sb + (size_t)r * D + c4), s[m]);
  }
  *reinterpret_cast<float4*>(&red[rg][c4]) = acc;
  __syncthreads();

  if (t < D) {
    float num = 0.f;
#pragma unroll
    for (int g = 0; g < RPP; ++g) num += red[g][t];
    float conv;
    if (WCAP > 0) {
      conv = w0 * vv[t];
#pragma unroll
      for (int i = 0; i < WCAP - 1; ++i)                   // window row i holds the value W-1-i steps back
        if (i < W - 1) conv = fmaf(wc[i], to_f32(wr[i]), conv);
#pragma unroll
      for (int i = 0; i < WCAP - 2; ++i)
        if (i + 2 < W) wb[(size_t)i * D + t] = wr[i + 1];
    } else {
      // one pass over the window in batches of eight rows: all loads of a batch are in flight together; row i is
      // used for its tap and then stored one place down (a batch only overwrites rows it or an earlier one has read)
      const float* wg = w + ((size_t)h * D + t) * W;
      conv = wg[0] * vv[t];
      for (int base = 0; base < W - 1; base += 8) {
        T r[8];
        float g[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (base + i < W - 1) {
            r[i] = wb[(size_t)(base + i) * D + t];
            g[i] = wg[W - 1 - (base + i)];
          }
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (base + i < W - 1) {
            conv = fmaf(g[i], to_f32(r[i]), conv);
            if (base + i >= 1) wb[(size_t)(base + i - 1) * D + t] = r[i];
          }
      }
    }
    if (W > 1) wb[(size_t)(W - 2) * D + t] = v[vec + t];
    o[vec + t] = from_f32<T>(num / (den + eps) + conv);
  }
  if (h == 0 && t == 0) pos[bh / H] += 1;
}

template <typename T, int D>
static cudaError_t launch_decode_t(la_ctx* ctx, int B, const void* q, const void* k, const void* v, const float* w,
                                   const la_state& st, void* o, cudaStream_t s) {
  const la_config& c = ctx->cfg;
  dim3 grid(B * c.H), block(256);
  const bool elu = c.phi == LA_PHI_ELU1;
  auto kern = c.conv_taps <= 4   ? (elu ? decode_kernel<T, D, LA_PHI_ELU1, 4> : decode_kernel<T, D, LA_PHI_RELU, 4>)
              : c.conv_taps <= 8 ? (elu ? decode_kernel<T, D, LA_PHI_ELU1, 8> : decode_kernel<T, D, LA_PHI_RELU, 8>)
                                 : (elu ? decode_kernel<T, D, LA_PHI_ELU1, 0> : decode_kernel<T, D, LA_PHI_RELU, 0>);
  ctx->launches += 1;
  return launch_pdl(kern, grid, block, 0, s, (const T*)q, (const T*)k, (const T*)v, w, st.S, st.z, (T*)st.win, st.pos,
                    (T*)o, c.H, c.conv_taps, c.eps);
}

cudaError_t launch_decode(la_ctx* ctx, int B, const void* q, const void* k, const void* v, const float* w,
                          const la_state& st, void* o, cudaStream_t s) {
  const la_config& c = ctx->cfg;
  if (c.io_dtype == LA_F32)
    return c.d == 64 ? launch_decode_t<float, 64>(ctx, B, q, k, v, w, st, o, s)
                     : launch_decode_t<float, 128>(ctx, B, q, k, v, w, st, o, s);
  return c.d == 64 ? launch_decode_t<__nv_bfloat16, 64>(ctx, B, q, k, v, w, st, o, s)
                   : launch_decode_t<__nv_bfloat16, 128>(ctx, B, q, k, v, w, st, o, s);
}

}  // namespace la
