// The three-branch block of Sec. 4.1 ("LA Augmentation for Autoregressive LLMs", Fig. "la_aug") on the CUDA cores.
//
// The sequence is cut into non-overlapping groups of C tokens.  For token i of group g
//     glob_i = phi(q_i)^T S_{<g} / (phi(q_i) . z_{<g} + eps)      middle branch: only the group-level cumulative sums
//                                                                 of the groups before g (0 where there is none)
//     loc_i  = sum_{j in g, j <= i} softmax_j(scale q_i . k_j) v_j  left branch: causal softmax attention in the group
//     conv_i = sum_{t<W} w[:, t] * v_{i-t}                         right branch: the masked depthwise convolution
//     o_i    = alpha glob_i + loc_i + conv_i.
// One CTA walks one (batch, head) chain group by group.  The keys and values of a group stay in shared memory; its
// queries pass through in blocks of QB rows: scores and the three products of a block are register-tiled fp32
// multiply-adds, the softmax runs one warp per row.  After the last block of a group the group's sum of
// phi(k) v^T is added to the state, which every thread holds a square block of in registers for the whole chain.
// All arithmetic is fp32 (phi(k) is kept in the io type, like the operands of the tensor-core prefill).
#include "la_common.cuh"

namespace la {
namespace grp {

constexpr int kThreads = 512;

template <typename T> struct Vec4;           // four consecutive elements of the io type
template <> struct Vec4<float> {
  float4 x;
  __device__ __forceinline__ float4 f() const { return x; }
  static __device__ __forceinline__ Vec4 from(float4 a) { return Vec4{a}; }
};
template <> struct Vec4<__nv_bfloat16> {
  uint2 x;
  __device__ __forceinline__ float4 f() const {
    return make_float4(__uint_as_float(x.x << 16), __uint_as_float(x.x & 0xffff0000u), __uint_as_float(x.y << 16),
                       __uint_as_float(x.y & 0xffff0000u));
  }
  static __device__ __forceinline__ Vec4 from(float4 a) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
    return Vec4{make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi))};
  }
};

// Rows of a query block: the 512 threads form D/4 column groups (four channels each) times 2048/D row groups.
template <typename T, int D> struct Shape {
  static constexpr int kColGroups = D / 4;
  static constexpr int kRowGroups = kThreads / kColGroups;
  static constexpr int QB = (sizeof(T) == 4 && D == 128) ? 16 : 32;     // rows per query block
  static constexpr int RT = QB / kRowGroups;                            // rows per thread
  static constexpr int SBA = D / 32, SBC = D / 16;                      // a thread's block of S: SBA rows x SBC columns
  static constexpr int kMaxGroup = (32768 / (D * (int)sizeof(T))) < 256 ? (32768 / (D * (int)sizeof(T))) : 256;
};

template <typename T, int D> __host__ __device__ inline size_t smem_bytes(int C, int W) {
  using Sh = Shape<T, D>;
  size_t b = 0;
  b += (size_t)2 * C * D * sizeof(T);                       // k, phi(k)
  b += (size_t)(C + W - 1 + 3) * D * sizeof(T);             // W-1 rows before the group, v, three rows of zeros
  b += (size_t)2 * Sh::QB * D * sizeof(T);                  // q, phi(q) of a block
  b += (size_t)Sh::QB * (((C + 3) & ~3) + 1) * sizeof(float);   // scores of a block (rows padded to four floats), then their row sums
  b += (size_t)D * D * sizeof(float) + D * sizeof(float);   // S, z before the group
  b += (size_t)W * D * sizeof(float);                       // taps
  b += (size_t)Sh::QB * sizeof(float);                      // phi(q) . z
  return b + 16;
}

template <typename T, int D, int PHI>
__global__ void __launch_bounds__(kThreads, 1)
prefill_grouped_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                       const float* __restrict__ w, float* __restrict__ S, float* __restrict__ z, T* __restrict__ win,
                       int64_t* __restrict__ pos, T* __restrict__ o, int H, int Tlen, int W, int C, float eps,
                       float alpha, float scale, int init) {
  using Sh = Shape<T, D>;
  constexpr int QB = Sh::QB, RT = Sh::RT, SBA = Sh::SBA, SBC = Sh::SBC, CG = Sh::kColGroups;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* ks = reinterpret_cast<T*>(smem_raw);                    // [C][D]
  T* fks = ks + (size_t)C * D;                               // [C][D]   phi(k)
  T* vs = fks + (size_t)C * D;                               // [W-1 + C + 3][D]: the product with P reads four rows at a time
  T* qs = vs + (size_t)(C + W - 1 + 3) * D;                  // [QB][D]
  T* fqs = qs + (size_t)QB * D;                              // [QB][D]  phi(q)
  const int CP = (C + 3) & ~3;                               // row pitch of P
  float* P = reinterpret_cast<float*>(fqs + (size_t)QB * D); // [QB][CP]
  float* rowsum = P + (size_t)QB * CP;                       // [QB]
  float* Ss = rowsum + QB;                                   // [D][D]
  float* zs = Ss + (size_t)D * D;                            // [D]
  float* ws = zs + D;                                        // [W][D]
  float* qz = ws + (size_t)W * D;                            // [QB]

  const int bh = blockIdx.x, h = bh % H, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t base = (size_t)bh * Tlen * D;
  const int tx = tid % CG, ty = tid / CG;                    // output tile of a block: rows ty*RT.., channels tx*4..
  const int sa = (tid / 16) * SBA, sc = (tid % 16) * SBC;    // this thread's block of S

  // ---- set-up: state, taps, the rows before the sequence ----
  float sreg[SBA][SBC];
  float zreg = 0.f;                                          // z[tid] for tid < D
#pragma unroll
  for (int a = 0; a < SBA; ++a)
#pragma unroll
    for (int c = 0; c < SBC; ++c) sreg[a][c] = init ? S[(size_t)bh * D * D + (size_t)(sa + a) * D + sc + c] : 0.f;
  if (tid < D) zreg = init ? z[(size_t)bh * D + tid] : 0.f;
  for (int idx = tid; idx < W * D; idx += kThreads) ws[idx] = w[((size_t)h * D + idx % D) * W + idx / D];
  for (int idx = tid; idx < (W - 1) * D; idx += kThreads)
    vs[idx] = init ? win[(size_t)bh * (W - 1) * D + idx] : from_f32<T>(0.f);
  bool have_state = init != 0;

  for (int g0 = 0; g0 < Tlen; g0 += C) {
    const int Cg = min(C, Tlen - g0);
    __syncthreads();                                         // the previous group's buffers are no longer read
    // ---- the group's keys and values; the state before the group ----
    for (int idx = tid; idx < Cg * D / 4; idx += kThreads) {
      const Vec4<T> kk = *reinterpret_cast<const Vec4<T>*>(k + base + (size_t)g0 * D + 4 * idx);
      const float4 f = kk.f();
      *reinterpret_cast<Vec4<T>*>(ks + 4 * idx) = kk;
      *reinterpret_cast<Vec4<T>*>(fks + 4 * idx) =
          Vec4<T>::from(make_float4(phi<PHI>(f.x), phi<PHI>(f.y), phi<PHI>(f.z), phi<PHI>(f.w)));
      *reinterpret_cast<Vec4<T>*>(vs + (size_t)(W - 1) * D + 4 * idx) =
          *reinterpret_cast<const Vec4<T>*>(v + base + (size_t)g0 * D + 4 * idx);
    }
    // three rows of zeros behind the group's last value: the product with P reads four rows at a time
    for (int idx = tid; idx < 3 * D; idx += kThreads) vs[(size_t)(W - 1 + Cg) * D + idx] = from_f32<T>(0.f);
#pragma unroll
    for (int a = 0; a < SBA; ++a)
#pragma unroll
      for (int c = 0; c < SBC; c += 4)
        *reinterpret_cast<float4*>(Ss + (sa + a) * D + sc + c) = make_float4(sreg[a][c], sreg[a][c + 1], sreg[a][c + 2], sreg[a][c + 3]);
    if (tid < D) zs[tid] = zreg;

    for (int r0 = 0; r0 < Cg; r0 += QB) {                    // query blocks of the group
      const int nr = min(QB, Cg - r0);
      __syncthreads();                                       // group data in place; previous block done with q, P
      for (int idx = tid; idx < QB * D / 4; idx += kThreads) {
        const int r = (4 * idx) / D;
        Vec4<T> qq = Vec4<T>::from(make_float4(0.f, 0.f, 0.f, 0.f)), fq = qq;
        if (r < nr) {
          qq = *reinterpret_cast<const Vec4<T>*>(q + base + (size_t)(g0 + r0) * D + 4 * idx);
          const float4 f = qq.f();
          fq = Vec4<T>::from(make_float4(phi<PHI>(f.x), phi<PHI>(f.y), phi<PHI>(f.z), phi<PHI>(f.w)));
        }
        *reinterpret_cast<Vec4<T>*>(qs + 4 * idx) = qq;
        *reinterpret_cast<Vec4<T>*>(fqs + 4 * idx) = fq;
      }
      __syncthreads();

      // ---- scores of the block: P[r][j] = scale q_r . k_j for j <= r0 + r (columns beyond stay unset) ----
      const int jmax = min(Cg, r0 + nr);                     // columns any row of this block can see
      for (int j = tx; j < jmax; j += CG) {
        if (j > r0 + ty * RT + RT - 1) continue;             // above the diagonal for all of this thread's rows
        float acc[RT];
#pragma unroll
        for (int i = 0; i < RT; ++i) acc[i] = 0.f;
#pragma unroll 4
        for (int e = 0; e < D; e += 4) {
          const float4 kk = reinterpret_cast<const Vec4<T>*>(ks + (size_t)j * D + e)->f();
#pragma unroll
          for (int i = 0; i < RT; ++i) {
            const float4 x = reinterpret_cast<const Vec4<T>*>(qs + (size_t)(ty * RT + i) * D + e)->f();
            acc[i] = fmaf(x.x, kk.x, fmaf(x.y, kk.y, fmaf(x.z, kk.z, fmaf(x.w, kk.w, acc[i]))));
          }
        }
#pragma unroll
        for (int i = 0; i < RT; ++i) P[(size_t)(ty * RT + i) * CP + j] = acc[i] * scale;
      }
      // phi(q) . z for the rows of the block (one warp per row, rows warp, warp + 8, ...)
      for (int r = warp; r < QB; r += kThreads / 32) {
        float part = 0.f;
        for (int e = lane; e < D; e += 32) part = fmaf(to_f32(fqs[(size_t)r * D + e]), zs[e], part);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
        if (lane == 0) qz[r] = part;
      }
      __syncthreads();

      // ---- causal softmax along each row (one warp per row); the row keeps exp(s - max), its sum goes aside ----
      for (int r = warp; r < nr; r += kThreads / 32) {
        const int last = r0 + r;                             // the row's own column
        float* row = P + (size_t)r * CP;
        float m = -INFINITY;
        for (int j = lane; j <= last; j += 32) m = fmaxf(m, row[j]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
        float sum = 0.f;
        for (int j = lane; j < ((jmax + 3) & ~3); j += 32) {     // (up to the padded end: the product reads four at a time)
          const float e = j <= last ? expf(row[j] - m) : 0.f;
          row[j] = e;
          sum += e;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        if (lane == 0) rowsum[r] = sum;
      }
      __syncthreads();

      // ---- the three branches for this thread's RT x 4 outputs ----
      float loc[RT][4], glo[RT][4];
#pragma unroll
      for (int i = 0; i < RT; ++i)
#pragma unroll
        for (int c = 0; c < 4; ++c) loc[i][c] = glo[i][c] = 0.f;
      const int jhi = min(jmax, r0 + ty * RT + RT);          // columns this thread's rows can see
      // loc += P V, four columns of P per step (the rows of P are padded to a multiple of four floats and columns
      // past a row's own hold zeros, so the last step may run past jhi)
      for (int j = 0; j < jhi; j += 4) {
        float4 vv[4], pp[RT];
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) vv[jj] = reinterpret_cast<const Vec4<T>*>(vs + (size_t)(W - 1 + j + jj) * D + 4 * tx)->f();
#pragma unroll
        for (int i = 0; i < RT; ++i) pp[i] = *reinterpret_cast<const float4*>(P + (size_t)(ty * RT + i) * CP + j);
#pragma unroll
        for (int i = 0; i < RT; ++i) {
          const float pj[4] = {pp[i].x, pp[i].y, pp[i].z, pp[i].w};
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            loc[i][0] = fmaf(pj[jj], vv[jj].x, loc[i][0]);
            loc[i][1] = fmaf(pj[jj], vv[jj].y, loc[i][1]);
            loc[i][2] = fmaf(pj[jj], vv[jj].z, loc[i][2]);
            loc[i][3] = fmaf(pj[jj], vv[jj].w, loc[i][3]);
          }
        }
      }
      if (have_state) {                                      // glo = phi(Q) S_{<g}
#pragma unroll 2
        for (int a = 0; a < D; a += 4) {                     // four features per step
          float4 s4[4], ff[RT];
#pragma unroll
          for (int aa = 0; aa < 4; ++aa) s4[aa] = *reinterpret_cast<const float4*>(Ss + (size_t)(a + aa) * D + 4 * tx);
#pragma unroll
          for (int i = 0; i < RT; ++i) ff[i] = reinterpret_cast<const Vec4<T>*>(fqs + (size_t)(ty * RT + i) * D + a)->f();
#pragma unroll
          for (int i = 0; i < RT; ++i) {
            const float fa[4] = {ff[i].x, ff[i].y, ff[i].z, ff[i].w};
#pragma unroll
            for (int aa = 0; aa < 4; ++aa) {
              glo[i][0] = fmaf(fa[aa], s4[aa].x, glo[i][0]);
              glo[i][1] = fmaf(fa[aa], s4[aa].y, glo[i][1]);
              glo[i][2] = fmaf(fa[aa], s4[aa].z, glo[i][2]);
              glo[i][3] = fmaf(fa[aa], s4[aa].w, glo[i][3]);
            }
          }
        }
      }
#pragma unroll
      for (int i = 0; i < RT; ++i) {
        const int r = ty * RT + i;
        if (r >= nr) continue;
        const int row = r0 + r;                              // row within the group; v row at W-1 + row
        const float den = qz[r] + eps;
        const float gs = (have_state && den != 0.f) ? alpha / den : 0.f;
        const float ls = 1.f / rowsum[r];
        float out[4] = {fmaf(gs, glo[i][0], ls * loc[i][0]), fmaf(gs, glo[i][1], ls * loc[i][1]),
                        fmaf(gs, glo[i][2], ls * loc[i][2]), fmaf(gs, glo[i][3], ls * loc[i][3])};
        for (int t = 0; t < W; ++t) {                        // masked depthwise convolution
          const float4 vv = reinterpret_cast<const Vec4<T>*>(vs + (size_t)(W - 1 + row - t) * D + 4 * tx)->f();
          const float4 w4 = *reinterpret_cast<const float4*>(ws + (size_t)t * D + 4 * tx);
          out[0] = fmaf(w4.x, vv.x, out[0]);
          out[1] = fmaf(w4.y, vv.y, out[1]);
          out[2] = fmaf(w4.z, vv.z, out[2]);
          out[3] = fmaf(w4.w, vv.w, out[3]);
        }
        *reinterpret_cast<Vec4<T>*>(o + base + (size_t)(g0 + row) * D + 4 * tx) =
            Vec4<T>::from(make_float4(out[0], out[1], out[2], out[3]));
      }
    }

    // ---- the group is complete: S += phi(K)^T V, z += column sums of phi(K) ----
    for (int j = 0; j < Cg; ++j) {
      float fa[SBA], vc[SBC];
      if (SBA == 4) {
        const float4 x = reinterpret_cast<const Vec4<T>*>(fks + (size_t)j * D + sa)->f();
        fa[0] = x.x; fa[1] = x.y; fa[SBA - 2] = x.z; fa[SBA - 1] = x.w;
      } else {
#pragma unroll
        for (int a = 0; a < SBA; ++a) fa[a] = to_f32(fks[(size_t)j * D + sa + a]);
      }
#pragma unroll
      for (int c = 0; c < SBC; c += 4) {
        const float4 y = reinterpret_cast<const Vec4<T>*>(vs + (size_t)(W - 1 + j) * D + sc + c)->f();
        vc[c] = y.x; vc[c + 1] = y.y; vc[c + 2] = y.z; vc[c + 3] = y.w;
      }
#pragma unroll
      for (int a = 0; a < SBA; ++a)
#pragma unroll
        for (int c = 0; c < SBC; ++c) sreg[a][c] = fmaf(fa[a], vc[c], sreg[a][c]);
    }
    if (tid < D)
      for (int j = 0; j < Cg; ++j) zreg += to_f32(fks[(size_t)j * D + tid]);
    have_state = true;
    __syncthreads();                                         // every read of v is done before the rows move
    // the last W-1 values of v move in front of the next group (ascending copy, source above target)
    for (int i = 0; i < W - 1; ++i)
      for (int c = tid; c < D; c += kThreads) vs[(size_t)i * D + c] = vs[(size_t)(i + Cg) * D + c];
  }
  __syncthreads();

  // ---- the state after all tokens ----
#pragma unroll
  for (int a = 0; a < SBA; ++a)
#pragma unroll
    for (int c = 0; c < SBC; ++c) S[(size_t)bh * D * D + (size_t)(sa + a) * D + sc + c] = sreg[a][c];
  if (tid < D) z[(size_t)bh * D + tid] = zreg;
  for (int idx = tid; idx < (W - 1) * D; idx += kThreads) win[(size_t)bh * (W - 1) * D + idx] = vs[idx];
  if (h == 0 && tid == 0) pos[bh / H] = (init ? pos[bh / H] : 0) + Tlen;
}

template <typename T, int D, int PHI>
static cudaError_t launch_t(la_ctx* ctx, int B, int Tlen, const void* q, const void* k, const void* v, const float* w,
                            int group, float alpha, float scale, int init, const la_state& st, void* o, cudaStream_t s) {
  const la_config& c = ctx->cfg;
  auto kern = prefill_grouped_kernel<T, D, PHI>;
  const size_t smem = smem_bytes<T, D>(group, c.conv_taps);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<dim3(B * c.H), dim3(kThreads), smem, s>>>((const T*)q, (const T*)k, (const T*)v, w, st.S, st.z, (T*)st.win,
                                                    st.pos, (T*)o, c.H, Tlen, c.conv_taps, group, c.eps, alpha, scale, init);
  ctx->launches += 1;
  return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t launch_phi(la_ctx* ctx, int B, int Tlen, const void* q, const void* k, const void* v, const float* w,
                              int group, float alpha, float scale, int init, const la_state& st, void* o, cudaStream_t s) {
  return ctx->cfg.phi == LA_PHI_ELU1
             ? launch_t<T, D, LA_PHI_ELU1>(ctx, B, Tlen, q, k, v, w, group, alpha, scale, init, st, o, s)
             : launch_t<T, D, LA_PHI_RELU>(ctx, B, Tlen, q, k, v, w, group, alpha, scale, init, st, o, s);
}

}  // namespace grp

int prefill_grouped_max_group(const la_config& c) {
  if (c.io_dtype == LA_F32) return c.d == 64 ? grp::Shape<float, 64>::kMaxGroup : grp::Shape<float, 128>::kMaxGroup;
  return c.d == 64 ? grp::Shape<__nv_bfloat16, 64>::kMaxGroup : grp::Shape<__nv_bfloat16, 128>::kMaxGroup;
}

cudaError_t launch_prefill_grouped(la_ctx* ctx, int B, int Tlen, const void* q, const void* k, const void* v,
                                   const float* w, int group, float alpha, float scale, int init, const la_state& st,
                                   void* o, cudaStream_t s) {
  const la_config& c = ctx->cfg;
  if (c.io_dtype == LA_F32)
    return c.d == 64 ? grp::launch_phi<float, 64>(ctx, B, Tlen, q, k, v, w, group, alpha, scale, init, st, o, s)
                     : grp::launch_phi<float, 128>(ctx, B, Tlen, q, k, v, w, group, alpha, scale, init, st, o, s);
  return c.d == 64 ? grp::launch_phi<__nv_bfloat16, 64>(ctx, B, Tlen, q, k, v, w, group, alpha, scale, init, st, o, s)
                   : grp::launch_phi<__nv_bfloat16, 128>(ctx, B, Tlen, q, k, v, w, group, alpha, scale, init, st, o, s);
}

}  // namespace la
