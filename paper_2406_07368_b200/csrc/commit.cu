// Commit of the accepted draft path (Sec. 4.2: later tokens interact with the verified
// tokens of earlier groups).  Per (sequence, head): rebuild the root-to-node path from
// the parent array (integer work, bit-exact), then stream the d x d state once, adding the
// rank-1 updates of all path tokens in order, and advance z, the convolution window and pos.
// The loads of the state are issued first, so that they are in flight while the path is rebuilt and the path
// tokens are gathered.
#include "la_common.cuh"

namespace la {

// The d x d state of one (sequence, head) unit is shared out among kCommitSplit CTAs (a band of rows each), so that
// a launch of few units still spreads evenly over the SMs; the first of them also advances z and the window.
constexpr int kCommitSplit = 4;

// Shared memory: phi(k) and v of the path tokens (max_depth rows each), then the integer tables.
struct CommitTables {
  int par[LA_MAX_NODES];
  int path[LA_MAX_NODES];
  int len;
  int bad;
};

template <typename T, int D, int PHI>
__global__ void __launch_bounds__(256)
commit_kernel(const T* __restrict__ k, const T* __restrict__ v, const int32_t* __restrict__ parent,
              const int32_t* __restrict__ accept, float* __restrict__ S, float* __restrict__ z, T* __restrict__ win,
              int64_t* __restrict__ pos, int32_t* __restrict__ path_out, int32_t* __restrict__ commit_len, int* status,
              int H, int N, int W, int max_depth) {
  constexpr int TPR = D / 4, RPP = 256 / TPR, ROWS = D / kCommitSplit, PASSES = ROWS / RPP;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float (*fk)[D] = reinterpret_cast<float (*)[D]>(smem_raw);
  float (*vv)[D] = fk + max_depth;
  CommitTables& sm = *reinterpret_cast<CommitTables*>(vv + max_depth);
  const int bh = blockIdx.x / kCommitSplit, part = blockIdx.x % kCommitSplit, b = bh / H, h = bh % H, t = threadIdx.x;

  pdl_wait();                      // the kernel before this one in the stream may still be running until here
  pdl_trigger();
  // The state is requested before anything else: the loads are in flight while the path is rebuilt.
  const int c4 = (t % TPR) * 4, rg = part * ROWS + t / TPR;   // this CTA's rows of S: part * ROWS .. + ROWS - 1
  float* Sb = S + (size_t)bh * D * D;
  float4 s[PASSES];
#pragma unroll
  for (int m = 0; m < PASSES; ++m) s[m] = __ldcs(reinterpret_cast<const float4*>(Sb + (size_t)(rg + RPP * m) * D + c4));

  if (t < N) sm.par[t] = parent[(size_t)b * N + t];
  __syncthreads();
  if (t == 0) {
    int a = accept[b], L = 0, bad = 0;
    if (a < -1 || a >= N) bad = 1;
    int m = bad ? -1 : a;
    while (m >= 0) {                       // m strictly decreases: terminates
      if (L >= max_depth) { bad = 1; break; }
      sm.path[L++] = m;
      const int p = sm.par[m];
      if (p < -1 || p >= m) { bad = 1; break; }
      m = p;
    }
    for (int i = 0; i < L / 2; ++i) {      // root first
      const int x = sm.path[i];
      sm.path[i] = sm.path[L - 1 - i];
      sm.path[L - 1 - i] = x;
    }
    sm.len = L;
    sm.bad = bad;
  }
  __syncthreads();
  if (sm.bad) {
    if (t == 0) report(status, LA_ERR_BAD_TREE);
    return;
  }
  const int L = sm.len;
  if (h == 0 && part == 0) {
    for (int i = t; i < max_depth; i += 256) path_out[(size_t)b * max_depth + i] = i < L ? sm.path[i] : -1;
    if (t == 0) commit_len[b] = L;
  }
  if (L == 0) return;

  const size_t base = (size_t)bh * N * D;
  for (int idx = t; idx < L * D; idx += 256) {
    const int l = idx / D, e = idx % D;
    const size_t g = base + (size_t)sm.path[l] * D + e;
    fk[l][e] = phi<PHI>(to_f32(k[g]));
    vv[l][e] = to_f32(v[g]);
  }
  __syncthreads();

  for (int l = 0; l < L; ++l) {
    const float4 v4 = *reinterpret_cast<const float4*>(&vv[l][c4]);
#pragma unroll
    for (int m = 0; m < PASSES; ++m) {
      const float a = fk[l][rg + RPP * m];
      s[m].x = fmaf(a, v4.x, s[m].x);
      s[m].y = fmaf(a, v4.y, s[m].y);
      s[m].z = fmaf(a, v4.z, s[m].z);
      s[m].w = fmaf(a, v4.w, s[m].w);
    }
  }
#pragma unroll
  for (int m = 0; m < PASSES; ++m) __stcs(reinterpret_cast<float4*>(Sb + (size_t)(rg + RPP * m) * D + c4), s[m]);

  if (part == 0 && t < D) {
    float zz = z[(size_t)bh * D + t];
    for (int l = 0; l < L; ++l) zz += fk[l][t];
    z[(size_t)bh * D + t] = zz;
    // window <- last W-1 entries of (window ++ v_path); ascending, source index above target
    T* wb = win + (size_t)bh * (W - 1) * D;
    for (int i = 0; i < W - 1; ++i) {
      const int src = L + i;
      wb[(size_t)i * D + t] = src < W - 1 ? wb[(size_t)src * D + t] : from_f32<T>(vv[src - (W - 1)][t]);
    }
  }
  if (h == 0 && part == 0 && t == 0) pos[b] += L;
}

template <typename T, int D, int PHI>
static cudaError_t launch_t(la_ctx* ctx, int B, int N, const void* k, const void* v, const int32_t* parent,
                            const int32_t* accept, const la_state& st, int32_t* path_out, int32_t* commit_len,
                            cudaStream_t s) {
  const la_config& c = ctx->cfg;
  auto kern = commit_kernel<T, D, PHI>;
  const size_t smem = (size_t)2 * c.max_depth * D * sizeof(float) + sizeof(CommitTables);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  ctx->launches += 1;
  return launch_pdl(kern, dim3(B * c.H * kCommitSplit), dim3(256), smem, s, (const T*)k, (const T*)v, parent, accept, st.S,
                    st.z, (T*)st.win, st.pos, path_out, commit_len, ctx->d_status, c.H, N, c.conv_taps, c.max_depth);
}

template <typename T, int D>
static cudaError_t launch_phi(la_ctx* ctx, int B, int N, const void* k, const void* v, const int32_t* parent,
                              const int32_t* accept, const la_state& st, int32_t* path_out, int32_t* commit_len,
                              cudaStream_t s) {
  return ctx->cfg.phi == LA_PHI_ELU1
             ? launch_t<T, D, LA_PHI_ELU1>(ctx, B, N, k, v, parent, accept, st, path_out, commit_len, s)
             : launch_t<T, D, LA_PHI_RELU>(ctx, B, N, k, v, parent, accept, st, path_out, commit_len, s);
}

cudaError_t launch_commit(la_ctx* ctx, int B, int N, const void* k, const void* v, const int32_t* parent,
                          const int32_t* accept, const la_state& st, int32_t* path_out, int32_t* commit_len,
                          cudaStream_t s) {
  const la_config& c = ctx->cfg;
  if (c.io_dtype == LA_F32)
    return c.d == 64 ? launch_phi<float, 64>(ctx, B, N, k, v, parent, accept, st, path_out, commit_len, s)
                     : launch_phi<float, 128>(ctx, B, N, k, v, parent, accept, st, path_out, commit_len, s);
  return c.d == 64 ? launch_phi<__nv_bfloat16, 64>(ctx, B, N, k, v, parent, accept, st, path_out, commit_len, s)
                   : launch_phi<__nv_bfloat16, 128>(ctx, B, N, k, v, parent, accept, st, path_out, commit_len, s);
}

}  // namespace la
