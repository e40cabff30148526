// Draft-tree verification (Sec. 4.2 "Proposed Solution", Sec. 5.3 shared cumulative-sum state).
// One CTA per (sequence, head).  The committed S is read once and serves all N nodes; each
// node adds the contributions of its ancestors and itself (tree mask) and convolves along its
// own ancestor chain, falling back to the committed window behind the tree.  Nothing in the
// state is written.
#include "la_common.cuh"

namespace la {

constexpr int kNodes = LA_MAX_NODES;

template <int D> struct VerifySmem {
  float fq[kNodes][D + 4];      // +4: rows land in different bank groups for 128-bit reads
  float fk[kNodes][D + 4];
  float v[kNodes][D];
  float A[kNodes][kNodes + 1];  // a[n][m] = phi(q_n).phi(k_m) for m in the ancestor-or-self set of n
  float w[LA_MAX_TAPS][D];
  float win[LA_MAX_TAPS - 1][D];
  float z[D];
  float den[kNodes];
  unsigned long long mask[kNodes];
  int par[kNodes];
  int depth[kNodes];
  int bad;
};

// PER_SEQ = false: `status` is one sticky word.  PER_SEQ = true: `status` has one word per sequence.
template <typename T, int D, int PHI, bool PER_SEQ = false>
__global__ void __launch_bounds__(256)
verify_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
              const int32_t* __restrict__ parent, const float* __restrict__ w, const float* __restrict__ S,
              const float* __restrict__ z, const T* __restrict__ win, T* __restrict__ o, int* status, int H, int N,
              int W, float eps) {
  constexpr int NG = 256 / D;            // thread groups, each owning all d output columns
  constexpr int NPG = kNodes / NG;       // nodes per group
  extern __shared__ __align__(16) unsigned char smem_raw[];
  VerifySmem<D>& sm = *reinterpret_cast<VerifySmem<D>*>(smem_raw);

  const int bh = blockIdx.x, b = bh / H, h = bh % H, t = threadIdx.x;

  // ---- tree preparation: ancestor-or-self masks and depths (integer work) ----
  if (t == 0) sm.bad = 0;
  if (t < N) sm.par[t] = parent[(size_t)b * N + t];
  __syncthreads();
  if (t < N) {
    unsigned long long mask = 0ull;
    int dep = 0, m = t;
    bool ok = true;
    while (m >= 0) {                     // m strictly decreases: at most N iterations
      mask |= 1ull << m;
      ++dep;
      const int p = sm.par[m];
      if (p < -1 || p >= m) { ok = false; break; }
      m = p;
    }
    sm.mask[t] = mask;
    sm.depth[t] = dep;
    if (!ok) sm.bad = 1;
  }
  __syncthreads();
  if (sm.bad) {
    if (t == 0) report(PER_SEQ ? status + b : status, LA_ERR_BAD_TREE);
    return;
  }

  // ---- stage phi(q), phi(k), v, z, the window and the taps ----
  const size_t base = (size_t)bh * N * D;
  for (int idx = t; idx < kNodes * D; idx += 256) {
    const int n = idx / D, e = idx % D;
    float a = 0.f, c = 0.f, x = 0.f;
    if (n < N) {
      a = phi<PHI>(to_f32(q[base + (size_t)n * D + e]));
      c = phi<PHI>(to_f32(k[base + (size_t)n * D + e]));
      x = to_f32(v[base + (size_t)n * D + e]);
    }
    sm.fq[n][e] = a;
    sm.fk[n][e] = c;
    sm.v[n][e] = x;
  }
  for (int idx = t; idx < W * D; idx += 256) sm.w[idx / D][idx % D] = w[((size_t)h * D + idx % D) * W + idx / D];
  for (int idx = t; idx < (W - 1) * D; idx += 256)
    sm.win[idx / D][idx % D] = to_f32(win[(size_t)bh * (W - 1) * D + idx]);
  if (t < D) sm.z[t] = z[(size_t)bh * D + t];
  __syncthreads();

  // ---- scores inside the tree, only where the mask allows ----
  for (int idx = t; idx < N * N; idx += 256) {
    const int n = idx / N, m = idx % N;
    if ((sm.mask[n] >> m) & 1ull) {
      float acc = 0.f;
#pragma unroll 8
      for (int e = 0; e < D; e += 4) {
        const float4 x = *reinterpret_cast<const float4*>(&sm.fq[n][e]);
        const float4 y = *reinterpret_cast<const float4*>(&sm.fk[m][e]);
        acc = fmaf(x.x, y.x, acc);
        acc = fmaf(x.y, y.y, acc);
        acc = fmaf(x.z, y.z, acc);
        acc = fmaf(x.w, y.w, acc);
      }
      sm.A[n][m] = acc;
    }
  }
  __syncthreads();
  if (t < N) {
    float den = 0.f;
    for (int e = 0; e < D; e += 4) {
      const float4 x = *reinterpret_cast<const float4*>(&sm.fq[t][e]);
      den = fmaf(x.x, sm.z[e], den);
      den = fmaf(x.y, sm.z[e + 1], den);
      den = fmaf(x.z, sm.z[e + 2], den);
      den = fmaf(x.w, sm.z[e + 3], den);
    }
    unsigned long long mk = sm.mask[t];
    while (mk) {
      const int m = __ffsll((long long)mk) - 1;
      mk &= mk - 1;
      den += sm.A[t][m];
    }
    sm.den[t] = den;
  }
  __syncthreads();

  // ---- phi(Q_tree) S against the committed state: S is read once for all nodes ----
  const int c = t % D, n0 = (t / D) * NPG;
  const float* Sb = S + (size_t)bh * D * D;
  float acc[NPG];
#pragma unroll
  for (int i = 0; i < NPG; ++i) acc[i] = 0.f;
  for (int a = 0; a < D; a += 4) {
    const float s0 = __ldg(Sb + (size_t)(a + 0) * D + c), s1 = __ldg(Sb + (size_t)(a + 1) * D + c);
    const float s2 = __ldg(Sb + (size_t)(a + 2) * D + c), s3 = __ldg(Sb + (size_t)(a + 3) * D + c);
#pragma unroll
    for (int i = 0; i < NPG; ++i) {
      const float4 f = *reinterpret_cast<const float4*>(&sm.fq[n0 + i][a]);
      acc[i] = fmaf(f.x, s0, acc[i]);
      acc[i] = fmaf(f.y, s1, acc[i]);
      acc[i] = fmaf(f.z, s2, acc[i]);
      acc[i] = fmaf(f.w, s3, acc[i]);
    }
  }

  // ---- ancestors, unfolded convolution, epilogue ----
#pragma unroll
  for (int i = 0; i < NPG; ++i) {
    const int n = n0 + i;
    if (n >= N) continue;
    float num = acc[i];
    unsigned long long mk = sm.mask[n];
    while (mk) {
      const int m = __ffsll((long long)mk) - 1;
      mk &= mk - 1;
      num = fmaf(sm.A[n][m], sm.v[m][c], num);
    }
    float conv = 0.f;
    int cur = n;
    const int dep = sm.depth[n];
    for (int tap = 0; tap < W; ++tap) {
      float u;
      if (cur >= 0) {
        u = sm.v[cur][c];
        cur = sm.par[cur];
      } else {
        u = sm.win[(W - 2) - (tap - dep)][c];       // v_{-(tap-dep+1)} of the committed prefix
      }
      conv = fmaf(sm.w[tap][c], u, conv);
    }
    o[base + (size_t)n * D + c] = from_f32<T>(num / (sm.den[n] + eps) + conv);
  }
}

template <typename T, int D, int PHI, bool PER_SEQ = false>
static cudaError_t launch_t(la_ctx* ctx, int B, int N, const void* q, const void* k, const void* v,
                            const int32_t* parent, const float* w, const la_state& st, void* o, cudaStream_t s) {
  const la_config& c = ctx->cfg;
  auto kern = verify_kernel<T, D, PHI, PER_SEQ>;
  const size_t smem = sizeof(VerifySmem<D>);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<dim3(B * c.H), dim3(256), smem, s>>>((const T*)q, (const T*)k, (const T*)v, parent, w, st.S, st.z,
                                               (const T*)st.win, (T*)o, ctx->d_status, c.H, N, c.conv_taps, c.eps);
  ctx->launches += 1;
  return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t launch_phi(la_ctx* ctx, int B, int N, const void* q, const void* k, const void* v,
                              const int32_t* parent, const float* w, const la_state& st, void* o, cudaStream_t s) {
  return ctx->cfg.phi == LA_PHI_ELU1 ? launch_t<T, D, LA_PHI_ELU1>(ctx, B, N, q, k, v, parent, w, st, o, s)
                                     : launch_t<T, D, LA_PHI_RELU>(ctx, B, N, q, k, v, parent, w, st, o, s);
}

cudaError_t launch_verify(la_ctx* ctx, int B, int N, const void* q, const void* k, const void* v,
                          const int32_t* parent, const float* w, const la_state& st, void* o, cudaStream_t s) {
  const la_config& c = ctx->cfg;
  if (c.io_dtype == LA_F32)
    return c.d == 64 ? launch_phi<float, 64>(ctx, B, N, q, k, v, parent, w, st, o, s)
                     : launch_phi<float, 128>(ctx, B, N, q, k, v, parent, w, st, o, s);
  return c.d == 64 ? launch_phi<__nv_bfloat16, 64>(ctx, B, N, q, k, v, parent, w, st, o, s)
                   : launch_phi<__nv_bfloat16, 128>(ctx, B, N, q, k, v, parent, w, st, o, s);
}

// ---- the same kernel with one status word per sequence (used by la_verify_tree_noalloc) ----
template <typename T, int D>
static cudaError_t launch_phi_per_seq(la_ctx* ctx, int B, int N, const void* q, const void* k, const void* v,
                                      const int32_t* parent, const float* w, const la_state& st, void* o,
                                      cudaStream_t s) {
  return ctx->cfg.phi == LA_PHI_ELU1
             ? launch_t<T, D, LA_PHI_ELU1, true>(ctx, B, N, q, k, v, parent, w, st, o, s)
             : launch_t<T, D, LA_PHI_RELU, true>(ctx, B, N, q, k, v, parent, w, st, o, s);
}

static cudaError_t launch_verify_per_seq(la_ctx* ctx, int B, int N, const void* q, const void* k, const void* v,
                                         const int32_t* parent, const float* w, const la_state& st, void* o,
                                         cudaStream_t s) {
  const la_config& c = ctx->cfg;
  if (c.io_dtype == LA_F32)
    return c.d == 64 ? launch_phi_per_seq<float, 64>(ctx, B, N, q, k, v, parent, w, st, o, s)
                     : launch_phi_per_seq<float, 128>(ctx, B, N, q, k, v, parent, w, st, o, s);
  return c.d == 64 ? launch_phi_per_seq<__nv_bfloat16, 64>(ctx, B, N, q, k, v, parent, w, st, o, s)
                   : launch_phi_per_seq<__nv_bfloat16, 128>(ctx, B, N, q, k, v, parent, w, st, o, s);
}

}  // namespace la

// =========================================================================================
// la_verify_tree_noalloc: tree verification for callers that must not allocate.
//
// The regular path reports device-side problems through a status word that la_create
// allocates with cudaMalloc.  Here that scratch lives in the library image instead: one
// status word per sequence in a fixed array that every GPU loading the library carries
// until the process exits (LA_NOALLOC_MAX_SEQ words = 4 KiB).
//
// In host code the name of a __device__ array is only a host-side handle, not an address
// the GPU can use, so the device address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and then handed to the kernel.
// =========================================================================================
#include <mutex>

static __device__ __align__(256) int g_noalloc_seq_status[LA_NOALLOC_MAX_SEQ];

namespace {

constexpr int kMaxDevices = 64;

// Device address of g_noalloc_seq_status on the current device `dev`; looked up on first use.
int* noalloc_scratch(int dev, cudaError_t* err) {
  static std::mutex mu;
  static int* addr[kMaxDevices] = {};
  std::lock_guard<std::mutex> lock(mu);
  *err = cudaSuccess;
  if (addr[dev] == nullptr) {
    void* p = nullptr;
    *err = cudaGetSymbolAddress(&p, g_noalloc_seq_status);
    if (*err != cudaSuccess) return nullptr;
    addr[dev] = static_cast<int*>(p);
  }
  return addr[dev];
}

inline bool ok16(const void* p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" la_status la_verify_tree_noalloc(const la_config* cfg, int32_t B, int32_t N, const void* q, const void* k,
                                            const void* v, const int32_t* parent, const float* conv_w,
                                            const la_state* st, void* o, int32_t* seq_status, void* stream) {
  if (!cfg || cfg->H < 1 || cfg->conv_taps < 1 || cfg->conv_taps > LA_MAX_TAPS) return LA_ERR_INVALID_ARG;
  if (cfg->phi != LA_PHI_ELU1 && cfg->phi != LA_PHI_RELU) return LA_ERR_INVALID_ARG;
  if (cfg->io_dtype != LA_F32 && cfg->io_dtype != LA_BF16) return LA_ERR_INVALID_ARG;
  if (!(cfg->eps >= 0.f) || cfg->eps > 3.0e38f) return LA_ERR_INVALID_ARG;
  if (cfg->d != 64 && cfg->d != 128) return LA_ERR_UNSUPPORTED;
  if (B < 1 || N < 1 || N > LA_MAX_NODES) return LA_ERR_INVALID_ARG;
  if (B > LA_NOALLOC_MAX_SEQ) return LA_ERR_TOO_LARGE;       // the fixed scratch has one word per sequence
  if (!ok16(q) || !ok16(k) || !ok16(v) || !ok16(conv_w) || !ok16(o) || !parent) return LA_ERR_INVALID_ARG;
  if (!st || !ok16(st->S) || !ok16(st->z) || (cfg->conv_taps > 1 && !ok16(st->win))) return LA_ERR_INVALID_ARG;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LA_ERR_CUDA;
  cudaError_t e;
  int* scratch = noalloc_scratch(dev, &e);
  if (!scratch) return LA_ERR_CUDA;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The array keeps what the previous call left in it: clear the words this call uses.
  if (cudaMemsetAsync(scratch, 0, sizeof(int) * B, s) != cudaSuccess) return LA_ERR_CUDA;
  la_ctx tmp{};
  tmp.cfg = *cfg;
  tmp.device = dev;
  tmp.d_status = scratch;
  if (la::launch_verify_per_seq(&tmp, B, N, q, k, v, parent, conv_w, *st, o, s) != cudaSuccess) return LA_ERR_CUDA;
  if (seq_status &&
      cudaMemcpyAsync(seq_status, scratch, sizeof(int) * B, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return LA_ERR_CUDA;
  return LA_OK;
}
