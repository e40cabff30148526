// Chunkwise-parallel prefill on the 5th-generation tensor cores (bf16 io, d = 128).
//
// Sec. 4.1: the sequence is cut into non-overlapping groups; inside a group the causally
// masked product phi(Q) phi(K)^T V is formed in parallel, between groups only the cumulative
// sums S = sum phi(k) v^T and z = sum phi(k) are carried.  One CTA walks one (batch, head)
// chain in tiles of 128 tokens.  Per tile:
//
//   TMA      Q, K, V tiles (128 x 128 bf16, two 64-column boxes each, 128-byte swizzle)
//   CUDA     phi applied in place on Q and K; den_inter = phi(Q) z; z += colsum phi(K)
//   tcgen05  P = phi(Q) phi(K)^T          (TMEM columns   0..127)
//            O = phi(Q) S_prev            (TMEM columns 128..255; S_prev as a bf16 copy in smem)
//   CUDA     P -> causal mask, row sums, bf16 -> smem
//   tcgen05  O += P V ;  S += phi(K)^T V  (S fp32 in TMEM columns 256..383 for the whole chain)
//   CUDA     o = O / den + conv(V)  -> smem -> TMA store;  S -> bf16 copy for the next tile
//
// Warps 0-7 do the CUDA-core work (thread = one tile row / TMEM lane, two column halves),
// warp 8 issues all TMA loads and all MMAs from one elected lane.  Every wait on an mbarrier
// is bounded; when one runs out the CTA records LA_ERR_TIMEOUT, stops issuing work, frees its
// TMEM and returns.
#include <cuda.h>

#include "la_common.cuh"

namespace la {
namespace tc {

constexpr int D = 128;
constexpr int TILE = 128;
constexpr int kComputeThreads = 256;
constexpr int kThreads = 288;
constexpr uint32_t BOX_BYTES = 128 * 128;          // 128 rows x 64 bf16
constexpr uint32_t TILE_BYTES = 2 * BOX_BYTES;
constexpr uint32_t P_COL = 0, O_COL = 128, S_COL = 256, TMEM_COLS = 512;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // one second per wait

// shared-memory map (offsets from a 1024-byte aligned base)
constexpr uint32_t OFF_Q = 0, OFF_K = TILE_BYTES, OFF_V0 = 2 * TILE_BYTES, /* second V buffer at 3 * TILE_BYTES */
                   OFF_P = 4 * TILE_BYTES, OFF_S = 5 * TILE_BYTES, OFF_SMALL = 6 * TILE_BYTES;

struct Small {
  float zs[D];
  float zpart[8][D];
  float den_inter[2][TILE];
  float den_intra[2][TILE];
  unsigned long long bars[8];
  uint32_t tmem_base;
  int abort;
  int pad[2];
};
enum { B_FULL_QK = 0, B_FULL_V0 = 1, B_FULL_V1 = 2, B_MMA1 = 3, B_MMA2 = 4, B_PHI = 5, B_P = 6, B_EPI = 7 };

__host__ __device__ constexpr uint32_t off_w() { return OFF_SMALL + (uint32_t)((sizeof(Small) + 15) / 16 * 16); }
__host__ __device__ inline uint32_t off_halo(int W) { return off_w() + (uint32_t)W * D * 4; }
__host__ __device__ inline uint32_t smem_bytes(int W) { return off_halo(W) + (uint32_t)(W > 1 ? W - 1 : 1) * D * 2 + 1024; }

// ---- PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
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
// Bounded wait.  Returns false (and raises the CTA's abort flag) when a second has passed or
// another thread has already given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
#pragma unroll 1
    for (int it = 0; it < 64; ++it)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort) return false;
    if (global_ns() - t0 > kWaitLimitNs) {
      *abort = 1;
      return false;
    }
  }
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

__device__ __forceinline__ void tma_load(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_store(const CUtensorMap* map, int x, int y, int z, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(map), "r"(x),
               "r"(y), "r"(z), "r"(src)
               : "memory");
}
__device__ __forceinline__ void tma_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)acc)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

#define LA_TMEM_LD32(taddr, r)                                                                                   \
  asm volatile(                                                                                                  \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                                  \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "                                  \
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"                  \
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),          \
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),    \
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),  \
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])   \
      : "r"(taddr)                                                                                               \
      : "memory")

#define LA_TMEM_ST32(taddr, r)                                                                                   \
  asm volatile(                                                                                                  \
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "                                                            \
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "                                 \
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"                         \
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),      \
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),            \
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),          \
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])           \
      : "memory")

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---- descriptors ----------------------------------------------------------------------------
// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading and stride byte offsets
// (all in 16-byte units), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Operand whose contraction index runs along the 128-byte rows (rows = M or N): step ks covers 16 elements.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t tile, int ks) {
  return smem_desc(tile + (uint32_t)(ks >> 2) * BOX_BYTES + (uint32_t)(ks & 3) * 32u, 16u, 1024u);
}
// Operand whose contraction index runs along the tile rows (rows = K, 128-byte rows hold M or N): step ks
// covers 16 rows; the two 64-element column boxes are BOX_BYTES apart.
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t tile, int ks) {
  return smem_desc(tile + (uint32_t)ks * 2048u, BOX_BYTES, 1024u);
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = 128.
__host__ __device__ constexpr uint32_t idesc(bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

// ---- bf16 packing ------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float lo_f(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float hi_f(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

template <int PHI> __device__ __forceinline__ float phi_fast(float x) {
  if (PHI == LA_PHI_ELU1) return x > 0.f ? x + 1.f : __expf(x);
  return fmaxf(x, 0.f);
}

// phi on 8 packed bf16 values; returns the rounded results packed, and their fp32 values in f[8].
template <int PHI> __device__ __forceinline__ uint4 phi8(uint4 u, float* f) {
  uint4 r;
  r.x = pack2(phi_fast<PHI>(lo_f(u.x)), phi_fast<PHI>(hi_f(u.x)));
  r.y = pack2(phi_fast<PHI>(lo_f(u.y)), phi_fast<PHI>(hi_f(u.y)));
  r.z = pack2(phi_fast<PHI>(lo_f(u.z)), phi_fast<PHI>(hi_f(u.z)));
  r.w = pack2(phi_fast<PHI>(lo_f(u.w)), phi_fast<PHI>(hi_f(u.w)));
  f[0] = lo_f(r.x); f[1] = hi_f(r.x); f[2] = lo_f(r.y); f[3] = hi_f(r.y);
  f[4] = lo_f(r.z); f[5] = hi_f(r.z); f[6] = lo_f(r.w); f[7] = hi_f(r.w);
  return r;
}

// Byte offset of 16-byte chunk `cc` (0..7) of row `row` inside one 128-byte-swizzled box.
__device__ __forceinline__ uint32_t swz(int row, int cc) { return (uint32_t)row * 128u + (uint32_t)((cc ^ (row & 7)) << 4); }

// ---- the kernel ------------------------------------------------------------------------------------
template <int PHI>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
                  const __grid_constant__ CUtensorMap mv, const __grid_constant__ CUtensorMap mo,
                  const float* __restrict__ w, float* __restrict__ S, float* __restrict__ z,
                  __nv_bfloat16* __restrict__ win, int64_t* __restrict__ pos, int* status, int H, int T, int W,
                  float eps, int init) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  Small& sm = *reinterpret_cast<Small*>(smem + OFF_SMALL);
  float* wsm = reinterpret_cast<float*>(smem + off_w());                       // [W][128]
  __nv_bfloat16* halo = reinterpret_cast<__nv_bfloat16*>(smem + off_halo(W));  // [W-1][128], oldest first
  volatile int* abort = &sm.abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.x, h = bh % H;
  const int nchunks = (T + TILE - 1) / TILE;
  uint32_t bar[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) bar[i] = smem_u32(&sm.bars[i]);

  // ---- set-up ----
  if (tid == 0) {
    mbar_init(bar[B_FULL_QK], 1);
    mbar_init(bar[B_FULL_V0], 1);
    mbar_init(bar[B_FULL_V1], 1);
    mbar_init(bar[B_MMA1], 1);
    mbar_init(bar[B_MMA2], 1);
    mbar_init(bar[B_PHI], kComputeThreads);
    mbar_init(bar[B_P], kComputeThreads);
    mbar_init(bar[B_EPI], kComputeThreads);
    sm.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int idx = tid; idx < W * D; idx += kThreads) wsm[idx] = w[((size_t)h * D + (idx % D)) * W + idx / D];
  for (int idx = tid; idx < (W - 1) * D; idx += kThreads)
    halo[idx] = init ? win[(size_t)bh * (W - 1) * D + idx] : __float2bfloat16_rn(0.f);
  if (tid < D) sm.zs[tid] = init ? z[(size_t)bh * D + tid] : 0.f;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 8) {
    // =============================== TMA + MMA issue (one lane) ===============================
    if (lane == 0) {
      bool ok = true;
      mbar_expect_tx(bar[B_FULL_QK], 2 * TILE_BYTES);
      tma_load(sbase + OFF_Q, &mq, 0, 0, bh, bar[B_FULL_QK]);
      tma_load(sbase + OFF_Q + BOX_BYTES, &mq, 64, 0, bh, bar[B_FULL_QK]);
      tma_load(sbase + OFF_K, &mk, 0, 0, bh, bar[B_FULL_QK]);
      tma_load(sbase + OFF_K + BOX_BYTES, &mk, 64, 0, bh, bar[B_FULL_QK]);
      for (int n = 0; n < 2 && n < nchunks; ++n) {
        mbar_expect_tx(bar[B_FULL_V0 + n], TILE_BYTES);
        tma_load(sbase + OFF_V0 + n * TILE_BYTES, &mv, 0, n * TILE, bh, bar[B_FULL_V0 + n]);
        tma_load(sbase + OFF_V0 + n * TILE_BYTES + BOX_BYTES, &mv, 64, n * TILE, bh, bar[B_FULL_V0 + n]);
      }
      for (int n = 0; n < nchunks && ok; ++n) {
        const uint32_t par = n & 1;
        const uint32_t vbuf = sbase + OFF_V0 + par * TILE_BYTES;
        const bool has_state = init || n > 0;
        ok = mbar_wait(bar[B_PHI], par, abort);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)   // P = phi(Q) phi(K)^T
          mma_bf16(tmem + P_COL, desc_kmajor(sbase + OFF_Q, ks), desc_kmajor(sbase + OFF_K, ks), idesc(false, false),
                   ks > 0);
        if (has_state) {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)   // O = phi(Q) S_prev
            mma_bf16(tmem + O_COL, desc_kmajor(sbase + OFF_Q, ks), desc_mnmajor(sbase + OFF_S, ks), idesc(false, true),
                     ks > 0);
        }
        mma_commit(bar[B_MMA1]);
        ok = mbar_wait(bar[B_P], par, abort) && mbar_wait(bar[B_FULL_V0 + par], (n >> 1) & 1, abort);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)   // O += (P o M) V
          mma_bf16(tmem + O_COL, desc_kmajor(sbase + OFF_P, ks), desc_mnmajor(vbuf, ks), idesc(false, true),
                   has_state || ks > 0);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)   // S += phi(K)^T V
          mma_bf16(tmem + S_COL, desc_mnmajor(sbase + OFF_K, ks), desc_mnmajor(vbuf, ks), idesc(true, true),
                   has_state || ks > 0);
        mma_commit(bar[B_MMA2]);
        if (n + 1 < nchunks) {
          ok = mbar_wait(bar[B_MMA1], par, abort);      // Q tile is free
          if (!ok) break;
          mbar_expect_tx(bar[B_FULL_QK], 2 * TILE_BYTES);
          tma_load(sbase + OFF_Q, &mq, 0, (n + 1) * TILE, bh, bar[B_FULL_QK]);
          tma_load(sbase + OFF_Q + BOX_BYTES, &mq, 64, (n + 1) * TILE, bh, bar[B_FULL_QK]);
          ok = mbar_wait(bar[B_MMA2], par, abort);      // K tile is free
          if (!ok) break;
          tma_load(sbase + OFF_K, &mk, 0, (n + 1) * TILE, bh, bar[B_FULL_QK]);
          tma_load(sbase + OFF_K + BOX_BYTES, &mk, 64, (n + 1) * TILE, bh, bar[B_FULL_QK]);
        }
        if (n + 2 < nchunks) {
          ok = mbar_wait(bar[B_EPI], par, abort);       // V buffer `par` is free
          if (!ok) break;
          mbar_expect_tx(bar[B_FULL_V0 + par], TILE_BYTES);
          tma_load(vbuf, &mv, 0, (n + 2) * TILE, bh, bar[B_FULL_V0 + par]);
          tma_load(vbuf + BOX_BYTES, &mv, 64, (n + 2) * TILE, bh, bar[B_FULL_V0 + par]);
        }
      }
    }
  } else {
    // =============================== CUDA-core work (256 threads) ===============================
    const int r = 32 * (warp & 3) + lane;         // tile row = TMEM lane
    const int hf = warp >> 2;                     // column half
    const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
    unsigned char* Qb = smem + OFF_Q + hf * BOX_BYTES;
    unsigned char* Pb = smem + OFF_P + hf * BOX_BYTES;
    unsigned char* Sb = smem + OFF_S + hf * BOX_BYTES;
    float* Sg = S + (size_t)bh * D * D + (size_t)r * D + 64 * hf;
    bool ok = true;

    if (init) {   // S -> TMEM (fp32) and -> bf16 copy in shared memory
#pragma unroll
      for (int qq = 0; qq < 2; ++qq) {
        uint32_t v[32];
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          const float4 x = *reinterpret_cast<const float4*>(Sg + 32 * qq + e);
          v[e] = __float_as_uint(x.x); v[e + 1] = __float_as_uint(x.y);
          v[e + 2] = __float_as_uint(x.z); v[e + 3] = __float_as_uint(x.w);
        }
        LA_TMEM_ST32(tmem + lane_addr + S_COL + 64 * hf + 32 * qq, v);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint4 u;
          u.x = pack2(__uint_as_float(v[8 * c]), __uint_as_float(v[8 * c + 1]));
          u.y = pack2(__uint_as_float(v[8 * c + 2]), __uint_as_float(v[8 * c + 3]));
          u.z = pack2(__uint_as_float(v[8 * c + 4]), __uint_as_float(v[8 * c + 5]));
          u.w = pack2(__uint_as_float(v[8 * c + 6]), __uint_as_float(v[8 * c + 7]));
          *reinterpret_cast<uint4*>(Sb + swz(r, 4 * qq + c)) = u;
        }
      }
      tmem_wait_st();
      tc_fence_before();
    }

    for (int n = 0; n < nchunks; ++n) {
      const uint32_t par = n & 1;
      const int valid = min(TILE, T - n * TILE);
      unsigned char* Vt = smem + OFF_V0 + par * TILE_BYTES;    // whole V tile (both boxes)
      const bool last = n + 1 == nchunks;

      // ---- phi on Q and K in place; den_inter = phi(Q).z_prev; column sums of phi(K) ----
      ok = ok && mbar_wait(bar[B_FULL_QK], par, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        float dot = 0.f;
#pragma unroll
        for (int cc = 0; cc < 8; ++cc) {
          uint4* p = reinterpret_cast<uint4*>(Qb + swz(r, cc));
          float f[8];
          *p = phi8<PHI>(*p, f);
          const float* zz = &sm.zs[64 * hf + 8 * cc];
#pragma unroll
          for (int e = 0; e < 8; ++e) dot = fmaf(f[e], zz[e], dot);
        }
        sm.den_inter[hf][r] = dot;

        const int ct = tid & 15, rg = tid >> 4;                 // chunk column 0..15, row group 0..15
        unsigned char* Kb = smem + OFF_K + (ct >> 3) * BOX_BYTES;
        float cs[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) cs[e] = 0.f;
#pragma unroll
        for (int m = 0; m < 8; ++m) {
          const int j = rg + 16 * m;
          uint4* p = reinterpret_cast<uint4*>(Kb + swz(j, ct & 7));
          if (j < valid) {
            float f[8];
            *p = phi8<PHI>(*p, f);
#pragma unroll
            for (int e = 0; e < 8; ++e) cs[e] += f[e];
          } else {
            *p = make_uint4(0u, 0u, 0u, 0u);                    // rows past the end contribute nothing
          }
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) cs[e] += __shfl_xor_sync(0xffffffffu, cs[e], 16);
        if (lane < 16) {
#pragma unroll
          for (int e = 0; e < 8; ++e) sm.zpart[warp][8 * ct + e] = cs[e];
        }
      }
      fence_proxy_async();
      tc_fence_before();
      mbar_arrive(bar[B_PHI]);
      if (tid == 0) tma_wait_read();                            // the previous output tile has left shared memory
      compute_sync();
      if (tid < D && ok) {
        float a = sm.zs[tid];
#pragma unroll
        for (int ww = 0; ww < 8; ++ww) a += sm.zpart[ww][tid];
        sm.zs[tid] = a;
      }

      // ---- P: causal mask, row sums, bf16 -> shared memory ----
      ok = ok && mbar_wait(bar[B_MMA1], par, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        tc_fence_after();
        float rowsum = 0.f;
#pragma unroll
        for (int qq = 0; qq < 2; ++qq) {
          const int col0 = 64 * hf + 32 * qq;
          uint32_t v[32];
          if (col0 <= 32 * (warp & 3) + 31) {                   // warp-uniform: some row of this warp reaches col0
            LA_TMEM_LD32(tmem + lane_addr + P_COL + col0, v);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = 0u;
          }
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int j = col0 + 8 * c + 2 * e;
              const float a = j <= r ? __uint_as_float(v[8 * c + 2 * e]) : 0.f;
              const float b = j + 1 <= r ? __uint_as_float(v[8 * c + 2 * e + 1]) : 0.f;
              pk[e] = pack2(a, b);
              rowsum += lo_f(pk[e]) + hi_f(pk[e]);
            }
            *reinterpret_cast<uint4*>(Pb + swz(r, 4 * qq + c)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
        sm.den_intra[hf][r] = rowsum;
      }
      fence_proxy_async();
      tc_fence_before();
      mbar_arrive(bar[B_P]);
      compute_sync();

      // ---- epilogue: o = O / den + conv(V); S -> bf16 copy (or to global after the last tile) ----
      ok = ok && mbar_wait(bar[B_MMA2], par, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        tc_fence_after();
        const float den = sm.den_intra[0][r] + sm.den_intra[1][r] + sm.den_inter[0][r] + sm.den_inter[1][r] + eps;
        const float rden = 1.f / den;
#pragma unroll
        for (int qq = 0; qq < 2; ++qq) {
          uint32_t v[32];
          LA_TMEM_LD32(tmem + lane_addr + O_COL + 64 * hf + 32 * qq, v);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int cc = 4 * qq + c;                          // chunk inside this half's box
            const int ch0 = 64 * hf + 8 * cc;                   // first channel of the chunk
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = __uint_as_float(v[8 * c + e]) * rden;
            for (int t = 0; t < W; ++t) {
              const int row = r - t;
              uint4 u;
              if (row >= 0) u = *reinterpret_cast<const uint4*>(Vt + hf * BOX_BYTES + swz(row, cc));
              else u = *reinterpret_cast<const uint4*>(halo + (W - 1 + row) * D + ch0);
              const float4 w0 = *reinterpret_cast<const float4*>(wsm + t * D + ch0);
              const float4 w1 = *reinterpret_cast<const float4*>(wsm + t * D + ch0 + 4);
              acc[0] = fmaf(w0.x, lo_f(u.x), acc[0]); acc[1] = fmaf(w0.y, hi_f(u.x), acc[1]);
              acc[2] = fmaf(w0.z, lo_f(u.y), acc[2]); acc[3] = fmaf(w0.w, hi_f(u.y), acc[3]);
              acc[4] = fmaf(w1.x, lo_f(u.z), acc[4]); acc[5] = fmaf(w1.y, hi_f(u.z), acc[5]);
              acc[6] = fmaf(w1.z, lo_f(u.w), acc[6]); acc[7] = fmaf(w1.w, hi_f(u.w), acc[7]);
            }
            *reinterpret_cast<uint4*>(Pb + swz(r, cc)) =
                make_uint4(pack2(acc[0], acc[1]), pack2(acc[2], acc[3]), pack2(acc[4], acc[5]), pack2(acc[6], acc[7]));
          }
        }
#pragma unroll
        for (int qq = 0; qq < 2; ++qq) {
          uint32_t v[32];
          LA_TMEM_LD32(tmem + lane_addr + S_COL + 64 * hf + 32 * qq, v);
          tmem_wait_ld();
          if (last) {
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              *reinterpret_cast<float4*>(Sg + 32 * qq + e) =
                  make_float4(__uint_as_float(v[e]), __uint_as_float(v[e + 1]), __uint_as_float(v[e + 2]),
                              __uint_as_float(v[e + 3]));
          } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint4 u;
              u.x = pack2(__uint_as_float(v[8 * c]), __uint_as_float(v[8 * c + 1]));
              u.y = pack2(__uint_as_float(v[8 * c + 2]), __uint_as_float(v[8 * c + 3]));
              u.z = pack2(__uint_as_float(v[8 * c + 4]), __uint_as_float(v[8 * c + 5]));
              u.w = pack2(__uint_as_float(v[8 * c + 6]), __uint_as_float(v[8 * c + 7]));
              *reinterpret_cast<uint4*>(Sb + swz(r, 4 * qq + c)) = u;
            }
          }
        }
      }
      fence_proxy_async();
      tc_fence_before();
      compute_sync();
      if (tid == 0 && ok) {
        tma_store(&mo, 0, n * TILE, bh, sbase + OFF_P);
        tma_store(&mo, 64, n * TILE, bh, sbase + OFF_P + BOX_BYTES);
        tma_commit();
      }
      if (tid < D && ok) {
        // halo <- last W-1 rows of (halo ++ valid rows of V); ascending, source index above target
        const unsigned char* Vc = Vt + (tid >> 6) * BOX_BYTES;
        const int cw = tid & 63;
        for (int i = 0; i < W - 1; ++i) {
          const int src = valid + i;
          __nv_bfloat16 x;
          if (src < W - 1) x = halo[src * D + tid];
          else x = *reinterpret_cast<const __nv_bfloat16*>(Vc + swz(src - (W - 1), cw >> 3) + (cw & 7) * 2);
          halo[i * D + tid] = x;
        }
      }
      mbar_arrive(bar[B_EPI]);
    }

    compute_sync();
    if (ok) {
      if (tid < D) {
        z[(size_t)bh * D + tid] = sm.zs[tid];
        for (int i = 0; i < W - 1; ++i) win[((size_t)bh * (W - 1) + i) * D + tid] = halo[i * D + tid];
      }
      if (tid == 0 && h == 0) pos[bh / H] = (init ? pos[bh / H] : 0) + T;
    }
    if (tid == 0) tma_wait_all();
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (sm.abort) {
    if (tid == 0) report(status, LA_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(2000);   // bounded grace period for copies still in flight
  }
  if (warp == 8) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

// ---- host side -------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// [BH, T, 128] bf16 viewed as a 3-D tensor; boxes of 64 columns x 128 rows x 1, 128-byte swizzle.
// Rows past T read as zeros and are clipped on store.
static bool make_map(CUtensorMap* m, const void* base, int BH, int T) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)T * D * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)TILE, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc

cudaError_t launch_prefill_tc(la_ctx* ctx, int B, int T, const void* q, const void* k, const void* v, const float* w,
                              int init, const la_state& st, void* o, cudaStream_t s, bool* handled) {
  const la_config& c = ctx->cfg;
  *handled = false;
  if (c.io_dtype != LA_BF16 || c.d != tc::D) return cudaSuccess;
  const int BH = B * c.H;
  CUtensorMap mq, mk, mv, mo;
  if (!tc::make_map(&mq, q, BH, T) || !tc::make_map(&mk, k, BH, T) || !tc::make_map(&mv, v, BH, T) ||
      !tc::make_map(&mo, o, BH, T))
    return cudaSuccess;   // no tensor-map support: the CUDA-core kernel takes over
  const size_t smem = tc::smem_bytes(c.conv_taps);
  auto kern = c.phi == LA_PHI_ELU1 ? tc::prefill_tc_kernel<LA_PHI_ELU1> : tc::prefill_tc_kernel<LA_PHI_RELU>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<dim3(BH), dim3(tc::kThreads), smem, s>>>(mq, mk, mv, mo, w, st.S, st.z, (__nv_bfloat16*)st.win, st.pos,
                                                  ctx->d_status, c.H, T, c.conv_taps, c.eps, init);
  ctx->launches += 1;
  *handled = true;
  return cudaGetLastError();
}

}  // namespace la
