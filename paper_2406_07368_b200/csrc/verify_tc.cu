// Draft-tree verification on the tensor cores (bf16 io, d = 128, N <= 64).
//
// Sec. 4.2 / Sec. 5.3: all N draft nodes of a sequence share the committed state.  The shared part
// of every node's numerator, phi(Q_tree) S, is one dense product; it is computed transposed,
//     O^T[c][n] = sum_a S[a][c] phi(q_n)[a],
// so that the fp32 state is the M x K operand exactly as it lies in memory: TMA brings the 128 x 128
// fp32 tile of S into shared memory (128-byte swizzle in 32-byte chunks) and tcgen05.mma consumes it as tf32 -- S is read
// from HBM once, without any conversion pass, while the CUDA cores prepare the tree.  The accumulator
// (128 channels x 64 nodes, fp32) lives in TMEM; each thread then owns one channel, adds the
// contributions of the node's ancestors and itself (tree mask), the unfolded convolution along the
// ancestor chain, and divides by the node's denominator.  Nothing of the state is written.  CTAs are persistent:
// while one warp group finishes a unit, another already prepares the next one.
#include <cuda.h>

#include <algorithm>

#include "la_common.cuh"

namespace la {
namespace vtc {

constexpr int D = 128, NMAX = LA_MAX_NODES;
constexpr int kMaxTaps = 8;                        // longer tap windows are served by the CUDA-core kernel
constexpr int kThreadsX = 256, kThreadsY = 256, kCtrlWarp = 16, kThreads = 544;
constexpr uint32_t S_BOX = 128 * 128;              // 128 rows x 32 fp32
constexpr uint32_t Q_BOX = NMAX * 128;             // 64 rows x 32 fp32
constexpr uint32_t TMEM_COLS = 128;                // two accumulators of 64 columns
constexpr unsigned long long kWaitLimitNs = 1000000000ull;

// What the epilogue of one unit reads; two copies, so that the next unit is prepared while this one is finished.
struct alignas(16) Buf {
  float A[NMAX][NMAX];                             // A[j][n] = phi(q_n) . phi(k of the ancestor of n at distance j); 0 past the chain
  float w[kMaxTaps][D];                            // taps of this unit's head
  float rden[NMAX];                                // 1 / (denominator + eps) per node
  __nv_bfloat16 vrows[NMAX + kMaxTaps - 1][D];     // rows 0..63 the draft values, rows 64.. the committed window
  unsigned char anc[NMAX][NMAX];                   // anc[j][n] = row of vrows holding the value at distance j behind n
  int max_depth;
  int bad;
  int pad[2];
};
// Scratch of the preparing group.
struct alignas(16) Prep {
  float fk[NMAX][D + 4];
  float z[D];
  int par[NMAX];
  int depth[NMAX];
  int pair_off[NMAX + 1];
  int scan_carry;
  unsigned char pair_n[NMAX * (NMAX + 1) / 2];
  unsigned char pair_j[NMAX * (NMAX + 1) / 2];
};
struct alignas(16) Ctl {
  unsigned long long bars[8];
  uint32_t tmem_base;
  int abort;
};
// The per-unit barriers come in pairs indexed by t & 1 (phase t >> 1): a barrier is not completed again before
// every waiter of its previous phase has passed, because the next completion depends on that waiter's own arrival.
enum { B_FULL_S = 0, B_MMA0 = 1, B_MMA1 = 2, B_XDONE0 = 3, B_XDONE1 = 4, B_EPI0 = 5, B_EPI1 = 6, kNumBars = 7 };
constexpr uint32_t OFF_S = 0, OFF_Q = 4 * S_BOX, OFF_PREP = OFF_Q + 4 * Q_BOX;
constexpr uint32_t OFF_BUF = OFF_PREP + (uint32_t)sizeof(Prep);
constexpr uint32_t OFF_CTL = OFF_BUF + 2 * (uint32_t)sizeof(Buf);
constexpr uint32_t kSmemBytes = OFF_CTL + (uint32_t)sizeof(Ctl) + 1024;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
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
// Bounded wait: false after one second (the CTA's abort flag is raised) or when another thread gave up.
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
// 128-byte swizzle: byte offset of 16-byte chunk `cc` of row `row` inside a box with 128-byte rows.
__device__ __forceinline__ uint32_t swz(int row, int cc) { return (uint32_t)row * 128u + (uint32_t)((cc ^ (row & 7)) << 4); }
// Shared-memory matrix descriptor; layout 2 = 128-byte swizzle in 16-byte chunks, 1 = 128-byte swizzle in 32-byte
// chunks (the only layout the hardware takes for a 32-bit operand whose M or N index is the contiguous one).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)layout << 61);
}
// Instruction descriptor: fp32 accumulate, tf32 x tf32, A with M contiguous (as S lies in memory), B with K
// contiguous, M = 128, N = 64.
constexpr uint32_t kIdesc = (1u << 4) | (2u << 7) | (2u << 10) | (1u << 15) | ((64u >> 3) << 17) | ((128u >> 4) << 24);

template <int PHI> __device__ __forceinline__ float phi_f(float x) {
  if (PHI == LA_PHI_ELU1) return x > 0.f ? x + 1.f : __expf(x);
  return fmaxf(x, 0.f);
}

__device__ __forceinline__ void sync_x() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Persistent kernel: CTA i handles units i, i + gridDim.x, ...  Three roles run concurrently:
//   group X (warps 0-7)  prepares unit t: tree tables, phi(q) as the tf32 operand, phi(k), scores, denominators;
//   warp 16 (one lane)   loads S of unit t by TMA and issues the tf32 product into TMEM accumulator t & 1;
//   group Y (warps 8-15) finishes unit t: tree terms, unfolded convolution, division, store --
// while group X already prepares unit t + 1 in the other copy of the per-unit tables.
template <int PHI>
__global__ void __launch_bounds__(kThreads, 1)
verify_tc_kernel(const __grid_constant__ CUtensorMap ms, const __nv_bfloat16* __restrict__ q,
                 const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                 const int32_t* __restrict__ parent, const float* __restrict__ w, const float* __restrict__ z,
                 const __nv_bfloat16* __restrict__ win, __nv_bfloat16* __restrict__ o, int* status, int H, int N, int W,
                 float eps, int units) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  Prep& pr = *reinterpret_cast<Prep*>(smem + OFF_PREP);
  Buf* bufs = reinterpret_cast<Buf*>(smem + OFF_BUF);
  Ctl& ctl = *reinterpret_cast<Ctl*>(smem + OFF_CTL);
  volatile int* abort = &ctl.abort;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nloc = (units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // units of this CTA
  uint32_t bar[kNumBars];
#pragma unroll
  for (int i = 0; i < kNumBars; ++i) bar[i] = smem_u32(&ctl.bars[i]);

  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar[B_FULL_S]) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar[B_MMA0]) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar[B_MMA1]) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar[B_XDONE0]), "r"(kThreadsX) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar[B_XDONE1]), "r"(kThreadsX) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar[B_EPI0]), "r"(kThreadsY) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar[B_EPI1]), "r"(kThreadsY) : "memory");
    ctl.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == kCtrlWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = ctl.tmem_base;

  if (warp == kCtrlWarp) {
    // =============================== TMA of S and the tf32 product (one lane) ===============================
    if (lane == 0) {
      auto load_s = [&](int t) {   // the committed state of unit t: four boxes of 32 columns
        const int u = (int)blockIdx.x + t * (int)gridDim.x;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar[B_FULL_S]), "r"(4 * S_BOX) : "memory");
#pragma unroll
        for (int x = 0; x < 4; ++x)
          asm volatile(
              "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
              ::"r"(sbase + OFF_S + x * S_BOX), "l"(&ms), "r"(32 * x), "r"(u * D), "r"(bar[B_FULL_S])
              : "memory");
      };
      if (nloc > 0) load_s(0);
      for (int t = 0; t < nloc; ++t) {
        const uint32_t par = t & 1, ph = (t >> 1) & 1;
        if (!mbar_wait(bar[B_XDONE0 + par], ph, abort) || !mbar_wait(bar[B_FULL_S], par, abort)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (!bufs[par].bad) {
#pragma unroll
          for (int ks = 0; ks < 16; ++ks) {    // 8 values of the contraction index a per step
            // S: 8 rows of a per step = two groups of 4 rows (512 B apart); the four 32-column boxes are S_BOX apart
            const uint64_t adesc = smem_desc(sbase + OFF_S + ks * 1024u, S_BOX, 512u, 1u);
            const uint64_t bdesc = smem_desc(sbase + OFF_Q + (ks >> 2) * Q_BOX + (ks & 3) * 32u, 16u, 1024u, 2u);
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "setp.ne.b32 p, %4, 0;\n\t"
                "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                ::"r"(tmem + par * 64u), "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"((uint32_t)(ks > 0))
                : "memory");
          }
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar[B_MMA0 + par]) : "memory");
        if (!mbar_wait(bar[B_MMA0 + par], ph, abort)) break;     // S and phi(Q) have been read
        if (t + 1 < nloc) load_s(t + 1);
      }
    }
  } else if (warp < 8) {
    // =============================== group X: prepare unit t ===============================
    bool ok = true;
    for (int t = 0; t < nloc; ++t) {
      const int u = (int)blockIdx.x + t * (int)gridDim.x, b = u / H, h = u % H;
      Buf& bf = bufs[t & 1];
      // this copy of the tables was last read by the epilogue of unit t - 2
      if (t >= 2) ok = ok && mbar_wait(bar[B_EPI0 + (t & 1)], ((t >> 1) - 1) & 1, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { mbar_arrive(bar[B_XDONE0 + (t & 1)]); continue; }

      // ---- q, k, v of the tree: all loads in flight before the tree is prepared ----
      const size_t base = (size_t)u * N * D;
      constexpr int ITERS = NMAX * (D / 4) / kThreadsX;      // 8 chunks of 4 values per thread
      uint2 uq[ITERS], uk[ITERS], uv[ITERS];
#pragma unroll
      for (int it = 0; it < ITERS; ++it) {
        const int idx = tid + it * kThreadsX, n = idx / (D / 4), a4 = (idx % (D / 4)) * 4;
        uq[it] = uk[it] = uv[it] = make_uint2(0u, 0u);
        if (n < N) {
          uq[it] = *reinterpret_cast<const uint2*>(q + base + (size_t)n * D + a4);
          uk[it] = *reinterpret_cast<const uint2*>(k + base + (size_t)n * D + a4);
          uv[it] = *reinterpret_cast<const uint2*>(v + base + (size_t)n * D + a4);
        }
      }

      // ---- tree preparation: ancestor chains and depths (integer work) ----
      if (tid < N) pr.par[tid] = parent[(size_t)b * N + tid];
      for (int idx = tid; idx < NMAX * NMAX; idx += kThreadsX) (&bf.A[0][0])[idx] = 0.f;
      if (tid == 0) { bf.max_depth = 0; bf.bad = 0; }
      sync_x();
      int my_dep = 0, my_off = 0;
      if (tid < NMAX) {
        if (tid < N) {
          int m = tid;
          bool good = true;
          while (m >= 0) {                     // m strictly decreases: at most N iterations
            bf.anc[my_dep++][tid] = (unsigned char)m;
            const int p = pr.par[m];
            if (p < -1 || p >= m) { good = false; break; }
            m = p;
          }
          if (!good) bf.bad = 1;
        }
        int x = my_dep;                        // exclusive prefix of the depths over the two warps that hold the nodes
#pragma unroll
        for (int o2 = 1; o2 < 32; o2 <<= 1) {
          const int y = __shfl_up_sync(0xffffffffu, x, o2);
          if (lane >= o2) x += y;
        }
        my_off = x - my_dep;
        if (tid == 31) pr.scan_carry = x;
        atomicMax(&bf.max_depth, my_dep);
        pr.depth[tid] = my_dep;
      }
      sync_x();
      const bool bad = bf.bad != 0;
      if (tid < NMAX && !bad) {
        if (tid >= 32) my_off += pr.scan_carry;
        pr.pair_off[tid] = my_off;
        if (tid == NMAX - 1) pr.pair_off[NMAX] = my_off + my_dep;
        const int jmax = max(bf.max_depth, W);
        for (int j = 0; j < my_dep; ++j) {
          pr.pair_n[my_off + j] = (unsigned char)tid;
          pr.pair_j[my_off + j] = (unsigned char)j;
        }
        for (int j = my_dep; j < jmax; ++j)    // behind the chain: the committed window while taps remain, else a dummy row
          bf.anc[j][tid] = (unsigned char)(tid < N && j < W ? NMAX + (W - 2) - (j - my_dep) : 0);
      }

      // ---- staging: phi(q) (fp32, swizzled: the B operand), phi(k), v, window, taps, z ----
      if (t >= 1) ok = mbar_wait(bar[B_MMA0 + ((t - 1) & 1)], ((t - 1) >> 1) & 1, abort);   // the previous product has read phi(Q)
      ok = __all_sync(0xffffffffu, ok);
      if (ok && !bad) {
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
          const int idx = tid + it * kThreadsX, n = idx / (D / 4), a4 = (idx % (D / 4)) * 4;
          float4 fq = make_float4(0.f, 0.f, 0.f, 0.f), fk = fq;
          if (n < N) {                                       // rows past N stay zero (phi(0) may be 1)
            fq = make_float4(phi_f<PHI>(__uint_as_float(uq[it].x << 16)), phi_f<PHI>(__uint_as_float(uq[it].x & 0xffff0000u)),
                             phi_f<PHI>(__uint_as_float(uq[it].y << 16)), phi_f<PHI>(__uint_as_float(uq[it].y & 0xffff0000u)));
            fk = make_float4(phi_f<PHI>(__uint_as_float(uk[it].x << 16)), phi_f<PHI>(__uint_as_float(uk[it].x & 0xffff0000u)),
                             phi_f<PHI>(__uint_as_float(uk[it].y << 16)), phi_f<PHI>(__uint_as_float(uk[it].y & 0xffff0000u)));
          }
          *reinterpret_cast<float4*>(smem + OFF_Q + (a4 >> 5) * Q_BOX + swz(n, (a4 & 31) >> 2)) = fq;
          *reinterpret_cast<float4*>(&pr.fk[n][a4]) = fk;
          *reinterpret_cast<uint2*>(&bf.vrows[n][a4]) = uv[it];
        }
        for (int idx = tid; idx < W * D; idx += kThreadsX) bf.w[idx / D][idx % D] = w[((size_t)h * D + idx % D) * W + idx / D];
        for (int idx = tid; idx < (W - 1) * D; idx += kThreadsX) bf.vrows[NMAX + idx / D][idx % D] = win[(size_t)u * (W - 1) * D + idx];
        if (tid < D) pr.z[tid] = z[(size_t)u * D + tid];
      }
      sync_x();

      // ---- scores of every (node, ancestor) pair, one pair per thread, then the denominators ----
      if (ok && !bad) {
        const int npairs = pr.pair_off[NMAX];
        for (int pi = tid; pi < npairs; pi += kThreadsX) {
          const int n = pr.pair_n[pi], j = pr.pair_j[pi], m = bf.anc[j][n];
          float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 8
          for (int e = 0; e < D; e += 4) {
            const float4 x = *reinterpret_cast<const float4*>(smem + OFF_Q + (e >> 5) * Q_BOX + swz(n, (e & 31) >> 2));
            const float4 y = *reinterpret_cast<const float4*>(&pr.fk[m][e]);
            a0 = fmaf(x.x, y.x, a0);
            a1 = fmaf(x.y, y.y, a1);
            a2 = fmaf(x.z, y.z, a2);
            a3 = fmaf(x.w, y.w, a3);
          }
          bf.A[j][n] = (a0 + a1) + (a2 + a3);
        }
      }
      sync_x();
      if (ok && !bad) {                         // four threads per node share the dot product with z (rows past N are zero)
        const int n = tid >> 2, part = tid & 3;
        float den = 0.f;
#pragma unroll
        for (int e = 32 * part; e < 32 * part + 32; e += 4) {
          const float4 x = *reinterpret_cast<const float4*>(smem + OFF_Q + (e >> 5) * Q_BOX + swz(n, (e & 31) >> 2));
          den = fmaf(x.x, pr.z[e], den);
          den = fmaf(x.y, pr.z[e + 1], den);
          den = fmaf(x.z, pr.z[e + 2], den);
          den = fmaf(x.w, pr.z[e + 3], den);
        }
        den += __shfl_xor_sync(0xffffffffu, den, 1);
        den += __shfl_xor_sync(0xffffffffu, den, 2);
        if (part == 0 && n < N) {
          for (int j = 0; j < pr.depth[n]; ++j) den += bf.A[j][n];
          bf.rden[n] = 1.f / (den + eps);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(bar[B_XDONE0 + (t & 1)]);    // unit t is ready for the product and for the epilogue
    }
  } else {
    // =============================== group Y: finish unit t (thread = channel c, 32 nodes per thread) ===============================
    const int wy = warp - 8;
    const int c = 32 * (wy & 3) + lane, n0 = 32 * (wy >> 2);
    bool ok = true;
    for (int t = 0; t < nloc; ++t) {
      const int u = (int)blockIdx.x + t * (int)gridDim.x;
      const Buf& bf = bufs[t & 1];
      ok = ok && mbar_wait(bar[B_XDONE0 + (t & 1)], (t >> 1) & 1, abort) && mbar_wait(bar[B_MMA0 + (t & 1)], (t >> 1) & 1, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (ok && bf.bad) {
        if (tid == kThreadsX) report(status, LA_ERR_BAD_TREE);
      } else if (ok && n0 < N) {               // warp-uniform
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const size_t base = (size_t)u * N * D;
        uint32_t acc[32];
        const uint32_t taddr = tmem + ((uint32_t)(32 * (wy & 3)) << 16) + (t & 1) * 64u + n0;
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
            "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
            "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
            : "=r"(acc[0]), "=r"(acc[1]), "=r"(acc[2]), "=r"(acc[3]), "=r"(acc[4]), "=r"(acc[5]), "=r"(acc[6]),
              "=r"(acc[7]), "=r"(acc[8]), "=r"(acc[9]), "=r"(acc[10]), "=r"(acc[11]), "=r"(acc[12]), "=r"(acc[13]),
              "=r"(acc[14]), "=r"(acc[15]), "=r"(acc[16]), "=r"(acc[17]), "=r"(acc[18]), "=r"(acc[19]), "=r"(acc[20]),
              "=r"(acc[21]), "=r"(acc[22]), "=r"(acc[23]), "=r"(acc[24]), "=r"(acc[25]), "=r"(acc[26]), "=r"(acc[27]),
              "=r"(acc[28]), "=r"(acc[29]), "=r"(acc[30]), "=r"(acc[31])
            : "r"(taddr)
            : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        // Walk the ancestor distance j in the outer loop: the value at distance j feeds both the tree term
        // (weight A[j][n]) and tap j of the unfolded convolution; behind the chain the taps read the committed
        // window.  Branch-free: weights are zero where a term does not apply.
        float conv[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) conv[i] = 0.f;
        const int jmax = max(bf.max_depth, W);
        for (int j = 0; j < jmax; ++j) {
          const float wj = j < W ? bf.w[j][c] : 0.f;
#pragma unroll
          for (int i = 0; i < 32; i += 4) {                  // four nodes per table load
            const float4 a4 = *reinterpret_cast<const float4*>(&bf.A[j][n0 + i]);
            const uint32_t r4 = *reinterpret_cast<const uint32_t*>(&bf.anc[j][n0 + i]);
            const float u0 = __bfloat162float(bf.vrows[r4 & 0xff][c]), u1 = __bfloat162float(bf.vrows[(r4 >> 8) & 0xff][c]);
            const float u2 = __bfloat162float(bf.vrows[(r4 >> 16) & 0xff][c]), u3 = __bfloat162float(bf.vrows[r4 >> 24][c]);
            acc[i] = __float_as_uint(fmaf(a4.x, u0, __uint_as_float(acc[i])));
            acc[i + 1] = __float_as_uint(fmaf(a4.y, u1, __uint_as_float(acc[i + 1])));
            acc[i + 2] = __float_as_uint(fmaf(a4.z, u2, __uint_as_float(acc[i + 2])));
            acc[i + 3] = __float_as_uint(fmaf(a4.w, u3, __uint_as_float(acc[i + 3])));
            conv[i] = fmaf(wj, u0, conv[i]);
            conv[i + 1] = fmaf(wj, u1, conv[i + 1]);
            conv[i + 2] = fmaf(wj, u2, conv[i + 2]);
            conv[i + 3] = fmaf(wj, u3, conv[i + 3]);
          }
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int n = n0 + i;
          if (n < N) o[base + (size_t)n * D + c] = __float2bfloat16_rn(fmaf(__uint_as_float(acc[i]), bf.rden[n], conv[i]));
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(bar[B_EPI0 + (t & 1)]);      // this copy of the tables and this accumulator may be reused
    }
  }

  // ---- teardown ----
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (ctl.abort) {
    if (tid == 0) report(status, LA_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(2000);   // bounded grace period for a copy still in flight
  }
  if (warp == kCtrlWarp) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) != cudaSuccess ||
        qr != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

}  // namespace vtc

cudaError_t launch_verify_tc(la_ctx* ctx, int B, int N, const void* q, const void* k, const void* v,
                             const int32_t* parent, const float* w, const la_state& st, void* o, cudaStream_t s,
                             bool* handled) {
  const la_config& c = ctx->cfg;
  *handled = false;
  if (c.io_dtype != LA_BF16 || c.d != vtc::D || c.conv_taps > vtc::kMaxTaps) return cudaSuccess;
  vtc::EncodeTiledFn fn = vtc::encode_fn();
  if (!fn) return cudaSuccess;
  const int BH = B * c.H;
  CUtensorMap ms;   // S viewed as [BH * 128 rows, 128 columns] fp32; boxes of 32 columns x 128 rows
  cuuint64_t dims[2] = {(cuuint64_t)vtc::D, (cuuint64_t)BH * vtc::D};
  cuuint64_t strides[1] = {(cuuint64_t)vtc::D * 4};
  cuuint32_t box[2] = {32, 128}, es[2] = {1, 1};
  if (fn(&ms, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, st.S, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
         CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) !=
      CUDA_SUCCESS)
    return cudaSuccess;
  auto kern = c.phi == LA_PHI_ELU1 ? vtc::verify_tc_kernel<LA_PHI_ELU1> : vtc::verify_tc_kernel<LA_PHI_RELU>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)vtc::kSmemBytes);
  if (e != cudaSuccess) return e;
  kern<<<dim3(std::min(BH, ctx->sm_count)), dim3(vtc::kThreads), vtc::kSmemBytes, s>>>(
      ms, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, parent, w, st.z,
      (const __nv_bfloat16*)st.win, (__nv_bfloat16*)o, ctx->d_status, c.H, N, c.conv_taps, c.eps, BH);
  ctx->launches += 1;
  *handled = true;
  return cudaGetLastError();
}

}  // namespace la
