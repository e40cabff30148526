// Draft-tree verification on the tensor cores (bf16 io, d = 128, N <= 64).
//
// Sec. 4.2 / Sec. 5.3: all N draft nodes of a sequence share the committed state and attend, among the draft
// tokens, to their ancestors and themselves only.  Per (sequence, head) unit everything that is a contraction
// runs as tcgen05.mma with the accumulators in TMEM:
//     P[n][m]    = phi(q_n) . phi(k_m)                              (bf16; 64 x 64 scores)
//     acc[c][n]  = sum_a S[a][c] phi(q_n)[a]                        (bf16; TMA brings the fp32 state into shared
//                                                                    memory, one warp group rounds it to bf16 in
//                                                                    the operand layout)
//     acc[c][n] += sum_m v_m[c] Pm[n][m]                            (bf16; Pm = P under the tree mask)
//     G_j[c][n]  = sum_m v_m[c] Sel_j[n][m]                         (bf16; Sel_j has a single one per row, at the
//                                                                    ancestor of n at distance j or at a row of the
//                                                                    committed window: an exact gather of the value
//                                                                    that tap j of the causal convolution reads)
// and the CUDA cores are left with phi, the tree walk, the mask, the denominators and
//     o[n][c] = acc[c][n] / (phi(q_n) . z + sum_m Pm[n][m] + eps) + sum_j w[j][c] G_j[c][n].
// Taps beyond the fourth (W > 4) are summed by the CUDA cores, from the same shared-memory copy of V and a table of
// the places they read, while the tensor cores work on the unit's products.  Nothing of the state is written.  CTAs are persistent: group X prepares
// unit t + 1 while group Y finishes unit t, and one thread feeds TMA and the tensor cores.
#include <cuda.h>

#include <algorithm>
#include <cstddef>

#include "la_common.cuh"

namespace la {
namespace vtc {

constexpr int D = 128, NMAX = LA_MAX_NODES;
constexpr int kMaxTaps = 4;                        // taps whose gathers run as tensor-core products
constexpr int kExtTaps = LA_MAX_TAPS - kMaxTaps;   // the others: gathered by the CUDA cores in the epilogue
constexpr int kThreadsX = 256, kThreadsY = 256, kCtrlWarp = 16, kTreeWarp = 17, kThreads = 576;
constexpr uint32_t S_BYTES = 128 * 128 * 4;        // the fp32 state of one unit, row-major
constexpr uint32_t SB_BOX = 128 * 128;             // 128 rows x 64 bf16
constexpr uint32_t Q_BOX = NMAX * 128;             // 64 rows x 64 bf16
constexpr uint32_t V_BOX = (NMAX + 32) * 128;      // 64 draft rows + 32 window rows (newest first) x 64 bf16
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t P_COL = 64, G_COL = 128;                // G_j at G_COL + 64 j
__host__ __device__ constexpr uint32_t acc_col(int t) { return (t & 1) ? 384u : 0u; }   // acc of unit t

// Small tables.  Those that group X writes and group Y reads exist twice (unit parity).
struct alignas(16) Tab {
  unsigned long long mask[2][NMAX];                // bit m of mask[n]: m is n or an ancestor of n
  float qz[2][NMAX];                               // phi(q_n) . z
  int bad[2];                                      // a parent index was out of range
  int pad0[2];
  float den_part[2][NMAX];                         // masked row sums of P, one per column half
  float rden[NMAX];                                // 1 / (denominator + eps)
  int par[NMAX];                                   // the parent array (private to the tree warp)
  unsigned short ext[2][kExtTaps][NMAX];           // where in a box of the V copy tap 4 + j of node n reads its row
                                                   // (row * 128 + ((row & 7) << 4); W > 4 only)
};
struct alignas(16) Ctl {
  unsigned long long bars[12];
  uint32_t tmem_base;
  int abort;
};
// XDONE comes as a pair indexed by the unit parity (phase t >> 1); every other barrier completes once per unit
// (phase t), and the protocol lets none complete again before the waiters of its previous phase have passed.
// XT (more than four taps only): group Y has taken the values of the later taps from the V copy and its tables.
enum { B_FULL_S = 0, B_FULL_V, B_XDONE0, B_XDONE1, B_SCONV, B_P, B_PS, B_SG, B_PMDONE, B_O, B_EPI, B_XT, kNumBars };
static_assert(kNumBars <= 12, "Ctl::bars");
constexpr uint32_t OFF_S = 0;                               // S as it lies in memory (fp32, rows = features)
constexpr uint32_t OFF_SB = OFF_S + S_BYTES;                // S as bf16: two boxes of 64 channels, rows = features
constexpr uint32_t OFF_QB = OFF_SB + 2 * SB_BOX;            // phi(Q) as bf16: two boxes of 64 features
constexpr uint32_t OFF_KB = OFF_QB + 2 * Q_BOX;             // phi(K) as bf16: likewise
constexpr uint32_t OFF_V = OFF_KB + 2 * Q_BOX;              // V: two boxes of 64 channels, rows = nodes, then window
constexpr uint32_t OFF_SEL = OFF_V + 2 * V_BOX;             // Sel_0 .. Sel_3 over the draft rows
constexpr uint32_t OFF_SELW = OFF_SEL + 4 * Q_BOX;          // row 64 j + n, column r: tap j of node n reads window row r
constexpr uint32_t OFF_PM = OFF_SELW + Q_BOX;               // masked scores, bf16
constexpr uint32_t OFF_TAB = OFF_PM + Q_BOX;
constexpr uint32_t OFF_CTL = OFF_TAB + (uint32_t)sizeof(Tab);
// Taps 4 .. W-1 of this unit's head, fp32 [W - 4][128 channels].
constexpr uint32_t OFF_WEXT = (OFF_CTL + (uint32_t)sizeof(Ctl) + 15u) & ~15u;
__host__ __device__ constexpr uint32_t smem_bytes(int W) { return OFF_WEXT + (W > kMaxTaps ? (uint32_t)(W - kMaxTaps) * D * 4 : 0u) + 1024; }
constexpr uint32_t kSmemBytes = smem_bytes(LA_MAX_TAPS);
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
static_assert(offsetof(Tab, rden) % 16 == 0, "rden is read four at a time");
static_assert(offsetof(Tab, ext) % 16 == 0, "the offsets of 8 nodes are read at a time");
static_assert(OFF_V % 1024 == 0 && V_BOX % 1024 == 0 && OFF_TAB % 16 == 0, "swizzled regions are 1024-byte aligned");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void sync_y() { asm volatile("bar.sync 2, 256;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 128-byte swizzle: byte offset of 16-byte chunk `cc` of row `row` inside a box with 128-byte rows.
__device__ __forceinline__ uint32_t swz(int row, int cc) { return (uint32_t)row * 128u + (uint32_t)((cc ^ (row & 7)) << 4); }
// Shared-memory matrix descriptor; layout 2 = 128-byte swizzle in 16-byte chunks, 0 = none (8 x 16-byte cores).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)layout << 61);
}
// Instruction descriptor: bf16 x bf16 with fp32 accumulate, M = 128, N = n; *_mn: the M (N) index is the contiguous
// one of that operand.
__host__ __device__ constexpr uint32_t idesc(bool a_mn, bool b_mn, uint32_t n = 64u) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((n >> 3) << 17) |
         ((128u >> 4) << 24);
}
__device__ __forceinline__ void mma(uint32_t d, uint64_t a, uint64_t b, uint32_t id, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d), "l"(a), "l"(b), "r"(id),
      "r"((uint32_t)accumulate)
      : "memory");
}
// The window selectors: 256 rows (64 j + n) x 16 columns, no swizzle: cores of 8 rows x 8 columns (128 bytes), the two
// cores of a row group side by side, row groups 256 bytes apart.
__device__ __forceinline__ uint32_t selw_offset(int row, int col) {
  return (uint32_t)(row >> 3) * 256u + (uint32_t)(col >> 3) * 128u + (uint32_t)(row & 7) * 16u + (uint32_t)(col & 7) * 2u;
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive TMEM columns of this thread's lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// phi on two packed bf16 values, in packed arithmetic; the results are bf16.  elu + 1:
// x + 1 where x > 0, 2^(x log2 e) elsewhere, merged with a lane mask.  ReLU: packed max.
// 8 consecutive TMEM columns of this thread's lane; the caller waits once for all the loads it has issued.
__device__ __forceinline__ void tmem_ld8_issue(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
template <int PHI> __device__ __forceinline__ uint32_t phi2(uint32_t u) {
  if (PHI == LA_PHI_ELU1) {
    uint32_t y, e, xp1, mask;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(y) : "r"(u), "r"(0x3fb93fb9u));        // log2(e) in bf16
    asm("ex2.approx.ftz.bf16x2 %0, %1;" : "=r"(e) : "r"(y));
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(xp1) : "r"(u), "r"(0x3f803f80u));
    asm("set.gt.u32.bf16x2 %0, %1, %2;" : "=r"(mask) : "r"(u), "r"(0u));
    return (xp1 & mask) | (e & ~mask);
  }
  uint32_t r;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(u), "r"(0u));
  return r;
}
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Persistent kernel: CTA i handles units i, i + gridDim.x, ...  Roles:
//   group X (warps 0-7)  unit t: phi(q), phi(k) as bf16 operands, phi(q) . z; rounds S to bf16;
//   warp 17              unit t: walks the tree; writes the tree masks, the selection matrices and the window rows;
//   warp 16 (one lane)   TMA of S and V; every tcgen05.mma;
//   group Y (warps 8-15) masks the scores, forms the denominators, and writes the outputs.
template <int PHI, bool EXT>   // EXT: more than kMaxTaps live taps
__global__ void __launch_bounds__(kThreads, 1)
verify_tc_kernel(const __grid_constant__ CUtensorMap ms, const __grid_constant__ CUtensorMap mv,
                 const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                 const int32_t* __restrict__ parent, const float* __restrict__ w, const float* __restrict__ z,
                 const __nv_bfloat16* __restrict__ win, __nv_bfloat16* __restrict__ o, int* status, int H, int N, int W,
                 float eps, int units) {
  extern __shared__ unsigned char smem_dyn[];
  // (an offset into the array rather than an integer cast: the compiler then knows that these are shared-memory
  // addresses: 32-bit arithmetic, ld.shared / st.shared)
  unsigned char* smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  Tab& tab = *reinterpret_cast<Tab*>(smem + OFF_TAB);
  Ctl& ctl = *reinterpret_cast<Ctl*>(smem + OFF_CTL);
  volatile int* abort = &ctl.abort;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nloc = (units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // units of this CTA
  uint32_t bar[kNumBars];
#pragma unroll
  for (int i = 0; i < kNumBars; ++i) bar[i] = smem_u32(&ctl.bars[i]);

  // ---- set-up: barriers, TMEM, the constant parts of the operands ----
  if (tid == 0) {
    mbar_init(bar[B_FULL_S], 1);
    mbar_init(bar[B_FULL_V], 1);
    mbar_init(bar[B_XDONE0], kThreadsX + 32);
    mbar_init(bar[B_XDONE1], kThreadsX + 32);
    mbar_init(bar[B_SCONV], kThreadsX);
    mbar_init(bar[B_P], 1);
    mbar_init(bar[B_PS], 1);
    mbar_init(bar[B_SG], 1);
    mbar_init(bar[B_PMDONE], kThreadsY);
    mbar_init(bar[B_O], 1);
    mbar_init(bar[B_EPI], kThreadsY);
    mbar_init(bar[B_XT], kThreadsY);
    ctl.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // selection matrices and masked scores start as zeros; so do the 16 window rows below the draft rows of V
  for (uint32_t i = tid; i < (OFF_TAB - OFF_SEL) / 16; i += kThreads)
    *reinterpret_cast<uint4*>(smem + OFF_SEL + i * 16) = make_uint4(0u, 0u, 0u, 0u);
  for (uint32_t i = tid; i < 2 * 32 * 128 / 16; i += kThreads)
    *reinterpret_cast<uint4*>(smem + OFF_V + (i >> 8) * V_BOX + NMAX * 128 + (i & 255) * 16) = make_uint4(0u, 0u, 0u, 0u);
  if (warp == kCtrlWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl.tmem_base;
  pdl_wait();                                // everything above touched shared memory and TMEM only
  pdl_trigger();

  if (warp == kCtrlWarp) {
    // =============================== TMA and the tensor cores (one lane) ===============================
    if (lane == 0) {
      auto load_s = [&](int t) {   // the committed state of unit t, 128 x 128 fp32 in one copy
        const int u = (int)blockIdx.x + t * (int)gridDim.x;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar[B_FULL_S]), "r"(S_BYTES) : "memory");
        asm volatile(
            "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
            ::"r"(sbase + OFF_S), "l"(&ms), "r"(0), "r"(u * D), "r"(bar[B_FULL_S])
            : "memory");
      };
      auto load_v = [&](int t) {   // the draft values of unit t: two boxes of 64 channels x 64 nodes (rows past N: zeros)
        const int u = (int)blockIdx.x + t * (int)gridDim.x;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar[B_FULL_V]), "r"(2 * Q_BOX) : "memory");
#pragma unroll
        for (int x = 0; x < 2; ++x)
          asm volatile(
              "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
              ::"r"(sbase + OFF_V + x * V_BOX), "l"(&mv), "r"(64 * x), "r"(0), "r"(u), "r"(bar[B_FULL_V])
              : "memory");
      };
      constexpr uint32_t kIdP = idesc(false, false), kIdV = idesc(true, false);
      load_s(0);
      load_v(0);
      for (int t = 0; t < nloc; ++t) {
        const uint32_t par = t & 1;
        if (!mbar_wait(bar[B_XDONE0 + par], (t >> 1) & 1, abort)) break;
        tc_fence_after();
        const bool good = tab.bad[par] == 0;
        if (good) {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {     // P[n][m]: 16 values of the feature index per step
            const uint32_t off = (ks >> 2) * Q_BOX + (ks & 3) * 32u;
            mma(tmem + P_COL, smem_desc(sbase + OFF_QB + off, 16u, 1024u, 2u), smem_desc(sbase + OFF_KB + off, 16u, 1024u, 2u),
                kIdP, ks > 0);
          }
        }
        mma_commit(bar[B_P]);
        if (!mbar_wait(bar[B_SCONV], par, abort)) break;   // the bf16 copy of S is in place, the fp32 one consumed
        if (t + 1 < nloc) load_s(t + 1);
        tc_fence_after();
        if (good) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)       // acc[c][n] = sum_a S[a][c] phi(q_n)[a]: 16 rows of S per step
            mma(tmem + acc_col(t), smem_desc(sbase + OFF_SB + kk * 2048u, SB_BOX, 1024u, 2u),
                smem_desc(sbase + OFF_QB + (kk >> 2) * Q_BOX + (kk & 3) * 32u, 16u, 1024u, 2u), kIdV, kk > 0);
        }
        mma_commit(bar[B_PS]);
        // G of unit t - 1 has been read (this unit's accumulator was last read two units ago)
        if (t >= 1 && !mbar_wait(bar[B_EPI], (t - 1) & 1, abort)) break;
        if (!mbar_wait(bar[B_FULL_V], par, abort)) break;
        tc_fence_after();
        if (good) {
          // G_j[c][n], the value tap j reads for node n, for all taps at once: the selection matrices lie one after
          // the other, so they form one operand of 64 W rows and the products land in 64 W consecutive columns
          const uint32_t idG = idesc(true, false, 64u * (uint32_t)min(W, kMaxTaps));
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)       // 16 draft rows per step
            mma(tmem + G_COL, smem_desc(sbase + OFF_V + kk * 2048u, V_BOX, 1024u, 2u),
                smem_desc(sbase + OFF_SEL + kk * 32u, 16u, 1024u, 2u), idG, kk > 0);
          if (W > 1)                           // the window rows
            mma(tmem + G_COL, smem_desc(sbase + OFF_V + NMAX * 128u, V_BOX, 1024u, 2u),
                smem_desc(sbase + OFF_SELW, 128u, 256u, 0u), idG, true);
        }
        mma_commit(bar[B_SG]);
        if (!mbar_wait(bar[B_PMDONE], par, abort)) break;
        tc_fence_after();
        if (good) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)       // acc[c][n] += sum_m v_m[c] Pm[n][m]
            mma(tmem + acc_col(t), smem_desc(sbase + OFF_V + kk * 2048u, V_BOX, 1024u, 2u),
                smem_desc(sbase + OFF_PM + kk * 32u, 16u, 1024u, 2u), kIdV, true);
        }
        mma_commit(bar[B_O]);
        if (!mbar_wait(bar[B_O], par, abort)) break;       // V has been read by the tensor cores
        // with more than four taps group Y reads V too
        if (EXT && !mbar_wait(bar[B_XT], par, abort)) break;
        if (t + 1 < nloc) load_v(t + 1);
      }
    }
  } else if (warp == kTreeWarp) {
    // =============================== the tree of unit t (one warp, nodes lane and lane + 32) ===============================
    for (int n = lane; n < NMAX; n += 32)                   // Sel_0 is the identity: tap 0 reads the node's own value
      *reinterpret_cast<unsigned short*>(smem + OFF_SEL + swz(n, n >> 3) + (n & 7) * 2) = 0x3F80;
    uint32_t prev[2][3];                                    // where the ones of this lane's nodes were put for the last unit
#pragma unroll
    for (int i = 0; i < 6; ++i) prev[i / 3][i % 3] = 0xffffffffu;
    bool ok = true;
    // the parents of this lane's two nodes, requested one unit ahead (right after the previous unit's walk)
    auto load_par = [&](int t2, int& p0, int& p1) {
      const int b2 = ((int)blockIdx.x + t2 * (int)gridDim.x) / H;
      p0 = lane < N ? parent[(size_t)b2 * N + lane] : -1;
      p1 = lane + 32 < N ? parent[(size_t)b2 * N + lane + 32] : -1;
    };
    int pn0 = -1, pn1 = -1;
    if (nloc > 0) load_par(0, pn0, pn1);
    for (int t = 0; t < nloc; ++t) {
      const int u = (int)blockIdx.x + t * (int)gridDim.x, par = t & 1;
      tab.par[lane] = pn0;
      tab.par[lane + 32] = pn1;
      uint32_t wv[6];                                       // the committed window (up to three rows: W <= 4) in flight early
#pragma unroll
      for (int i = 0; i < 6; ++i) {
        const int idx = lane + 32 * i;
        wv[i] = (!EXT && idx < 64 * (W - 1)) ? *reinterpret_cast<const uint32_t*>(win + (size_t)u * (W - 1) * D + 2 * idx)
                                                      : 0u;
      }
      // more than four taps: the window is up to 31 rows, 16 bytes per lane and load, 8 loads in flight at a time
      const uint4* wsrc = reinterpret_cast<const uint4*>(win + (size_t)u * (W - 1) * D);
      const int wtotal = EXT ? (W - 1) * 16 : 0;
      uint4 wq[8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (EXT && lane + 32 * i < wtotal) wq[i] = wsrc[lane + 32 * i];
      __syncwarp();
      // ---- each lane follows the parents of its two nodes (integer work), both chains in one loop so that their
      //      loads overlap.  With more than four taps the walk also notes where taps 4 .. W-1 read: the ancestor at
      //      distance j while the chain lasts, then rows of the committed window, newest first.  (This parity's table
      //      was last read two units ago, and the wait for that lies an iteration back.) ----
      unsigned long long mask[2] = {0ull, 0ull};
      int depth[2] = {0, 0}, anc[2][3] = {{0, 0, 0}, {0, 0, 0}};
      bool good = true;
      int mm[2] = {lane < N ? lane : -1, lane + 32 < N ? lane + 32 : -1};
      while (mm[0] >= 0 || mm[1] >= 0) {                    // every step lowers the live indices: at most N iterations
#pragma unroll
        for (int s2 = 0; s2 < 2; ++s2) {
          const int m = mm[s2];
          if (m >= 0) {
            mask[s2] |= 1ull << m;
            if (depth[s2] == 1) anc[s2][0] = m;
            if (depth[s2] == 2) anc[s2][1] = m;
            if (depth[s2] == 3) anc[s2][2] = m;
            if (EXT && depth[s2] >= kMaxTaps && depth[s2] < W)
              tab.ext[par][depth[s2] - kMaxTaps][lane + 32 * s2] = (unsigned short)(m * 128 + ((m & 7) << 4));
            ++depth[s2];
            const int p = tab.par[m];
            if (p < -1 || p >= m) {
              good = false;
              mm[s2] = -1;
            } else {
              mm[s2] = p;
            }
          }
        }
      }
      const bool bad_any = __any_sync(0xffffffffu, !good);
      if (EXT) {
#pragma unroll
        for (int s2 = 0; s2 < 2; ++s2) {
          const int n = lane + 32 * s2;
          // behind the chain: window rows; nodes past N are read like the others and never stored: any row will do
          for (int kk = max(n < N ? depth[s2] : 0, kMaxTaps); kk < W; ++kk) {
            const int row = n < N ? NMAX + kk - depth[s2] : 0;
            tab.ext[par][kk - kMaxTaps][n] = (unsigned short)(row * 128 + ((row & 7) << 4));
          }
        }
      }
      __syncwarp();
      if (t + 1 < nloc) load_par(t + 1, pn0, pn1);           // in flight during the waits and the writes below

      // ---- the selection matrices and the window rows of unit t - 1 have been consumed      __syncwarp();

      // ---- the selection matrices and the window rows of unit t - 1 have been consumed (and with them everything
      //      issued before: this parity's tables were last read two units ago) ----
      if (t >= 1) ok = ok && mbar_wait(bar[B_SG], (t - 1) & 1, abort);
      // with more than four taps group Y reads the window rows and the V copy of unit t - 1 as well
      if (EXT && t >= 1) ok = ok && mbar_wait(bar[B_XT], (t - 1) & 1, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        if (lane == 0) tab.bad[par] = bad_any ? 1 : 0;
#pragma unroll
        for (int s2 = 0; s2 < 2; ++s2) {
          const int n = lane + 32 * s2;
          tab.mask[par][n] = mask[s2];
#pragma unroll
          for (int j = 1; j < kMaxTaps; ++j) {              // one entry per (node, tap): clear the last unit's, set this unit's
            uint32_t& pv = prev[s2][j - 1];
            if (pv != 0xffffffffu) *reinterpret_cast<unsigned short*>(smem + pv) = 0;
            pv = 0xffffffffu;
            if (n < N && j < W) {
              if (j < depth[s2]) {
                const int a = anc[s2][j - 1];
                pv = OFF_SEL + j * Q_BOX + swz(n, a >> 3) + (a & 7) * 2;
              } else {                                      // behind the chain: the committed window, newest row first
                pv = OFF_SELW + selw_offset(64 * j + n, j - depth[s2]);
              }
              *reinterpret_cast<unsigned short*>(smem + pv) = 0x3F80;
            }
          }
        }
        // the window below the draft rows of both channel halves, newest row first: row NMAX + p holds the value
        // p + 1 steps behind the first draft token
        if (!EXT) {
#pragma unroll
          for (int i = 0; i < 6; ++i) {
            const int idx = lane + 32 * i, p = (W - 2) - (idx >> 6), c2 = (idx & 63) * 2;
            if (idx < 64 * (W - 1))
              *reinterpret_cast<uint32_t*>(smem + OFF_V + (c2 >> 6) * V_BOX + swz(NMAX + p, (c2 & 63) >> 3) + (c2 & 7) * 2) = wv[i];
          }
        } else {
          for (int base = 0; base < wtotal; base += 256) {
            if (base > 0) {
#pragma unroll
              for (int i = 0; i < 8; ++i)
                if (base + lane + 32 * i < wtotal) wq[i] = wsrc[base + lane + 32 * i];
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int idx = base + lane + 32 * i;          // row idx >> 4 of the window (oldest first), channels 8 (idx & 15) ...
              if (idx < wtotal)
                *reinterpret_cast<uint4*>(smem + OFF_V + ((idx & 15) >> 3) * V_BOX + swz(NMAX + (W - 2) - (idx >> 4), idx & 7)) = wq[i];
            }
          }
        }
      }
      proxy_fence();
      mbar_arrive(bar[B_XDONE0 + par]);
    }
  } else if (warp < 8) {
    // =============================== group X: phi(q), phi(k) and the bf16 copy of S of unit t ===============================
    bool ok = true;
    uint2 pq[8], pk[8];
    float4 z4;
    auto load_qk = [&](int t2) {                            // row n = warp + 8 it, 4 features per lane
      const int u = (int)blockIdx.x + t2 * (int)gridDim.x;
      const size_t base = (size_t)u * N * D;
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const int n = warp + 8 * it;
        pq[it] = pk[it] = make_uint2(0u, 0u);
        if (n < N) {
          pq[it] = *reinterpret_cast<const uint2*>(q + base + (size_t)n * D + lane * 4);
          pk[it] = *reinterpret_cast<const uint2*>(k + base + (size_t)n * D + lane * 4);
        }
      }
      z4 = *reinterpret_cast<const float4*>(z + (size_t)u * D + lane * 4);
    };
    load_qk(0);
    for (int t = 0; t < nloc; ++t) {
      const int par = t & 1;
      // ---- everything that needs no shared memory happens while the tensor cores still read unit t - 1 ----
      float part[8];                                         // this lane's share of phi(q_n) . z, n = warp + 8 it
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        if (warp + 8 * it < N) {                             // rows past N stay zero (phi(0) may be 1)
          pq[it] = make_uint2(phi2<PHI>(pq[it].x), phi2<PHI>(pq[it].y));
          pk[it] = make_uint2(phi2<PHI>(pk[it].x), phi2<PHI>(pk[it].y));
        }
        part[it] = fmaf(bf_lo(pq[it].x), z4.x, fmaf(bf_hi(pq[it].x), z4.y, fmaf(bf_lo(pq[it].y), z4.z, bf_hi(pq[it].y) * z4.w)));
      }
      // Sum over the lanes, eight rows at once: each exchange halves the rows a lane carries, so that after three of
      // them lane l holds row (l >> 2) & 7 and two plain steps finish the sum.
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const bool up = lane & 16;
        const float got = __shfl_xor_sync(0xffffffffu, up ? part[i] : part[i + 4], 16);
        part[i] = (up ? part[i + 4] : part[i]) + got;
      }
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const bool up = lane & 8;
        const float got = __shfl_xor_sync(0xffffffffu, up ? part[i] : part[i + 2], 8);
        part[i] = (up ? part[i + 2] : part[i]) + got;
      }
      float qz;
      {
        const bool up = lane & 4;
        const float got = __shfl_xor_sync(0xffffffffu, up ? part[0] : part[1], 4);
        qz = (up ? part[1] : part[0]) + got;
        qz += __shfl_xor_sync(0xffffffffu, qz, 2);
        qz += __shfl_xor_sync(0xffffffffu, qz, 1);
      }

      // ---- phi(Q), phi(K) and the bf16 copy of S of unit t - 1 have been consumed ----
      if (t >= 1) ok = ok && mbar_wait(bar[B_PS], (t - 1) & 1, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          const uint32_t offb = (lane >> 4) * Q_BOX + swz(warp + 8 * it, (lane & 15) >> 1) + (lane & 1) * 8;
          *reinterpret_cast<uint2*>(smem + OFF_QB + offb) = pq[it];
          *reinterpret_cast<uint2*>(smem + OFF_KB + offb) = pk[it];
        }
        if ((lane & 3) == 0) tab.qz[par][warp + 8 * ((lane >> 2) & 7)] = qz;
      }
      proxy_fence();
      mbar_arrive(bar[B_XDONE0 + par]);
      if (t + 1 < nloc) load_qk(t + 1);                      // in flight during the conversion below

      // ---- S of unit t has landed: round it to bf16 in the operand layout (rows = features, channels contiguous) ----
      ok = ok && mbar_wait(bar[B_FULL_S], par, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
#pragma unroll 8
        for (int it = 0; it < 16; ++it) {
          const int a = warp + 8 * it;                         // row a, channels 4 lane .. 4 lane + 3
          const float4 s4 = *reinterpret_cast<const float4*>(smem + OFF_S + a * 512 + lane * 16);
          *reinterpret_cast<uint2*>(smem + OFF_SB + (lane >> 4) * SB_BOX + swz(a, (lane & 15) >> 1) + (lane & 1) * 8) =
              make_uint2(pack2(s4.x, s4.y), pack2(s4.z, s4.w));
        }
      }
      proxy_fence();
      mbar_arrive(bar[B_SCONV]);
    }
  } else if (warp < 16) {
    // =============================== group Y: finish unit t ===============================
    const int ty = tid - kThreadsX, wy = warp - 8;
    const int q4 = wy & 3;                                   // this warp reads TMEM lanes 32 q4 .. 32 q4 + 31
    const int c = 32 * q4 + lane, n0 = 32 * (wy >> 2);       // epilogue: channel c, nodes n0 .. n0 + 31
    bool ok = true;
    for (int t = 0; t < nloc; ++t) {
      const int u = (int)blockIdx.x + t * (int)gridDim.x, h = u % H, par = t & 1;
      float wt[kMaxTaps];                                    // taps of channel c
#pragma unroll
      for (int j = 0; j < kMaxTaps; ++j) wt[j] = w[((size_t)h * D + c) * W + min(j, W - 1)];   // used where j < W

      if (EXT) {
        // The later taps of this head: its [128][W] block is read as it lies in memory, by all threads.  (Every
        // thread has left the last unit's sums, which read these; the barrier below publishes the new ones.)
        float* wext = reinterpret_cast<float*>(smem + OFF_WEXT);
        const float* wh = w + (size_t)h * D * W + kMaxTaps;
#pragma unroll 4
        for (int e = ty; e < D * (W - kMaxTaps); e += kThreadsY)   // tap 4 + (e >> 7) of channel e & 127
          wext[e] = wh[(e & (D - 1)) * W + (e >> 7)];
      }

      ok = ok && mbar_wait(bar[B_XDONE0 + par], (t >> 1) & 1, abort) && mbar_wait(bar[B_P], par, abort);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      const bool good = ok && tab.bad[par] == 0;
      // ---- scores under the tree mask: lane = node n, this warp's half of the columns m ----
      if (good && q4 < 2) {
        const int n = 32 * q4 + lane, hc = wy >> 2;
        uint32_t p[32];
        tmem_ld32(tmem + ((uint32_t)(32 * q4) << 16) + P_COL + 32u * hc, p);
        const uint32_t bits = (uint32_t)(tab.mask[par][n] >> (32 * hc));
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float x = (bits >> i) & 1u ? __uint_as_float(p[i]) : 0.f;
          sum += x;
          p[i] = __float_as_uint(x);
        }
        tab.den_part[hc][n] = hc == 0 ? sum + tab.qz[par][n] : sum;   // phi(q_n) . z joins the first half
#pragma unroll
        for (int cc = 0; cc < 4; ++cc)                       // 8 bf16 per 16-byte chunk of row n
          *reinterpret_cast<uint4*>(smem + OFF_PM + swz(n, 4 * hc + cc)) =
              make_uint4(pack2(__uint_as_float(p[8 * cc]), __uint_as_float(p[8 * cc + 1])),
                         pack2(__uint_as_float(p[8 * cc + 2]), __uint_as_float(p[8 * cc + 3])),
                         pack2(__uint_as_float(p[8 * cc + 4]), __uint_as_float(p[8 * cc + 5])),
                         pack2(__uint_as_float(p[8 * cc + 6]), __uint_as_float(p[8 * cc + 7])));
      }
      tc_fence_before();
      proxy_fence();
      mbar_arrive(bar[B_PMDONE]);
      sync_y();
      if (ty < NMAX) tab.rden[ty] = 1.f / (tab.den_part[0][ty] + tab.den_part[1][ty] + eps);
      float ex[EXT ? 32 : 1];                                // more than four taps: what taps 4 .. W-1 add to nodes n0 .. n0 + 31
      if (EXT) {
        // Each thread sums the later taps of its channel over its 32 nodes.  The values come straight from the
        // shared-memory copy of V (draft rows, then window rows), at the places the tree warp tabulated.  None of this
        // needs a product of this unit: it runs while the tensor cores work.
        // For these sums lane 4 g + o of a warp takes channels 4 g ... 4 g + 3 of the warp's 32 and nodes 8 o ... 8 o + 7 of
        // its 32: one 8-byte load brings four channels of a node's row, so a tap costs 8 loads per thread instead of
        // 32.  A 4 x 4 transpose inside each group of four lanes (two exchange steps) then hands every lane the sums
        // of its own channel for all 32 nodes, which is how the epilogue below holds them.
        const float* wext = reinterpret_cast<const float*>(smem + OFF_WEXT);
        ok = ok && mbar_wait(bar[B_FULL_V], par, abort);     // the draft rows of V have landed
        ok = __all_sync(0xffffffffu, ok);
#pragma unroll
        for (int i = 0; i < 32; ++i) ex[i] = 0.f;
        if (good && ok) {                                    // (the same for every lane of the warp)
          const int cb = 32 * q4 + (lane & ~3), o = lane & 3;             // first of the four channels; node octet
          const unsigned char* vq = smem + OFF_V + (cb >> 6) * V_BOX + (cb & 7) * 2;
          const uint32_t cx = (uint32_t)((cb & 63) >> 3) << 4;            // the channels' 16-byte piece, before the swizzle
#pragma unroll 1
          for (int j = kMaxTaps; j < W; ++j) {
            const float4 wj = *reinterpret_cast<const float4*>(wext + (j - kMaxTaps) * D + cb);
            const uint4 o4 = *reinterpret_cast<const uint4*>(&tab.ext[par][j - kMaxTaps][n0 + 8 * o]);   // 8 nodes
            const uint32_t offs[8] = {o4.x & 0xffffu, o4.x >> 16, o4.y & 0xffffu, o4.y >> 16,
                                      o4.z & 0xffffu, o4.z >> 16, o4.w & 0xffffu, o4.w >> 16};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint2 x = *reinterpret_cast<const uint2*>(vq + (offs[i] ^ cx));
              ex[i] = fmaf(wj.x, __uint_as_float(x.x << 16), ex[i]);
              ex[8 + i] = fmaf(wj.y, __uint_as_float(x.x & 0xffff0000u), ex[8 + i]);
              ex[16 + i] = fmaf(wj.z, __uint_as_float(x.y << 16), ex[16 + i]);
              ex[24 + i] = fmaf(wj.w, __uint_as_float(x.y & 0xffff0000u), ex[24 + i]);
            }
          }
          // ex[8 r + i]: channel cb + r, node 8 o + i  ->  ex[8 o' + i]: channel cb + o (this lane's own), node 8 o' + i
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float a0 = ex[i], a1 = ex[8 + i], a2 = ex[16 + i], a3 = ex[24 + i];
            const bool odd1 = o & 1, odd2 = o & 2;
            float t0 = __shfl_xor_sync(0xffffffffu, odd1 ? a0 : a1, 1);
            float t1 = __shfl_xor_sync(0xffffffffu, odd1 ? a2 : a3, 1);
            if (odd1) { a0 = t0; a2 = t1; } else { a1 = t0; a3 = t1; }
            t0 = __shfl_xor_sync(0xffffffffu, odd2 ? a0 : a2, 2);
            t1 = __shfl_xor_sync(0xffffffffu, odd2 ? a1 : a3, 2);
            if (odd2) { a0 = t0; a1 = t1; } else { a2 = t0; a3 = t1; }
            ex[i] = a0; ex[8 + i] = a1; ex[16 + i] = a2; ex[24 + i] = a3;
          }
        }
        mbar_arrive(bar[B_XT]);
      }

      ok = ok && mbar_wait(bar[B_O], par, abort);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      sync_y();
      if (good && n0 < N) {                                  // warp-uniform (good implies ok)
        const uint32_t lane_base = tmem + ((uint32_t)(32 * q4) << 16) + n0;
        const int odd = lane & 1;
        uint32_t pairs[EXT ? 1 : 16];                        // two adjacent channels of node n0 + 2 i + odd
        __nv_bfloat16* orow = o + ((size_t)u * N + n0 + odd) * D + (c - odd);
#pragma unroll
        for (int part = 0; part < 4; ++part) {               // 8 nodes at a time, all their TMEM loads in flight at once
          const int nb = n0 + 8 * part;
          uint32_t ra[8], rg[kMaxTaps][8];
          tmem_ld8_issue(lane_base + acc_col(t) + 8u * part, ra);
#pragma unroll
          for (int j = 0; j < kMaxTaps; ++j)
            if (j < W) tmem_ld8_issue(lane_base + G_COL + 64u * j + 8u * part, rg[j]);
          tmem_ld_wait();
          float out[8];
#pragma unroll
          for (int i = 0; i < 8; i += 4) {
            const float4 rd = *reinterpret_cast<const float4*>(&tab.rden[nb + i]);
            out[i] = __uint_as_float(ra[i]) * rd.x;
            out[i + 1] = __uint_as_float(ra[i + 1]) * rd.y;
            out[i + 2] = __uint_as_float(ra[i + 2]) * rd.z;
            out[i + 3] = __uint_as_float(ra[i + 3]) * rd.w;
          }
#pragma unroll
          for (int j = 0; j < kMaxTaps; ++j)
            if (j < W) {
#pragma unroll
              for (int i = 0; i < 8; ++i) out[i] = fmaf(wt[j], __uint_as_float(rg[j][i]), out[i]);
            }
          if (EXT) {                                         // taps beyond the fourth: summed above
#pragma unroll
            for (int i = 0; i < 8; ++i) out[i] += ex[8 * part + i];
          }
          // Two neighbouring lanes trade values so that each stores two adjacent channels of one node: the even
          // lane takes node nb + i, the odd lane node nb + i + 1.
#pragma unroll
          for (int i = 0; i < 8; i += 2) {
            const float give = odd ? out[i] : out[i + 1];
            const float got = __shfl_xor_sync(0xffffffffu, give, 1);
            const uint32_t pr = odd ? pack2(got, out[i + 1]) : pack2(out[i], got);
            if (EXT) {                                         // (the later taps' sums need the registers: store at once)
              if (nb + i + odd < N) *reinterpret_cast<uint32_t*>(orow + (size_t)(8 * part + i) * D) = pr;
            } else {
              pairs[4 * part + i / 2] = pr;
            }
          }
        }
        // the accumulators are free again before the outputs leave: the barrier's release would wait for the stores
        tc_fence_before();
        mbar_arrive(bar[B_EPI]);
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (!EXT && n0 + 2 * i + odd < N) *reinterpret_cast<uint32_t*>(orow + (size_t)(2 * i) * D) = pairs[i];
      } else {
        if (ok && !good && ty == 0) report(status, LA_ERR_BAD_TREE);
        tc_fence_before();
        mbar_arrive(bar[B_EPI]);
      }
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (ctl.abort) {
    if (tid == 0) report(status, LA_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(2000);   // bounded grace period for a copy still in flight
  }
  if (warp == kCtrlWarp) {
    __syncwarp();
    tc_fence_after();
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
  if (c.io_dtype != LA_BF16 || c.d != vtc::D) return cudaSuccess;
  vtc::EncodeTiledFn fn = vtc::encode_fn();
  if (!fn) return cudaErrorNotSupported;   // the driver cannot encode tensor maps: reported, never a silent slow path
  const int BH = B * c.H;
  const cuuint32_t es[3] = {1, 1, 1};
  CUtensorMap ms;   // S viewed as [BH * 128 rows, 128 columns] fp32; one unit per box, no swizzle
  {
    const cuuint64_t dims[2] = {(cuuint64_t)vtc::D, (cuuint64_t)BH * vtc::D};
    const cuuint64_t strides[1] = {(cuuint64_t)vtc::D * 4};
    const cuuint32_t box[2] = {128, 128};
    if (fn(&ms, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, st.S, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
           CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorNotSupported;
  }
  CUtensorMap mv;   // V viewed as [BH][N][128] bf16; boxes of 64 channels x 64 nodes (nodes past N read as zeros)
  {
    const cuuint64_t dims[3] = {(cuuint64_t)vtc::D, (cuuint64_t)N, (cuuint64_t)BH};
    const cuuint64_t strides[2] = {(cuuint64_t)vtc::D * 2, (cuuint64_t)N * vtc::D * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)vtc::NMAX, 1};
    if (fn(&mv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(v), dims, strides, box, es,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorNotSupported;
  }
  const bool elu = c.phi == LA_PHI_ELU1;
  auto kern = c.conv_taps <= vtc::kMaxTaps
                  ? (elu ? vtc::verify_tc_kernel<LA_PHI_ELU1, false> : vtc::verify_tc_kernel<LA_PHI_RELU, false>)
                  : (elu ? vtc::verify_tc_kernel<LA_PHI_ELU1, true> : vtc::verify_tc_kernel<LA_PHI_RELU, true>);
  const uint32_t smem = vtc::smem_bytes(c.conv_taps);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  e = launch_pdl(kern, dim3(std::min(BH, ctx->sm_count)), dim3(vtc::kThreads), smem, s, ms, mv,
                 (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, parent, w, (const float*)st.z,
                 (const __nv_bfloat16*)st.win, (__nv_bfloat16*)o, ctx->d_status, c.H, N, c.conv_taps, c.eps, BH);
  ctx->launches += 1;
  *handled = true;
  return e;
}

}  // namespace la
