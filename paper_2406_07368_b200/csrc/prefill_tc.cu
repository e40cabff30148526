// Chunkwise-parallel prefill on the 5th-generation tensor cores (bf16 io, d = 128).
//
// Sec. 4.1: the sequence is cut into non-overlapping groups; inside a group the causally
// masked product phi(Q) phi(K)^T V is formed in parallel, between groups only the cumulative
// sums S = sum phi(k) v^T and z = sum phi(k) are carried.  One CTA walks one (batch, head)
// chain in tiles of 128 tokens:
//     O = phi(Q) S_prev + (P o M) V,   den = phi(Q) . z_prev + rowsum(P o M),   S += phi(K)^T V,   z += colsum phi(K).
// The matrix products run on the tensor cores, and z rides along with them: V is extended by a column of ones
// ([S | z] += phi(K)^T [V | 1], a 16-column unswizzled operand block), and the K tile by a row that holds z_prev, so
// that the score product delivers phi(q) . z_prev as one more column of P.  The row sums of the masked P are taken
// by the threads that mask it.  Per tile n:
//
//   TMA      Q, K, V tiles (128 x 128 bf16, two 64-column boxes each, 128-byte swizzle)
//   group A  phi(Q) -> TMEM and phi(K) in place (packed bf16x2 arithmetic)
//   tcgen05  [P | phi(q) . z_prev] = phi(Q) [phi(K); z_prev]^T     (144 columns: 128 tokens, z_prev, 15 unused)
//            [S | z] += phi(K)^T [V | 1]               (fp32 in TMEM for the whole chain)
//            O = phi(Q) S_prev                         (S_prev is a bf16 copy in shared memory)
//   group A  phi on K of tile n+1 (K is double-buffered), while the tensor cores form the scores;
//            P -> causal mask, row sums (+ the z column), bf16 -> TMEM (the A operand of the next product);
//            the rows of v before the next tile -> a halo buffer;  S -> bf16 copy, z -> the K buffer of tile n+1
//   tcgen05  O += (P o M) V
//   group B  o = O / (den + eps) + conv(V) -> the tile's V buffer;  TMA stores it to global memory
// (More than 5 taps: a second epilogue, which forms the tap sums by channel pair and stages the outputs in the tile's
// K buffer; three-branch mode, GRP: the score product on the raw q and k and a causal softmax instead of the mask.)
//
// Four roles run concurrently: group A (warps 8-15), group B (warps 0-7), warp 16, whose elected lane issues
// every MMA and the Q loads, and warp 17, one lane of which issues the V loads and the output stores (a store has
// to have read its buffer before the buffer is reloaded: that wait must not hold up the products) and another the
// K reloads.  While group B finishes tile n, group A already works on tile n+1.  Every wait on an mbarrier is bounded; when one runs out the CTA
// records LA_ERR_TIMEOUT, stops issuing work, frees its TMEM and returns.
#include <cuda.h>

#include <algorithm>
#include <type_traits>

#include "la_common.cuh"

namespace la {
namespace tc {

constexpr int D = 128;
constexpr int TILE = 128;
constexpr int kThreadsB = 256;                     // group B: warps 0-7
constexpr int kThreadsA = 256;                     // group A: warps 8-15
constexpr int kCtrlWarp = 16, kCopyWarp = 17;
constexpr int kThreads = 576;
constexpr uint32_t BOX_BYTES = 128 * 128;          // 128 rows x 64 bf16
constexpr uint32_t TILE_BYTES = 2 * BOX_BYTES;
// A K buffer carries 8 more rows below the 128 token rows of each box, the first of which (row 128) holds z_prev as
// bf16: the score product runs with N = 144 and its column 128 is phi(q) . z_prev.  Columns 129-143 are never read,
// so rows 129-135 hold whatever they hold and rows 136-143 are simply the first kilobyte of what follows the box.
constexpr uint32_t KBOX_BYTES = (128 + 8) * 128;
constexpr uint32_t KBUF_BYTES = 2 * KBOX_BYTES;
// TMEM columns: P (144 fp32 columns: the scores and, in column 128, phi(q) . z_prev), O and S (128 each); phi(Q) as
// packed bf16 pairs (64 columns); a 16-column block whose first column is z.  phi(Q) is the A operand of two products and goes from the registers
// that computed it straight to TMEM, so that the Q buffer in shared memory is free for the next tile as soon as it
// has been read.  The masked P goes back as packed bf16 pairs
// into the columns its own fp32 values came from: each thread overwrites only columns of its own row that it has
// already read (row r, tokens 64 hf + 32 qq ... + 31 -> columns 64 hf + 16 qq ... + 15).
constexpr uint32_t P_COL = 0, QZ_COL = 128, O_COL = 144, S_COL = 272, FQ_COL = 400 /* 64 columns */, Z_COL = 464,
                   TMEM_COLS = 512;

// shared-memory map (offsets from a 1024-byte aligned base)
constexpr uint32_t OFF_Q = 0, OFF_V0 = TILE_BYTES, /* second V buffer at 2 * TILE_BYTES */ OFF_S = 3 * TILE_BYTES,
                   OFF_K0 = 4 * TILE_BYTES, OFF_K1 = OFF_K0 + KBUF_BYTES,
                   OFF_ONES = OFF_K1 + KBUF_BYTES, // [128 x 16] bf16, column 0 = 1: the extension of V
                   OFF_DEN = OFF_ONES + 4096,      // [2][2][128] fp32: halves of the denominator of tile n in slot n & 1
                   OFF_SMALL = OFF_DEN + 2048;

struct Small {
  unsigned long long bars[20];
  uint32_t tmem_base;
  int abort;
  int pad[2];
};
// full_*: TMA landed.  PHI / PDONE / SB: arrivals of group A.  EPI0 / EPI1: arrivals of group B (the accumulator
// has been read; tiles alternate between the two).
// STAGED0 / STAGED1: group B has written a tile's outputs into that V buffer (the control lane stores them).
// MMA_P / MMA_S / MMA_Q / MMA_O: tcgen05.commit after P; after [S|z] += phi(K)^T [V|1] (K buffer free);
// after O = phi(Q) S_prev; after O += P V (MMA_O0 / MMA_O1, tiles alternate).
// A barrier that one role waits on while another role can run a tile ahead exists once per tile parity, so that a
// waiter is never more than one phase behind.
enum { B_FULL_K0 = 0, B_FULL_V0 = 1, B_FULL_V1 = 2, B_MMA_P = 3, B_MMA_S = 4, B_MMA_O0 = 5, B_MMA_O1 = 6, B_PHI = 7,
       B_PDONE = 8, B_SB = 9, B_EPI0 = 10, B_EPI1 = 11, B_MMA_Q = 12, B_FULL_Q = 13, B_FULL_K1 = 14, B_STAGED0 = 15,
       B_STAGED1 = 16, B_HALO = 17, kNumBars = 18 };

__host__ __device__ constexpr uint32_t off_w() { return OFF_SMALL + (uint32_t)((sizeof(Small) + 15) / 16 * 16); }
__host__ __device__ inline uint32_t off_halo(int W) { return off_w() + (uint32_t)W * D * 4; }
// Three halo buffers (the rows of v before a tile, for the convolution).  Where group B fills them itself, tile n reads
// buffer n & 1 and fills the other; where group A fills them (short windows of the exact layer), tile n reads buffer
// n % 3 and group A fills (n + 1) % 3 meanwhile, which the epilogue of tile n - 1 no longer reads.
__host__ __device__ inline uint32_t smem_bytes(int W) { return off_halo(W) + 3u * (uint32_t)(W > 1 ? W - 1 : 1) * D * 2 + 1024; }
// The three-branch mode keeps 4 KB more behind the halo rows: z before the tile as fp32 [128], the halves of
// phi(q) . z [2][128], and each half-row's running maximum and sum of the softmax [2][128] x 2.
constexpr uint32_t kGrpScratch = 4096;
// The epilogue for longer tap windows ("long" below) keeps the taps padded with zeros to whole groups of 8 and ONE
// halo buffer, updated in place, of as many rows as the padded taps reach back (the rows before the window stay 0).
__host__ __device__ inline uint32_t long_taps(int W) { return ((uint32_t)W + 7u) & ~7u; }
__host__ __device__ inline uint32_t off_halo_long(int W) { return off_w() + long_taps(W) * D * 4; }
__host__ __device__ inline uint32_t smem_bytes_long(int W) { return off_halo_long(W) + (long_taps(W) - 1) * D * 2 + 1024; }
__host__ __device__ inline uint32_t off_grp(int W, bool lng = false) {
  return ((lng ? smem_bytes_long(W) : smem_bytes(W)) - 1024 + 15u) & ~15u;
}
__host__ __device__ inline uint32_t smem_bytes_grp(int W, bool lng = false) { return off_grp(W, lng) + kGrpScratch + 1024; }
// Which windows take the long epilogue: above 5 taps it is the faster of the two (measured on 128 chains of 2048
// tokens: 6 taps 126 us either way, 8 taps 132 against 154 us, 16 taps 126 against 254, 32 taps 162 against 686).
// The three-branch mode compiles the short epilogue for 3 taps only.
inline bool long_epilogue(int W, bool grouped = false) { return grouped ? W != 3 : W > 5; }

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
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void sync_group_b() { asm volatile("bar.sync 2, 256;" ::: "memory"); }
__device__ __forceinline__ void sync_group_a() { asm volatile("bar.sync 5, 256;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void sync_half_b(int hf) {
  if (hf) asm volatile("bar.sync 4, 128;" ::: "memory");
  else asm volatile("bar.sync 3, 128;" ::: "memory");
}

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
// The same with the A operand read from TMEM (rows in lanes, two bf16 per 32-bit column).
__device__ __forceinline__ void mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, bool acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"((uint32_t)acc)
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

__device__ __forceinline__ uint32_t tmem_ld1(uint32_t taddr) {
  uint32_t v;
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(v) : "r"(taddr) : "memory");
  return v;
}
__device__ __forceinline__ void tmem_st1(uint32_t taddr, uint32_t v) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%0], {%1};" ::"r"(taddr), "r"(v) : "memory");
}
#define LA_TMEM_ST16(taddr, r)                                                                                   \
  asm volatile(                                                                                                  \
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "                                                            \
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"                                 \
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),      \
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])             \
      : "memory")

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---- descriptors ----------------------------------------------------------------------------
// Shared-memory matrix descriptor: start address, leading and stride byte offsets (16-byte units),
// descriptor version 1, layout type (2 = 128-byte swizzle, 0 = no swizzle).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)layout << 61);
}
// Operand whose contraction index runs along the 128-byte rows (rows = M or N): step ks covers 16 elements.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t tile, int ks) {
  return smem_desc(tile + (uint32_t)(ks >> 2) * BOX_BYTES + (uint32_t)(ks & 3) * 32u, 16u, 1024u, 2u);
}
// Operand whose contraction index runs along the tile rows (rows = K, 128-byte rows hold M or N): step ks
// covers 16 rows; the two 64-element column boxes are BOX_BYTES apart.
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t tile, int ks) {
  return smem_desc(tile + (uint32_t)ks * 2048u, BOX_BYTES, 1024u, 2u);
}
// The 16-column extensions ([128 rows = K] x [16 = N], no swizzle): 8 x 8 cores of 128 bytes, the two cores of
// one 8-row group side by side (stride 128 B along N), 8-row groups 256 B apart (stride along K).
__device__ __forceinline__ uint64_t desc_ext(uint32_t tile, int ks) {
  return smem_desc(tile + (uint32_t)ks * 512u, 256u, 128u, 0u);
}
__device__ __forceinline__ uint32_t ext_offset(int k, int n) {   // byte offset of element (k, n) in such a block
  return (uint32_t)(k >> 3) * 256u + (uint32_t)(n >> 3) * 128u + (uint32_t)(k & 7) * 16u + (uint32_t)(n & 7) * 2u;
}
// The same descriptors split into their two 32-bit words: the steps of a product differ only in the start-address
// field of the low word (by a constant, and the field cannot overflow below 256 KB), so the issuing lane forms the
// words of step 0 once per tile and adds a constant per step.
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes) {
  return ((addr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
constexpr uint32_t kDescHiSw128 = ((1024u >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);   // SBO 1024, version 1, 128-byte swizzle
__host__ __device__ constexpr uint32_t kstep_kmajor(int ks, uint32_t box = BOX_BYTES) { return ((uint32_t)(ks >> 2) * box + (uint32_t)(ks & 3) * 32u) >> 4; }
__host__ __device__ constexpr uint32_t kstep_mnmajor(int ks) { return ((uint32_t)ks * 2048u) >> 4; }
__device__ __forceinline__ uint64_t desc64(uint32_t lo) { return ((uint64_t)kDescHiSw128 << 32) | lo; }
// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = n.
__host__ __device__ constexpr uint32_t idesc(bool a_mn, bool b_mn, uint32_t n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// ---- bf16 packing ------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float lo_f(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float hi_f(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// phi on two packed bf16 values, entirely in packed arithmetic.  elu+1: x + 1 where x > 0 (one correctly
// rounded bf16 addition), 2^(x log2 e) elsewhere; the two are merged with a lane mask.  The exponent argument is
// formed by one fused multiply (x * log2e_hi + x * log2e_lo would not help: the product is rounded to bf16
// either way), so exp(x) carries a relative error of about |x| 2^-9 on top of the bf16 rounding of the result --
// below one bf16 ulp for |x| < 1, and in absolute terms largest where exp(x) is close to 1.  ReLU: packed max.
template <int PHI> __device__ __forceinline__ uint32_t phi2(uint32_t u) {
  if (PHI == LA_PHI_ELU1) {
    uint32_t y, e, xp1, mask;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(y) : "r"(u), "r"(0x3fb93fb9u));        // log2(e) = 1.4453 in bf16
    asm("ex2.approx.ftz.bf16x2 %0, %1;" : "=r"(e) : "r"(y));
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(xp1) : "r"(u), "r"(0x3f803f80u));
    asm("set.gt.u32.bf16x2 %0, %1, %2;" : "=r"(mask) : "r"(u), "r"(0u));
    return (xp1 & mask) | (e & ~mask);
  }
  uint32_t r;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(u), "r"(0u));
  return r;
}
template <int PHI> __device__ __forceinline__ uint4 phi8(uint4 u) {
  return make_uint4(phi2<PHI>(u.x), phi2<PHI>(u.y), phi2<PHI>(u.z), phi2<PHI>(u.w));
}

// Byte offset of 16-byte chunk `cc` (0..7) of row `row` inside one 128-byte-swizzled box.
__device__ __forceinline__ uint32_t swz(int row, int cc) { return (uint32_t)row * 128u + (uint32_t)((cc ^ (row & 7)) << 4); }

// ---- the kernel ------------------------------------------------------------------------------------
// Convolution part of the epilogue for one 8-channel chunk: acc[e] += sum_t w[t][ch] v_{row-t}[ch], two channels per
// packed fp32 multiply-add (each half is the IEEE fused multiply-add of the scalar instruction).
__device__ __forceinline__ float2 bf2(uint32_t u) { return make_float2(lo_f(u), hi_f(u)); }
template <int WT>
__device__ __forceinline__ void conv8(float2* acc, int W, int r, int cc, int ch0, const unsigned char* Vbox,
                                      const __nv_bfloat16* halo, const float* wsm) {
  const int taps = WT > 0 ? WT : W;
#pragma unroll
  for (int t = 0; t < taps; ++t) {
    const int row = r - t;
    uint4 u;
    if (row >= 0) u = *reinterpret_cast<const uint4*>(Vbox + swz(row, cc));
    else u = *reinterpret_cast<const uint4*>(halo + (W - 1 + row) * D + ch0);
    const float4 w0 = *reinterpret_cast<const float4*>(wsm + t * D + ch0);
    const float4 w1 = *reinterpret_cast<const float4*>(wsm + t * D + ch0 + 4);
    acc[0] = __ffma2_rn(make_float2(w0.x, w0.y), bf2(u.x), acc[0]);
    acc[1] = __ffma2_rn(make_float2(w0.z, w0.w), bf2(u.y), acc[1]);
    acc[2] = __ffma2_rn(make_float2(w1.x, w1.y), bf2(u.z), acc[2]);
    acc[3] = __ffma2_rn(make_float2(w1.z, w1.w), bf2(u.w), acc[3]);
  }
}

// Long-window epilogue: one thread owns a pair of channels and 32 consecutive rows of the tile, in four blocks of 8.
// conv_block adds one group of 8 taps to the 8 sums of block BLK: the 15 rows of v that those taps reach are each
// read once, as one packed pair, and feed up to 8 of the sums.  Where the rows come from is fixed at compile time:
//   ALL_V  the V buffer: pg[k] = the thread's column at (its first row - 8 g), for rows = k mod 8 (the swizzle)
//   ALL_H  the halo column: hq = its row 8 (BLK - g) - 7
//   MIXED  (g = BLK, first 32 rows of the tile) rows -7 ... -1 from the halo (hq = its row -7), rows 0 ... 7 from V
// so that every load is one instruction with an immediate offset.
template <int I, int N, typename F>
__device__ __forceinline__ void static_for(F&& f) {           // f(integral_constant<int, I>) ... for I, I + 1, ..., N - 1
  if constexpr (I < N) {
    f(std::integral_constant<int, I>{});
    static_for<I + 1, N>(f);
  }
}
enum { ALL_V = 0, MIXED = 1, ALL_H = 2 };
// (Shared-memory addresses as 32-bit numbers and explicit ld.shared / st.shared: one register per address.)
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ float2 lds_f2(uint32_t a) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }
template <int BLK, int KIND>
__device__ __forceinline__ void conv_block(float2 (&acc)[8], uint32_t wtap, const uint32_t (&pg)[8], uint32_t hq) {
  float2 wg[8];
  static_for<0, 8>([&](auto tc_) {
    constexpr int t = decltype(tc_)::value;
    wg[t] = lds_f2(wtap + t * (D * 4));
  });
  static_for<0, 15>([&](auto ic) {
    constexpr int i = decltype(ic)::value;
    uint32_t u;
    if constexpr (KIND == ALL_V) {
      constexpr int rel = 8 * BLK - 7 + i;        // row, from the thread's first row, before the 8 g rows of the group
      u = lds32(pg[rel & 7] + rel * 128);
    } else if constexpr (KIND == ALL_H || i < 7) {
      u = lds32(hq + i * (D * 2));
    } else {
      u = lds32(pg[i - 7] + (i - 7) * 128);
    }
    const float2 x = bf2(u);
    static_for<0, 8>([&](auto tc_) {
      constexpr int tau = decltype(tc_)::value;   // tap (within the group) that links input row i to sum jj
      constexpr int jj = i - 7 + tau;
      if constexpr (jj >= 0 && jj < 8) acc[jj] = __ffma2_rn(wg[tau], x, acc[jj]);
    });
  });
}
// All tap groups of block BLK (rows 8 BLK ... 8 BLK + 7 of the thread), then the sums are added to the attention
// term that waits in the output tile.  FIRST: the thread owns the first 32 rows of the tile (rows before them
// come from the halo, hend = the halo column just past its last row).
template <int BLK, bool FIRST>
__device__ __forceinline__ void conv_rows(uint32_t wcol, const uint32_t (&pv)[8], uint32_t sthr, int cc, uint32_t hend, int ngroups) {
  float2 acc[8];
#pragma unroll
  for (int jj = 0; jj < 8; ++jj) acc[jj] = make_float2(0.f, 0.f);
#pragma unroll 1
  for (int g = 0; g < ngroups; ++g) {
    const uint32_t wtap = wcol + g * (8 * D * 4);
    if (!FIRST || g < BLK) {
      uint32_t pg[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) pg[k] = pv[k] - g * 1024;
      conv_block<BLK, ALL_V>(acc, wtap, pg, 0u);
    } else if (g == BLK) {
      conv_block<BLK, MIXED>(acc, wtap, pv, hend - 7 * (D * 2));
    } else {
      conv_block<BLK, ALL_H>(acc, wtap, pv, hend + (8 * (BLK - g) - 7) * (D * 2));
    }
  }
  uint32_t lav[8];                                // the attention terms of the 8 rows, all loads in flight at once
#pragma unroll
  for (int jj = 0; jj < 8; ++jj) lav[jj] = lds32(sthr + (8 * BLK + jj) * 128 + ((cc ^ jj) << 4));
#pragma unroll
  for (int jj = 0; jj < 8; ++jj) {
    const float2 la = bf2(lav[jj]);
    sts32(sthr + (8 * BLK + jj) * 128 + ((cc ^ jj) << 4), pack2(acc[jj].x + la.x, acc[jj].y + la.y));
  }
}

__device__ __forceinline__ uint4 pack8(const uint32_t* v) {
  return make_uint4(pack2(__uint_as_float(v[0]), __uint_as_float(v[1])), pack2(__uint_as_float(v[2]), __uint_as_float(v[3])),
                    pack2(__uint_as_float(v[4]), __uint_as_float(v[5])), pack2(__uint_as_float(v[6]), __uint_as_float(v[7])));
}

// GRP: the three-branch block of Sec. 4.1 with the group equal to the 128-token tile: the score product runs on the raw
// q and k and its rows go through a causal softmax (left branch); the products with the state of the earlier tiles are
// the group-exclusive linear attention (middle branch: there is no intra-tile linear term); both land in one
// accumulator, the probabilities pre-scaled by (phi(q).z_prev + eps) / alpha so that one row factor finishes both.
template <int PHI, int WT, bool GRP = false>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
                  const __grid_constant__ CUtensorMap mv, const __grid_constant__ CUtensorMap mo,
                  const float* __restrict__ w, float* __restrict__ S, float* __restrict__ z,
                  __nv_bfloat16* __restrict__ win, int64_t* __restrict__ pos,
                  int* status, int H, int Ttot, int W, float eps, int init, int nseg,
                  int seg_len, float* __restrict__ S_fin, float* __restrict__ z_fin, float alpha, float sm_scale,
                  int tstep) {
  extern __shared__ unsigned char smem_dyn[];
  // (an offset into the array rather than an integer cast: the compiler then knows that these are shared-memory
  // addresses: 32-bit arithmetic, ld.shared / st.shared)
  unsigned char* smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  Small& sm = *reinterpret_cast<Small*>(smem + OFF_SMALL);
  constexpr bool LONG = WT < 0;                  // the epilogue for longer tap windows
  constexpr bool HALO_A = !GRP && WT > 0;        // group A copies the rows before the next tile aside (it has the time)
  float* wsm = reinterpret_cast<float*>(smem + off_w());                       // [W][128] ([W up to a multiple of 8][128] if LONG)
  // two halo buffers [W-1][128], oldest row first: tile n reads buffer n&1 and writes buffer (n+1)&1 (LONG: one buffer)
  __nv_bfloat16* halo0 = reinterpret_cast<__nv_bfloat16*>(smem + (LONG ? off_halo_long(W) : off_halo(W)));
  const int halo_elems = (W > 1 ? W - 1 : 1) * D;
  volatile int* abort = &sm.abort;
  // three-branch mode only: z before the tile (fp32), the halves of phi(q) . z, the halves of the softmax statistics
  float* zs = reinterpret_cast<float*>(smem + off_grp(W, LONG));               // [128]
  float* dgh = zs + D;                                                         // [2][128]
  float2* mlh = reinterpret_cast<float2*>(dgh + 2 * D);                        // [2][128] (max, sum)
  const bool use_glob = GRP && alpha != 0.f;     // alpha = 0: the global branch is switched off altogether

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // A launch covers BH chains cut into nseg segments of seg_len tokens (nseg = 1: whole chains).  Unit u owns
  // tokens [y0, y0 + T) of chain bh; state, window and z of a unit are addressed by u.
  const int u = blockIdx.x, bh = u / nseg, h = bh % H;
  const int y0 = (u % nseg) * seg_len, T = min(seg_len, Ttot - y0);
  // tstep: tokens per tile, 128 except for three-branch groups shorter than that, which take one partly filled tile
  // each (the TMA boxes are then tstep rows high; the rows below hold zeros or values that the causal mask discards).
  const int nchunks = (T + tstep - 1) / tstep;
  const uint32_t tile_tx = (uint32_t)tstep * 256u;            // bytes a tile's two boxes bring
  const uint32_t bar0 = smem_u32(&sm.bars[0]);    // barrier i lives at bar0 + 8 i

  // ---- set-up ----
  if (tid == 0) {
    mbar_init((bar0 + 8u * (B_FULL_K0)), 1);
    mbar_init((bar0 + 8u * (B_FULL_K1)), 1);
    mbar_init((bar0 + 8u * (B_FULL_Q)), 1);
    mbar_init((bar0 + 8u * (B_FULL_V0)), 1);
    mbar_init((bar0 + 8u * (B_FULL_V1)), 1);
    mbar_init((bar0 + 8u * (B_MMA_P)), 1);
    mbar_init((bar0 + 8u * (B_MMA_S)), 1);
    mbar_init((bar0 + 8u * (B_MMA_O0)), 1);
    mbar_init((bar0 + 8u * (B_MMA_O1)), 1);
    mbar_init((bar0 + 8u * (B_PHI)), kThreadsA);
    mbar_init((bar0 + 8u * (B_PDONE)), kThreadsA);
    mbar_init((bar0 + 8u * (B_SB)), kThreadsA);
    mbar_init((bar0 + 8u * (B_EPI0)), kThreadsB);
    mbar_init((bar0 + 8u * (B_EPI1)), kThreadsB);
    mbar_init((bar0 + 8u * (B_MMA_Q)), 1);
    mbar_init((bar0 + 8u * (B_STAGED0)), kThreadsB);
    mbar_init((bar0 + 8u * (B_STAGED1)), kThreadsB);
    mbar_init((bar0 + 8u * (B_HALO)), kThreadsA);
    sm.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kCtrlWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int idx = tid; idx < (LONG ? (int)long_taps(W) : W) * D; idx += kThreads)
    wsm[idx] = idx < W * D ? w[((size_t)h * D + (idx % D)) * W + idx / D] : 0.f;
  if (LONG) {                                    // [long_taps - 1][128]: zeros, then the W-1 rows of the window
    const int lead = ((int)long_taps(W) - W) * D;
    for (int idx = tid; idx < ((int)long_taps(W) - 1) * D; idx += kThreads)
      halo0[idx] = init && idx >= lead ? win[(size_t)u * (W - 1) * D + idx - lead] : __float2bfloat16_rn(0.f);
  } else
  for (int idx = tid; idx < (W - 1) * D; idx += kThreads)
    halo0[idx] = init ? win[(size_t)u * (W - 1) * D + idx] : __float2bfloat16_rn(0.f);
  float* denbuf = reinterpret_cast<float*>(smem + OFF_DEN);
  for (int idx = tid; idx < 4096 / 16; idx += kThreads)                        // the 16-column block of ones <- 0
    reinterpret_cast<uint4*>(smem + OFF_ONES)[idx] = make_uint4(0u, 0u, 0u, 0u);
  if (GRP && tstep < TILE) {                                                   // partly filled tiles: rows tstep-127 of V <- 0
    const int per_box = (TILE - tstep) * 8;                                    // 16-byte pieces per box
    for (int idx = tid; idx < 4 * per_box; idx += kThreads)
      reinterpret_cast<uint4*>(smem + OFF_V0 + (idx / per_box) * BOX_BYTES + tstep * 128)[idx % per_box] = make_uint4(0u, 0u, 0u, 0u);
  }
  for (int idx = tid; idx < 4 * 1024 / 16; idx += kThreads)                    // rows 128-135 of the four K boxes <- 0
    reinterpret_cast<uint4*>(smem + OFF_K0 + (idx >> 6) * KBOX_BYTES + BOX_BYTES)[idx & 63] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  if (tid < TILE) {
    *reinterpret_cast<__nv_bfloat16*>(smem + OFF_ONES + ext_offset(tid, 0)) = __float2bfloat16_rn(1.f);
    if (GRP) zs[tid] = init ? z[(size_t)u * D + tid] : 0.f;
    else if (init)                                // z before tile 0: row 128 of the first K buffer (feature tid)
      *reinterpret_cast<__nv_bfloat16*>(smem + OFF_K0 + (tid >> 6) * KBOX_BYTES + BOX_BYTES + (tid & 63) * 2) =
          __float2bfloat16_rn(z[(size_t)u * D + tid]);
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == kCtrlWarp) {
    // =============================== MMA issue, the Q and K loads (one lane) ===============================
    if (lane == 0) {
      bool ok = true;
      mbar_expect_tx((bar0 + 8u * (B_FULL_Q)), tile_tx);
      tma_load(sbase + OFF_Q, &mq, 0, y0, bh, (bar0 + 8u * (B_FULL_Q)));
      tma_load(sbase + OFF_Q + BOX_BYTES, &mq, 64, y0, bh, (bar0 + 8u * (B_FULL_Q)));
      for (int n = 0; n < nchunks; ++n) {
        const uint32_t par = n & 1;
        const uint32_t vbuf = sbase + OFF_V0 + par * TILE_BYTES;
        const uint32_t kbuf = sbase + (par ? OFF_K1 : OFF_K0);
        const bool has_state = init || n > 0;
        // low descriptor words of step 0: K read along its rows (K-major), K, V and the S copy down their rows
        const uint32_t k_km = desc_lo(kbuf, 16u);
        const uint32_t k_mn = desc_lo(kbuf, KBOX_BYTES), v_mn = desc_lo(vbuf, BOX_BYTES), s_mn = desc_lo(sbase + OFF_S, BOX_BYTES);
        if (GRP) {
          // scores of the raw q and k, both operands from shared memory as TMA delivered them; group A applies phi
          // only once this product is complete
          ok = mbar_wait((bar0 + 8u * (B_FULL_Q)), par, abort) &&
               mbar_wait((bar0 + 8u * (par ? B_FULL_K1 : B_FULL_K0)), (n >> 1) & 1, abort);
          if (!ok) break;
          const uint32_t q_km = desc_lo(sbase + OFF_Q, 16u);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            mma_bf16(tmem + P_COL, desc64(q_km + kstep_kmajor(ks)), desc64(k_km + kstep_kmajor(ks, KBOX_BYTES)),
                     idesc(false, false, 128), ks > 0);
          mma_commit((bar0 + 8u * (B_MMA_P)));
        }
        ok = mbar_wait((bar0 + 8u * (B_PHI)), par, abort);   // phi(Q) of tile n is in TMEM, phi(K) in place
        if (!ok) break;
        tc_fence_after();
        // The Q buffer has been read by then (phi(Q) lives in TMEM): its reload, which sets the pace, goes out first.
        if (n + 1 < nchunks) {
          mbar_expect_tx((bar0 + 8u * (B_FULL_Q)), tile_tx);
          tma_load(sbase + OFF_Q, &mq, 0, y0 + (n + 1) * tstep, bh, (bar0 + 8u * (B_FULL_Q)));
          tma_load(sbase + OFF_Q + BOX_BYTES, &mq, 64, y0 + (n + 1) * tstep, bh, (bar0 + 8u * (B_FULL_Q)));
        }
        if (!GRP) {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)   // [P | phi(q).z_prev] = phi(Q) [phi(K); z_prev]^T; 16 channels of phi(Q) = 8 columns
            mma_bf16_ts(tmem + P_COL, tmem + FQ_COL + 8 * ks, desc64(k_km + kstep_kmajor(ks, KBOX_BYTES)),
                        idesc(false, false, 144), ks > 0);
          mma_commit((bar0 + 8u * (B_MMA_P)));
        }
        // The state update needs nothing from the previous tile's epilogue: it fills the time until that epilogue
        // has read the accumulator.
        ok = mbar_wait((bar0 + 8u * (B_FULL_V0 + par)), (n >> 1) & 1, abort);
        if (!ok) break;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {     // [S | z] += phi(K)^T [V | 1]
          const uint64_t kd = desc64(k_mn + kstep_mnmajor(ks));
          mma_bf16(tmem + S_COL, kd, desc64(v_mn + kstep_mnmajor(ks)), idesc(true, true, 128), has_state || ks > 0);
          mma_bf16(tmem + Z_COL, kd, desc_ext(sbase + OFF_ONES, ks), idesc(true, true, 16), has_state || ks > 0);
        }
        mma_commit((bar0 + 8u * (B_MMA_S)));
        // the bf16 copy of S before tile n is complete after n + 1 arrivals; the accumulator is free once the
        // epilogue of tile n-1 has read it
        ok = mbar_wait((bar0 + 8u * (B_SB)), par, abort);
        if (ok && n >= 1) ok = mbar_wait((bar0 + 8u * (B_EPI0 + (par ^ 1))), ((n - 1) >> 1) & 1, abort);
        if (!ok) break;
        tc_fence_after();
        if (has_state && (!GRP || use_glob)) {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)     // O = phi(Q) S_prev
            mma_bf16_ts(tmem + O_COL, tmem + FQ_COL + 8 * ks, desc64(s_mn + kstep_mnmajor(ks)), idesc(false, true, 128), ks > 0);
        }
        mma_commit((bar0 + 8u * (B_MMA_Q)));
        ok = mbar_wait((bar0 + 8u * (B_PDONE)), par, abort);               // masked P of tile n is in TMEM
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)       // O += (P o M) V; 16 tokens of every row of P = 8 columns
          mma_bf16_ts(tmem + O_COL, tmem + P_COL + (ks < 4 ? 8 * ks : 64 + 8 * (ks - 4)), desc64(v_mn + kstep_mnmajor(ks)),
                      idesc(false, true, 128), (has_state && (!GRP || use_glob)) || ks > 0);
        mma_commit((bar0 + 8u * (B_MMA_O0 + par)));
        // P of the next tile overwrites the columns that the last product of this tile reads
        ok = mbar_wait((bar0 + 8u * (B_MMA_O0 + par)), (n >> 1) & 1, abort);
        if (!ok) break;
      }
    }
  } else if (warp == kCopyWarp) {
    // =============================== the first K loads, the V loads, output stores (one lane) ===============================
    // A lane of its own, so that waiting for a store to have read its buffer never holds up the issue of products.
    if (lane == 0) {
      bool ok = true;
      for (int n = 0; n < 2 && n < nchunks; ++n) {
        const uint32_t kb = sbase + (n ? OFF_K1 : OFF_K0), kbar = bar0 + 8u * (n ? B_FULL_K1 : B_FULL_K0);
        mbar_expect_tx(kbar, tile_tx);
        tma_load(kb, &mk, 0, y0 + n * tstep, bh, kbar);
        tma_load(kb + KBOX_BYTES, &mk, 64, y0 + n * tstep, bh, kbar);
      }
      for (int n = 0; n < 2 && n < nchunks; ++n) {
        mbar_expect_tx((bar0 + 8u * (B_FULL_V0 + n)), tile_tx);
        tma_load(sbase + OFF_V0 + n * TILE_BYTES, &mv, 0, y0 + n * tstep, bh, (bar0 + 8u * (B_FULL_V0 + n)));
        tma_load(sbase + OFF_V0 + n * TILE_BYTES + BOX_BYTES, &mv, 64, y0 + n * tstep, bh, (bar0 + 8u * (B_FULL_V0 + n)));
      }
      for (int n = 0; n < nchunks; ++n) {
        const uint32_t par = n & 1;
        // the outputs of tile n are staged in its V buffer: store them; once they have been read the buffer takes
        // tile n+2
        ok = mbar_wait((bar0 + 8u * (B_STAGED0 + par)), (n >> 1) & 1, abort);
        if (!ok) break;
        const uint32_t vb = sbase + OFF_V0 + par * TILE_BYTES;
        if (LONG) {
          // the outputs wait in the token rows of this tile's K buffer; every tap has been taken from its V buffer
          const uint32_t kb = sbase + (par ? OFF_K1 : OFF_K0), kbar = bar0 + 8u * (par ? B_FULL_K1 : B_FULL_K0);
          tma_store(&mo, 0, y0 + n * tstep, bh, kb);
          tma_store(&mo, 64, y0 + n * tstep, bh, kb + KBOX_BYTES);
          tma_commit();
          if (n + 2 < nchunks) {
            mbar_expect_tx((bar0 + 8u * (B_FULL_V0 + par)), tile_tx);
            tma_load(vb, &mv, 0, y0 + (n + 2) * tstep, bh, (bar0 + 8u * (B_FULL_V0 + par)));
            tma_load(vb + BOX_BYTES, &mv, 64, y0 + (n + 2) * tstep, bh, (bar0 + 8u * (B_FULL_V0 + par)));
            tma_wait_read();
            mbar_expect_tx(kbar, tile_tx);
            tma_load(kb, &mk, 0, y0 + (n + 2) * tstep, bh, kbar);
            tma_load(kb + KBOX_BYTES, &mk, 64, y0 + (n + 2) * tstep, bh, kbar);
          }
          continue;
        }
        tma_store(&mo, 0, y0 + n * tstep, bh, vb);               // rows past the end of the sequence are clipped
        tma_store(&mo, 64, y0 + n * tstep, bh, vb + BOX_BYTES);
        tma_commit();
        if (n + 2 < nchunks) {
          tma_wait_read();
          mbar_expect_tx((bar0 + 8u * (B_FULL_V0 + par)), tile_tx);
          tma_load(vb, &mv, 0, y0 + (n + 2) * tstep, bh, (bar0 + 8u * (B_FULL_V0 + par)));
          tma_load(vb + BOX_BYTES, &mv, 64, y0 + (n + 2) * tstep, bh, (bar0 + 8u * (B_FULL_V0 + par)));
        }
      }
      tma_wait_all();                             // every store is complete before the CTA exits
    } else if (lane == 1 && !LONG) {
      // A lane of its own for the K reloads (short-window mode): the K buffer of tile n is free the moment its state
      // update completes, and phi(K) of tile n+2 is wanted early -- neither the issuing lane nor the store lane
      // should have to stand by for that moment.
      for (int n = 0; n + 2 < nchunks; ++n) {
        const uint32_t par = n & 1;
        if (!mbar_wait((bar0 + 8u * (B_MMA_S)), par, abort)) break;
        const uint32_t kbuf = sbase + (par ? OFF_K1 : OFF_K0), kbar = bar0 + 8u * (par ? B_FULL_K1 : B_FULL_K0);
        mbar_expect_tx(kbar, tile_tx);
        tma_load(kbuf, &mk, 0, y0 + (n + 2) * tstep, bh, kbar);
        tma_load(kbuf + KBOX_BYTES, &mk, 64, y0 + (n + 2) * tstep, bh, kbar);
      }
    }
  } else if (warp >= 8) {
    // =============================== group A: phi, P, [S|z] snapshot (256 threads) ===============================
    const int ta = tid - kThreadsB;               // 0..255
    const int wa = warp - 8;                      // 0..7
    const int r = 32 * (wa & 3) + lane;           // tile row = TMEM lane
    const int hf = wa >> 2;                       // column half
    const uint32_t lane_addr = (uint32_t)(32 * (wa & 3)) << 16;
    unsigned char* Qb = smem + OFF_Q + hf * BOX_BYTES;
    unsigned char* Sb = smem + OFF_S + hf * BOX_BYTES;
    float* Sg = S + (size_t)u * D * D + (size_t)r * D + 64 * hf;
    // Where the state after this unit goes: its own slot, or -- for the last segment of a chain that was cut -- the
    // caller's state (the pre-pass does not visit last segments: nobody starts from their sums).
    const bool to_caller = nseg > 1 && (u % nseg) == nseg - 1;
    float* Sout = to_caller ? S_fin + (size_t)bh * D * D + (size_t)r * D + 64 * hf : Sg;
    float* zout = to_caller ? z_fin + (size_t)bh * D : z + (size_t)u * D;
    bool ok = true;

    if (init) {   // S -> TMEM (fp32) and bf16 copy in shared memory (z was copied during set-up)
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
        for (int c = 0; c < 4; ++c) *reinterpret_cast<uint4*>(Sb + swz(r, 4 * qq + c)) = pack8(v + 8 * c);
      }
      if (hf == 0) {
        tmem_st1(tmem + lane_addr + Z_COL, __float_as_uint(z[(size_t)u * D + r]));
#pragma unroll
        for (int c = 1; c < 16; ++c) tmem_st1(tmem + lane_addr + Z_COL + c, 0u);
      }
      tmem_wait_st();
    }
    fence_proxy_async();
    tc_fence_before();
    mbar_arrive((bar0 + 8u * (B_SB)));                       // phase 0: the state before tile 0 is in place

    // phi on the K tile of tile m, in place; rows at or beyond the end of the sequence become zero
    auto phi_k = [&](int m, bool go) {
      if (!go) return;
      const int valid = min(tstep, T - m * tstep);
      const int ct = ta & 15, rg = ta >> 4;                     // chunk column 0..15, row group 0..15
      unsigned char* Kb = smem + ((m & 1) ? OFF_K1 : OFF_K0) + (ct >> 3) * KBOX_BYTES;
      uint4 x[8];                                               // all eight loads first: they do not wait for the stores
#pragma unroll
      for (int i = 0; i < 8; ++i) x[i] = *reinterpret_cast<const uint4*>(Kb + swz(rg + 16 * i, ct & 7));
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int j = rg + 16 * i;
        *reinterpret_cast<uint4*>(Kb + swz(j, ct & 7)) = j < valid ? phi8<PHI>(x[i]) : make_uint4(0u, 0u, 0u, 0u);
      }
    };
    if (!GRP) {
      ok = mbar_wait((bar0 + 8u * (B_FULL_K0)), 0, abort);
      ok = __all_sync(0xffffffffu, ok);
      phi_k(0, ok);
    }

    for (int n = 0; n < nchunks; ++n) {
      const uint32_t par = n & 1;
      const bool last = n + 1 == nchunks;

      // ---- phi on Q in place (phi on K of this tile was done one iteration earlier) ----
      ok = ok && mbar_wait((bar0 + 8u * (B_FULL_Q)), par, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (GRP) sync_group_a();                    // z of the previous snapshot (written by other threads) is in place
      // phi(q) of row r, this thread's 64 channels: 32 packed pairs = 32 TMEM columns of lane r.  (The products of
      // tile n-1 that read these columns are complete: the snapshot at the end of the previous iteration waited for them.)
      uint32_t fq[32];
      if (ok) {
#pragma unroll
        for (int cc = 0; cc < 8; ++cc) {
          const uint4 f = phi8<PHI>(*reinterpret_cast<const uint4*>(Qb + swz(r, cc)));
          fq[4 * cc] = f.x; fq[4 * cc + 1] = f.y; fq[4 * cc + 2] = f.z; fq[4 * cc + 3] = f.w;
        }
        LA_TMEM_ST32(tmem + lane_addr + FQ_COL + 32 * hf, fq);
        if (GRP) {                                // this half of phi(q) . z_prev, z in fp32
          float dg = 0.f;
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float4 z4 = *reinterpret_cast<const float4*>(zs + 64 * hf + 2 * e);
            dg = fmaf(lo_f(fq[e]), z4.x, fmaf(hi_f(fq[e]), z4.y, fmaf(lo_f(fq[e + 1]), z4.z, fmaf(hi_f(fq[e + 1]), z4.w, dg))));
          }
          dgh[hf * D + r] = dg;
        }
        tmem_wait_st();
      }
      if (GRP) {
        // phi on K of this tile, in place: the score product runs on the raw q and k, so K may be touched only once
        // that product is complete (phi(Q) above reads the Q buffer and writes TMEM: it ran beside the product)
        ok = ok && mbar_wait((bar0 + 8u * (par ? B_FULL_K1 : B_FULL_K0)), (n >> 1) & 1, abort) &&
             mbar_wait((bar0 + 8u * (B_MMA_P)), par, abort);
        ok = __all_sync(0xffffffffu, ok);
        phi_k(n, ok);
      }
      fence_proxy_async();                        // (phi(K) of this tile, written one iteration earlier)
      tc_fence_before();
      mbar_arrive((bar0 + 8u * (B_PHI)));
      float dpart = 0.f;                          // this half of the row sum of the masked P

      // ---- phi on K of the next tile, while the tensor cores form the scores of this one.  (Not with the long-window
      //      epilogue: there the K buffer comes back late, after the outputs staged in it have left, and waiting for
      //      it here would hold up the mask; see below.) ----
      if (!GRP && !LONG && !last) {
        ok = ok && mbar_wait((bar0 + 8u * (((n + 1) & 1) ? B_FULL_K1 : B_FULL_K0)), ((n + 1) >> 1) & 1, abort);
        ok = __all_sync(0xffffffffu, ok);
        phi_k(n + 1, ok);
      }

      // ---- P: causal mask, packed bf16 -> TMEM ----
      if (!GRP) ok = ok && mbar_wait((bar0 + 8u * (B_MMA_P)), par, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (!GRP && ok) {
        tc_fence_after();
#pragma unroll
        for (int qq = 0; qq < 2; ++qq) {
          const int col0 = 64 * hf + 32 * qq;
          uint32_t v[32], pk[16];
          float ps0 = 0.f, ps1 = 0.f;
          if (col0 <= 32 * (wa & 3) + 31) {                     // warp-uniform: some row of this warp reaches col0
            LA_TMEM_LD32(tmem + P_COL + lane_addr + col0, v);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const float p0 = col0 + 2 * e <= r ? __uint_as_float(v[2 * e]) : 0.f;
              const float p1 = col0 + 2 * e + 1 <= r ? __uint_as_float(v[2 * e + 1]) : 0.f;
              pk[e] = pack2(p0, p1);
              ps0 += p0;
              ps1 += p1;
            }
            dpart += ps0 + ps1;
          } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) pk[e] = 0u;
          }
          LA_TMEM_ST16(tmem + P_COL + lane_addr + 64 * hf + 16 * qq, pk);
        }
        if (hf == 1) {                            // phi(q) . z_prev, delivered by the score product as column 128
          dpart += __uint_as_float(tmem_ld1(tmem + lane_addr + QZ_COL));
          tmem_wait_ld();
        }
        // (slot n & 1 was last read by the epilogue of tile n-2, before the arrival that released the accumulator to
        // tile n-1, whose products were complete before P of this tile was issued)
        denbuf[(par * 2 + hf) * D + r] = dpart;
        tmem_wait_st();
      }
      if (GRP) {
        // ---- P: causal softmax along the rows.  A row's 128 columns belong to two threads (halves): each takes the
        // running maximum and sum of its half, the halves meet through shared memory, and a second pass writes
        // exp(s - max) / sum back as bf16 -- times (phi(q) . z_prev + eps) / alpha where the global branch is alive, so
        // that the epilogue's one row factor alpha / (phi(q) . z_prev + eps) finishes both branches.
        const float c2 = sm_scale * 1.4426950408889634f;       // scores -> exponents of two
        float m_run = -INFINITY, l_run = 0.f;
        if (ok) {
          tc_fence_after();
#pragma unroll
          for (int qq = 0; qq < 2; ++qq) {
            const int col0 = 64 * hf + 32 * qq;
            if (col0 <= 32 * (wa & 3) + 31) {                   // warp-uniform: some row of this warp reaches col0
              uint32_t v[32];
              LA_TMEM_LD32(tmem + P_COL + lane_addr + col0, v);
              tmem_wait_ld();
              float bm = -INFINITY;
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (col0 + e <= r) bm = fmaxf(bm, __uint_as_float(v[e]) * c2);
              if (bm > -INFINITY) {
                const float mn = fmaxf(m_run, bm);
                float acc = 0.f;
#pragma unroll
                for (int e = 0; e < 32; ++e)
                  if (col0 + e <= r) acc += ex2(__uint_as_float(v[e]) * c2 - mn);
                l_run = l_run * ex2(m_run - mn) + acc;
                m_run = mn;
              }
            }
          }
        }
        mlh[hf * D + r] = make_float2(m_run, l_run);
        sync_group_a();
        const float2 oth = mlh[(hf ^ 1) * D + r];
        const float m = fmaxf(m_run, oth.x);                    // finite: the row's own column lies in one of the halves
        const float l = l_run * ex2(m_run - m) + oth.y * ex2(oth.x - m);
        const float den = dgh[r] + dgh[D + r] + eps;
        const bool has_g = use_glob && (init || n > 0) && den != 0.f;
        const float rs = has_g ? den / alpha : 1.f;
        const float f = rs / l;
        if (ok) {
#pragma unroll
          for (int qq = 0; qq < 2; ++qq) {
            const int col0 = 64 * hf + 32 * qq;
            uint32_t pk[16];
            if (col0 <= 32 * (wa & 3) + 31) {
              uint32_t v[32];
              LA_TMEM_LD32(tmem + P_COL + lane_addr + col0, v);
              tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                const float p0 = col0 + 2 * e <= r ? ex2(__uint_as_float(v[2 * e]) * c2 - m) * f : 0.f;
                const float p1 = col0 + 2 * e + 1 <= r ? ex2(__uint_as_float(v[2 * e + 1]) * c2 - m) * f : 0.f;
                pk[e] = pack2(p0, p1);
              }
            } else {
#pragma unroll
              for (int e = 0; e < 16; ++e) pk[e] = 0u;
            }
            LA_TMEM_ST16(tmem + P_COL + lane_addr + 64 * hf + 16 * qq, pk);
          }
          // the epilogue's row factor is 1 / (the two halves + its eps): the factor here, nothing else
          denbuf[(par * 2 + hf) * D + r] = hf == 0 ? rs : 0.f;
          tmem_wait_st();
        }
      }
      tc_fence_before();
      mbar_arrive((bar0 + 8u * (B_PDONE)));

      if (!GRP && LONG && !last) {                // long-window epilogue: phi on K of the next tile after the mask
        ok = ok && mbar_wait((bar0 + 8u * (((n + 1) & 1) ? B_FULL_K1 : B_FULL_K0)), ((n + 1) >> 1) & 1, abort);
        ok = __all_sync(0xffffffffu, ok);
        phi_k(n + 1, ok);
      }

      // ---- the rows of v before the next tile: the last W-1 of (halo ++ valid rows of this tile's V), 16 bytes per
      //      thread, in the time this group would otherwise wait for the state update ----
      if (HALO_A) {
        ok = ok && mbar_wait((bar0 + 8u * (B_FULL_V0 + par)), (n >> 1) & 1, abort);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
          const int valid = min(tstep, T - n * tstep);
          const __nv_bfloat16* halo = halo0 + (n % 3) * halo_elems;
          __nv_bfloat16* halo_next = halo0 + ((n + 1) % 3) * halo_elems;
          const unsigned char* Vt = smem + OFF_V0 + par * TILE_BYTES;
          for (int idx = ta; idx < 16 * (W - 1); idx += kThreadsA) {
            const int i = idx >> 4, c16 = idx & 15, src = valid + i;
            uint4 x;
            if (src < W - 1) x = *reinterpret_cast<const uint4*>(halo + src * D + 8 * c16);
            else x = *reinterpret_cast<const uint4*>(Vt + (c16 >> 3) * BOX_BYTES + swz(src - (W - 1), c16 & 7));
            *reinterpret_cast<uint4*>(halo_next + i * D + 8 * c16) = x;
          }
        }
        mbar_arrive((bar0 + 8u * (B_HALO)));
      }

      // ---- S_n: bf16 copy for the next tile, or the final state to global memory ----
      // S_n is final after MMA_S; the old copy may be overwritten once O = phi(Q) S_prev has read it
      ok = ok && mbar_wait((bar0 + 8u * (B_MMA_S)), par, abort) && mbar_wait((bar0 + 8u * (B_MMA_Q)), par, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        tc_fence_after();
        uint32_t zbits = 0u;
        if (hf == 0) zbits = tmem_ld1(tmem + lane_addr + Z_COL);
#pragma unroll
        for (int qq = 0; qq < 2; ++qq) {
          uint32_t v[32];
          LA_TMEM_LD32(tmem + lane_addr + S_COL + 64 * hf + 32 * qq, v);
          tmem_wait_ld();
          if (last) {
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              *reinterpret_cast<float4*>(Sout + 32 * qq + e) =
                  make_float4(__uint_as_float(v[e]), __uint_as_float(v[e + 1]), __uint_as_float(v[e + 2]),
                              __uint_as_float(v[e + 3]));
          } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) *reinterpret_cast<uint4*>(Sb + swz(r, 4 * qq + c)) = pack8(v + 8 * c);
          }
        }
        if (hf == 0) {
          const float zz = __uint_as_float(zbits);
          if (last) zout[r] = zz;
          else if (GRP) zs[r] = zz;               // fp32, for phi(q) . z of the next tile
          else                                    // row 128 of the K buffer of tile n+1 (its token rows are in place already)
            *reinterpret_cast<__nv_bfloat16*>(smem + (((n + 1) & 1) ? OFF_K1 : OFF_K0) + (r >> 6) * KBOX_BYTES + BOX_BYTES +
                                              (r & 63) * 2) = __float2bfloat16_rn(zz);
        }
      }
      fence_proxy_async();
      tc_fence_before();
      mbar_arrive((bar0 + 8u * (B_SB)));
    }
  } else {
    // =============================== group B: epilogue (256 threads) ===============================
    const int r = 32 * (warp & 3) + lane;         // tile row = TMEM lane
    const int hf = warp >> 2;                     // column half
    const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
    bool ok = true;
    if constexpr (LONG) {
      // Two phases per tile.  (1) Row by row, as the accumulator's lanes dictate: the attention term O / den goes,
      // rounded to bf16, into the token rows of this tile's K buffer, which every product has finished with (its
      // reload for tile n + 2 waits, in this mode, until the outputs have left).  (2) Channel pair by channel pair:
      // thread (cp, jq) owns channels 2 cp, 2 cp + 1 and rows 32 jq ... 32 jq + 31, forms the tap sums of 16 rows at a
      // time in registers (every row of v it needs is read once per group of 8 taps, and the taps of a group sit in
      // registers), adds the attention term and writes the output over it.  The shared-memory traffic of a tile no
      // longer grows with rows x taps x 16 bytes, and the V buffer is never written.
      const int cp = tid & 63, jq = tid >> 6;
      const int cc = (cp & 31) >> 2;                                         // 16-byte piece of the pair in its box row
      const uint32_t colv = (uint32_t)(cp >> 5) * BOX_BYTES + (uint32_t)(cp & 3) * 4u + (uint32_t)jq * 4096u;
      const uint32_t colk = (uint32_t)(cp >> 5) * KBOX_BYTES + (uint32_t)(cp & 3) * 4u + (uint32_t)jq * 4096u;
      const int lead = (int)long_taps(W) - W;                                // rows of zeros at the head of the halo
      const uint32_t hcol = sbase + off_halo_long(W) + 4u * cp;
      const uint32_t hend = hcol + (long_taps(W) - 1) * (D * 2);
      const uint32_t wcol = sbase + off_w() + 8u * cp;
      const int ngroups = (W + 7) >> 3;
      for (int n = 0; n < nchunks; ++n) {
        const uint32_t par = n & 1;
        const int valid = min(tstep, T - n * tstep);
        const uint32_t vthr = sbase + OFF_V0 + par * TILE_BYTES + colv;       // this thread's column at its first row
        unsigned char* stage = smem + (par ? OFF_K1 : OFF_K0);
        ok = ok && mbar_wait((bar0 + 8u * (B_MMA_O0 + par)), (n >> 1) & 1, abort);   // also: every product that reads K or V is done
        ok = __all_sync(0xffffffffu, ok);
        uint32_t v[32];
        float rden = 0.f;
        if (ok) {
          tc_fence_after();
          LA_TMEM_LD32(tmem + lane_addr + O_COL + 64 * hf, v);
          const float den = denbuf[(par * 2) * D + r] + denbuf[(par * 2 + 1) * D + r];
          rden = 1.f / (den + (GRP ? 0.f : eps));
        }
        unsigned char* Lb = stage + hf * KBOX_BYTES;
#pragma unroll
        for (int qq = 0; qq < 2; ++qq) {
          if (ok) {
            tmem_wait_ld();
            uint4 la[4];
#pragma unroll
            for (int c = 0; c < 4; ++c)
              la[c] = make_uint4(pack2(__uint_as_float(v[8 * c]) * rden, __uint_as_float(v[8 * c + 1]) * rden),
                                 pack2(__uint_as_float(v[8 * c + 2]) * rden, __uint_as_float(v[8 * c + 3]) * rden),
                                 pack2(__uint_as_float(v[8 * c + 4]) * rden, __uint_as_float(v[8 * c + 5]) * rden),
                                 pack2(__uint_as_float(v[8 * c + 6]) * rden, __uint_as_float(v[8 * c + 7]) * rden));
            if (qq == 0) LA_TMEM_LD32(tmem + lane_addr + O_COL + 64 * hf + 32, v);
#pragma unroll
            for (int c = 0; c < 4; ++c) *reinterpret_cast<uint4*>(Lb + swz(r, 4 * qq + c)) = la[c];
          }
        }
        tc_fence_before();
        mbar_arrive((bar0 + 8u * (B_EPI0 + par)));           // this accumulator has been read
        ok = ok && mbar_wait((bar0 + 8u * (B_FULL_V0 + par)), (n >> 1) & 1, abort);
        ok = __all_sync(0xffffffffu, ok);
        sync_group_b();                                      // the attention term of every row is in place
        if (ok) {
          uint32_t pv[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) pv[k] = vthr + ((cc ^ k) << 4);
          const uint32_t sthr = sbase + (par ? OFF_K1 : OFF_K0) + colk;
          const int mine = valid - 32 * jq;                  // rows of this thread that hold tokens
          if (jq == 0) {
            if (mine > 0) conv_rows<0, true>(wcol, pv, sthr, cc, hend, ngroups);
            if (mine > 8) conv_rows<1, true>(wcol, pv, sthr, cc, hend, ngroups);
            if (mine > 16) conv_rows<2, true>(wcol, pv, sthr, cc, hend, ngroups);
            if (mine > 24) conv_rows<3, true>(wcol, pv, sthr, cc, hend, ngroups);
            // The rows before the next tile: the last W-1 of (halo ++ valid rows of v), in place.  This thread is the
            // only one that reads or writes this column of the halo (the rows of the other threads start at 32, and
            // no window reaches back further than 31 rows).
            for (int i = 0; i < W - 1; ++i) {
              const int src = valid - (W - 1) + i;
              const uint32_t x = src >= 0 ? lds32(vthr + src * 128 + ((cc ^ (src & 7)) << 4)) : lds32(hend + src * (D * 2));
              sts32(hcol + (lead + i) * (D * 2), x);
            }
          } else {
            if (mine > 0) conv_rows<0, false>(wcol, pv, sthr, cc, hend, ngroups);
            if (mine > 8) conv_rows<1, false>(wcol, pv, sthr, cc, hend, ngroups);
            if (mine > 16) conv_rows<2, false>(wcol, pv, sthr, cc, hend, ngroups);
            if (mine > 24) conv_rows<3, false>(wcol, pv, sthr, cc, hend, ngroups);
          }
        }
        fence_proxy_async();
        mbar_arrive((bar0 + 8u * (B_STAGED0 + par)));
      }
    } else
    for (int n = 0; n < nchunks; ++n) {
      const uint32_t par = n & 1;
      const int valid = min(tstep, T - n * tstep);
      const unsigned char* Vt = smem + OFF_V0 + par * TILE_BYTES;
      // rows before this tile, addressed so that row -1 is the last of W-1 rows
      const __nv_bfloat16* halo = halo0 + (HALO_A ? n % 3 : (int)par) * halo_elems;
      __nv_bfloat16* halo_next = halo0 + (par ^ 1) * halo_elems;    // rows before the next tile
      ok = ok && mbar_wait((bar0 + 8u * (B_FULL_V0 + par)), (n >> 1) & 1, abort);
      // (HALO_A: group A has read the last rows of this tile's V, and with that filled the halo of the tile before)
      if (HALO_A) ok = ok && mbar_wait((bar0 + 8u * (B_HALO)), par, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (ok && !HALO_A) {
        // next halo <- last W-1 rows of (halo ++ valid rows of V), 16 bytes (8 channels) per thread; each half of the
        // group copies its own 64 channels
        const unsigned char* Vc = Vt + hf * BOX_BYTES;
        for (int idx = tid & 127; idx < 8 * (W - 1); idx += 128) {
          const int i = idx >> 3, c8 = idx & 7, src = valid + i;
          uint4 x;
          if (src < W - 1) x = *reinterpret_cast<const uint4*>(halo + src * D + 64 * hf + 8 * c8);
          else x = *reinterpret_cast<const uint4*>(Vc + swz(src - (W - 1), c8));
          *reinterpret_cast<uint4*>(halo_next + i * D + 64 * hf + 8 * c8) = x;
        }
      }
      ok = ok && mbar_wait((bar0 + 8u * (B_MMA_O0 + par)), (n >> 1) & 1, abort);   // also: every product that reads V is done
      ok = __all_sync(0xffffffffu, ok);
      // The outputs leave through the V buffer of this tile, 16-byte column by column: a column is overwritten (same
      // swizzled layout) once every thread of this half has taken its taps from it, so that a thread holds one
      // column of outputs at a time; the control lane then stores whole rows with one TMA store per box.  The two
      // halves of the group (64 channels each) share nothing and synchronise separately.
      // The accumulator is read 32 columns at a time; each load is issued as early as its registers are free, so
      // that its latency passes behind the barrier and the arithmetic in between.
      uint32_t v[32];
      if (ok) {
        tc_fence_after();
        LA_TMEM_LD32(tmem + lane_addr + O_COL + 64 * hf, v);
      }
      if (!HALO_A) sync_half_b(hf);               // the next halo is complete before any row of V is overwritten
      float rden = 0.f;
      if (ok) {
        // row sum of the masked P + phi(q) . z_prev, both halves gathered by the masking threads
        const float den = denbuf[(par * 2) * D + r] + denbuf[(par * 2 + 1) * D + r];
        rden = 1.f / (den + (GRP ? 0.f : eps));   // (three-branch mode: the masking threads left the finished factor)
      }
      unsigned char* Ob = smem + OFF_V0 + par * TILE_BYTES + hf * BOX_BYTES;
#pragma unroll
      for (int qq = 0; qq < 2; ++qq) {
        if (ok) tmem_wait_ld();
        if (qq == 1) {
          tc_fence_before();
          mbar_arrive((bar0 + 8u * (B_EPI0 + par)));         // this accumulator has been read
        }
#pragma unroll
        for (int c2 = 0; c2 < 2; ++c2) {          // two columns per barrier
          uint4 outp[2];
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int c = 2 * c2 + j;
            const int cc = 4 * qq + c;                          // chunk inside this half's box
            const int ch0 = 64 * hf + 8 * cc;                   // first channel of the chunk
            outp[j] = make_uint4(0u, 0u, 0u, 0u);
            if (ok && r < valid) {                              // rows past the tile's tokens stage zeros
              float2 acc[4];
#pragma unroll
              for (int e = 0; e < 4; ++e)
                acc[e] = __fmul2_rn(make_float2(__uint_as_float(v[8 * c + 2 * e]), __uint_as_float(v[8 * c + 2 * e + 1])),
                                    make_float2(rden, rden));
              conv8<WT>(acc, W, r, cc, ch0, Vt + hf * BOX_BYTES, halo, wsm);
              outp[j] = make_uint4(pack2(acc[0].x, acc[0].y), pack2(acc[1].x, acc[1].y), pack2(acc[2].x, acc[2].y),
                                   pack2(acc[3].x, acc[3].y));
            }
          }
          if (qq == 0 && c2 == 1 && ok)           // the first 32 columns have been used: fetch the other 32
            LA_TMEM_LD32(tmem + lane_addr + O_COL + 64 * hf + 32, v);
          sync_half_b(hf);                        // these two columns of this half have been read by all of its rows
          if (ok) {
#pragma unroll
            for (int j = 0; j < 2; ++j) *reinterpret_cast<uint4*>(Ob + swz(r, 4 * qq + 2 * c2 + j)) = outp[j];
          }
        }
      }
      fence_proxy_async();
      mbar_arrive((bar0 + 8u * (B_STAGED0 + par)));
    }
    sync_group_b();                               // both halves of the last halo are complete
    if (ok && tid < D) {
      // the window to carry on: the last W-1 values of (incoming window ++ this unit's v)
      const __nv_bfloat16* halo = halo0 + (LONG ? ((int)long_taps(W) - W) * D : (HALO_A ? nchunks % 3 : nchunks & 1) * halo_elems);
      for (int i = 0; i < W - 1; ++i) win[((size_t)u * (W - 1) + i) * D + tid] = halo[i * D + tid];
      if (tid == 0 && h == 0 && nseg == 1) pos[bh / H] = (init ? pos[bh / H] : 0) + T;
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (sm.abort) {
    if (tid == 0) report(status, LA_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(2000);   // bounded grace period for copies still in flight
  }
  if (warp == kCtrlWarp) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

// ---- sequence split: local state of a segment ------------------------------------------------------
// For chains too few to fill the GPU the sequence is cut into segments that run as separate CTAs.  This
// kernel computes, for one segment, only its own contribution [dS | dz] = sum phi(k) [v | 1]^T (K and V are
// read, phi applied to K, one product per tile) and stores it in fp32.  A prefix sum over the segments
// (prefix_kernel) turns the contributions into the state each segment starts from.
constexpr int kStateThreads = 288;       // 8 compute warps + 1 issue warp
constexpr uint32_t ST_OFF_K = 0, ST_OFF_V = 2 * TILE_BYTES, ST_OFF_ONES = 4 * TILE_BYTES, ST_OFF_SMALL = ST_OFF_ONES + 4096;
constexpr uint32_t kStateSmem = ST_OFF_SMALL + 256 + 1024;
enum { SB_FULL_K0 = 0, SB_FULL_K1, SB_FULL_V0, SB_FULL_V1, SB_PHI, SB_MMA, kStateBars };

template <int PHI>
__global__ void __launch_bounds__(kStateThreads, 1)
segment_state_kernel(const __grid_constant__ CUtensorMap mk, const __grid_constant__ CUtensorMap mv,
                     float* __restrict__ S_out, float* __restrict__ z_out, int* status, int Ttot, int nseg,
                     int seg_len, int nrun) {
  extern __shared__ unsigned char smem_dyn[];
  // (an offset into the array rather than an integer cast: the compiler then knows that these are shared-memory
  // addresses: 32-bit arithmetic, ld.shared / st.shared)
  unsigned char* smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + ST_OFF_SMALL);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + ST_OFF_SMALL + 128);
  volatile int* abort = reinterpret_cast<int*>(smem + ST_OFF_SMALL + 132);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // The launch visits the first nrun of a chain's nseg segments (all of them, or all but the last, whose sums no
  // other segment starts from); results go to slot bh * nseg + segment.
  const int bh = blockIdx.x / nrun, sg = blockIdx.x % nrun, u = bh * nseg + sg;
  const int y0 = sg * seg_len, T = min(seg_len, Ttot - y0);
  const int nchunks = (T + TILE - 1) / TILE;
  const uint32_t bar0 = smem_u32(&bars[0]);       // barrier i lives at bar0 + 8 i

  if (tid == 0) {
    for (int i = 0; i < 4; ++i) mbar_init((bar0 + 8u * (i)), 1);
    mbar_init((bar0 + 8u * (SB_PHI)), 256);
    mbar_init((bar0 + 8u * (SB_MMA)), 1);
    *abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int idx = tid; idx < 4096 / 16; idx += kStateThreads)
    reinterpret_cast<uint4*>(smem + ST_OFF_ONES)[idx] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  if (tid < TILE) *reinterpret_cast<__nv_bfloat16*>(smem + ST_OFF_ONES + ext_offset(tid, 0)) = __float2bfloat16_rn(1.f);
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  constexpr uint32_t SCOL = 0, ZCOL = 128;

  if (warp == 8) {
    if (lane == 0) {
      auto load_tile = [&](int n) {
        const uint32_t b2 = n & 1;
        mbar_expect_tx((bar0 + 8u * (SB_FULL_K0 + b2)), TILE_BYTES);
        tma_load(sbase + ST_OFF_K + b2 * TILE_BYTES, &mk, 0, y0 + n * TILE, bh, (bar0 + 8u * (SB_FULL_K0 + b2)));
        tma_load(sbase + ST_OFF_K + b2 * TILE_BYTES + BOX_BYTES, &mk, 64, y0 + n * TILE, bh, (bar0 + 8u * (SB_FULL_K0 + b2)));
        mbar_expect_tx((bar0 + 8u * (SB_FULL_V0 + b2)), TILE_BYTES);
        tma_load(sbase + ST_OFF_V + b2 * TILE_BYTES, &mv, 0, y0 + n * TILE, bh, (bar0 + 8u * (SB_FULL_V0 + b2)));
        tma_load(sbase + ST_OFF_V + b2 * TILE_BYTES + BOX_BYTES, &mv, 64, y0 + n * TILE, bh, (bar0 + 8u * (SB_FULL_V0 + b2)));
      };
      for (int n = 0; n < 2 && n < nchunks; ++n) load_tile(n);
      for (int n = 0; n < nchunks; ++n) {
        const uint32_t b2 = n & 1;
        if (!mbar_wait((bar0 + 8u * (SB_PHI)), n & 1, abort) || !mbar_wait((bar0 + 8u * (SB_FULL_V0 + b2)), (n >> 1) & 1, abort)) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {     // [dS | dz] += phi(K)^T [V | 1]
          const uint64_t kd = desc_mnmajor(sbase + ST_OFF_K + b2 * TILE_BYTES, ks);
          mma_bf16(tmem + SCOL, kd, desc_mnmajor(sbase + ST_OFF_V + b2 * TILE_BYTES, ks), idesc(true, true, 128), n > 0 || ks > 0);
          mma_bf16(tmem + ZCOL, kd, desc_ext(sbase + ST_OFF_ONES, ks), idesc(true, true, 16), n > 0 || ks > 0);
        }
        mma_commit((bar0 + 8u * (SB_MMA)));
        if (!mbar_wait((bar0 + 8u * (SB_MMA)), n & 1, abort)) break;       // both buffers of this tile are free
        if (n + 2 < nchunks) load_tile(n + 2);
      }
    }
  } else {
    bool ok = true;
    for (int n = 0; n < nchunks; ++n) {
      const int valid = min(TILE, T - n * TILE);
      ok = ok && mbar_wait((bar0 + 8u * (SB_FULL_K0 + (n & 1))), (n >> 1) & 1, abort);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        const int ct = tid & 15, rg = tid >> 4;
        unsigned char* Kb = smem + ST_OFF_K + (n & 1) * TILE_BYTES + (ct >> 3) * BOX_BYTES;
        uint4 x[8];                                             // all eight loads first: they do not wait for the stores
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = *reinterpret_cast<const uint4*>(Kb + swz(rg + 16 * i, ct & 7));
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int j = rg + 16 * i;
          *reinterpret_cast<uint4*>(Kb + swz(j, ct & 7)) = j < valid ? phi8<PHI>(x[i]) : make_uint4(0u, 0u, 0u, 0u);
        }
      }
      fence_proxy_async();
      mbar_arrive((bar0 + 8u * (SB_PHI)));
    }
    // Wait for the last two products in turn (tile L was loaded only after product L-2 had completed, so the
    // barrier is at phase L-1 or later here and a parity wait cannot be fooled by an older phase).
    for (int n = max(0, nchunks - 2); n < nchunks; ++n) ok = ok && mbar_wait((bar0 + 8u * (SB_MMA)), n & 1, abort);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      const int r = 32 * (warp & 3) + lane, hf = warp >> 2;
      const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
      float* Sg = S_out + (size_t)u * D * D + (size_t)r * D + 64 * hf;
#pragma unroll
      for (int qq = 0; qq < 2; ++qq) {
        uint32_t v[32];
        LA_TMEM_LD32(tmem + lane_addr + SCOL + 64 * hf + 32 * qq, v);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; e += 4)
          *reinterpret_cast<float4*>(Sg + 32 * qq + e) = make_float4(__uint_as_float(v[e]), __uint_as_float(v[e + 1]),
                                                                     __uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
      }
      if (hf == 0) {
        const uint32_t zz = tmem_ld1(tmem + lane_addr + ZCOL);
        tmem_wait_ld();
        z_out[(size_t)u * D + r] = __uint_as_float(zz);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort) {
    if (tid == 0) report(status, LA_ERR_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(2000);
  }
  if (warp == 8) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
  }
}

// Exclusive prefix over the segments of one chain, in place: on return S_seg[bh][s] / z_seg[bh][s] hold the state
// segment s starts from and win_seg its incoming window; win / pos of the caller get their final values here, S / z
// of the caller are written by the last segment's block of the main pass (the sums of last segments are not
// computed beforehand, so their slots are not read).
// grid = (BH, d*d / 1024), 256 threads, four consecutive elements of S per thread.
__global__ void __launch_bounds__(256)
prefix_kernel(float* __restrict__ S_seg, float* __restrict__ z_seg, __nv_bfloat16* __restrict__ win_seg,
              const __nv_bfloat16* __restrict__ v, float* __restrict__ S, float* __restrict__ z,
              __nv_bfloat16* __restrict__ win, int64_t* __restrict__ pos, int H, int Ttot, int W, int nseg, int seg_len,
              int init) {
  const int bh = blockIdx.x, e4 = (blockIdx.y * 256 + threadIdx.x) * 4;
  // Loads in batches of sixteen segments, all in flight at once; only the additions are sequential.
  float4 run = init ? *reinterpret_cast<const float4*>(S + (size_t)bh * D * D + e4) : make_float4(0.f, 0.f, 0.f, 0.f);
  for (int sg0 = 0; sg0 < nseg; sg0 += 16) {
    float4 d[16];
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (sg0 + j < nseg - 1) d[j] = *reinterpret_cast<const float4*>(S_seg + ((size_t)bh * nseg + sg0 + j) * D * D + e4);
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (sg0 + j < nseg) {
        *reinterpret_cast<float4*>(S_seg + ((size_t)bh * nseg + sg0 + j) * D * D + e4) = run;
        if (sg0 + j < nseg - 1) { run.x += d[j].x; run.y += d[j].y; run.z += d[j].z; run.w += d[j].w; }
      }
  }
  if (blockIdx.y == 0 && threadIdx.x < D) {
    const int c = threadIdx.x;
    float rz = init ? z[(size_t)bh * D + c] : 0.f;
    for (int sg0 = 0; sg0 < nseg; sg0 += 8) {
      float d[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (sg0 + j < nseg - 1) d[j] = z_seg[((size_t)bh * nseg + sg0 + j) * D + c];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (sg0 + j < nseg) {
          z_seg[((size_t)bh * nseg + sg0 + j) * D + c] = rz;
          if (sg0 + j < nseg - 1) rz += d[j];
        }
    }
    if (c == 0 && bh % H == 0) pos[bh / H] = (init ? pos[bh / H] : 0) + Ttot;
  }
  // Incoming windows: the W-1 values of v before each segment; before the first one the caller's window or zeros.
  // One element per thread over all blocks of this chain.  The thread that reads the caller's window entry (i, c)
  // is also the one that overwrites it with the final window: the last W-1 values of v (Ttot >= W-1 whenever the
  // split is used).
  const int per_chain = nseg * (W - 1) * D;
  for (int idx = blockIdx.y * 256 + threadIdx.x; idx < per_chain; idx += gridDim.y * 256) {
    const int c = idx % D, i = (idx / D) % (W - 1), sg = idx / (D * (W - 1));
    const int t = sg * seg_len - (W - 1) + i;
    __nv_bfloat16 x = __float2bfloat16_rn(0.f);
    if (t >= 0) x = v[((size_t)bh * Ttot + t) * D + c];
    else if (init) x = win[((size_t)bh * (W - 1) + i) * D + c];          // sg == 0: t = i - (W-1)
    win_seg[(((size_t)bh * nseg + sg) * (W - 1) + i) * D + c] = x;
    if (sg == 0) win[((size_t)bh * (W - 1) + i) * D + c] = v[((size_t)bh * Ttot + Ttot - (W - 1) + i) * D + c];
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
static bool make_map(CUtensorMap* m, const void* base, int BH, int T, int box_rows = TILE) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)T * D * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc

template <int PHI>
static cudaError_t launch_w(const la_config& c, int units, int T, const CUtensorMap& mq, const CUtensorMap& mk,
                            const CUtensorMap& mv, const CUtensorMap& mo, const float* w, int init, float* S, float* z,
                            __nv_bfloat16* win, int64_t* pos, int* status, int nseg, int seg_len,
                            float* S_fin, float* z_fin, cudaStream_t s, bool grouped = false, float alpha = 1.f,
                            float sm_scale = 1.f, int tstep = tc::TILE) {
  const bool lng = tc::long_epilogue(c.conv_taps, grouped);
  const size_t smem = grouped ? tc::smem_bytes_grp(c.conv_taps, lng) : lng ? tc::smem_bytes_long(c.conv_taps) : tc::smem_bytes(c.conv_taps);
  void (*kern)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, const float*, float*, float*, __nv_bfloat16*, int64_t*,
               int*, int, int, int, float, int, int, int, float*, float*, float, float, int);
  if (grouped) {
    kern = lng ? tc::prefill_tc_kernel<PHI, -1, true> : tc::prefill_tc_kernel<PHI, 3, true>;
  } else
  switch (c.conv_taps) {     // short windows: the tap loop unrolled; the others: the long epilogue
    case 1: kern = tc::prefill_tc_kernel<PHI, 1>; break;
    case 2: kern = tc::prefill_tc_kernel<PHI, 2>; break;
    case 3: kern = tc::prefill_tc_kernel<PHI, 3>; break;
    case 4: kern = tc::prefill_tc_kernel<PHI, 4>; break;
    case 5: kern = tc::prefill_tc_kernel<PHI, 5>; break;
    default: kern = tc::prefill_tc_kernel<PHI, -1>; break;
  }
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<dim3(units), dim3(tc::kThreads), smem, s>>>(mq, mk, mv, mo, w, S, z, win, pos, status, c.H, T,
                                                     c.conv_taps, c.eps, init, nseg, seg_len, S_fin, z_fin, alpha, sm_scale, tstep);
  return cudaGetLastError();
}

// Segments per chain for a launch of BH chains of T tokens: 1 unless the chains are too few to fill the GPU and
// long enough to cut (every segment a multiple of 128 tokens, at least 1024).
static void plan_split(const la_ctx* ctx, int BH, int T, int* nseg, int* seg_len) {
  *nseg = 1;
  *seg_len = T;
  if (2 * BH > ctx->sm_count || T < 2048) return;
  // One wave of thread blocks: as many segments per chain as fit on the SMs at once.  (Measured on 32 chains of
  // 32768 tokens: 4 segments per chain 418 us, 9 segments (two waves) 432 us, 13: 456, 18: 483 -- a second wave
  // never fills as well as the first, and every segment costs a 64 KB state written and read back.)
  int n = std::min(ctx->sm_count / BH, T / 1024);
  if (n < 2) return;
  const int len = ((T + n - 1) / n + tc::TILE - 1) / tc::TILE * tc::TILE;
  n = (T + len - 1) / len;
  if (n < 2) return;
  *nseg = n;
  *seg_len = len;
}
static size_t split_bytes(const la_config& c, int BH, int nseg) {
  return (size_t)BH * nseg * ((size_t)tc::D * tc::D * 4 + tc::D * 4 + (size_t)(c.conv_taps > 1 ? c.conv_taps - 1 : 1) * tc::D * 2);
}

size_t prefill_workspace_bytes(const la_ctx* ctx, int B, int T) {
  const la_config& c = ctx->cfg;
  if (c.io_dtype != LA_BF16 || c.d != tc::D) return 0;
  int nseg, seg_len;
  plan_split(ctx, B * c.H, T, &nseg, &seg_len);
  return nseg > 1 ? split_bytes(c, B * c.H, nseg) : 0;
}

cudaError_t launch_prefill_tc(la_ctx* ctx, int B, int T, const void* q, const void* k, const void* v, const float* w,
                              int init, const la_state& st, void* o, cudaStream_t s, bool* handled) {
  const la_config& c = ctx->cfg;
  *handled = false;
  if (c.io_dtype != LA_BF16 || c.d != tc::D) return cudaSuccess;
  if ((tc::long_epilogue(c.conv_taps) ? tc::smem_bytes_long(c.conv_taps) : tc::smem_bytes(c.conv_taps)) > 227u * 1024u)
    return cudaSuccess;                                                  // (does not happen up to LA_MAX_TAPS)
  const int BH = B * c.H;
  CUtensorMap mq, mk, mv, mo;
  if (!tc::make_map(&mq, q, BH, T) || !tc::make_map(&mk, k, BH, T) || !tc::make_map(&mv, v, BH, T) ||
      !tc::make_map(&mo, o, BH, T))
    return cudaErrorNotSupported;   // the driver cannot encode tensor maps: reported, never a silent slow path
  int nseg, seg_len;
  plan_split(ctx, BH, T, &nseg, &seg_len);
  if (nseg > 1 && (ctx->ws == nullptr || ctx->ws_bytes < split_bytes(c, BH, nseg) || T < c.conv_taps)) nseg = 1, seg_len = T;
  const bool elu = c.phi == LA_PHI_ELU1;
  cudaError_t e;
  if (nseg == 1) {
    e = elu ? launch_w<LA_PHI_ELU1>(c, BH, T, mq, mk, mv, mo, w, init, st.S, st.z, (__nv_bfloat16*)st.win, st.pos,
                                    ctx->d_status, 1, T, nullptr, nullptr, s)
            : launch_w<LA_PHI_RELU>(c, BH, T, mq, mk, mv, mo, w, init, st.S, st.z, (__nv_bfloat16*)st.win, st.pos,
                                    ctx->d_status, 1, T, nullptr, nullptr, s);
    ctx->launches += 1;
    *handled = true;
    return e;
  }
  // Sequence split: local states of all segments, prefix over the segments, then every segment as its own CTA.
  const int units = BH * nseg;
  float* S_seg = static_cast<float*>(ctx->ws);
  float* z_seg = S_seg + (size_t)units * tc::D * tc::D;
  __nv_bfloat16* win_seg = reinterpret_cast<__nv_bfloat16*>(z_seg + (size_t)units * tc::D);
  auto skern = elu ? tc::segment_state_kernel<LA_PHI_ELU1> : tc::segment_state_kernel<LA_PHI_RELU>;
  e = cudaFuncSetAttribute(skern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kStateSmem);
  if (e != cudaSuccess) return e;
  skern<<<dim3(BH * (nseg - 1)), dim3(tc::kStateThreads), tc::kStateSmem, s>>>(mk, mv, S_seg, z_seg, ctx->d_status, T, nseg,
                                                                               seg_len, nseg - 1);
  tc::prefix_kernel<<<dim3(BH, tc::D * tc::D / 1024), dim3(256), 0, s>>>(S_seg, z_seg, win_seg, (const __nv_bfloat16*)v, st.S,
                                                                          st.z, (__nv_bfloat16*)st.win, st.pos, c.H, T,
                                                                          c.conv_taps, nseg, seg_len, init);
  e = elu ? launch_w<LA_PHI_ELU1>(c, units, T, mq, mk, mv, mo, w, 1, S_seg, z_seg, win_seg, st.pos, ctx->d_status, nseg,
                                  seg_len, st.S, st.z, s)
          : launch_w<LA_PHI_RELU>(c, units, T, mq, mk, mv, mo, w, 1, S_seg, z_seg, win_seg, st.pos, ctx->d_status, nseg,
                                  seg_len, st.S, st.z, s);
  ctx->launches += 3;
  *handled = true;
  return e;
}

// The three-branch block on the tensor cores: bf16 io, d = 128, groups of 32 to 128 tokens (one tile per group, partly
// filled below 128: a group of 64 runs the tensor cores half empty and still beats the CUDA-core kernel seven times;
// below 32 that kernel takes over), and few enough taps for the 4 KB of extra shared memory.  Sets *handled to false otherwise (the CUDA-core kernel takes those).
cudaError_t launch_prefill_grouped_tc(la_ctx* ctx, int B, int T, const void* q, const void* k, const void* v, const float* w,
                                      int group, float alpha, float scale, int init, const la_state& st, void* o,
                                      cudaStream_t s, bool* handled) {
  const la_config& c = ctx->cfg;
  *handled = false;
  if (c.io_dtype != LA_BF16 || c.d != tc::D || group < 32 || group > tc::TILE) return cudaSuccess;
  if (tc::smem_bytes_grp(c.conv_taps, tc::long_epilogue(c.conv_taps, true)) > 227u * 1024u) return cudaSuccess;
  const int BH = B * c.H;
  CUtensorMap mq, mk, mv, mo;
  if (!tc::make_map(&mq, q, BH, T, group) || !tc::make_map(&mk, k, BH, T, group) || !tc::make_map(&mv, v, BH, T, group) ||
      !tc::make_map(&mo, o, BH, T, group))
    return cudaErrorNotSupported;
  cudaError_t e = c.phi == LA_PHI_ELU1
                      ? launch_w<LA_PHI_ELU1>(c, BH, T, mq, mk, mv, mo, w, init, st.S, st.z, (__nv_bfloat16*)st.win, st.pos,
                                              ctx->d_status, 1, T, nullptr, nullptr, s, true, alpha, scale, group)
                      : launch_w<LA_PHI_RELU>(c, BH, T, mq, mk, mv, mo, w, init, st.S, st.z, (__nv_bfloat16*)st.win, st.pos,
                                              ctx->d_status, 1, T, nullptr, nullptr, s, true, alpha, scale, group);
  ctx->launches += 1;
  *handled = true;
  return e;
}

// The sums of one segment on the tensor cores (bf16 io, d = 128): the kernel of the sequence split with one segment
// per (batch, head) chain.
cudaError_t launch_segment_state_tc(la_ctx* ctx, int B, int T, const void* k, const void* v, float* dS, float* dz,
                                    cudaStream_t s, bool* handled) {
  const la_config& c = ctx->cfg;
  *handled = false;
  if (c.io_dtype != LA_BF16 || c.d != tc::D) return cudaSuccess;
  const int BH = B * c.H;
  CUtensorMap mk, mv;
  if (!tc::make_map(&mk, k, BH, T) || !tc::make_map(&mv, v, BH, T)) return cudaErrorNotSupported;
  auto skern = c.phi == LA_PHI_ELU1 ? tc::segment_state_kernel<LA_PHI_ELU1> : tc::segment_state_kernel<LA_PHI_RELU>;
  cudaError_t e = cudaFuncSetAttribute(skern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kStateSmem);
  if (e != cudaSuccess) return e;
  skern<<<dim3(BH), dim3(tc::kStateThreads), tc::kStateSmem, s>>>(mk, mv, dS, dz, ctx->d_status, T, 1, T, 1);
  ctx->launches += 1;
  *handled = true;
  return cudaGetLastError();
}

}  // namespace la
