// Causal multi-head attention backward on the 5th-generation tensor cores (tcgen05 + TMEM + TMA),
// bf16, head width 64 or 128, sequence length a multiple of 128.  Two kernels, no atomics,
// bit-reproducible (product counts below are for head width 64; at 128 every operand tile is two
// 64-feature blocks, the contractions over features take twice the products and dQ, dK, dV are two
// 64-column blocks each):
//
//   attn_bwd_dkv_t5_kernel   persistent CTAs; for each 128-row key tile of a (sequence, head) it walks the
//       query tiles i >= key tile and keeps dK, dV as fp32 accumulators in tensor memory:
//         S^T = K Q^T, dP^T = V dO^T                (M128 N128 K16 x4 each, operands K-major)
//         P^T = exp(S^T/sqrt(dh) - lse[q]),  dS^T = P^T (dP^T - D[q])      (one thread per key row; the
//                                                    results go back to tensor memory as bf16)
//         dV += P^T dO,  dK += dS^T Q               (M128 N64 K16 x8 each; left operand read from
//                                                    tensor memory, dO and Q used as loaded:
//                                                    MN-major right operands)
//   attn_bwd_dq_t5_kernel    persistent CTAs; for each 128-row query tile of a (sequence, head) it walks the
//       key tiles j <= query tile and keeps dQ in tensor memory:
//         S = Q K^T, dP = dO V^T,  dS = P (dP - D[row]),  dQ += dS K   (K as loaded: MN-major)
//
// D[row] = sum(dO * O) is computed by the dQ kernel from its staged dO and O tiles and left in global
// memory for the dK/dV kernel, which runs second (head width 128: shared memory has no room for O,
// both kernels read D from global memory, where a small kernel has put it beforehand).
// Warp roles (struct Roles below): warp 0 TMA producer, warp 1 tensor-memory owner + issuer of the score
// products, then the element-wise warps (thread = accumulator lane; four warps per lane quarter at head
// width 64, two at 128), one warp that issues the accumulating products, four warps that move finished
// accumulators to global memory, and in the dK/dV kernel at head width 64 one warp that prepares the row
// statistics of each stage.  At head width 64 the statistics enter the score products as one more
// contraction step ("augmented contraction" below), so the element-wise threads never read them.
// All mbarrier waits are bounded (tc_common.cuh); on expiry a code is left in `status`.
#include "host_common.h"
#include "tc_common.cuh"

namespace sl {
namespace {

using namespace tc;

constexpr int DH = 64;
constexpr int BT = 128;                   // rows of a query tile and of a key tile
constexpr int TILE = BT * DH * 2;         // 16 KB: one [128 x 64] bf16 tile
constexpr int OUT_THREADS = 128;
// Warp roles: warp 0 TMA, warp 1 score products, then the element-wise warps (EWQ per accumulator lane
// quarter, each computing CW of a half's 64 columns), one warp for the accumulating products, and four
// output warps that move finished accumulators to global memory.  Head width 64 takes four
// element-wise warps per quarter: the element-wise work is a chain of dependent instructions per element,
// and two warps per scheduler left it waiting on its own latencies for half of the time.  Head width 128
// keeps two (P^T and dS^T are written over the score columns there, chunk by chunk of 32).
template <int DHT> struct Roles {
  static constexpr int EWQ = DHT == 64 ? 4 : 2;
  static constexpr int CW = 64 / EWQ;
  static constexpr int EW_THREADS = 128 * EWQ;
  static constexpr int ACC_WARP = 2 + 4 * EWQ;
  static constexpr int OUT_WARP0 = ACC_WARP + 1;
  // Head width 64 folds the row statistics into the score products (see "augmented contraction" below);
  // one more warp turns them into the operand rows that carries them.
  static constexpr bool AUG = DHT == 64;
  static constexpr int STAT_WARP = OUT_WARP0 + 4;               // dK/dV kernel only
  static constexpr int NTHREADS_DQ = (OUT_WARP0 + 4) * 32;
  static constexpr int NTHREADS_DKV = (OUT_WARP0 + 4 + (AUG ? 1 : 0)) * 32;
};

// Augmented contraction.  The element-wise threads need exp(scale * S - lse) and dP - D, where lse and D
// belong to the query (a row of the dQ kernel's tiles, a column of the dK/dV kernel's).  Both shifts are
// rank-one terms, so the tensor core adds them: each score product takes one more 16-deep step whose
// operands are a constant tile of ones and a tile that holds, per query, -lse/scale and -D, each as a sum of
// two bf16 values (hi + lo: the pair carries 16 mantissa bits, the products with 1 are exact and the
// accumulation is fp32).  The accumulators then hold S - lse/scale and dP - D, and an element costs the
// element-wise threads two multiplications, one exponential and the conversions.
// These tiles are [128 rows x 16] bf16, K-major without swizzle: 8-row groups of 256 bytes, in a group the
// 16-byte rows of columns 0..7 (128 bytes) and then those of columns 8..15.  Columns: 0, 1 = -lse/scale
// (hi, lo), 2, 3 = -D (hi, lo), the rest zero; the constant tiles have ones in columns 0, 1 (for S) or 2, 3
// (for dP).
constexpr int AUG_TILE = 128 * 16 * 2;
constexpr uint32_t DESC_HI_AUG = (uint32_t)(256 >> 4) | (1u << 14);           // 8-row groups 256 bytes apart, no swizzle
__device__ __forceinline__ uint32_t desc_lo_aug(uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | ((uint32_t)(128 >> 4) << 16); }
__device__ __forceinline__ void tc_mma_aug(uint32_t d_tmem, uint32_t alo, uint32_t blo, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, 1, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(alo), "r"(blo), "r"(DESC_HI_AUG), "r"(idesc) : "memory");
}
// byte offset of row r's columns 0..7 inside such a tile
__device__ __forceinline__ uint32_t aug_row(int r) { return (uint32_t)(r >> 3) * 256u + (uint32_t)(r & 7) * 16u; }
// -x as hi + lo, two bf16 values in one word (hi in the low half)
__device__ __forceinline__ uint32_t neg_split(float x) {
  const __nv_bfloat16 hi = __float2bfloat16_rn(-x);
  const __nv_bfloat16 lo = __float2bfloat16_rn(-x - __bfloat162float(hi));
  return (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(lo) << 16);
}
// zeroes `bytes` of shared memory and writes the two constant tiles: ones in columns 0, 1 / in columns 2, 3
__device__ __forceinline__ void aug_init(uint8_t* ones_s, uint8_t* ones_d, int rows, uint8_t* zero, int zero_bytes) {
  for (int i = threadIdx.x; i < zero_bytes / 16; i += blockDim.x) reinterpret_cast<uint4*>(zero)[i] = make_uint4(0u, 0u, 0u, 0u);
  for (int i = threadIdx.x; i < rows * 2; i += blockDim.x) {       // 16-byte pieces: row i / 2, columns 0..7 or 8..15
    const int r = i >> 1;
    const uint32_t off = aug_row(r) + (uint32_t)(i & 1) * 128u;
    const uint32_t one2 = 0x3F803F80u;
    *reinterpret_cast<uint4*>(ones_s + off) = make_uint4((i & 1) ? 0u : one2, 0u, 0u, 0u);
    *reinterpret_cast<uint4*>(ones_d + off) = make_uint4(0u, (i & 1) ? 0u : one2, 0u, 0u);
  }
}
constexpr int TMEM_COLS = 512;
constexpr uint32_t IDESC_64KK = make_idesc(BT, DH);                   // [128 x 64] products, both operands K-major
constexpr uint32_t IDESC_64MN = make_idesc(BT, DH) | (1u << 16);      // [128 x 64] products, right operand MN-major
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// 16 consecutive tensor-memory columns of this thread's lane
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
// 8 packed words of this thread's lane to 8 consecutive tensor-memory columns
__device__ __forceinline__ void tc_st8(uint32_t taddr, const uint32_t* w) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
      ::"r"(taddr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
}
template <int CW> __device__ __forceinline__ void tc_ld_cw(uint32_t taddr, float* v) {
  if constexpr (CW == 32) tc_ld32(taddr, v); else tc_ld16(taddr, v);
}
template <int CW> __device__ __forceinline__ void tc_st_cw(uint32_t taddr, const uint32_t* w) {   // CW / 2 packed words
  if constexpr (CW == 32) tc_st16(taddr, w); else tc_st8(taddr, w);
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
}
// one row (lane r) of a [128 x 64] bf16 tile in the 128-byte-swizzled layout: 16-byte chunk jj
__device__ __forceinline__ void st_row_chunk(uint32_t tile, int r, uint32_t jj, const uint32_t* w) {
  const uint32_t addr = tile + (uint32_t)r * 128u + ((jj ^ ((uint32_t)r & 7u)) << 4);
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
}
// Operand descriptors are passed as their address-carrying lower halves (desc_lo); the upper half
// is the same constant for the K-major tiles and for the MN-major ones (128-byte rows, 128-byte
// swizzle, 8-row groups 1024 bytes apart), so a product costs the issuing thread two adds.
//
// 4 products [128 x 64] += A[:, 64h .. 64h+63] * B rows [64h, 64h + 64): one half of the contraction
// over a 128-row tile.  A (P^T, dS^T or dS, bf16) lives in tensor memory at a_tmem: 128 contraction
// elements = 64 columns, so half h starts 32 columns in and each product advances 8 columns.  B is an
// MN-major tile used as loaded (lower descriptor half blo); 16 of its rows = 2048 bytes = 128 units.
// With SPREAD the 64 columns of A are not side by side: each 32-column chunk of the fp32 tile they
// were computed from holds 16 of them in its first half, so half h starts 64 columns in and the
// third product hops to the next chunk.
template <bool SPREAD = false>
__device__ __forceinline__ void mma_acc_half(uint32_t d_tmem, uint32_t a_tmem, uint32_t blo, int h, bool fresh) {
  const uint32_t a0 = a_tmem + (uint32_t)((SPREAD ? 64 : 32) * h), b0 = blo + (uint32_t)(512 * h);
  constexpr uint32_t HOP = SPREAD ? 32u : 16u;
  tc_mma_ts_lo(d_tmem, a0, b0, IDESC_64MN, fresh ? 0u : 1u);
  tc_mma_ts_lo(d_tmem, a0 + 8, b0 + 128, IDESC_64MN, 1u);
  tc_mma_ts_lo(d_tmem, a0 + HOP, b0 + 256, IDESC_64MN, 1u);
  tc_mma_ts_lo(d_tmem, a0 + HOP + 8, b0 + 384, IDESC_64MN, 1u);
}
// 4 products [128 x 64] = A[128 x 64] * (rows [64h, 64h + 64) of the K-major tile at blo)^T:
// one half (64 columns) of a [128 x 128] score tile.  64 rows of 128 bytes = 512 descriptor units.
__device__ __forceinline__ void mma_score_half(uint32_t d_tmem, uint32_t alo, uint32_t blo, int h, bool fresh = true) {
  const uint32_t b0 = blo + (uint32_t)(512 * h);
  tc_mma_lo(d_tmem, alo, b0, IDESC_64KK, fresh ? 0u : 1u);
  tc_mma_lo_acc(d_tmem, alo + 2, b0 + 2, IDESC_64KK);
  tc_mma_lo_acc(d_tmem, alo + 4, b0 + 4, IDESC_64KK);
  tc_mma_lo_acc(d_tmem, alo + 6, b0 + 6, IDESC_64KK);
}

struct BwdParams {
  int T, H, d;
  float scale;             // 1/sqrt(dh)
  const float* lse;        // [nseq, H, T] natural log
  int nitems;              // nseq * H (sequence, head) items, shared out over the CTAs
  const float* rowdot;     // [nseq, H, T]: D[row] = sum(dO * O), read by the dK/dV kernel
  float* rowdot_out;       // the same buffer, written by the dQ kernel (which runs first)
  int* status;
};

#define T5_SETUP(NBARS, CNT128_A, CNT128_B, CNT128_C, CNT128_D, CNT_OUT, CNT2_LO, CNT2_HI, CNT_OUT_LO, CNT_OUT_HI)                                                     \
  extern __shared__ uint8_t smem_raw[];                                                                   \
  const uint32_t raw = smem_u32(smem_raw);                                                                \
  const uint32_t base = (raw + 1023u) & ~1023u;                                                           \
  uint8_t* base_ptr = smem_raw + (base - raw);                                                            \
  const uint32_t bar = base + OFF_BAR;                                                                    \
  auto B = [&](int i) { return bar + 8u * i; };                                                           \
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + OFF_BAR + 8 * NBARS);    \
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + OFF_BAR + 8 * NBARS + 8);         \
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;                                             \
  if (threadIdx.x == 0) {                                                                                 \
    for (int i = 0; i < NBARS; ++i)                                                                       \
      mbar_init(B(i), (i == CNT128_A || i == CNT128_B || i == CNT128_C || i == CNT128_D) ? EW_THREADS : (i == CNT_OUT || (i >= CNT_OUT_LO && i < CNT_OUT_HI)) ? OUT_THREADS \
                      : (i >= CNT2_LO && i < CNT2_HI) ? 2 : 1);                                           \
    *abort_flag = 0;                                                                                      \
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");                                    \
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");                                          \
  }                                                                                                       \
  if (warp == 1) {                                                                                        \
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"                      \
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)TMEM_COLS) : "memory");           \
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");              \
  }                                                                                                       \
  tc_fence_before();                                                                                      \
  __syncthreads();                                                                                        \
  tc_fence_after();                                                                                       \
  const uint32_t tmem_base = *tmem_slot;

#define T5_TEARDOWN()                                                                                     \
  __syncwarp();                                                                                           \
  if (*abort_flag) { for (int i = 0; i < 2000; ++i) __nanosleep(1000); }                                  \
  tc_fence_before();                                                                                      \
  __syncthreads();                                                                                        \
  if (warp == 1) {                                                                                        \
    tc_fence_after();                                                                                     \
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory"); \
  }

// parity to wait on for "the n-th completion (0-based) of this barrier has happened"
__device__ __forceinline__ uint32_t done(int n) { return (uint32_t)n & 1u; }
// parity to wait on before the n-th use of a slot whose release is signalled once per use
__device__ __forceinline__ uint32_t freed(int n) { return ((uint32_t)n & 1u) ^ 1u; }

// ==========================================================================================
// dK, dV
// ==========================================================================================
namespace dkv {
enum { KV_FULL = 0 /*+buffer*/, KV_FULL1, KV_EMPTY /*+buffer*/, KV_EMPTY1, QD_FULL /*+s*/, QD_FULL1, QD_FULL2,
       QD_EMPTY /*+s*/, QD_EMPTY1, QD_EMPTY2, S_FULL /*+half*/, S_FULL1, S_FREE /*+half*/, S_FREE1,
       P_READY /*+half*/, P_READY1, P_FREE /*+half*/, P_FREE1, ACC_FULL, ACC_FREE, AUG_READY /*+s*/, AUG_READY1, AUG_READY2,
       N_BARS };
// Head width 64: K, V of a key tile are double buffered (the next key tile's arrive during this
// one's last steps); Q, dO and the row statistics of a step go through a ring of three stages; P^T
// and dS^T have tensor-memory columns of their own.
// Head width 128: every operand is two 64-feature blocks and dK, dV take 128 columns each, which
// fills tensor memory next to S^T and dP^T.  P^T and dS^T are then written over the S^T and dP^T
// columns they were computed from (each thread over the first half of its own 32-column chunk), and
// a half of S^T / dP^T is only recomputed once the accumulating products that read it have
// finished.  Shared memory holds one K / V buffer, two Q / dO stages and a two-block staging area
// through which dK and then dV leave.
template <int DHT> struct Cfg {
  static constexpr int NB = DHT / 64;
  static constexpr bool ALIAS = DHT == 128;
  static constexpr int KVB = DHT == 64 ? 2 : 1;
  static constexpr int RINGN = DHT == 64 ? 3 : 2;
  static constexpr int OFF_KV = 0;                                  // buffer kb: K blocks at +kb*2*NB*TILE, V blocks after them
  static constexpr int OFF_QD = KVB * 2 * NB * TILE;                // stage s: Q blocks at +s*2*NB*TILE, dO blocks after them
  static constexpr int OFF_OUT = OFF_QD + RINGN * 2 * NB * TILE;    // two blocks staged for the TMA stores
  static constexpr int OFF_STAT = OFF_OUT + 2 * TILE;               // stage s: lse at +s*1024, D at +512
  static constexpr int OFF_AUG = OFF_STAT + RINGN * 1024;           // ones for S^T, ones for dP^T, then one tile per stage
  static constexpr int OFF_BAR = OFF_AUG + (DHT == 64 ? (2 + RINGN) * AUG_TILE : 0);
  static constexpr int USED = OFF_BAR + 256;
  static constexpr int SMEM = DHT == 64 ? USED + 1024 : 232448;     // width 128 takes all a CTA can have
};
}  // namespace dkv

template <int DHT>
__global__ void __launch_bounds__(Roles<DHT>::NTHREADS_DKV, 1)
attn_bwd_dkv_t5_kernel(const __grid_constant__ CUtensorMap mapQKV, const __grid_constant__ CUtensorMap mapDO,
                       const __grid_constant__ CUtensorMap mapDQKV, BwdParams p) {
  using namespace dkv;
  using C = Cfg<DHT>;
  constexpr int CW = Roles<DHT>::CW, EW_THREADS = Roles<DHT>::EW_THREADS, ACC_WARP = Roles<DHT>::ACC_WARP,
                OUT_WARP0 = Roles<DHT>::OUT_WARP0, STAT_WARP = Roles<DHT>::STAT_WARP, OFF_AUG = C::OFF_AUG;
  constexpr bool AUG = Roles<DHT>::AUG;
  constexpr int NB = C::NB, KVB = C::KVB, RINGN = C::RINGN, OFF_KV = C::OFF_KV, OFF_QD = C::OFF_QD, OFF_OUT = C::OFF_OUT,
                OFF_STAT = C::OFF_STAT, OFF_BAR = C::OFF_BAR;
  constexpr bool ALIAS = C::ALIAS;
  {
    // the tiles start at the next 1024-byte boundary of the dynamic shared memory: leave, with a
    // code, if what is left after that does not hold them (nothing has been set up yet)
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw0 = smem_u32(smem_raw);
    if ((((raw0 + 1023u) & ~1023u) - raw0) + (uint32_t)C::USED > (uint32_t)C::SMEM) {
      if (threadIdx.x == 0) atomicExch(p.status, 90);
      return;
    }
  }
  T5_SETUP(N_BARS, S_FREE, S_FREE1, P_READY, P_READY1, ACC_FREE, QD_EMPTY, QD_EMPTY + RINGN, 0, 0)
  if (AUG) {
    aug_init(base_ptr + OFF_AUG, base_ptr + OFF_AUG + AUG_TILE, BT, base_ptr + OFF_AUG + 2 * AUG_TILE, RINGN * AUG_TILE);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
  }
  const int nq = p.T / BT;
  // persistent: the work units are (item, tile) pairs, item = (sequence, head).  The grid is a multiple of
  // nq CTAs; in round t the CTAs nq*s .. nq*s + nq-1 take the nq tiles of one item (the s-th of the round's
  // block of items), so an item's Q, K, V and dO are read from memory once and found in L2 by its other
  // tiles, which run at about the same time; which tile a CTA takes rotates with the round, so that every
  // CTA gets the same mix of long and short tiles.  Every role walks its units in one flat loop, so loads
  // for the next unit are issued while this one ends.
  const int ipb = (int)gridDim.x / nq, slot = (int)blockIdx.x / nq, pos = (int)blockIdx.x % nq;
  const int my_tiles = (slot < ipb && slot < p.nitems) ? (p.nitems - slot + ipb - 1) / ipb : 0;
  const uint32_t tS = tmem_base, tDP = tmem_base + 128u, tDV = tmem_base + 256u, tDK = tmem_base + 256u + (uint32_t)DHT;
  // P^T, dS^T (bf16): 64 columns each after dK, or on top of S^T and dP^T
  const uint32_t tPT = ALIAS ? tS : tmem_base + 384u, tDST = ALIAS ? tDP : tmem_base + 448u;

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      int s = 0, n = 0;                            // ring stage and how often it has been used
      for (int tk = 0; tk < my_tiles && ok; ++tk) {
        const int item = tk * ipb + slot, kt = (pos + tk) % nq;
        const int h = item % p.H, b = item / p.H;      // this CTA walks several (sequence, head) items
        const int seq_row0 = b * p.T;
        const size_t stat0 = ((size_t)b * p.H + h) * p.T;
        (void)seq_row0; (void)stat0;
        const int kb = tk % KVB;
        if (!mbar_wait(B(KV_EMPTY + kb), freed(tk / KVB), abort_flag, p.status, 41)) { ok = false; break; }
        mbar_expect_tx(B(KV_FULL + kb), 2 * NB * TILE);
        const uint32_t kv = base + OFF_KV + kb * 2 * NB * TILE;
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          tma_load_2d(kv + nb * TILE, &mapQKV, B(KV_FULL + kb), p.d + h * DHT + 64 * nb, seq_row0 + kt * BT);
          tma_load_2d(kv + (NB + nb) * TILE, &mapQKV, B(KV_FULL + kb), 2 * p.d + h * DHT + 64 * nb, seq_row0 + kt * BT);
        }
        for (int i = kt; i < nq; ++i) {
          if (!mbar_wait(B(QD_EMPTY + s), freed(n), abort_flag, p.status, 42)) { ok = false; break; }
          mbar_expect_tx(B(QD_FULL + s), 2 * NB * TILE + 1024);
          const uint32_t qd = base + OFF_QD + s * 2 * NB * TILE;
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) {
            tma_load_2d(qd + nb * TILE, &mapQKV, B(QD_FULL + s), h * DHT + 64 * nb, seq_row0 + i * BT);
            tma_load_2d(qd + (NB + nb) * TILE, &mapDO, B(QD_FULL + s), h * DHT + 64 * nb, seq_row0 + i * BT);
          }
          bulk_load(base + OFF_STAT + s * 1024, p.lse + stat0 + (size_t)i * BT, 512, B(QD_FULL + s));
          bulk_load(base + OFF_STAT + s * 1024 + 512, p.rowdot + stat0 + (size_t)i * BT, 512, B(QD_FULL + s));
          if (++s == RINGN) { s = 0; ++n; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- score products: S^T = K Q^T, dP^T = V dO^T ----------------
    // Half hh (64 query columns) of a step needs the step's Q/dO stage and the previous step's reads
    // of that half done.  The halves are separate products so that the next step's first half is
    // computed while the element-wise warps still work on this step's second.  The accumulating
    // products are issued by another thread (warp ACC_WARP): one thread cannot issue 32 products of
    // 48 cycles each per step next to the busy element-wise warps.
    if (lane == 0) {
      bool ok = true;
      int it = 0, s = 0, n = 0;
      const uint32_t lo_kv = desc_lo(base + OFF_KV), lo_qd = desc_lo(base + OFF_QD), lo_aug = desc_lo_aug(base + OFF_AUG);
      constexpr uint32_t TILE16 = TILE >> 4;
      for (int tk = 0; tk < my_tiles && ok; ++tk) {
        const int item = tk * ipb + slot, kt = (pos + tk) % nq;
        const int h = item % p.H, b = item / p.H;      // this CTA walks several (sequence, head) items
        const int seq_row0 = b * p.T;
        const size_t stat0 = ((size_t)b * p.H + h) * p.T;
        (void)seq_row0; (void)stat0;
        const int kb = tk % KVB;
        const uint32_t lo_k = lo_kv + (uint32_t)(kb * 2 * NB) * TILE16, lo_v = lo_k + (uint32_t)NB * TILE16;
        if (!mbar_wait(B(KV_FULL + kb), done(tk / KVB), abort_flag, p.status, 45)) { ok = false; break; }
        for (int i = kt; i < nq && ok; ++i, ++it) {
          const uint32_t lo_q = lo_qd + (uint32_t)(s * 2 * NB) * TILE16, lo_do = lo_q + (uint32_t)NB * TILE16;
          if (!mbar_wait(B(QD_FULL + s), done(n), abort_flag, p.status, 43)) { ok = false; break; }
          if (AUG && !mbar_wait(B(AUG_READY + s), done(n), abort_flag, p.status, 52)) { ok = false; break; }
          const uint32_t lo_aq = lo_aug + (uint32_t)((2 + s) * AUG_TILE >> 4);      // this stage's -lse/scale, -D rows
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            // the half's columns are free once read (own P^T columns) or, where P^T and dS^T lie on
            // top of them, once the accumulating products of the previous step have used those
            if (!mbar_wait(B((ALIAS ? P_FREE : S_FREE) + hh), freed(it), abort_flag, p.status, 44)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int nb = 0; nb < NB; ++nb)           // contraction over the head's features, 64 per block
              mma_score_half(tS + 64u * hh, lo_k + (uint32_t)nb * TILE16, lo_q + (uint32_t)nb * TILE16, hh, nb == 0);
            // one more step: ones x (-lse/scale) of the half's 64 queries (8 row groups = 2048 bytes per half)
            if (AUG) tc_mma_aug(tS + 64u * hh, lo_aug, lo_aq + (uint32_t)(128 * hh), IDESC_64KK);
#pragma unroll
            for (int nb = 0; nb < NB; ++nb)
              mma_score_half(tDP + 64u * hh, lo_v + (uint32_t)nb * TILE16, lo_do + (uint32_t)nb * TILE16, hh, nb == 0);
            if (AUG) tc_mma_aug(tDP + 64u * hh, lo_aug + (uint32_t)(AUG_TILE >> 4), lo_aq + (uint32_t)(128 * hh), IDESC_64KK);
            tc_commit(B(S_FULL + hh));
          }
          if (ok) tc_commit(B(QD_EMPTY + s));        // second arrival comes from the accumulating thread
          if (++s == RINGN) { s = 0; ++n; }
        }
        if (ok) tc_commit(B(KV_EMPTY + kb));         // K, V are read by these products only
      }
    }
  } else if (warp == ACC_WARP) {
    // ---------------- accumulating products: dV += P^T dO, dK += dS^T Q ----------------
    if (lane == 0) {
      bool ok = true;
      int it = 0, s = 0, n = 0;
      const uint32_t lo_qd = desc_lo(base + OFF_QD);
      constexpr uint32_t TILE16 = TILE >> 4;
      for (int tk = 0; tk < my_tiles && ok; ++tk) {
        const int item = tk * ipb + slot, kt = (pos + tk) % nq;
        const int h = item % p.H, b = item / p.H;      // this CTA walks several (sequence, head) items
        const int seq_row0 = b * p.T;
        const size_t stat0 = ((size_t)b * p.H + h) * p.T;
        (void)seq_row0; (void)stat0;
        // the accumulators of the previous key tile must have been read
        if (!mbar_wait(B(ACC_FREE), freed(tk), abort_flag, p.status, 46)) { ok = false; break; }
        for (int i = kt; i < nq && ok; ++i, ++it) {
          const uint32_t lo_q = lo_qd + (uint32_t)(s * 2 * NB) * TILE16, lo_do = lo_q + (uint32_t)NB * TILE16;
          if (!mbar_wait(B(QD_FULL + s), done(n), abort_flag, p.status, 43)) { ok = false; break; }
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            if (!mbar_wait(B(P_READY + hh), done(it), abort_flag, p.status, 47)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int nb = 0; nb < NB; ++nb)           // one 64-column block of dV per block of dO
              mma_acc_half<ALIAS>(tDV + 64u * nb, tPT, lo_do + (uint32_t)nb * TILE16, hh, i == kt && hh == 0);
#pragma unroll
            for (int nb = 0; nb < NB; ++nb)
              mma_acc_half<ALIAS>(tDK + 64u * nb, tDST, lo_q + (uint32_t)nb * TILE16, hh, i == kt && hh == 0);
            tc_commit(B(P_FREE + hh));
          }
          if (ok) tc_commit(B(QD_EMPTY + s));
          if (++s == RINGN) { s = 0; ++n; }
        }
        if (ok) tc_commit(B(ACC_FULL));
      }
    }
  } else if (warp < ACC_WARP) {
    // ---------------- element-wise warps (2 .. ACC_WARP - 1) ----------------
    const int q4 = warp & 3;
    const int wsel = (warp - 2) >> 2;            // which of the EWQ warps of this accumulator lane quarter
    const int r = q4 * 32 + lane;                // key row inside the tile = accumulator lane
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const float scale_log2 = p.scale * LOG2E;
    const uint64_t sc2 = pack2(scale_log2, scale_log2), nlog2 = pack2(-LOG2E, -LOG2E), neg1 = pack2(-1.f, -1.f);
    bool ok = true;
    int it = 0, s = 0, n = 0;
    for (int tk = 0; tk < my_tiles; ++tk) {
      const int item = tk * ipb + slot, kt = (pos + tk) % nq;
      const int h = item % p.H, b = item / p.H;      // this CTA walks several (sequence, head) items
      const int seq_row0 = b * p.T;
      const size_t stat0 = ((size_t)b * p.H + h) * p.T;
      (void)seq_row0; (void)stat0;
      for (int i = kt; i < nq && ok; ++i, ++it) {
        const float* Ls = reinterpret_cast<const float*>(base_ptr + OFF_STAT + s * 1024);
        const float* Ds = Ls + 128;
        (void)Ls; (void)Ds;
        // (with the statistics folded into the products these threads read nothing of the stage)
        if (!AUG && !mbar_wait(B(QD_FULL + s), done(n), abort_flag, p.status, 48)) { ok = false; break; }
        const bool diag = (i == kt);
        // The 128 query columns go in two halves of 64 (one CW-column chunk per warp and half): the
        // products that contract over the first half run while the second half is being computed.
#pragma unroll 1
        for (int hh = 0; hh < 2; ++hh) {
          const int c = hh * 64 + wsel * CW;
          if (!mbar_wait(B(S_FULL + hh), done(it), abort_flag, p.status, 49)) { ok = false; break; }
          // (with P^T on top of S^T, S_FULL already implies that the previous step's products are done)
          if (!ALIAS && !mbar_wait(B(P_FREE + hh), freed(it), abort_flag, p.status, 50)) { ok = false; break; }
          tc_fence_after();
          uint32_t pk[CW / 2], dk[CW / 2];
          // on the diagonal tile only queries >= this key count: chunks wholly before the warp's rows are zero
          if (!diag || c + CW > q4 * 32) {
            float sv[CW], dv[CW];
            tc_ld_cw<CW>(tS + lane_off + (uint32_t)c, sv);
            tc_ld_cw<CW>(tDP + lane_off + (uint32_t)c, dv);
            tc_wait_ld();
            if (!ALIAS) {                              // the values are in registers: this half of S^T, dP^T
              tc_fence_before();                       // may be overwritten by the next step's products
              mbar_arrive(B(S_FREE + hh));
            }
            // The causal mask goes onto the scores first (exp2(-inf) = 0), so that the element loop
            // below has no test in it: with one, every element is a basic block of its own and the
            // independent chains run one after another instead of interleaved.
            if (diag && c < q4 * 32 + 32) {
#pragma unroll
              for (int e = 0; e < CW; ++e) sv[e] = (c + e < r) ? -INFINITY : sv[e];
            }
            if constexpr (AUG) {
              // the accumulators hold S^T - lse/scale and dP^T - D already
#pragma unroll
              for (int e = 0; e < CW; e += 2) {
                float a0, a1, g0, g1;
                unpack2(mul2(pack2(sv[e], sv[e + 1]), sc2), a0, a1);
                const float p0 = ex2(a0), p1 = ex2(a1);
                unpack2(mul2(pack2(p0, p1), pack2(dv[e], dv[e + 1])), g0, g1);
                __nv_bfloat162 pa = __floats2bfloat162_rn(p0, p1), da = __floats2bfloat162_rn(g0, g1);
                pk[e >> 1] = *reinterpret_cast<uint32_t*>(&pa);
                dk[e >> 1] = *reinterpret_cast<uint32_t*>(&da);
              }
            } else {
#pragma unroll
            for (int e = 0; e < CW; e += 4) {
              // two elements per instruction: the row statistics come out of shared memory as pairs
              const ulonglong2 l4 = *reinterpret_cast<const ulonglong2*>(Ls + c + e);
              const ulonglong2 d4 = *reinterpret_cast<const ulonglong2*>(Ds + c + e);
              float a0, a1, a2, a3;
              unpack2(fma2(pack2(sv[e], sv[e + 1]), sc2, mul2(l4.x, nlog2)), a0, a1);
              unpack2(fma2(pack2(sv[e + 2], sv[e + 3]), sc2, mul2(l4.y, nlog2)), a2, a3);
              const float p0 = ex2(a0), p1 = ex2(a1), p2 = ex2(a2), p3 = ex2(a3);
              float g0, g1, g2, g3;
              unpack2(mul2(pack2(p0, p1), fma2(d4.x, neg1, pack2(dv[e], dv[e + 1]))), g0, g1);
              unpack2(mul2(pack2(p2, p3), fma2(d4.y, neg1, pack2(dv[e + 2], dv[e + 3]))), g2, g3);
              __nv_bfloat162 pa = __floats2bfloat162_rn(p0, p1), pb = __floats2bfloat162_rn(p2, p3);
              __nv_bfloat162 da = __floats2bfloat162_rn(g0, g1), db = __floats2bfloat162_rn(g2, g3);
              pk[e >> 1] = *reinterpret_cast<uint32_t*>(&pa);
              pk[(e >> 1) + 1] = *reinterpret_cast<uint32_t*>(&pb);
              dk[e >> 1] = *reinterpret_cast<uint32_t*>(&da);
              dk[(e >> 1) + 1] = *reinterpret_cast<uint32_t*>(&db);
            }
            }
          } else {
#pragma unroll
            for (int e = 0; e < CW / 2; ++e) { pk[e] = 0u; dk[e] = 0u; }
            if (!ALIAS) mbar_arrive(B(S_FREE + hh));
          }
          // CW bf16 = CW / 2 columns: packed side by side, or over the first half of the chunk just read
          const uint32_t pcol = ALIAS ? (uint32_t)c : (uint32_t)(c >> 1);
          tc_st_cw<CW>(tPT + lane_off + pcol, pk);
          tc_st_cw<CW>(tDST + lane_off + pcol, dk);
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(B(P_READY + hh));                // this half of P^T, dS^T is complete
        }
        if (!ok) break;
        if (++s == RINGN) { s = 0; ++n; }
      }
    }
  } else if (AUG && warp == STAT_WARP) {
    // ---------------- the queries' -lse/scale and -D of a stage as operand rows ----------------
    bool ok = true;
    int s = 0, n = 0;
    const float inv_scale = 1.0f / p.scale;
    for (int tk = 0; tk < my_tiles && ok; ++tk) {
      const int kt = (pos + tk) % nq;
      for (int i = kt; i < nq; ++i) {
        if (!mbar_wait(B(QD_FULL + s), done(n), abort_flag, p.status, 53)) { ok = false; break; }
        const float* Ls = reinterpret_cast<const float*>(base_ptr + OFF_STAT + s * 1024);
        const float* Ds = Ls + 128;
        uint8_t* rows = base_ptr + OFF_AUG + (2 + s) * AUG_TILE;
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) {
          const int j = lane + 32 * k4;
          *reinterpret_cast<uint2*>(rows + aug_row(j)) = make_uint2(neg_split(Ls[j] * inv_scale), neg_split(Ds[j]));
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(B(AUG_READY + s));
        if (++s == RINGN) { s = 0; ++n; }
      }
    }
  } else if (warp >= OUT_WARP0 && warp < OUT_WARP0 + 4) {
    // ---------------- output: dK (scaled) and dV of a finished key tile ----------------
    // Own warps, so that the element-wise warps go on with the next key tile while the last
    // products of this one drain: tensor memory -> bf16 -> shared memory -> TMA stores.
    const int q4 = warp & 3;
    const int r = q4 * 32 + lane;
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    bool ok = true;
    for (int tk = 0; tk < my_tiles; ++tk) {
      const int item = tk * ipb + slot, kt = (pos + tk) % nq;
      const int h = item % p.H, b = item / p.H;      // this CTA walks several (sequence, head) items
      const int seq_row0 = b * p.T;
      const size_t stat0 = ((size_t)b * p.H + h) * p.T;
      (void)seq_row0; (void)stat0;
      if (ok && !mbar_wait(B(ACC_FULL), done(tk), abort_flag, p.status, 51)) ok = false;
      if (ok) tc_fence_after();
      // dK (scaled), then dV, in 64-column blocks through the two staging tiles; two blocks per store
#pragma unroll
      for (int blk = 0; blk < 2 * NB; ++blk) {
        const int which = blk / NB, nb = blk % NB, slot = blk & 1;
        if (ok) {
          const uint32_t tsrc = (which == 0 ? tDK : tDV) + (uint32_t)(64 * nb);
          const float mul = which == 0 ? p.scale : 1.0f;
#pragma unroll
          for (int c = 0; c < 64; c += 32) {
            float v[32];
            tc_ld32(tsrc + lane_off + (uint32_t)c, v);
            tc_wait_ld();
#pragma unroll
            for (uint32_t jj = 0; jj < 4; ++jj) {
              uint32_t w[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                __nv_bfloat162 ob = __floats2bfloat162_rn(v[8 * jj + 2 * e] * mul, v[8 * jj + 2 * e + 1] * mul);
                w[e] = *reinterpret_cast<uint32_t*>(&ob);
              }
              st_row_chunk(base + OFF_OUT + slot * TILE, r, (uint32_t)(c >> 3) + jj, w);
            }
          }
          if (blk == 2 * NB - 1) {
            tc_fence_before();
            mbar_arrive(B(ACC_FREE));
          }
        }
        if (slot == 1) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          asm volatile("bar.sync 1, 128;" ::: "memory");         // the four output warps (always reached)
          if (ok && warp == OUT_WARP0 && lane == 0) {
            const int pw = (blk - 1) / NB, pnb = (blk - 1) % NB;
            tma_store_2d(&mapDQKV, base + OFF_OUT, (pw + 1) * p.d + h * DHT + 64 * pnb, seq_row0 + kt * BT);
            tma_store_2d(&mapDQKV, base + OFF_OUT + TILE, (which + 1) * p.d + h * DHT + 64 * nb, seq_row0 + kt * BT);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
      }
    }
    if (warp == OUT_WARP0 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }
  T5_TEARDOWN()
}

// ==========================================================================================
// dQ
// ==========================================================================================
namespace dq {
enum { QO_FULL = 0 /*+buffer*/, QO_FULL1, QO_EMPTY /*+buffer*/, QO_EMPTY1, KV_FULL /*+s*/, KV_FULL1, KV_FULL2,
       KV_EMPTY /*+s*/, KV_EMPTY1, KV_EMPTY2, S_FULL /*+half*/, S_FULL1, S_FREE /*+half*/, S_FREE1,
       P_READY /*+half*/, P_READY1, P_FREE /*+half*/, P_FREE1, ACC_FULL, ACC_FREE, AUG_READY /*+buffer*/, AUG_READY1, N_BARS };
// Head width 64: Q, dO and O of a query tile are double buffered (O only serves D[row] = sum(dO * O),
// which the kernel then computes for itself and leaves in global memory for the dK/dV kernel); K, V
// of a step go through a ring of three stages.  Head width 128: every operand is two 64-feature
// blocks, so shared memory holds one Q / dO buffer and a ring of two K / V stages, and D[row] is read
// from global memory (computed beforehand by a kernel of its own).
template <int DHT> struct Cfg {
  static constexpr int NB = DHT / 64;
  static constexpr bool HAS_O = DHT == 64;
  static constexpr int QOB = DHT == 64 ? 2 : 1;                 // Q / dO (/ O) buffers
  static constexpr int RINGN = DHT == 64 ? 3 : 2;               // K / V stages
  static constexpr int QO_TILES = (HAS_O ? 3 : 2) * NB;         // blocks per buffer: Q, then dO, then O
  static constexpr int OFF_QO = 0;
  static constexpr int OFF_KV = QOB * QO_TILES * TILE;          // stage s: K blocks at +s*2*NB*TILE, V blocks after them
  static constexpr int OFF_OUT = OFF_KV + RINGN * 2 * NB * TILE;   // dQ staged for the TMA store
  static constexpr int OFF_AUG = OFF_OUT + NB * TILE;              // ones for S, ones for dP (64 key rows each), then one tile per Q buffer
  static constexpr int OFF_BAR = OFF_AUG + (DHT == 64 ? AUG_TILE + QOB * AUG_TILE : 0);
  static constexpr int SMEM = OFF_BAR + 256 + 1024;
};
}  // namespace dq

template <int DHT>
__global__ void __launch_bounds__(Roles<DHT>::NTHREADS_DQ, 1)
attn_bwd_dq_t5_kernel(const __grid_constant__ CUtensorMap mapQKV, const __grid_constant__ CUtensorMap mapDO,
                      const __grid_constant__ CUtensorMap mapO, const __grid_constant__ CUtensorMap mapDQKV, BwdParams p) {
  using namespace dq;
  using C = Cfg<DHT>;
  constexpr int CW = Roles<DHT>::CW, EW_THREADS = Roles<DHT>::EW_THREADS, ACC_WARP = Roles<DHT>::ACC_WARP,
                OUT_WARP0 = Roles<DHT>::OUT_WARP0, OFF_AUG = C::OFF_AUG;
  constexpr bool AUG = Roles<DHT>::AUG;
  static_assert(!AUG || C::HAS_O, "the statistics warp computes D from the staged O tile");
  constexpr int NB = C::NB, QOB = C::QOB, RINGN = C::RINGN, QO_TILES = C::QO_TILES, OFF_QO = C::OFF_QO, OFF_KV = C::OFF_KV,
                OFF_OUT = C::OFF_OUT, OFF_BAR = C::OFF_BAR;
  constexpr bool HAS_O = C::HAS_O;
  T5_SETUP(N_BARS, S_FREE, S_FREE1, P_READY, P_READY1, ACC_FREE, KV_EMPTY, KV_EMPTY + RINGN, AUG_READY, AUG_READY + 2)
  if (AUG) {
    // the two constant tiles need 64 rows each (a half's key columns): they share one tile's room
    aug_init(base_ptr + OFF_AUG, base_ptr + OFF_AUG + AUG_TILE / 2, 64, base_ptr + OFF_AUG + AUG_TILE, QOB * AUG_TILE);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
  }
  const int nq = p.T / BT;
  // persistent: the work units are (item, tile) pairs, item = (sequence, head).  The grid is a multiple of
  // nq CTAs; in round t the CTAs nq*s .. nq*s + nq-1 take the nq tiles of one item (the s-th of the round's
  // block of items), so an item's Q, K, V and dO are read from memory once and found in L2 by its other
  // tiles, which run at about the same time; which tile a CTA takes rotates with the round, so that every
  // CTA gets the same mix of long and short tiles.  Every role walks its units in one flat loop, so loads
  // for the next unit are issued while this one ends.
  const int ipb = (int)gridDim.x / nq, slot = (int)blockIdx.x / nq, pos = (int)blockIdx.x % nq;
  const int my_tiles = (slot < ipb && slot < p.nitems) ? (p.nitems - slot + ipb - 1) / ipb : 0;
  const uint32_t tS = tmem_base, tDP = tmem_base + 128u, tDQ = tmem_base + 256u;      // dQ: DHT columns
  const uint32_t tDS = tmem_base + 256u + (uint32_t)DHT;               // dS: bf16, 64 columns

  // query tiles are walked from the last (most key tiles) to the first
  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      int s = 0, n = 0;
      for (int tq = 0; tq < my_tiles && ok; ++tq) {
        const int item = tq * ipb + slot, qi = (pos + tq) % nq;
        const int h = item % p.H, b = item / p.H;      // this CTA walks several (sequence, head) items
        const int seq_row0 = b * p.T;
        const size_t stat0 = ((size_t)b * p.H + h) * p.T;
        (void)seq_row0; (void)stat0;
        const int i = nq - 1 - qi, qb = tq % QOB;
        if (!mbar_wait(B(QO_EMPTY + qb), freed(tq / QOB), abort_flag, p.status, 61)) { ok = false; break; }
        mbar_expect_tx(B(QO_FULL + qb), QO_TILES * TILE);
        const uint32_t qo = base + OFF_QO + qb * QO_TILES * TILE;
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          tma_load_2d(qo + nb * TILE, &mapQKV, B(QO_FULL + qb), h * DHT + 64 * nb, seq_row0 + i * BT);
          tma_load_2d(qo + (NB + nb) * TILE, &mapDO, B(QO_FULL + qb), h * DHT + 64 * nb, seq_row0 + i * BT);
          if (HAS_O) tma_load_2d(qo + (2 * NB + nb) * TILE, &mapO, B(QO_FULL + qb), h * DHT + 64 * nb, seq_row0 + i * BT);
        }
        for (int j = 0; j <= i; ++j) {
          if (!mbar_wait(B(KV_EMPTY + s), freed(n), abort_flag, p.status, 62)) { ok = false; break; }
          mbar_expect_tx(B(KV_FULL + s), 2 * NB * TILE);
          const uint32_t kv = base + OFF_KV + s * 2 * NB * TILE;
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) {
            tma_load_2d(kv + nb * TILE, &mapQKV, B(KV_FULL + s), p.d + h * DHT + 64 * nb, seq_row0 + j * BT);
            tma_load_2d(kv + (NB + nb) * TILE, &mapQKV, B(KV_FULL + s), 2 * p.d + h * DHT + 64 * nb, seq_row0 + j * BT);
          }
          if (++s == RINGN) { s = 0; ++n; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- score products: S = Q K^T, dP = dO V^T, in halves of 64 key columns ----------------
    if (lane == 0) {
      bool ok = true;
      int it = 0, s = 0, n = 0;
      const uint32_t lo_qo = desc_lo(base + OFF_QO), lo_kv = desc_lo(base + OFF_KV), lo_aug = desc_lo_aug(base + OFF_AUG);
      constexpr uint32_t TILE16 = TILE >> 4;
      for (int tq = 0; tq < my_tiles && ok; ++tq) {
        const int item = tq * ipb + slot, qi = (pos + tq) % nq;
        const int h = item % p.H, b = item / p.H;      // this CTA walks several (sequence, head) items
        const int seq_row0 = b * p.T;
        const size_t stat0 = ((size_t)b * p.H + h) * p.T;
        (void)seq_row0; (void)stat0;
        const int steps = nq - qi;               // key tiles 0 .. i, i = nq-1-qi
        const int qb = tq % QOB;
        const uint32_t lo_q = lo_qo + (uint32_t)(qb * QO_TILES) * TILE16, lo_do = lo_q + (uint32_t)NB * TILE16;
        if (!mbar_wait(B(QO_FULL + qb), done(tq / QOB), abort_flag, p.status, 65)) { ok = false; break; }
        const uint32_t lo_aq = lo_aug + (uint32_t)((1 + qb) * AUG_TILE >> 4);       // this tile's -lse/scale, -D rows
        for (int st = 0; st < steps && ok; ++st, ++it) {
          const uint32_t lo_k = lo_kv + (uint32_t)(s * 2 * NB) * TILE16;
          if (!mbar_wait(B(KV_FULL + s), done(n), abort_flag, p.status, 63)) { ok = false; break; }
          // The rows with -lse/scale and -D are written by the statistics warp once Q, dO and O have arrived.
          // In a tile's first step both halves' products over the features are issued before that is waited
          // for, so the statistics are computed while the tensor pipe already works on the tile.
          const bool late_aug = AUG && st == 0;
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            if (!mbar_wait(B(S_FREE + hh), freed(it), abort_flag, p.status, 64)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int nb = 0; nb < NB; ++nb)           // contraction over the head's features, 64 per block
              mma_score_half(tS + 64u * hh, lo_q + (uint32_t)nb * TILE16, lo_k + (uint32_t)nb * TILE16, hh, nb == 0);
#pragma unroll
            for (int nb = 0; nb < NB; ++nb)
              mma_score_half(tDP + 64u * hh, lo_do + (uint32_t)nb * TILE16, lo_k + (uint32_t)(NB + nb) * TILE16, hh, nb == 0);
            if (AUG && !late_aug) {
              // one more step: (-lse/scale of the queries) x ones, then (-D) x ones
              tc_mma_aug(tS + 64u * hh, lo_aq, lo_aug, IDESC_64KK);
              tc_mma_aug(tDP + 64u * hh, lo_aq, lo_aug + (uint32_t)(AUG_TILE / 2 >> 4), IDESC_64KK);
            }
            if (!late_aug) tc_commit(B(S_FULL + hh));
          }
          if (ok && late_aug) {
            if (!mbar_wait(B(AUG_READY + qb), done(tq / QOB), abort_flag, p.status, 72)) { ok = false; break; }
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
              tc_mma_aug(tS + 64u * hh, lo_aq, lo_aug, IDESC_64KK);
              tc_mma_aug(tDP + 64u * hh, lo_aq, lo_aug + (uint32_t)(AUG_TILE / 2 >> 4), IDESC_64KK);
              tc_commit(B(S_FULL + hh));
            }
          }
          if (ok) tc_commit(B(KV_EMPTY + s));        // second arrival comes from the accumulating thread
          if (++s == RINGN) { s = 0; ++n; }
        }
        if (ok) tc_commit(B(QO_EMPTY + qb));         // Q, dO are read by these products only
      }
    }
  } else if (warp == ACC_WARP) {
    // ---------------- accumulating products: dQ += dS K ----------------
    if (lane == 0) {
      bool ok = true;
      int it = 0, s = 0, n = 0;
      const uint32_t lo_kv = desc_lo(base + OFF_KV);
      constexpr uint32_t TILE16 = TILE >> 4;
      for (int tq = 0; tq < my_tiles && ok; ++tq) {
        const int item = tq * ipb + slot, qi = (pos + tq) % nq;
        const int h = item % p.H, b = item / p.H;      // this CTA walks several (sequence, head) items
        const int seq_row0 = b * p.T;
        const size_t stat0 = ((size_t)b * p.H + h) * p.T;
        (void)seq_row0; (void)stat0;
        const int steps = nq - qi;
        if (!mbar_wait(B(ACC_FREE), freed(tq), abort_flag, p.status, 66)) { ok = false; break; }
        for (int st = 0; st < steps && ok; ++st, ++it) {
          const uint32_t lo_k = lo_kv + (uint32_t)(s * 2 * NB) * TILE16;
          if (!mbar_wait(B(KV_FULL + s), done(n), abort_flag, p.status, 63)) { ok = false; break; }
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            if (!mbar_wait(B(P_READY + hh), done(it), abort_flag, p.status, 67)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int nb = 0; nb < NB; ++nb)           // one 64-column block of dQ per block of K
              mma_acc_half(tDQ + 64u * nb, tDS, lo_k + (uint32_t)nb * TILE16, hh, st == 0 && hh == 0);
            tc_commit(B(P_FREE + hh));
          }
          if (ok) tc_commit(B(KV_EMPTY + s));
          if (++s == RINGN) { s = 0; ++n; }
        }
        if (ok) tc_commit(B(ACC_FULL));
      }
    }
  } else if (warp < ACC_WARP) {
    // ---------------- element-wise warps (2 .. ACC_WARP - 1) ----------------
    const int q4 = warp & 3;
    const int wsel = (warp - 2) >> 2;            // which of the EWQ warps of this accumulator lane quarter
    const int r = q4 * 32 + lane;                // query row inside the tile
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const float scale_log2 = p.scale * LOG2E;
    const uint64_t sc2 = pack2(scale_log2, scale_log2);
    bool ok = true;
    int it = 0;
    for (int tq = 0; tq < my_tiles; ++tq) {
      const int item = tq * ipb + slot, qi = (pos + tq) % nq;
      const int h = item % p.H, b = item / p.H;      // this CTA walks several (sequence, head) items
      const int seq_row0 = b * p.T;
      const size_t stat0 = ((size_t)b * p.H + h) * p.T;
      (void)seq_row0; (void)stat0;
      const int i = nq - 1 - qi;
      // (with the statistics folded into the products these threads need neither lse nor D)
      const float L2 = AUG ? 0.f : p.lse[stat0 + (size_t)i * BT + r] * LOG2E;
      // D[row] = sum(dO * O) from the staged tiles: both have the same swizzle, so 16-byte chunk j of
      // one row holds the same eight columns in both
      float Dr = 0.f;
      if (AUG) {
      } else if (!HAS_O) {
        Dr = p.rowdot[stat0 + (size_t)i * BT + r];
      } else {
        const int qb = tq % QOB;
        if (!mbar_wait(B(QO_FULL + qb), done(tq / QOB), abort_flag, p.status, 71)) ok = false;
        if (ok) {
          const uint8_t* dorow = base_ptr + OFF_QO + qb * 3 * TILE + TILE + r * 128;
          const uint8_t* orow = dorow + TILE;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int jj = (j ^ (r & 7)) << 4;       // lanes of a warp spread over all banks
            const uint4 a = *reinterpret_cast<const uint4*>(dorow + jj);
            const uint4 bq = *reinterpret_cast<const uint4*>(orow + jj);
            const uint32_t* aw = reinterpret_cast<const uint32_t*>(&a);
            const uint32_t* bw = reinterpret_cast<const uint32_t*>(&bq);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              Dr = fmaf(__uint_as_float(aw[e] << 16), __uint_as_float(bw[e] << 16), Dr);
              Dr = fmaf(__uint_as_float(aw[e] & 0xffff0000u), __uint_as_float(bw[e] & 0xffff0000u), Dr);
            }
          }
          if (wsel == 0) p.rowdot_out[stat0 + (size_t)i * BT + r] = Dr;
        }
      }
      const uint64_t nl2 = pack2(-L2, -L2), nd2 = pack2(-Dr, -Dr);
      for (int j = 0; j <= i && ok; ++j, ++it) {
        const bool diag = (j == i);
#pragma unroll 1
        for (int hh = 0; hh < 2; ++hh) {
          const int c = hh * 64 + wsel * CW;
          if (!mbar_wait(B(S_FULL + hh), done(it), abort_flag, p.status, 68)) { ok = false; break; }
          if (!mbar_wait(B(P_FREE + hh), freed(it), abort_flag, p.status, 69)) { ok = false; break; }
          tc_fence_after();
          uint32_t dk[CW / 2];
          // on the diagonal tile only keys <= this query count: chunks wholly after the warp's rows are zero
          if (!diag || c < q4 * 32 + 32) {
            float sv[CW], dv[CW];
            tc_ld_cw<CW>(tS + lane_off + (uint32_t)c, sv);
            tc_ld_cw<CW>(tDP + lane_off + (uint32_t)c, dv);
            tc_wait_ld();
            tc_fence_before();                  // the values are in registers: the next step's products
            mbar_arrive(B(S_FREE + hh));        // may overwrite this half of S and dP
            if (diag && c + CW > q4 * 32 + 1) { // mask on the scores: the element loop stays free of tests
#pragma unroll
              for (int e = 0; e < CW; ++e) sv[e] = (c + e > r) ? -INFINITY : sv[e];
            }
#pragma unroll
            for (int e = 0; e < CW; e += 2) {
              float a0, a1, g0, g1;
              if constexpr (AUG) {      // the accumulators hold S - lse/scale and dP - D already
                unpack2(mul2(pack2(sv[e], sv[e + 1]), sc2), a0, a1);
              } else {
                unpack2(fma2(pack2(sv[e], sv[e + 1]), sc2, nl2), a0, a1);
              }
              const float p0 = ex2(a0), p1 = ex2(a1);
              if constexpr (AUG) {
                unpack2(mul2(pack2(p0, p1), pack2(dv[e], dv[e + 1])), g0, g1);
              } else {
                unpack2(mul2(pack2(p0, p1), add2(pack2(dv[e], dv[e + 1]), nd2)), g0, g1);
              }
              __nv_bfloat162 db = __floats2bfloat162_rn(g0, g1);
              dk[e >> 1] = *reinterpret_cast<uint32_t*>(&db);
            }
          } else {
#pragma unroll
            for (int e = 0; e < CW / 2; ++e) dk[e] = 0u;
            mbar_arrive(B(S_FREE + hh));
          }
          tc_st_cw<CW>(tDS + lane_off + (uint32_t)(c >> 1), dk);
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(B(P_READY + hh));
        }
        if (!ok) break;
      }
    }
  } else if (warp >= OUT_WARP0 && warp < OUT_WARP0 + 4) {
    // ---------------- output: dQ (scaled) of a finished query tile (own warps, see the dK/dV kernel) ----------------
    const int q4 = warp & 3;
    const int r = q4 * 32 + lane;
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    bool ok = true;
    // These warps idle while a tile's products run, so they also prepare the next tile's row statistics
    // (one thread per query row): D[row] = sum(dO * O) from the staged tiles, left in global memory for the
    // dK/dV kernel, and the operand row that carries -lse/scale and -D into the tile's score products.
    const float inv_scale = 1.0f / p.scale;
    auto statistics = [&](int t) {
      const int item = t * ipb + slot, qi = (pos + t) % nq;
      const int h = item % p.H, b = item / p.H;
      const size_t row = ((size_t)b * p.H + h) * p.T + (size_t)(nq - 1 - qi) * BT + r;
      const int qb = t % QOB;
      const float L = p.lse[row];
      if (!mbar_wait(B(QO_FULL + qb), done(t / QOB), abort_flag, p.status, 73)) { ok = false; return; }
      // dO and O tiles have the same swizzle, so 16-byte chunk j of one row holds the same eight columns in both
      const uint8_t* dorow = base_ptr + OFF_QO + qb * QO_TILES * TILE + TILE + r * 128;
      const uint8_t* orow = dorow + TILE;
      float Dr = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int jj = (j ^ (r & 7)) << 4;       // lanes of a warp spread over all banks
        const uint4 av = *reinterpret_cast<const uint4*>(dorow + jj);
        const uint4 bv = *reinterpret_cast<const uint4*>(orow + jj);
        const uint32_t* aw = reinterpret_cast<const uint32_t*>(&av);
        const uint32_t* bw = reinterpret_cast<const uint32_t*>(&bv);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          Dr = fmaf(__uint_as_float(aw[e] << 16), __uint_as_float(bw[e] << 16), Dr);
          Dr = fmaf(__uint_as_float(aw[e] & 0xffff0000u), __uint_as_float(bw[e] & 0xffff0000u), Dr);
        }
      }
      p.rowdot_out[row] = Dr;
      *reinterpret_cast<uint2*>(base_ptr + OFF_AUG + (1 + qb) * AUG_TILE + aug_row(r)) = make_uint2(neg_split(L * inv_scale), neg_split(Dr));
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(B(AUG_READY + qb));
    };
    if (AUG && my_tiles > 0) statistics(0);
    for (int tq = 0; tq < my_tiles; ++tq) {
      const int item = tq * ipb + slot, qi = (pos + tq) % nq;
      const int h = item % p.H, b = item / p.H;      // this CTA walks several (sequence, head) items
      const int seq_row0 = b * p.T;
      const size_t stat0 = ((size_t)b * p.H + h) * p.T;
      (void)seq_row0; (void)stat0;
      const int i = nq - 1 - qi;
      // (the next tile's Q, dO and O were requested when the tile before this one had been read: they arrive
      // long before this tile's accumulator is complete)
      if (AUG && ok && tq + 1 < my_tiles) statistics(tq + 1);
      if (ok && !mbar_wait(B(ACC_FULL), done(tq), abort_flag, p.status, 70)) ok = false;
      if (ok) {
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < DHT; c += 32) {
          float v[32];
          tc_ld32(tDQ + lane_off + (uint32_t)c, v);
          tc_wait_ld();
#pragma unroll
          for (uint32_t jj = 0; jj < 4; ++jj) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              __nv_bfloat162 ob = __floats2bfloat162_rn(v[8 * jj + 2 * e] * p.scale, v[8 * jj + 2 * e + 1] * p.scale);
              w[e] = *reinterpret_cast<uint32_t*>(&ob);
            }
            st_row_chunk(base + OFF_OUT + (uint32_t)(c >> 6) * TILE, r, (uint32_t)((c & 63) >> 3) + jj, w);
          }
        }
        tc_fence_before();
        mbar_arrive(B(ACC_FREE));
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("bar.sync 1, 128;" ::: "memory");         // the four output warps (always reached)
      if (ok && warp == OUT_WARP0 && lane == 0) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) tma_store_2d(&mapDQKV, base + OFF_OUT + nb * TILE, h * DHT + 64 * nb, seq_row0 + i * BT);
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
    }
    if (warp == OUT_WARP0 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }
  T5_TEARDOWN()
}

PerDeviceOnce g_once;

bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols) {
  return cached_map_2d(m, ptr, rows, cols, cols, 64, (uint32_t)BT, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

// kernel attributes are per device: set them the first time each device launches
bool init_device() {
  const int dev = current_device();
  if (dev < 0 || !tensor_map_encoder()) return false;
  if (!g_once.needed(dev)) return true;
  if (cudaFuncSetAttribute(attn_bwd_dkv_t5_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, dkv::Cfg<64>::SMEM) != cudaSuccess) return false;
  if (cudaFuncSetAttribute(attn_bwd_dkv_t5_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, dkv::Cfg<128>::SMEM) != cudaSuccess) return false;
  if (cudaFuncSetAttribute(attn_bwd_dq_t5_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, dq::Cfg<64>::SMEM) != cudaSuccess) return false;
  if (cudaFuncSetAttribute(attn_bwd_dq_t5_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, dq::Cfg<128>::SMEM) != cudaSuccess) return false;
  g_once.done(dev);
  return true;
}

}  // namespace

cudaError_t attention_bwd_t5(const void* qkv, const void* o, const float* lse, const void* d_o, int nseq, int T, int H,
                             int d, void* dqkv, float* rowdot, int* status, cudaStream_t st) {
  if (!attention_t5_supported(DT_BF16, T, H, d)) return cudaErrorInvalidValue;
  if (!init_device()) return cudaErrorInitializationError;
  const int sms = num_sms();
  if (!status) status = library_status_word();
  if (!status || sms < 1) return cudaErrorInitializationError;
  CUtensorMap mQKV, mDO, mO, mDQKV;
  const uint64_t rows = (uint64_t)nseq * T;
  if (!make_map(&mQKV, qkv, rows, (uint64_t)3 * d) || !make_map(&mDO, d_o, rows, (uint64_t)d) ||
      !make_map(&mO, o, rows, (uint64_t)d) || !make_map(&mDQKV, dqkv, rows, (uint64_t)3 * d))
    return cudaErrorInvalidValue;
  BwdParams p;
  p.T = T; p.H = H; p.d = d; p.scale = 1.0f / sqrtf((float)DH); p.lse = lse; p.rowdot = rowdot; p.rowdot_out = rowdot;
  p.status = status;
  p.nitems = nseq * H;
  const int nq = T / BT, units = p.nitems * nq;
  dim3 grid((unsigned)(((units < sms ? units : sms) / nq) * nq));   // one persistent CTA per SM, whole items per round
  // dQ first: it leaves D[row] = sum(dO * O) in `rowdot` for the dK/dV kernel
  attn_bwd_dq_t5_kernel<64><<<grid, Roles<64>::NTHREADS_DQ, dq::Cfg<64>::SMEM, st>>>(mQKV, mDO, mO, mDQKV, p);
  attn_bwd_dkv_t5_kernel<64><<<grid, Roles<64>::NTHREADS_DKV, dkv::Cfg<64>::SMEM, st>>>(mQKV, mDO, mDQKV, p);
  return cudaGetLastError();
}

// Heads of width 128: D[row] = sum(dO * O) must already be in `rowdot` (both kernels read it).
bool attention_bwd_t5_128_supported(int dt, int T, int H, int d) {
  return dt == DT_BF16 && H > 0 && d % H == 0 && d / H == 128 && T >= BT && T % BT == 0 && T / BT <= 64;
}

cudaError_t attention_bwd_t5_128(const void* qkv, const float* lse, const void* d_o, const float* rowdot, int nseq,
                                    int T, int H, int d, void* dqkv, int* status, cudaStream_t st) {
  if (!attention_bwd_t5_128_supported(DT_BF16, T, H, d)) return cudaErrorInvalidValue;
  if (!init_device()) return cudaErrorInitializationError;
  const int sms = num_sms();
  if (!status) status = library_status_word();
  if (!status || sms < 1) return cudaErrorInitializationError;
  CUtensorMap mQKV, mDO, mDQKV;
  const uint64_t rows = (uint64_t)nseq * T;
  if (!make_map(&mQKV, qkv, rows, (uint64_t)3 * d) || !make_map(&mDO, d_o, rows, (uint64_t)d) ||
      !make_map(&mDQKV, dqkv, rows, (uint64_t)3 * d))
    return cudaErrorInvalidValue;
  BwdParams p;
  p.T = T; p.H = H; p.d = d; p.scale = 1.0f / sqrtf(128.0f); p.lse = lse; p.rowdot = rowdot; p.rowdot_out = nullptr;
  p.status = status;
  p.nitems = nseq * H;
  const int nq = T / BT, units = p.nitems * nq;
  dim3 grid((unsigned)(((units < sms ? units : sms) / nq) * nq));
  attn_bwd_dq_t5_kernel<128><<<grid, Roles<128>::NTHREADS_DQ, dq::Cfg<128>::SMEM, st>>>(mQKV, mDO, mDO /* unused */, mDQKV, p);
  attn_bwd_dkv_t5_kernel<128><<<grid, Roles<128>::NTHREADS_DKV, dkv::Cfg<128>::SMEM, st>>>(mQKV, mDO, mDQKV, p);
  return cudaGetLastError();
}

}  // namespace sl
