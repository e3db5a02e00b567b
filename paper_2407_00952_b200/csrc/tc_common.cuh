// Device-side building blocks shared by the tcgen05 linear-layer kernels: mbarrier / TMA / tcgen05
// PTX wrappers, shared-memory operand descriptors and the epilogue of one 32-column chunk.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"

namespace sl {
namespace tc {

constexpr int BM = 128;           // accumulator rows per CTA (the 128 lanes of tensor memory)
constexpr int BK = 64;            // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int GROUP_M = 16;       // output tiles are walked in bands of GROUP_M tile rows
constexpr unsigned long long WAIT_LIMIT_NS = 4000000000ull;
// Shared-memory operand descriptor of a K-major tile with 128-byte rows, 128-byte swizzle and groups
// of 8 rows 1024 bytes apart, split into its constant upper half and the address-carrying lower half.
constexpr uint32_t DESC_HI = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | (1u << 16); }

struct TcParams {
  int M, N, K;                    // K counts the main contraction only
  int num_kb;                     // K / 64
  int ext_blocks;                 // blocks of 64 in the rank-r extension
  int ext_last_mmas;              // MMAs (of 16) in the last extension block
  int gap_kb_begin, gap_kb;       // blocks of 64 columns skipped in X and W from block gap_kb_begin on
  int rows_per_group;             // 0: one group
  int w_group_rows;               // rows between groups in W (0: shared)
  int we_group_rows;              // rows between groups in We
  int tiles_m, tiles_n;
  int epi, gelu_tanh;
  const bf16* bias;
  const bf16* R; long long ldr;
  bf16* Y; long long ldy;
  bf16* Z; long long ldz;
  int* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Arrive on a barrier given by a shared::cluster address (own CTA or the peer of a CTA pair).
// Default (CTA-scope) release: what the arrival publishes are tensor-memory reads, which the
// tcgen05 fence before it orders.  A cluster-scope release here waited for the warp's output
// stores in flight, about 2,600 cycles per tile.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the limit expired or another role of this CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, int code) {
  if (mbar_try(bar, parity)) return true;
  unsigned long long t0 = global_ns();
  uint32_t spins = 0;
  while (!mbar_try(bar, parity)) {
    if ((++spins & 1023u) == 0) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > WAIT_LIMIT_NS) {
        *abort_flag = 1;
        atomicCAS(status, 0, code);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// Load issued inside a CTA pair: the completion may be signalled on the partner's barrier
// (bar is a shared::cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Commit of a CTA pair's products; arrives on the barrier at this offset in every CTA of `mask`.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, uint16_t mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// The same products with the operand descriptors passed as 32-bit halves.  The issuing thread runs
// alone in its warp, so every instruction between two tcgen05.mma costs several cycles during which
// the tensor pipe can run dry: with the descriptors rebuilt per product the pipe reached 128 cycles
// of work per 190; with the upper half constant (DESC_HI) and the lower half advanced by one add,
// consecutive products issue back to back.  `accumulate` = 0 overwrites the accumulator.
__device__ __forceinline__ void tc_mma_lo(uint32_t d_tmem, uint32_t alo, uint32_t blo, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(alo), "r"(blo), "r"(DESC_HI), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_mma_lo_acc(uint32_t d_tmem, uint32_t alo, uint32_t blo, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, 1, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(alo), "r"(blo), "r"(DESC_HI), "r"(idesc) : "memory");
}
__device__ __forceinline__ void tc_mma_pair_lo(uint32_t d_tmem, uint32_t alo, uint32_t blo, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(alo), "r"(blo), "r"(DESC_HI), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_mma_pair_lo_acc(uint32_t d_tmem, uint32_t alo, uint32_t blo, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, 1, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(alo), "r"(blo), "r"(DESC_HI), "r"(idesc) : "memory");
}
// Left operand taken from tensor memory (row = lane, two bf16 per 32-bit column, 16 elements of K
// = 8 columns), right operand from shared memory through its descriptor's lower half.
__device__ __forceinline__ void tc_mma_ts_lo(uint32_t d_tmem, uint32_t a_tmem, uint32_t blo, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(blo), "r"(DESC_HI), "r"(idesc), "r"(accumulate) : "memory");
}
// 16 packed words of this thread's lane to 16 consecutive tensor-memory columns
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t* w) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]),
        "r"(w[8]), "r"(w[9]), "r"(w[10]), "r"(w[11]), "r"(w[12]), "r"(w[13]), "r"(w[14]), "r"(w[15]) : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// tanh-form GELU and its derivative without a test of the form (see epilogue_chunk)
__device__ __forceinline__ float gelu_tanh_tc(float z) {
  const float u = z * fmaf(0.7978845608028654f * 0.044715f, z * z, 0.7978845608028654f);
  const float hz = 0.5f * z;
  return fmaf(hz, tanh_fast(u), hz);
}
__device__ __forceinline__ float gelu_grad_tanh_tc(float z) {
  const float z2 = z * z;
  const float u = z * fmaf(0.7978845608028654f * 0.044715f, z2, 0.7978845608028654f);
  const float t = tanh_fast(u);
  const float du = fmaf(0.7978845608028654f * 0.134145f, z2, 0.7978845608028654f);
  const float hz = 0.5f * z;
  return fmaf(hz * du, fmaf(-t, t, 1.0f), fmaf(0.5f, t, 0.5f));
}
// The same two functions on pairs of values with the packed fp32 instructions of this architecture
// (one instruction per pair; the hyperbolic tangent stays one special-function instruction per
// value).  The epilogue warps share their schedulers with the threads that feed the tensor pipe, so
// every instruction saved here is issue time given back to them.
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
// the two bf16 halves of a 32-bit word as a packed pair of floats
__device__ __forceinline__ uint64_t bf16x2_to_f32x2(uint32_t w) {
  return pack2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ void gelu_tanh_pair(float& a, float& b) {
  const uint64_t c1 = pack2(0.7978845608028654f, 0.7978845608028654f);
  const uint64_t c2 = pack2(0.7978845608028654f * 0.044715f, 0.7978845608028654f * 0.044715f);
  const uint64_t half = pack2(0.5f, 0.5f);
  const uint64_t z = pack2(a, b);
  const uint64_t u = mul2(z, fma2(mul2(z, z), c2, c1));
  float u0, u1;
  unpack2(u, u0, u1);
  const uint64_t t = pack2(tanh_fast(u0), tanh_fast(u1));
  const uint64_t hz = mul2(z, half);
  unpack2(fma2(hz, t, hz), a, b);
}
// (a, b) *= gelu'(z) for the two bf16 values of zw
__device__ __forceinline__ void mul_gelu_grad_tanh_pair(float& a, float& b, uint32_t zw) {
  const uint64_t c1 = pack2(0.7978845608028654f, 0.7978845608028654f);
  const uint64_t c2 = pack2(0.7978845608028654f * 0.044715f, 0.7978845608028654f * 0.044715f);
  const uint64_t c3 = pack2(0.7978845608028654f * 0.134145f, 0.7978845608028654f * 0.134145f);
  const uint64_t half = pack2(0.5f, 0.5f), one = pack2(1.0f, 1.0f), neg1 = pack2(-1.0f, -1.0f);
  const uint64_t z = bf16x2_to_f32x2(zw);
  const uint64_t z2 = mul2(z, z);
  const uint64_t u = mul2(z, fma2(z2, c2, c1));
  float u0, u1;
  unpack2(u, u0, u1);
  const uint64_t t = pack2(tanh_fast(u0), tanh_fast(u1));
  const uint64_t hzdu = mul2(mul2(z, half), fma2(z2, c3, c1));
  const uint64_t sech2 = fma2(mul2(t, t), neg1, one);
  const uint64_t g = fma2(hzdu, sech2, fma2(t, half, half));
  unpack2(mul2(pack2(a, b), g), a, b);
}
__device__ __forceinline__ float gelu_tc(float z, bool tanh_form) {
  if (tanh_form) {
    float u = 0.7978845608028654f * (z + 0.044715f * z * z * z);
    return 0.5f * z * (1.0f + tanh_fast(u));
  }
  return gelu_f(z, false);
}
__device__ __forceinline__ float gelu_grad_tc(float z, bool tanh_form) {
  if (tanh_form) {
    float u = 0.7978845608028654f * (z + 0.044715f * z * z * z);
    float t = tanh_fast(u);
    float du = 0.7978845608028654f * (1.0f + 0.134145f * z * z);
    return 0.5f * (1.0f + t) + 0.5f * z * (1.0f - t * t) * du;
  }
  return gelu_grad_f(z, false);
}

// Shared-memory operand descriptor: K-major tile whose rows are 128 bytes, 128-byte swizzle,
// groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);      // start address, 16-byte units
  d |= (uint64_t)1 << 16;                        // leading byte offset (unused for this layout)
  d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                        // 128-byte swizzle
  return d;
}

// kind::f16 instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major
__host__ __device__ constexpr uint32_t make_idesc(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// Output-tile walk: bands of GROUP_M tile rows, rows fastest inside a band.
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int& tm, int& tn) {
  const int band_tiles = GROUP_M * tiles_n;
  int band = tile / band_tiles, in = tile % band_tiles;
  int m_first = band * GROUP_M;
  int rows = min(GROUP_M, tiles_m - m_first);
  tm = m_first + in % rows;
  tn = in / rows;
}

// Bytes of shared memory the epilogue warps use to stage output chunks: 8 warps x 2 buffers x
// (32 rows x 64 bytes).
constexpr int EPI_STAGE_BYTES = 8 * 2 * 2048;

// One 32-row x 32-column bf16 chunk: registers -> shared (64-byte swizzle, conflict-free 16-byte
// stores) -> global through a TMA store.  Rows of the output are written as full 64-byte segments
// by the copy engine instead of 32 scattered 16-byte stores per warp instruction, which keeps the
// L1 data path free for the tensor core's operand reads.  `packed` holds this thread's row
// (lane = row).  The buffer is reused once the bulk group that read it has finished reading.
__device__ __forceinline__ void stage_and_store(uint32_t sbuf, const CUtensorMap* map, const uint32_t* packed,
                                                int lane, int n, int m_warp0) {
  if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
  __syncwarp();
  const uint32_t row = sbuf + (uint32_t)lane * 64u;
  const uint32_t sw = ((uint32_t)lane >> 1) & 3u;
#pragma unroll
  for (uint32_t j = 0; j < 4; ++j) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + ((j ^ sw) << 4)), "r"(packed[4 * j]),
                 "r"(packed[4 * j + 1]), "r"(packed[4 * j + 2]), "r"(packed[4 * j + 3]) : "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncwarp();
  if (lane == 0) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(sbuf), "r"(n), "r"(m_warp0) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  }
}
__device__ __forceinline__ void epilogue_drain(int lane) {
  if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  __syncwarp();
}

// The second epilogue operand (residual, or the saved pre-activation) of columns [n, n+32) of row m.
// Issued one chunk ahead of its use so that its latency overlaps the previous chunk's work.
__device__ __forceinline__ void load_r_chunk(const TcParams& p, int m, int n, uint4* r) {
  const bf16* rrow = p.R + (size_t)m * p.ldr + n;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (n + 8 * j < p.N) r[j] = *reinterpret_cast<const uint4*>(rrow + 8 * j);
    else r[j] = make_uint4(0u, 0u, 0u, 0u);
  }
}

// Bias of columns [n, n+32) (zeros past the last column, or when the layer has none).  Every lane
// reads the same 64 bytes; issued ahead of its use because nothing hides a global load's latency
// inside a chunk.
__device__ __forceinline__ void load_bias_chunk(const TcParams& p, int n, uint4* b) {
  const bool have = p.bias != nullptr && p.epi != EPI_MUL_GELUGRAD;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (have && n + 8 * j < p.N) b[j] = __ldg(reinterpret_cast<const uint4*>(p.bias + n + 8 * j));
    else b[j] = make_uint4(0u, 0u, 0u, 0u);
  }
}

// Epilogue of 32 accumulator columns [n, n+32) of row m (= m_warp0 + lane): bias (bcur, from
// load_bias_chunk), activation / residual (rpre: the row's second operand, zero past the last
// column), bf16 output through the staging buffers `stage` (this warp's two 2 KB buffers).
// Every per-element loop below is free of branches: the form of the epilogue is tested once per
// chunk, so that the 32 independent element chains can be interleaved by the instruction scheduler
// (with a test inside the loop each element is a basic block of its own and runs serially).
// Columns past N carry garbage that the TMA store clips.
// A warp barrier between runs of independent arithmetic.  The epilogue's element loops are long runs
// of instructions that never wait for each other, and two warps issuing such runs on one scheduler
// keep the single threads that feed the tensor pipe (TMA producer, MMA issuer) off it: in a
// stand-alone loop, bursts of four products took 574-620 cycles instead of 512 next to two warps of
// plain fp32 chains per scheduler, and 512 again with this barrier after every 32 of their
// instructions.
__device__ __forceinline__ void epi_yield() { __syncwarp(); }

__device__ __forceinline__ void epilogue_chunk(const TcParams& p, float* v, const uint4* bcur, const uint4* rpre, int n,
                                               bool tanh_form, uint32_t stage, int& buf, const CUtensorMap* mapY,
                                               const CUtensorMap* mapZ, int m_warp0, int lane) {
  if (p.bias != nullptr && p.epi != EPI_MUL_GELUGRAD) {      // warp-uniform; layers without a bias skip 64 instructions
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const bf16* bp = reinterpret_cast<const bf16*>(&bcur[j]);
#pragma unroll
      for (int i = 0; i < 8; ++i) v[8 * j + i] += __bfloat162float(bp[i]);
      if (j & 1) epi_yield();
    }
  }
  uint32_t packed[16];
  if (p.epi == EPI_BIAS_GELU) {
    float zr[32];                       // the pre-activation as stored (rounded to bf16)
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      __nv_bfloat162 z2 = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      packed[i] = *reinterpret_cast<uint32_t*>(&z2);
      zr[2 * i] = __low2float(z2);
      zr[2 * i + 1] = __high2float(z2);
    }
    epi_yield();
    if (tanh_form) {
#pragma unroll
      for (int i = 0; i < 32; i += 2) {
        v[i] = zr[i]; v[i + 1] = zr[i + 1]; gelu_tanh_pair(v[i], v[i + 1]);
        if ((i & 6) == 6) epi_yield();
      }
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = gelu_f(zr[i], false);
    }
    stage_and_store(stage + (uint32_t)buf * 2048u, mapZ, packed, lane, n, m_warp0);
    buf ^= 1;
  } else if (p.epi == EPI_BIAS_RESID) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const bf16* rp = reinterpret_cast<const bf16*>(&rpre[j]);
#pragma unroll
      for (int i = 0; i < 8; ++i) v[8 * j + i] += __bfloat162float(rp[i]);
      if (j & 1) epi_yield();
    }
  } else if (p.epi == EPI_MUL_GELUGRAD) {
    if (tanh_form) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t* rw = reinterpret_cast<const uint32_t*>(&rpre[j]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          mul_gelu_grad_tanh_pair(v[8 * j + 2 * i], v[8 * j + 2 * i + 1], rw[i]);
          if (i & 1) epi_yield();
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bf16* rp = reinterpret_cast<const bf16*>(&rpre[j]);
#pragma unroll
        for (int i = 0; i < 8; ++i) v[8 * j + i] *= gelu_grad_f(__bfloat162float(rp[i]), false);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    __nv_bfloat162 y2 = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    packed[i] = *reinterpret_cast<uint32_t*>(&y2);
  }
  epi_yield();
  stage_and_store(stage + (uint32_t)buf * 2048u, mapY, packed, lane, n, m_warp0);
  buf ^= 1;
}

// Per-warp epilogue state carried across tiles: staging buffer in use and the prefetched second
// operand (valid for the chunk at row block pm, column pn).
struct EpiState {
  uint4 rnext[4];
  int pm = -1, pn = -1;
  int buf = 0;
};

// This warp's share of one output tile: columns [n0 + c_begin, n0 + c_end) of the 32 rows starting
// at m_warp0, accumulator lanes at tensor-memory address t_row.  (m_next, n_next) is the first chunk
// this warp will process in its next tile (m_next < 0: none); its second operand is requested while
// the last chunk of this tile is being worked on.
__device__ __forceinline__ void epilogue_tile(const TcParams& p, uint32_t t_row, int m_warp0, int lane, int n0,
                                              int c_begin, int c_end, int m_next, int n_next, bool tanh_form,
                                              uint32_t stage, EpiState& st, const CUtensorMap* mapY,
                                              const CUtensorMap* mapZ) {
  const bool need_r = p.epi == EPI_BIAS_RESID || p.epi == EPI_MUL_GELUGRAD;
  const int m = m_warp0 + lane;
#pragma unroll 1
  for (int c = c_begin; c < c_end; c += 32) {
    const int n = n0 + c;
    if (n >= p.N) break;                    // warp-uniform
    uint4 rcur[4];
    if (need_r) {
      if (st.pm == m_warp0 && st.pn == n) {
#pragma unroll
        for (int j = 0; j < 4; ++j) rcur[j] = st.rnext[j];
      } else {
        load_r_chunk(p, m, n, rcur);
      }
      if (c + 32 < c_end && n + 32 < p.N) {
        load_r_chunk(p, m, n + 32, st.rnext); st.pm = m_warp0; st.pn = n + 32;
      } else if (m_next >= 0 && n_next < p.N) {
        load_r_chunk(p, m_next + lane, n_next, st.rnext); st.pm = m_next; st.pn = n_next;
      }
    }
    uint4 bcur[4];
    load_bias_chunk(p, n, bcur);
    float v[32];
    tc_ld32(t_row + (uint32_t)c, v);
    tc_wait_ld();
    epilogue_chunk(p, v, bcur, rcur, n, tanh_form, stage, st.buf, mapY, mapZ, m_warp0, lane);
  }
}

// Same, with the second epilogue operand already in shared memory: `rtile` holds this CTA's
// [128 rows x 256 columns] block of R as four [128 x 64] tiles in the 128-byte-swizzled layout a
// TMA load produces (rtile == 0: the epilogue has no second operand).  row = this thread's row
// inside the CTA tile.
__device__ __forceinline__ void epilogue_tile_smem_r(const TcParams& p, uint32_t t_row, int m_warp0, int lane, int n0,
                                                     int c_begin, int c_end, bool tanh_form, uint32_t stage, int& buf,
                                                     const CUtensorMap* mapY, const CUtensorMap* mapZ, uint32_t rtile,
                                                     int row, const uint4* bfirst) {
  uint4 bcur[4], bnext[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) bnext[j] = bfirst[j];
#pragma unroll 1
  for (int c = c_begin; c < c_end; c += 32) {
    const int n = n0 + c;
    if (n >= p.N) break;                    // warp-uniform
#pragma unroll
    for (int j = 0; j < 4; ++j) bcur[j] = bnext[j];
    if (c + 32 < c_end) load_bias_chunk(p, n + 32, bnext);
    uint4 rcur[4];
    if (rtile) {
      const uint32_t rrow = rtile + (uint32_t)(c >> 6) * (uint32_t)(BM * BK * 2) + (uint32_t)row * 128u;
      const uint32_t cb = (uint32_t)((c & 63) >> 3);
#pragma unroll
      for (uint32_t j = 0; j < 4; ++j) {
        const uint32_t a = rrow + (((cb + j) ^ ((uint32_t)row & 7u)) << 4);
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(rcur[j].x), "=r"(rcur[j].y), "=r"(rcur[j].z), "=r"(rcur[j].w) : "r"(a) : "memory");
      }
    }
    float v[32];
    tc_ld32(t_row + (uint32_t)c, v);
    tc_wait_ld();
    epilogue_chunk(p, v, bcur, rcur, n, tanh_form, stage, buf, mapY, mapZ, m_warp0, lane);
  }
}

}  // namespace tc
}  // namespace sl
