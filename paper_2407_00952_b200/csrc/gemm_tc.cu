// Linear-layer kernels for sm_100a: bf16 operands staged in shared memory by TMA, products issued
// with tcgen05.mma from one thread, fp32 accumulators in tensor memory, epilogue read back with
// tcgen05.ld.  Persistent CTAs walk the output tiles; the accumulator is double buffered in tensor
// memory so that the epilogue of one tile overlaps the products of the next.
//
//   Y[M,N] = epilogue( X[M,K] W[N,K]^T  +  Xe[M,Ke] We[N,Ke]^T )
//
// The second term is the rank-r LoRA path: it enters as extra blocks of the contraction, read
// through a second pair of tensor maps whose rows are selected by the row group (client) of the
// tile, so K clients with their own adapters share one pass over the frozen W.
//
// Two kernels:
//   gemm_tc_pair_kernel   CTA pairs (cluster of 2, tcgen05 cta_group::2): a pair owns a 256 x 256
//                         tile; each CTA stages its 128 rows of X and one half (128 rows) of the W
//                         tile, the leader issues 256 x 256 x 16 products that read both CTAs'
//                         shared memory and write both CTAs' tensor memory.  32 KB per CTA per
//                         64-deep block (131 FLOP per byte from L2), 6 stages.
//   gemm_tc_kernel<BN>    one CTA per tile of 128 x BN (BN 256 / 128 / 64): narrow outputs (the
//                         rank-r down projections) and shapes the pair kernel does not take.
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = tensor-memory owner + MMA issuer,
// warps 2..9 = epilogue (a warp reads the 32 accumulator lanes its warp id modulo 4 selects; the
// two warps of a lane quarter take one half of the tile's columns each).
// Every wait on an mbarrier is bounded: when it expires the kernel records a code in `status`,
// stops issuing work, waits briefly for copies in flight, frees its tensor memory and returns.
#include "host_common.h"
#include "tc_common.cuh"

namespace sl {
namespace {

using namespace tc;

constexpr int NUM_THREADS = 320;

// ------------------------------------------------------------------------------------------
// one CTA per tile
// ------------------------------------------------------------------------------------------
template <int BN, bool DEEP = false> struct Cfg {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  // BN 64 is the HBM-bound rank-r down projection: two CTAs per SM (three stages each) keep every
  // SM streaming when the tiles do not fill whole waves of one CTA per SM.  DEEP is for the case
  // with fewer tiles than SMs (few tokens, wide rows): then a CTA has an SM to itself and what
  // limits it is the bytes it keeps in flight, so it takes an eight-stage ring.
  static constexpr int CTAS_PER_SM = (BN == 64 && !DEEP) ? 2 : 1;
  static constexpr int STAGES = BN == 64 ? (DEEP ? 8 : 3) : ((196608 / STAGE_BYTES) > 8 ? 8 : (196608 / STAGE_BYTES));
  static constexpr int TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
  static constexpr uint32_t IDESC = make_idesc(BM, BN);
};

template <int BN, bool DEEP = false>
__global__ void __launch_bounds__(NUM_THREADS, Cfg<BN, DEEP>::CTAS_PER_SM)
gemm_tc_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW,
               const __grid_constant__ CUtensorMap mapXe, const __grid_constant__ CUtensorMap mapWe,
               const __grid_constant__ CUtensorMap mapY, const __grid_constant__ CUtensorMap mapZ, TcParams p) {
  using C = Cfg<BN, DEEP>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t epi_base = base + C::STAGES * C::STAGE_BYTES;     // output staging of the epilogue warps
  const uint32_t bar_base = epi_base + EPI_STAGE_BYTES;
  // barrier slots: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + 2 + a); };
  uint8_t* tail = base_ptr + C::STAGES * C::STAGE_BYTES + EPI_STAGE_BYTES + 8 * (2 * C::STAGES + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)C::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int num_tiles = p.tiles_m * p.tiles_n;
  const int kb_total = p.num_kb + p.ext_blocks;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int tm, tn; tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
        const int m0 = tm * BM, n0 = tn * BN;
        const int g = p.rows_per_group > 0 ? m0 / p.rows_per_group : 0;
        const int w_row = g * p.w_group_rows + n0;
        const int we_row = g * p.we_group_rows + n0;
        for (int kb = 0; kb < kb_total; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 1)) { ok = false; break; }
          mbar_expect_tx(full_bar(stage), C::STAGE_BYTES);
          const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
          if (kb < p.num_kb) {
            const int kc = (kb < p.gap_kb_begin ? kb : kb + p.gap_kb) * BK;
            tma_load_2d(sa, &mapX, full_bar(stage), kc, m0);
            tma_load_2d(sb, &mapW, full_bar(stage), kc, w_row);
          } else {
            const int e = kb - p.num_kb;
            tma_load_2d(sa, &mapXe, full_bar(stage), e * BK, m0);
            tma_load_2d(sb, &mapWe, full_bar(stage), e * BK, we_row);
          }
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int as = 0; uint32_t aphase = 0;
      bool ok = true;
      const uint32_t a_lo0 = desc_lo(base);
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        if (!mbar_wait(tempty_bar(as), aphase ^ 1u, abort_flag, p.status, 2)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * BN);
        // main contraction: four products per block, issued back to back (advancing 16 elements
        // along K inside the swizzled row = +32 bytes = +2 in descriptor units)
        for (int kb = 0; kb < p.num_kb; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 3)) { ok = false; break; }
          const uint32_t alo = a_lo0 + (uint32_t)stage * (uint32_t)(C::STAGE_BYTES >> 4);
          const uint32_t blo = alo + (uint32_t)(C::A_BYTES >> 4);
          tc_mma_lo(d_tmem, alo, blo, C::IDESC, (uint32_t)kb);
          tc_mma_lo_acc(d_tmem, alo + 2, blo + 2, C::IDESC);
          tc_mma_lo_acc(d_tmem, alo + 4, blo + 4, C::IDESC);
          tc_mma_lo_acc(d_tmem, alo + 6, blo + 6, C::IDESC);
          tc_commit(empty_bar(stage));          // frees the stage once these products have read it
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        // rank-r extension: the last block may hold fewer than four products
        for (int kb = p.num_kb; kb < kb_total && ok; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 3)) { ok = false; break; }
          const uint32_t alo = a_lo0 + (uint32_t)stage * (uint32_t)(C::STAGE_BYTES >> 4);
          const uint32_t blo = alo + (uint32_t)(C::A_BYTES >> 4);
          const int nmma = kb == kb_total - 1 ? p.ext_last_mmas : BK / UMMA_K;
#pragma unroll 1
          for (int k = 0; k < nmma; ++k) tc_mma_lo_acc(d_tmem, alo + 2 * k, blo + 2 * k, C::IDESC);
          tc_commit(empty_bar(stage));
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull_bar(as));               // accumulator complete
        if (++as == 2) { as = 0; aphase ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue ----------------
    const int q = warp & 3;                     // lanes [32q, 32q+32) of tensor memory
    const int half = (warp - 2) >> 2;           // two warps share a lane quarter and split the columns
    const int c_begin = half * (BN / 2), c_end = c_begin + BN / 2;
    int as = 0; uint32_t aphase = 0;
    const bool tanh_form = p.gelu_tanh != 0;
    const uint32_t stage = epi_base + (uint32_t)(warp - 2) * 4096u;   // this warp's two staging buffers
    EpiState est;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      int tm, tn; tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
      const int m_warp0 = tm * BM + q * 32;
      const int n0 = tn * BN;
      int m_next = -1, n_next = 0;
      if (tile + (int)gridDim.x < num_tiles) {
        int tm2, tn2; tile_coords(tile + gridDim.x, p.tiles_m, p.tiles_n, tm2, tn2);
        m_next = tm2 * BM + q * 32; n_next = tn2 * BN + c_begin;
      }
      if (!mbar_wait(tfull_bar(as), aphase, abort_flag, p.status, 4)) { ok = false; break; }
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BN);
      epilogue_tile(p, t_row, m_warp0, lane, n0, c_begin, c_end, m_next, n_next, tanh_form, stage, est, &mapY, &mapZ);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(as));
      if (++as == 2) { as = 0; aphase ^= 1u; }
    }
    epilogue_drain(lane);
  }

  // ---------------- teardown ----------------
  __syncwarp();
  if (*abort_flag) {
    // give copies and products already in flight time to land before shared / tensor memory go away
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------------------
// CTA pairs
// ------------------------------------------------------------------------------------------
// NEED_R: the epilogue has a second operand R (residual, or the pre-activation for GELU').  Its
// [128 x 256] block per CTA tile is brought into shared memory by the producer warp with TMA about
// one tile ahead of its use, so the epilogue never waits on a global load; the room comes from a
// shorter operand ring (4 stages instead of 6).
template <bool NEED_R> struct PairCfg {
  static constexpr int BN = 256;                       // tile columns of the pair
  static constexpr int A_BYTES = BM * BK * 2;          // this CTA's 128 rows of X
  static constexpr int B_BYTES = (BN / 2) * BK * 2;    // this CTA's half of the W tile
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = NEED_R ? 4 : 6;
  static constexpr int R_BYTES = NEED_R ? BM * BN * 2 : 0;
  static constexpr int TMEM_COLS = 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + R_BYTES + EPI_STAGE_BYTES + 1024 + 256;
  static constexpr uint32_t IDESC = make_idesc(2 * BM, BN);
};

template <bool NEED_R>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW,
                    const __grid_constant__ CUtensorMap mapXe, const __grid_constant__ CUtensorMap mapWe,
                    const __grid_constant__ CUtensorMap mapY, const __grid_constant__ CUtensorMap mapZ,
                    const __grid_constant__ CUtensorMap mapR, TcParams p) {
  using C = PairCfg<NEED_R>;
  constexpr int BN = C::BN;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t r_base = base + C::STAGES * C::STAGE_BYTES;       // second epilogue operand of the current tile
  const uint32_t epi_base = r_base + C::R_BYTES;                   // output staging of the epilogue warps
  const uint32_t bar_base = epi_base + EPI_STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };                         // used in the leader
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };          // one per CTA
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + a); };      // one per CTA
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + 2 + a); }; // used in the leader
  const uint32_t rfull_bar = bar_base + 8u * (2 * C::STAGES + 4), rempty_bar = rfull_bar + 8u;   // one per CTA
  uint8_t* tail = base_ptr + C::STAGES * C::STAGE_BYTES + C::R_BYTES + EPI_STAGE_BYTES + 8 * (2 * C::STAGES + 6);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();           // 0 = leader of the pair
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 16); }
    mbar_init(rfull_bar, 1); mbar_init(rempty_bar, 8);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    // both CTAs of the pair allocate together
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)C::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                // the partner's barriers are initialised too
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int num_tiles = p.tiles_m * p.tiles_n;       // tiles of 256 x 256
  const int kb_total = p.num_kb + p.ext_blocks;

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs) ----------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int tcount = 0;                              // tiles this CTA has started
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
        int tm, tn; tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
        const int m0 = tm * 2 * BM + (int)rank * BM, n0 = tn * BN + (int)rank * (BN / 2);
        const int g = p.rows_per_group > 0 ? m0 / p.rows_per_group : 0;
        const int w_row = g * p.w_group_rows + n0;
        const int we_row = g * p.we_group_rows + n0;
        // R block of this tile: issued as soon as the epilogue has released the buffer (checked
        // between operand blocks so that the operand ring never waits for it)
        bool r_pending = NEED_R;
        auto issue_r = [&](bool blocking) -> bool {
          if (!r_pending) return true;
          const uint32_t par = ((uint32_t)tcount & 1u) ^ 1u;
          if (blocking) { if (!mbar_wait(rempty_bar, par, abort_flag, p.status, 15)) return false; }
          else if (!mbar_try(rempty_bar, par)) return true;
          mbar_expect_tx(rfull_bar, C::R_BYTES);
#pragma unroll
          for (int j = 0; j < BN / BK; ++j)
            tma_load_2d(r_base + j * (BM * BK * 2), &mapR, rfull_bar, tn * BN + j * BK, m0);
          r_pending = false;
          return true;
        };
        for (int kb = 0; kb < kb_total; ++kb) {
          issue_r(false);
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 11)) { ok = false; break; }
          // the leader's barrier collects the bytes of both CTAs' copies
          if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * C::STAGE_BYTES);
          const uint32_t leader_full = map_to_cta(full_bar(stage), 0);
          const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
          if (kb < p.num_kb) {
            tma_load_2d_pair(sa, &mapX, leader_full, kb * BK, m0);
            tma_load_2d_pair(sb, &mapW, leader_full, kb * BK, w_row);
          } else {
            const int e = kb - p.num_kb;
            tma_load_2d_pair(sa, &mapXe, leader_full, e * BK, m0);
            tma_load_2d_pair(sb, &mapWe, leader_full, e * BK, we_row);
          }
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok && !issue_r(true)) ok = false;
        ++tcount;
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (leader only) ----------------
    if (lane == 0 && rank == 0) {
      int stage = 0; uint32_t phase = 0;
      int as = 0; uint32_t aphase = 0;
      bool ok = true;
      const uint32_t a_lo0 = desc_lo(base);
      for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
        if (!mbar_wait(tempty_bar(as), aphase ^ 1u, abort_flag, p.status, 12)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * BN);
        for (int kb = 0; kb < p.num_kb; ++kb) {    // four products per block, issued back to back
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 13)) { ok = false; break; }
          const uint32_t alo = a_lo0 + (uint32_t)stage * (uint32_t)(C::STAGE_BYTES >> 4);
          const uint32_t blo = alo + (uint32_t)(C::A_BYTES >> 4);
          tc_mma_pair_lo(d_tmem, alo, blo, C::IDESC, (uint32_t)kb);
          tc_mma_pair_lo_acc(d_tmem, alo + 2, blo + 2, C::IDESC);
          tc_mma_pair_lo_acc(d_tmem, alo + 4, blo + 4, C::IDESC);
          tc_mma_pair_lo_acc(d_tmem, alo + 6, blo + 6, C::IDESC);
          tc_commit_pair(empty_bar(stage), 3);     // frees the stage in both CTAs
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        for (int kb = p.num_kb; kb < kb_total && ok; ++kb) {   // rank-r extension
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 13)) { ok = false; break; }
          const uint32_t alo = a_lo0 + (uint32_t)stage * (uint32_t)(C::STAGE_BYTES >> 4);
          const uint32_t blo = alo + (uint32_t)(C::A_BYTES >> 4);
          const int nmma = kb == kb_total - 1 ? p.ext_last_mmas : BK / UMMA_K;
#pragma unroll 1
          for (int k = 0; k < nmma; ++k) tc_mma_pair_lo_acc(d_tmem, alo + 2 * k, blo + 2 * k, C::IDESC);
          tc_commit_pair(empty_bar(stage), 3);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(tfull_bar(as), 3);          // accumulator halves complete in both CTAs
        if (++as == 2) { as = 0; aphase ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue (both CTAs, own 128 rows) ----------------
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    const int c_begin = half * (BN / 2), c_end = c_begin + BN / 2;
    int as = 0; uint32_t aphase = 0;
    const bool tanh_form = p.gelu_tanh != 0;
    const uint32_t stage = epi_base + (uint32_t)(warp - 2) * 4096u;   // this warp's two staging buffers
    int buf = 0, tcount = 0;
    bool ok = true;
    for (int tile = pair; tile < num_tiles && ok; tile += npairs, ++tcount) {
      int tm, tn; tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
      const int m_warp0 = tm * 2 * BM + (int)rank * BM + q * 32;
      const int n0 = tn * BN;
      uint4 bfirst[4];
      load_bias_chunk(p, n0 + c_begin, bfirst);       // in flight while the accumulator is awaited
      if (!mbar_wait(tfull_bar(as), aphase, abort_flag, p.status, 14)) { ok = false; break; }
      if (NEED_R && !mbar_wait(rfull_bar, (uint32_t)tcount & 1u, abort_flag, p.status, 16)) { ok = false; break; }
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BN);
      epilogue_tile_smem_r(p, t_row, m_warp0, lane, n0, c_begin, c_end, tanh_form, stage, buf, &mapY, &mapZ,
                           NEED_R ? r_base : 0u, q * 32 + lane, bfirst);
      if (NEED_R) { __syncwarp(); if (lane == 0) mbar_arrive(rempty_bar); }   // 8 warps release the R buffer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(as), 0));   // 16 arrivals free the stage
      if (++as == 2) { as = 0; aphase ^= 1u; }
    }
    epilogue_drain(lane);
  }

  // ---------------- teardown ----------------
  __syncwarp();
  if (*abort_flag) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                // neither CTA leaves while its partner may still touch it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
  }
}

// ---- host side -----------------------------------------------------------------------------
// CTA pairs that can be resident at once, per device (0: pair kernel unavailable there)
int g_max_pairs[MAX_DEVICES] = {};
PerDeviceOnce g_pair_once;

// 2-D bf16 tensor [rows, cols] with leading dimension ld (elements); box = 64 columns x box_rows rows.
bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
  return cached_map_2d(m, ptr, rows, cols, ld, (uint32_t)BK, box_rows, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// Output map: bf16 [rows, cols], box = 32 columns x 32 rows, 64-byte swizzle (the epilogue's staging layout).
bool make_out_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld) {
  return cached_map_2d(m, ptr, rows, cols, ld, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

int max_pairs() {
  const int dev = current_device();
  return dev < 0 ? 0 : g_max_pairs[dev];
}

int pick_bn(const GemmArgs& a) {
  if (a.N % 256 == 0) return 256;
  if (a.N <= 64) return 64;
  if (a.N <= 128) return 128;
  return 256;
}

bool pair_ok(const GemmArgs& a) {
  if (max_pairs() < 1 || a.k_gap_len > 0) return false;
  if (a.M % (2 * BM) != 0 || a.N < 256) return false;
  if (a.rows_per_group > 0 && a.rows_per_group % (2 * BM) != 0) return false;
  return true;
}

// Fills the parameters both kernels share and encodes the tensor maps; box rows of the W maps differ.
bool prepare(const GemmArgs& a, int* status, int w_box_rows, CUtensorMap* mX, CUtensorMap* mW, CUtensorMap* mXe,
             CUtensorMap* mWe, CUtensorMap* mY, CUtensorMap* mZ, TcParams* p) {
  const int G = a.rows_per_group > 0 ? a.M / a.rows_per_group : 1;
  const int w_rows = a.w_rows > 0 ? a.w_rows : a.N;
  if (!make_map(mX, a.X, a.M, a.K + a.k_gap_len, a.ldx, BM)) return false;
  if (!make_map(mW, a.W, a.w_grouped ? (uint64_t)G * a.N : (uint64_t)w_rows, a.K + a.k_gap_len, a.ldw, w_box_rows)) return false;
  p->M = a.M; p->N = a.N; p->K = a.K; p->num_kb = a.K / BK;
  p->gap_kb = a.k_gap_len / BK;
  p->gap_kb_begin = a.k_gap_len > 0 ? a.k_gap_begin / BK : p->num_kb;
  if (a.Ke > 0) {
    const uint64_t ke_cols = (uint64_t)((a.Ke + BK - 1) / BK) * BK;
    if (!make_map(mXe, a.Xe, a.M, ke_cols, a.ldxe, BM)) return false;
    if (!make_map(mWe, a.We, a.we_grouped ? (uint64_t)G * a.N : (uint64_t)a.N, ke_cols, a.ldwe, w_box_rows)) return false;
    p->ext_blocks = (a.Ke + BK - 1) / BK;
    p->ext_last_mmas = (a.Ke - (p->ext_blocks - 1) * BK) / UMMA_K;
  } else {
    *mXe = *mX; *mWe = *mW;
    p->ext_blocks = 0; p->ext_last_mmas = 0;
  }
  if (!make_out_map(mY, a.Y, a.M, a.N, a.ldy)) return false;
  if (a.epi == EPI_BIAS_GELU) { if (!make_out_map(mZ, a.Z, a.M, a.N, a.ldz)) return false; }
  else *mZ = *mY;
  p->rows_per_group = a.rows_per_group;
  p->w_group_rows = a.w_grouped ? a.N : 0;
  p->we_group_rows = a.we_grouped ? a.N : 0;
  p->epi = a.epi; p->gelu_tanh = a.gelu_tanh;
  p->bias = (const bf16*)a.bias; p->R = (const bf16*)a.R; p->ldr = a.ldr;
  p->Y = (bf16*)a.Y; p->ldy = a.ldy; p->Z = (bf16*)a.Z; p->ldz = a.ldz;
  p->status = status;
  return true;
}

template <int BN, bool DEEP = false>
cudaError_t launch(const GemmArgs& a, int* status, cudaStream_t st) {
  using C = Cfg<BN, DEEP>;
  const int sms = num_sms();
  if (BN == 64 && !DEEP && (a.M / BM) * ((a.N + BN - 1) / BN) <= sms) return launch<64, true>(a, status, st);
  static PerDeviceOnce once;                    // one per instantiation; attributes are per device
  const int dev = current_device();
  if (once.needed(dev)) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN, DEEP>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    once.done(dev);
  }
  CUtensorMap mX, mW, mXe, mWe, mY, mZ;
  TcParams p;
  if (!prepare(a, status, BN, &mX, &mW, &mXe, &mWe, &mY, &mZ, &p)) return cudaErrorInvalidValue;
  p.tiles_m = a.M / BM; p.tiles_n = (a.N + BN - 1) / BN;
  const int tiles = p.tiles_m * p.tiles_n;
  const int slots = sms * C::CTAS_PER_SM;
  const int grid = tiles < slots ? tiles : slots;
  gemm_tc_kernel<BN, DEEP><<<grid, NUM_THREADS, C::SMEM_BYTES, st>>>(mX, mW, mXe, mWe, mY, mZ, p);
  return cudaGetLastError();
}

cudaError_t launch_pair(const GemmArgs& a, int* status, cudaStream_t st) {
  constexpr int BN = PairCfg<false>::BN;
  CUtensorMap mX, mW, mXe, mWe, mY, mZ, mR;
  TcParams p;
  if (!prepare(a, status, BN / 2, &mX, &mW, &mXe, &mWe, &mY, &mZ, &p)) return cudaErrorInvalidValue;
  p.tiles_m = a.M / (2 * BM); p.tiles_n = (a.N + BN - 1) / BN;
  const int tiles = p.tiles_m * p.tiles_n;
  const int pairs = tiles < max_pairs() ? tiles : max_pairs();
  const bool need_r = a.epi == EPI_BIAS_RESID || a.epi == EPI_MUL_GELUGRAD;
  if (need_r) {
    if (!make_map(&mR, a.R, a.M, a.N, a.ldr, BM)) return cudaErrorInvalidValue;
    gemm_tc_pair_kernel<true><<<2 * pairs, NUM_THREADS, PairCfg<true>::SMEM_BYTES, st>>>(mX, mW, mXe, mWe, mY, mZ, mR, p);
  } else {
    mR = mY;
    gemm_tc_pair_kernel<false><<<2 * pairs, NUM_THREADS, PairCfg<false>::SMEM_BYTES, st>>>(mX, mW, mXe, mWe, mY, mZ, mR, p);
  }
  return cudaGetLastError();
}

}  // namespace

int gemm_tc_init() {
  if (!tensor_map_encoder()) return -1;
  const int dev = current_device(), sms = num_sms();
  if (dev < 0 || sms < 1) return -1;
  if (!g_pair_once.needed(dev)) return 0;
  // how many CTA pairs fit on this device at once (the pair kernel is persistent: one wave)
  g_max_pairs[dev] = 0;
  if (cudaFuncSetAttribute(gemm_tc_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairCfg<false>::SMEM_BYTES) == cudaSuccess &&
      cudaFuncSetAttribute(gemm_tc_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairCfg<true>::SMEM_BYTES) == cudaSuccess) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sms & ~1); cfg.blockDim = dim3(NUM_THREADS); cfg.dynamicSmemBytes = PairCfg<true>::SMEM_BYTES;
    cudaLaunchAttribute at;
    at.id = cudaLaunchAttributeClusterDimension;
    at.val.clusterDim.x = 2; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
    cfg.attrs = &at; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_tc_pair_kernel<true>, &cfg) == cudaSuccess && n > 0)
      g_max_pairs[dev] = n < sms / 2 ? n : sms / 2;
    cudaGetLastError();
  }
  g_pair_once.done(dev);
  return 0;
}

bool gemm_tc_supported(const GemmArgs& a) {
  auto al16 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
  if (!tensor_map_encoder() || a.dtype != DT_BF16) return false;
  if (a.M < BM || a.M % BM != 0 || a.K < BK || a.K % BK != 0 || a.N < 8 || a.N % 8 != 0) return false;
  if (a.rows_per_group > 0 && (a.rows_per_group % BM != 0 || a.M % a.rows_per_group != 0)) return false;
  if (a.ldx % 8 || a.ldw % 8 || a.ldy % 8) return false;
  if (a.k_gap_len < 0 || a.k_gap_begin < 0 || a.k_gap_len % BK || a.k_gap_begin % BK || a.k_gap_begin > a.K) return false;
  if (!al16(a.X) || !al16(a.W) || !al16(a.Y)) return false;
  if (a.bias && !al16(a.bias)) return false;
  if (a.epi == EPI_BIAS_GELU && (!a.Z || a.ldz % 8 || !al16(a.Z))) return false;
  if ((a.epi == EPI_BIAS_RESID || a.epi == EPI_MUL_GELUGRAD) && (!a.R || a.ldr % 8 || !al16(a.R))) return false;
  if (a.Ke > 0) {
    if (a.Ke % UMMA_K != 0 || !a.Xe || !a.We || a.ldxe % 8 || a.ldwe % 8 || !al16(a.Xe) || !al16(a.We)) return false;
    if ((int64_t)((a.Ke + BK - 1) / BK) * BK > a.ldxe || (int64_t)((a.Ke + BK - 1) / BK) * BK > a.ldwe) return false;
  }
  return true;
}

cudaError_t gemm_tc(const GemmArgs& a, int* status, cudaStream_t st) {
  if (!gemm_tc_supported(a)) return cudaErrorInvalidValue;
  if (pair_ok(a)) return launch_pair(a, status, st);
  switch (pick_bn(a)) {
    case 256: return launch<256>(a, status, st);
    case 128: return launch<128>(a, status, st);
    default: return launch<64>(a, status, st);
  }
}

}  // namespace sl
