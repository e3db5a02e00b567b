// Causal multi-head attention forward for heads of width 64 on the 5th-generation tensor cores
// (tcgen05 + TMEM + TMA), bf16, sequence length a multiple of 128.
//
// Persistent CTAs, two per SM.  The work units are 128-row query tiles of (sequence, head) items; the
// tiles of one item run on neighbouring CTAs at about the same time (K and V come from memory once).
// A query tile walks its keys in HALF-STEPS of 64 keys:
//   S  = Q K^T      tcgen05.mma M128 N64 K16 x4 into one of two 64-column score buffers
//   softmax         ONE thread per query row reads its 64 scores from tensor memory once, keeps them in
//                   registers for the row maximum and the exponentials (no second read, no exchange
//                   between threads), and writes P (bf16) back to tensor memory
//   O += P V        tcgen05.mma M128 N64 K16 x4, P read from tensor memory, V used as loaded (MN-major)
// The score and P buffers are double buffered, so the products of half-step i+1 and i+2 run while the
// softmax threads work on half-step i, and the score buffer is released as soon as it has been read.
// O stays in tensor memory for the whole query tile.  It is rescaled only when a row's running maximum
// has moved by more than 2^8 since the reference maximum its exponentials are taken against: the
// exponentials and the row sum use that (stale) reference, which cancels in O / l at the end, and the
// bound keeps every P below 2^8.  Output rows (128 bytes each) go from registers straight to memory.
// Warp roles (192 threads): warp 0 TMA producer, warp 1 tensor-memory owner + MMA issuer, warps 2..5
// softmax (warp w owns accumulator lanes 32*(w%4)..+31).
// All mbarrier waits are bounded (see tc_common.cuh); on expiry a code is left in `status`.
#include "host_common.h"
#include "tc_common.cuh"

namespace sl {
namespace {

using namespace tc;

constexpr int BQ = 128;                   // query rows per tile
constexpr int BKV = 128;                  // key rows per TMA tile (two half-steps)
constexpr int HK = 64;                    // keys per half-step
constexpr int DH = 64;
constexpr int TILE = BQ * 64 * 2;         // 16 KB: one [128 x 64] bf16 block
constexpr int THREADS = 192;
constexpr int SM_THREADS = 128;
constexpr int OFF_Q = 0, OFF_K = 2 * TILE, OFF_V = 4 * TILE, OFF_BAR = 6 * TILE;
constexpr int SMEM = 6 * TILE + 256 + 1024;
constexpr int TMEM_COLS = 256;            // S0 [0,64) S1 [64,128) O [128,192) P0 [192,224) P1 [224,256)
constexpr uint32_t IDESC_S = make_idesc(BQ, HK);
constexpr uint32_t IDESC_PV = make_idesc(BQ, DH) | (1u << 16);   // B operand (V) MN-major
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;
constexpr float RESCALE_STEP = 8.0f;      // log2 of the largest P the stale reference maximum may produce

enum { Q_FULL = 0 /*+2*/, Q_EMPTY = 2 /*+2*/, K_FULL = 4 /*+2*/, K_EMPTY = 6 /*+2*/, V_FULL = 8 /*+2*/, V_EMPTY = 10 /*+2*/,
       S_FULL = 12 /*+2*/, S_FREE = 14 /*+2*/, P_READY = 16 /*+2*/, P_FREE = 18 /*+2*/, O_FREE = 20, N_BARS = 21 };

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

struct F64Params {
  int T, H, d;
  int nitems;              // nseq * H (sequence, head) items, shared out over the CTAs
  float scale_log2;
  bf16* o;
  float* lse;
  int* status;
};

__global__ void __launch_bounds__(THREADS, 2)
attn_fwd_t5_h64_kernel(const __grid_constant__ CUtensorMap mapQKV, F64Params p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t bar = base + OFF_BAR;
  auto B = [&](int i) { return bar + 8u * i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + OFF_BAR + 8 * N_BARS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + OFF_BAR + 8 * N_BARS + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = p.T / BQ;
  // Work units are (item, query tile) pairs.  The grid is a multiple of nq CTAs; in round t the CTAs
  // nq*s .. nq*s + nq-1 take the nq query tiles of one item (s-th item of the round's block of items), so an
  // item's K and V are read from memory once and found in L2 by its other tiles, which run at about the
  // same time.  Which of the item's tiles a CTA takes rotates with the round, so that every CTA gets the
  // same mix of long and short tiles.
  const int ipb = (int)gridDim.x / nq;             // items per round
  const int slot = (int)blockIdx.x / nq, pos = (int)blockIdx.x % nq;
  const int my_tiles = (slot < ipb && slot < p.nitems) ? (p.nitems - slot + ipb - 1) / ipb : 0;
  auto qt_of = [&](int tq) { return (pos + tq) % nq; };
  auto item_of = [&](int tq) { return tq * ipb + slot; };
  auto head_of = [&](int tq) { return item_of(tq) % p.H; };
  auto row0_of = [&](int tq) { return (item_of(tq) / p.H) * p.T; };

  if (threadIdx.x == 0) {
    for (int i = 0; i < N_BARS; ++i) {
      const bool by_threads = (i >= S_FREE && i < S_FREE + 2) || (i >= P_READY && i < P_READY + 2) || i == O_FREE;
      mbar_init(B(i), by_threads ? SM_THREADS : 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tS = tmem_base, tO = tmem_base + 128u, tP = tmem_base + 192u;

  if (warp == 0) {
    // ---------------- TMA producer: Q per query tile (two buffers), K and V per 128 keys (two stages) ----------------
    if (lane == 0) {
      bool ok = true;
      int ks = 0;                                   // 128-key steps issued so far
      for (int tq = 0; tq < my_tiles && ok; ++tq) {
        const int qt = qt_of(tq), h = head_of(tq), seq_row0 = row0_of(tq);
        const int qs = tq & 1;
        if (!mbar_wait(B(Q_EMPTY + qs), (((uint32_t)(tq >> 1)) & 1u) ^ 1u, abort_flag, p.status, 20)) { ok = false; break; }
        mbar_expect_tx(B(Q_FULL + qs), TILE);
        tma_load_2d(base + OFF_Q + qs * TILE, &mapQKV, B(Q_FULL + qs), h * DH, seq_row0 + qt * BQ);
        for (int j = 0; j <= qt && ok; ++j, ++ks) {
          const int s = ks & 1;
          const uint32_t par = (((uint32_t)(ks >> 1)) & 1u) ^ 1u;
          if (!mbar_wait(B(K_EMPTY + s), par, abort_flag, p.status, 21)) { ok = false; break; }
          mbar_expect_tx(B(K_FULL + s), TILE);
          tma_load_2d(base + OFF_K + s * TILE, &mapQKV, B(K_FULL + s), p.d + h * DH, seq_row0 + j * BKV);
          if (!mbar_wait(B(V_EMPTY + s), par, abort_flag, p.status, 22)) { ok = false; break; }
          mbar_expect_tx(B(V_FULL + s), TILE);
          tma_load_2d(base + OFF_V + s * TILE, &mapQKV, B(V_FULL + s), 2 * p.d + h * DH, seq_row0 + j * BKV);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    // Half-steps are numbered `it` over the CTA's whole work; S(it) goes to score buffer it & 1, P(it)
    // comes from P buffer it & 1.  Issue order: S(0), S(1), then PV(it), S(it + 2) for it = 0, 1, ...
    if (lane == 0) {
      bool ok = true;
      const uint32_t lo_q0 = desc_lo(base + OFF_Q), lo_k0 = desc_lo(base + OFF_K), lo_v0 = desc_lo(base + OFF_V);
      constexpr uint32_t TILE16 = TILE >> 4;
      // cursor of the score products (runs two half-steps ahead of the PV cursor)
      int s_tq = 0, s_hs = 0, s_it = 0, s_ks = 0;
      auto issue_S = [&]() -> bool {
        if (s_tq >= my_tiles) return true;
        const int qt = qt_of(s_tq), nhs = 2 * (qt + 1);
        const int half = s_hs & 1, st = s_ks & 1, sb = s_it & 1, qs = s_tq & 1;
        if (s_hs == 0 && !mbar_wait(B(Q_FULL + qs), (uint32_t)(s_tq >> 1) & 1u, abort_flag, p.status, 25)) return false;
        if (half == 0 && !mbar_wait(B(K_FULL + st), (uint32_t)(s_ks >> 1) & 1u, abort_flag, p.status, 23)) return false;
        if (!mbar_wait(B(S_FREE + sb), (((uint32_t)(s_it >> 1)) & 1u) ^ 1u, abort_flag, p.status, 24)) return false;
        tc_fence_after();
        const uint32_t a = lo_q0 + (uint32_t)qs * TILE16;
        const uint32_t b = lo_k0 + (uint32_t)st * TILE16 + (uint32_t)half * 512u;     // 64 key rows = 8192 bytes
        const uint32_t d = tS + (uint32_t)(sb * HK);
        tc_mma_lo(d, a, b, IDESC_S, 0u);
        tc_mma_lo_acc(d, a + 2, b + 2, IDESC_S);
        tc_mma_lo_acc(d, a + 4, b + 4, IDESC_S);
        tc_mma_lo_acc(d, a + 6, b + 6, IDESC_S);
        if (half == 1) tc_commit(B(K_EMPTY + st));
        if (s_hs == nhs - 1) tc_commit(B(Q_EMPTY + qs));
        tc_commit(B(S_FULL + sb));
        ++s_it;
        if (half == 1) ++s_ks;
        if (++s_hs == nhs) { s_hs = 0; ++s_tq; }
        return true;
      };
      ok = issue_S() && issue_S();
      int it = 0, ks = 0;
      for (int tq = 0; tq < my_tiles && ok; ++tq) {
        const int nhs = 2 * (qt_of(tq) + 1);
        for (int hs = 0; hs < nhs && ok; ++hs, ++it) {
          const int half = hs & 1, st = ks & 1, pb = it & 1;
          if (!mbar_wait(B(P_READY + pb), (uint32_t)(it >> 1) & 1u, abort_flag, p.status, 26)) { ok = false; break; }
          if (half == 0 && !mbar_wait(B(V_FULL + st), (uint32_t)(ks >> 1) & 1u, abort_flag, p.status, 27)) { ok = false; break; }
          // the first product of a query tile overwrites O: the previous tile's O must have been read
          if (hs == 0 && !mbar_wait(B(O_FREE), ((uint32_t)tq & 1u) ^ 1u, abort_flag, p.status, 28)) { ok = false; break; }
          tc_fence_after();
          const uint32_t v = lo_v0 + (uint32_t)st * TILE16 + (uint32_t)half * 512u;   // 64 key rows = 8192 bytes
          const uint32_t a = tP + (uint32_t)(pb * 32);
#pragma unroll
          for (int k = 0; k < HK / UMMA_K; ++k)       // 16 keys = 8 columns of P = 2048 bytes of V per product
            tc_mma_ts_lo(tO, a + (uint32_t)(8 * k), v + (uint32_t)(128 * k), IDESC_PV, (hs | k) != 0 ? 1u : 0u);
          tc_commit(B(P_FREE + pb));                  // also says: O holds the products up to this half-step
          if (half == 1) { tc_commit(B(V_EMPTY + st)); ++ks; }
          ok = issue_S();                             // the score product two half-steps ahead
        }
      }
    }
  } else {
    // ---------------- softmax / output: one thread per query row ----------------
    const int q = warp & 3;
    const int r = q * 32 + lane;                 // row inside the tile = accumulator lane
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    bool ok = true;
    int it = 0;
    // The output of a finished query tile is written one half-step late: its last product is still running
    // when its last P has been handed over, so the thread first does the next tile's first half-step (whose
    // scores are waiting already) and only then reads O, frees it and writes the row.
    bool pend = false;
    float pend_m = 0.f, pend_l = 1.f;
    int pend_tq = 0;
    auto finish_tile = [&](int tq_done, float m_fin, float l_fin, int it_after) -> bool {
      // the tile's last product is half-step it_after - 1: its commit on its P buffer's barrier is the next
      // phase this thread has not yet waited for there
      if (!mbar_wait(B(P_FREE + ((it_after - 1) & 1)), (uint32_t)((it_after - 1) >> 1) & 1u, abort_flag, p.status, 30)) return false;
      tc_fence_after();
      float o_acc[DH];
      tc_ld32(tO + lane_off, o_acc);
      tc_ld32(tO + lane_off + 32u, o_acc + 32);
      tc_wait_ld();
      tc_fence_before();
      mbar_arrive(B(O_FREE));                      // O may be overwritten by the next query tile
      const int qt = qt_of(tq_done), h = head_of(tq_done), seq_row0 = row0_of(tq_done), b = seq_row0 / p.T;
      const float inv = 1.0f / l_fin;
      bf16* orow = p.o + (size_t)(seq_row0 + qt * BQ + r) * p.d + (size_t)h * DH;
#pragma unroll
      for (int jj = 0; jj < DH / 8; ++jj) {
        uint4 w;
        uint32_t* wp = reinterpret_cast<uint32_t*>(&w);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          __nv_bfloat162 ob = __floats2bfloat162_rn(o_acc[8 * jj + 2 * i] * inv, o_acc[8 * jj + 2 * i + 1] * inv);
          wp[i] = *reinterpret_cast<uint32_t*>(&ob);
        }
        *reinterpret_cast<uint4*>(orow + 8 * jj) = w;
      }
      p.lse[((size_t)b * p.H + h) * p.T + (size_t)qt * BQ + r] = (m_fin + log2f(l_fin)) * LN2;
      return true;
    };
    for (int tq = 0; tq < my_tiles && ok; ++tq) {
      const int qt = qt_of(tq), nhs = 2 * (qt + 1);
      float m_run = -INFINITY;                   // running maximum of the scaled scores (log2 domain)
      float m_ref = -INFINITY;                   // the maximum the exponentials are taken against
      float l_run = 0.f;
      for (int hs = 0; hs < nhs && ok; ++hs, ++it) {
        const int sb = it & 1;
        const uint32_t par = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(B(S_FULL + sb), par, abort_flag, p.status, 29)) { ok = false; break; }
        tc_fence_after();
        float v[HK];
        tc_ld32(tS + lane_off + (uint32_t)(sb * HK), v);
        tc_ld32(tS + lane_off + (uint32_t)(sb * HK + 32), v + 32);
        tc_wait_ld();
        tc_fence_before();
        mbar_arrive(B(S_FREE + sb));             // the scores are in registers: the buffer may be overwritten
        uint32_t pk[HK / 2];
        float psum = 0.f;
        // Rows 128 qt + r see keys 64 hs + i only up to the diagonal.  In the last half-step the first 64
        // rows see nothing (their warps write zeros), in the one before it the last 64 rows see everything.
        const bool dead = (hs == nhs - 1) && q < 2;
        if (!dead) {
          if (hs >= nhs - 2 && ((hs == nhs - 2) ? q < 2 : true)) {
            const int lim = r - 64 * (hs - (nhs - 2));         // last visible key of this half-step
#pragma unroll
            for (int i = 0; i < HK; ++i) v[i] = (i > lim) ? -INFINITY : v[i];
          }
          float m4[4] = {max3(v[0], v[1], v[2]), max3(v[3], v[4], v[5]), max3(v[6], v[7], v[8]), max3(v[9], v[10], v[11])};
#pragma unroll
          for (int i = 12; i < 60; i += 8) {     // three-input maxima, four chains
            m4[0] = max3(m4[0], v[i], v[i + 1]); m4[1] = max3(m4[1], v[i + 2], v[i + 3]);
            m4[2] = max3(m4[2], v[i + 4], v[i + 5]); m4[3] = max3(m4[3], v[i + 6], v[i + 7]);
          }
          m4[0] = max3(m4[0], v[60], v[61]); m4[1] = max3(m4[1], v[62], v[63]);
          const float mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
          const float m_new = fmaxf(m_run, mx * p.scale_log2);   // finite: key 0 is visible to every row
          m_run = m_new;
          if (hs == 0) {
            m_ref = m_new;
          } else {
            const bool need = m_new - m_ref > RESCALE_STEP;
            if (__any_sync(0xffffffffu, need)) {
              // O must hold the products up to half-step it - 1 (the next one waits for P_READY below).  That
              // product's commit on its P buffer's barrier is the next phase this thread has not yet seen
              // there (it waits on each of the two barriers every other half-step), so the parity is safe.
              if (!mbar_wait(B(P_FREE + ((it - 1) & 1)), (uint32_t)((it - 1) >> 1) & 1u, abort_flag, p.status, 30)) { ok = false; break; }
              tc_fence_after();
              const float corr = need ? ex2(m_ref - m_new) : 1.0f;
#pragma unroll
              for (int oc = 0; oc < DH; oc += 32) {
                float ov[32];
                tc_ld32(tO + lane_off + (uint32_t)oc, ov);
                tc_wait_ld();
                uint32_t w[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) w[i] = __float_as_uint(ov[i] * corr);
                tc_st16(tO + lane_off + (uint32_t)oc, w);
                tc_st16(tO + lane_off + (uint32_t)(oc + 16), w + 16);
              }
              l_run *= corr;
              if (need) m_ref = m_new;
            }
          }
          // exponentials on pairs: one packed multiply-add and one packed add per two scores
          const uint64_t sc2 = pack2(p.scale_log2, p.scale_log2), nm2 = pack2(-m_ref, -m_ref);
          uint64_t ps2 = pack2(0.f, 0.f);
#pragma unroll
          for (int i = 0; i < HK; i += 2) {
            float a0, a1;
            unpack2(fma2(pack2(v[i], v[i + 1]), sc2, nm2), a0, a1);
            const float p0 = ex2(a0), p1 = ex2(a1);
            ps2 = add2(ps2, pack2(p0, p1));
            __nv_bfloat162 pb2 = __floats2bfloat162_rn(p0, p1);
            pk[i >> 1] = *reinterpret_cast<uint32_t*>(&pb2);
          }
          float s0, s1;
          unpack2(ps2, s0, s1);
          psum = s0 + s1;
        } else {
#pragma unroll
          for (int i = 0; i < HK / 2; ++i) pk[i] = 0u;
        }
        // P buffer of this parity: the product that read it two half-steps ago must be done
        if (!mbar_wait(B(P_FREE + sb), par ^ 1u, abort_flag, p.status, 31)) { ok = false; break; }
        tc_fence_after();
        tc_st16(tP + lane_off + (uint32_t)(sb * 32), pk);
        tc_st16(tP + lane_off + (uint32_t)(sb * 32 + 16), pk + 16);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(B(P_READY + sb));
        l_run += psum;
        if (hs == 0 && pend) {                   // the previous tile's output (its products are done by now)
          if (!finish_tile(pend_tq, pend_m, pend_l, it)) { ok = false; break; }
          pend = false;
        }
      }
      pend = true; pend_m = m_ref; pend_l = l_run; pend_tq = tq;
    }
    if (ok && pend) finish_tile(pend_tq, pend_m, pend_l, it);
  }

  // ---------------- teardown ----------------
  __syncwarp();
  if (*abort_flag) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

PerDeviceOnce g_once;

}  // namespace

cudaError_t attention_fwd_t5_h64(const void* qkv, int nseq, int T, int H, int d, void* o, float* lse, int* status,
                                 cudaStream_t st) {
  if (H < 1 || d != H * DH || T < BQ || T % BQ != 0) return cudaErrorInvalidValue;
  const int dev = current_device(), sms = num_sms();
  if (dev < 0 || sms < 1 || !tensor_map_encoder()) return cudaErrorInitializationError;
  if (g_once.needed(dev)) {
    if (cudaFuncSetAttribute(attn_fwd_t5_h64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess)
      return cudaErrorInitializationError;
    g_once.done(dev);
  }
  if (!status) status = library_status_word();
  if (!status) return cudaErrorInitializationError;
  CUtensorMap mQKV;
  if (!cached_map_2d(&mQKV, qkv, (uint64_t)nseq * T, (uint64_t)3 * d, (uint64_t)3 * d, 64, BQ, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B))
    return cudaErrorInvalidValue;
  F64Params p;
  p.T = T; p.H = H; p.d = d; p.scale_log2 = LOG2E / sqrtf((float)DH); p.o = (bf16*)o; p.lse = lse; p.status = status;
  p.nitems = nseq * H;
  const int nq = T / BQ, units = p.nitems * nq, cap = 2 * sms;
  const int grid = ((units < cap ? units : cap) / nq) * nq;          // a multiple of nq: whole items per round
  if (grid < nq) return cudaErrorInvalidValue;
  attn_fwd_t5_h64_kernel<<<grid, THREADS, SMEM, st>>>(mQKV, p);
  return cudaGetLastError();
}

}  // namespace sl
