// Causal multi-head attention forward on the 5th-generation tensor cores (tcgen05 + TMEM + TMA),
// bf16, head width 64 or 128, sequence length a multiple of 128.
//
// Persistent CTAs (two per SM at head width 64, one at 128, where every operand tile is two
// 64-feature blocks and O takes 128 tensor-memory columns).  The work units are 128-row query tiles
// of (sequence, head) items, longest first, dealt round-robin to the CTAs (K/V tiles are re-read
// from L2); with two CTAs on an SM the softmax of one overlaps the products of the other.
// Per 128-row key tile:
//   S  = Q K^T      tcgen05.mma M128 N128 K16 x4 per 64 features, both operands K-major from TMA-swizzled tiles
//   softmax         two threads per query row read their halves of S from tensor memory (twice:
//                   row max, then exponentials), keep the running max / sum, write P (bf16) back to
//                   tensor memory
//   O' = P V        tcgen05.mma M128 N64 K16 x8 per 64 output features, P read from tensor memory; V is used as loaded
//                   ([key, feature] rows, i.e. an MN-major operand), no transpose
//   O += P V        accumulates in tensor memory over the key tiles of a query tile; before a step's
//                   product the row's two threads rescale their halves of the columns of O in place by the
//                   factor the new running maximum implies
// Warp roles (320 threads): warp 0 TMA producer, warp 1 tensor-memory owner + MMA issuer,
// warps 2..9 softmax: two threads per query row (warp w owns accumulator lanes 32*(w%4)..+31, warps
// 2..5 the first half of the score and output columns, warps 6..9 the second).
// All mbarrier waits are bounded (see tc_common.cuh); on expiry a code is left in `status`.
#include "host_common.h"
#include "tc_common.cuh"

namespace sl {
namespace {

using namespace tc;

constexpr int BQ = 128;                   // query rows per tile
constexpr int BKV = 128;                  // key rows per step
constexpr int TILE = BQ * 64 * 2;         // 16 KB: one [128 x 64] bf16 block; a head of width DH is DH / 64 blocks
constexpr int T5_THREADS = 320;           // TMA warp, MMA warp, eight softmax warps (two threads per row)
constexpr int SM_THREADS = 256;
// Head width 64: two CTAs per SM (83 KB, 256 tensor-memory columns each).  Head width 128: every
// operand is two blocks, O takes 128 columns, one CTA per SM.
template <int DH> struct FwdCfg {
  static constexpr int NB = DH / 64;
  static constexpr int OFF_Q = 0, OFF_K = NB * TILE, OFF_V = 3 * NB * TILE, OFF_P = 4 * NB * TILE /* output staging */,
                       OFF_BAR = 5 * NB * TILE,
                       OFF_X = OFF_BAR + 256 /* half-row maxima and sums exchanged by the two threads of a row: 4 KB */;
  static constexpr int SMEM = 5 * NB * TILE + 256 + 4096 + 1024;     // tiles + barriers + exchange + alignment slack
  static constexpr int TMEM_COLS = DH == 64 ? 256 : 512;             // S [0,128), O [128,128+DH), P (bf16) after it
  static constexpr int CTAS_PER_SM = DH == 64 ? 2 : 1;
};
constexpr uint32_t IDESC_S = make_idesc(BQ, BKV);
constexpr uint32_t IDESC_PV = make_idesc(BQ, 64) | (1u << 16);   // one 64-column block of O; B operand MN-major
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

// barrier slots
enum { Q_FULL = 0, Q_EMPTY = 1, K_FULL = 2 /*+stage*/, K_EMPTY = 4 /*+stage*/, V_FULL = 6, V_EMPTY = 7,
       S_FULL = 8, S_FREE = 9, P_READY = 10, O_FULL = 11, O_FREE = 12, X_MAX = 13, X_SUM = 14, N_BARS = 15 };

// Operand descriptors are passed to the products as their address-carrying lower halves (desc_lo);
// the upper half is the same constant for the K-major tiles (Q, K, P) and for V, which is used as
// loaded ([key, feature] rows = an MN-major right operand with 128-byte rows and 128-byte swizzle,
// groups of 8 key rows 1024 bytes apart).
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct T5Params {
  int T, H, d;
  int nitems;              // nseq * H (sequence, head) items, shared out over the CTAs
  float scale_log2;
  float* lse;
  int* status;
};

// The CTA's work is a flat sequence of (query tile, key tile) steps: query tiles nq-1 .. 0, for
// each the key tiles 0 .. qt.  `it` counts steps, `iq` counts query tiles; barrier parities derive
// from these counters so that every role stays in lock step without sharing state.
template <int DH>
__global__ void __launch_bounds__(T5_THREADS, FwdCfg<DH>::CTAS_PER_SM)
attn_fwd_t5_kernel(const __grid_constant__ CUtensorMap mapQKV, const __grid_constant__ CUtensorMap mapO, T5Params p) {
  using C = FwdCfg<DH>;
  constexpr int NB = C::NB, OFF_Q = C::OFF_Q, OFF_K = C::OFF_K, OFF_V = C::OFF_V, OFF_P = C::OFF_P, OFF_BAR = C::OFF_BAR,
                OFF_X = C::OFF_X, TMEM_COLS = C::TMEM_COLS;
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
  // persistent: the work units are (query tile, item) pairs, item = (sequence, head), ordered by
  // falling cost (the last query tile of every item first: it has the most key tiles); this CTA
  // takes units blockIdx.x, blockIdx.x + gridDim.x, ..., so every CTA gets the same mix of long and
  // short tiles.  Every role walks its units in one flat sequence tq = 0 .. my_tiles - 1, so the loads
  // of the next unit are issued while the current one ends.
  const int n_units = p.nitems * nq;
  const int my_tiles = (int)blockIdx.x < n_units ? (n_units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  auto unit_of = [&](int tq) { return (int)blockIdx.x + tq * (int)gridDim.x; };
  auto qt_of = [&](int tq) { return nq - 1 - unit_of(tq) / p.nitems; };
  auto item_of = [&](int tq) { return unit_of(tq) % p.nitems; };
  auto head_of = [&](int tq) { return item_of(tq) % p.H; };
  auto row0_of = [&](int tq) { return (item_of(tq) / p.H) * p.T; };

  if (threadIdx.x == 0) {
    for (int i = 0; i < N_BARS; ++i)
      mbar_init(B(i), (i == S_FREE || i == P_READY || i == O_FREE || i == X_MAX || i == X_SUM) ? SM_THREADS : 1);
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
  const uint32_t tS = tmem_base, tO = tmem_base + 128u, tP = tmem_base + 128u + (uint32_t)DH;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      bool ok = true;
      int it = 0;                                   // running step index of the K loads issued
      auto load_K = [&](int step, int j, int h, int seq_row0) -> bool {
        const int s = step & 1;
        if (!mbar_wait(B(K_EMPTY + s), (((uint32_t)(step >> 1)) & 1u) ^ 1u, abort_flag, p.status, 21)) return false;
        mbar_expect_tx(B(K_FULL + s), NB * TILE);
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
          tma_load_2d(base + OFF_K + (s * NB + nb) * TILE, &mapQKV, B(K_FULL + s), p.d + h * DH + 64 * nb, seq_row0 + j * BKV);
        return true;
      };
      for (int tq = 0; tq < my_tiles && ok; ++tq) {
        const int qt = qt_of(tq);
        const int h = head_of(tq), seq_row0 = row0_of(tq);
        // Q of this query tile (the buffer is free once the previous tile's last S product is done)
        if (!mbar_wait(B(Q_EMPTY), ((uint32_t)tq & 1u) ^ 1u, abort_flag, p.status, 20)) { ok = false; break; }
        mbar_expect_tx(B(Q_FULL), NB * TILE);
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
          tma_load_2d(base + OFF_Q + nb * TILE, &mapQKV, B(Q_FULL), h * DH + 64 * nb, seq_row0 + qt * BQ);
        if (tq == 0) ok = load_K(0, 0, h, seq_row0);   // K runs one step ahead of V
        for (int j = 0; j <= qt && ok; ++j, ++it) {
          // next step's K: the next key tile, or key tile 0 of the next query tile (maybe of the next item)
          if (j < qt) ok = load_K(it + 1, j + 1, h, seq_row0);
          else if (tq + 1 < my_tiles) ok = load_K(it + 1, 0, head_of(tq + 1), row0_of(tq + 1));
          if (!ok) break;
          if (!mbar_wait(B(V_EMPTY), ((uint32_t)it & 1u) ^ 1u, abort_flag, p.status, 22)) { ok = false; break; }
          mbar_expect_tx(B(V_FULL), NB * TILE);
#pragma unroll
          for (int nb = 0; nb < NB; ++nb)
            tma_load_2d(base + OFF_V + nb * TILE, &mapQKV, B(V_FULL), 2 * p.d + h * DH + 64 * nb, seq_row0 + j * BKV);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      bool ok = true;
      const uint32_t lo_q = desc_lo(base + OFF_Q), lo_k0 = desc_lo(base + OFF_K), lo_v = desc_lo(base + OFF_V);
      constexpr uint32_t TILE16 = TILE >> 4;
      // S of step `step`; first_of_q: wait for the query tile iq; last_of_q: release the Q buffer
      auto issue_S = [&](int step, int tq, bool first_of_q, bool last_of_q) -> bool {
        const int s = step & 1;
        if (first_of_q && !mbar_wait(B(Q_FULL), (uint32_t)tq & 1u, abort_flag, p.status, 25)) return false;
        if (!mbar_wait(B(K_FULL + s), (uint32_t)(step >> 1) & 1u, abort_flag, p.status, 23)) return false;
        if (!mbar_wait(B(S_FREE), ((uint32_t)step & 1u) ^ 1u, abort_flag, p.status, 24)) return false;
        tc_fence_after();
        const uint32_t lo_k = lo_k0 + (uint32_t)(s * NB) * TILE16;
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {                    // 64 features per block; 16 elements = +32 bytes = +2 units
          const uint32_t a = lo_q + (uint32_t)nb * TILE16, bq = lo_k + (uint32_t)nb * TILE16;
          tc_mma_lo(tS, a, bq, IDESC_S, nb != 0 ? 1u : 0u);
          tc_mma_lo_acc(tS, a + 2, bq + 2, IDESC_S);
          tc_mma_lo_acc(tS, a + 4, bq + 4, IDESC_S);
          tc_mma_lo_acc(tS, a + 6, bq + 6, IDESC_S);
        }
        tc_commit(B(K_EMPTY + s));
        if (last_of_q) tc_commit(B(Q_EMPTY));
        tc_commit(B(S_FULL));
        return true;
      };
      int it = 0;
      ok = issue_S(0, 0, true, qt_of(0) == 0);
      for (int tq = 0; tq < my_tiles && ok; ++tq) {
        const int qt = qt_of(tq);
        for (int j = 0; j <= qt && ok; ++j, ++it) {
          // next step's S overlaps this step's softmax
          if (j < qt) ok = issue_S(it + 1, tq, false, j + 1 == qt);
          else if (tq + 1 < my_tiles) ok = issue_S(it + 1, tq + 1, true, qt_of(tq + 1) == 0);
          if (!ok) break;
          if (!mbar_wait(B(P_READY), (uint32_t)it & 1u, abort_flag, p.status, 26)) { ok = false; break; }
          if (!mbar_wait(B(V_FULL), (uint32_t)it & 1u, abort_flag, p.status, 27)) { ok = false; break; }
          // the first product of a query tile overwrites O: the previous tile's O must have been read
          if (j == 0 && !mbar_wait(B(O_FREE), ((uint32_t)tq & 1u) ^ 1u, abort_flag, p.status, 28)) { ok = false; break; }
          tc_fence_after();
          // P is read from tensor memory (16 keys = 8 columns per product);
          // V advances 16 key rows = 2048 bytes = 128 units per product
#pragma unroll
          for (int nb = 0; nb < NB; ++nb)                    // one 64-column block of O per block of V
#pragma unroll
            for (int k = 0; k < BKV / UMMA_K; ++k)
              tc_mma_ts_lo(tO + (uint32_t)(64 * nb), tP + (uint32_t)(8 * k), lo_v + (uint32_t)nb * TILE16 + (uint32_t)(128 * k),
                           IDESC_PV, (j | k) != 0 ? 1u : 0u);
          tc_commit(B(V_EMPTY));      // V (and P) reusable
          tc_commit(B(O_FULL));       // this step's contribution is in O
        }
      }
    }
  } else {
    // ---------------- softmax / output: two threads per query row ----------------
    // Warps 2..5 take score columns [0, 64) and output columns [0, 32) of their lane quarter's rows,
    // warps 6..9 the other halves.  The two threads of a row exchange their half-row maxima through
    // shared memory once per step (barrier X_MAX) and their partial row sums once per query tile
    // (barrier X_SUM); everything else they do on their own halves.
    const int q = warp & 3;
    const int hf = (warp - 2) >> 2;              // which half of the columns
    const int r = q * 32 + lane;                 // row inside the tile = accumulator lane
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    float* xmax = reinterpret_cast<float*>(base_ptr + OFF_X);          // [2 steps][2 halves][128 rows]
    float* xsum = xmax + 2 * 2 * BQ;                                   // [2 tiles][2 halves][128 rows]
    bool ok = true;
    int it = 0;
    for (int tq = 0; tq < my_tiles; ++tq) {
      const int qt = qt_of(tq);
      const int h = head_of(tq), seq_row0 = row0_of(tq), b = seq_row0 / p.T;
      float m_run = -INFINITY, l_run = 0.f;      // l_run: this thread's half of the row sum
      for (int j = 0; j <= qt && ok; ++j, ++it) {
        if (!mbar_wait(B(S_FULL), (uint32_t)it & 1u, abort_flag, p.status, 29)) { ok = false; break; }
        tc_fence_after();
        const bool diag = (j == qt);
        // On the diagonal tile only columns <= r count; whole 32-column chunks beyond the row are
        // skipped (their probabilities are zero), the chunk that holds the diagonal is masked.
        const int c_last = diag ? (r & ~31) : (BKV - 32);       // last chunk with a live column
        const int c_lo = hf * (BKV / 2), c_hi = c_lo + BKV / 2;
        // pass 1: maximum of the raw scores of this half row (the scale is positive)
        float mx = -INFINITY;
#pragma unroll 1
        for (int c = c_lo; c < c_hi && c <= c_last; c += 32) {
          float v[32];
          tc_ld32(tS + lane_off + (uint32_t)c, v);
          tc_wait_ld();
          if (diag && c == c_last) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = (c + i > r) ? -INFINITY : v[i];
          }
          float m4[4] = {v[0], v[1], v[2], v[3]};          // four short chains instead of one of 32
#pragma unroll
          for (int i = 4; i < 32; i += 4) {
            m4[0] = fmaxf(m4[0], v[i]); m4[1] = fmaxf(m4[1], v[i + 1]);
            m4[2] = fmaxf(m4[2], v[i + 2]); m4[3] = fmaxf(m4[3], v[i + 3]);
          }
          mx = fmaxf(mx, fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])));
        }
        float* xm = xmax + (it & 1) * 2 * BQ;
        xm[hf * BQ + r] = mx;
        mbar_arrive(B(X_MAX));
        if (!mbar_wait(B(X_MAX), (uint32_t)it & 1u, abort_flag, p.status, 31)) { ok = false; break; }
        mx = fmaxf(mx, xm[(hf ^ 1) * BQ + r]);
        const float m_new = fmaxf(m_run, mx * p.scale_log2);   // finite: column 0 is never masked
        const float corr = ex2(m_run - m_new);
        // O stays in tensor memory and the products accumulate onto it; when the running maximum
        // moves, this thread's 32 columns of it are rescaled in place before this step's product
        // (which cannot start before P_READY below).  The previous step's product is long done.
        if (j > 0) {
          if (!mbar_wait(B(O_FULL), (uint32_t)(it - 1) & 1u, abort_flag, p.status, 30)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int oc = 0; oc < DH / 2; oc += 32) {
            float v[32];
            tc_ld32(tO + lane_off + (uint32_t)(hf * (DH / 2) + oc), v);
            tc_wait_ld();
            uint32_t w[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) w[i] = __float_as_uint(v[i] * corr);
            tc_st16(tO + lane_off + (uint32_t)(hf * (DH / 2) + oc), w);
            tc_st16(tO + lane_off + (uint32_t)(hf * (DH / 2) + oc + 16), w + 16);
          }
        }
        // pass 2: exponentials, partial row sum, P back to tensor memory
        float psum = 0.f;
#pragma unroll 1
        for (int c = c_lo; c < c_hi; c += 32) {
          uint32_t pk[16];
          if (c <= c_last) {
            float v[32];
            tc_ld32(tS + lane_off + (uint32_t)c, v);
            tc_wait_ld();
            if (diag && c == c_last) {          // mask on the scores: the element loop stays free of tests
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] = (c + i > r) ? -INFINITY : v[i];
            }
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float p0 = ex2(fmaf(v[i], p.scale_log2, -m_new)), p1 = ex2(fmaf(v[i + 1], p.scale_log2, -m_new));
              psum += p0 + p1;
              __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
              pk[i >> 1] = *reinterpret_cast<uint32_t*>(&pb);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = 0u;
          }
          tc_st16(tP + lane_off + (uint32_t)(c >> 1), pk);          // 32 bf16 = 16 columns of this row's lane
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(B(S_FREE));                      // S may be overwritten
        mbar_arrive(B(P_READY));                     // P complete in tensor memory
        l_run = l_run * corr + psum;
        m_run = m_new;
      }
      // row sum = the two partial sums; normalise, stage this thread's half of the output row in the
      // staging tile, one TMA store per query tile
      float l_tot = l_run;
      if (ok) {
        float* xs = xsum + (tq & 1) * 2 * BQ;
        xs[hf * BQ + r] = l_run;
        mbar_arrive(B(X_SUM));
        if (!mbar_wait(B(X_SUM), (uint32_t)tq & 1u, abort_flag, p.status, 32)) ok = false;
        else l_tot += xs[(hf ^ 1) * BQ + r];
      }
      // the tile's last product
      if (ok && !mbar_wait(B(O_FULL), (uint32_t)(it - 1) & 1u, abort_flag, p.status, 30)) ok = false;
      if (ok) {
        tc_fence_after();
        float o_acc[DH / 2];
#pragma unroll
        for (int oc = 0; oc < DH / 2; oc += 32) tc_ld32(tO + lane_off + (uint32_t)(hf * (DH / 2) + oc), o_acc + oc);
        tc_wait_ld();
        tc_fence_before();
        mbar_arrive(B(O_FREE));                      // O may be overwritten by the next query tile
        const float inv = 1.0f / l_tot;
#pragma unroll
        for (uint32_t jj = 0; jj < DH / 16; ++jj) {  // this thread's DH/2 columns as 16-byte chunks of 8
          uint32_t w[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 ob = __floats2bfloat162_rn(o_acc[8 * jj + 2 * i] * inv, o_acc[8 * jj + 2 * i + 1] * inv);
            w[i] = *reinterpret_cast<uint32_t*>(&ob);
          }
          const uint32_t gc = (uint32_t)(hf * (DH / 2)) + 8u * jj;          // first column of the chunk in the head
          const uint32_t orow = base + OFF_P + (gc >> 6) * TILE + (uint32_t)r * 128u;
          const uint32_t chunk = ((gc & 63u) >> 3) ^ ((uint32_t)r & 7u);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(orow + (chunk << 4)), "r"(w[0]), "r"(w[1]),
                       "r"(w[2]), "r"(w[3]) : "memory");
        }
        if (hf == 0) p.lse[((size_t)b * p.H + h) * p.T + (size_t)qt * BQ + r] = (m_run + log2f(l_tot)) * LN2;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("bar.sync 1, 256;" ::: "memory");         // the eight softmax warps (always reached)
      if (ok && warp == 2 && lane == 0) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
          asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                       ::"l"(&mapO), "r"(base + OFF_P + nb * TILE), "r"(h * DH + 64 * nb), "r"(seq_row0 + qt * BQ) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // staging reusable for the next tile
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
    }
    if (warp == 2 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
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

bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  return cached_map_2d(m, ptr, rows, cols, cols, 64, box_rows, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

// kernel attributes are per device: set them the first time each device launches
bool init_device() {
  const int dev = current_device();
  if (dev < 0 || !tensor_map_encoder()) return false;
  if (!g_once.needed(dev)) return true;
  if (cudaFuncSetAttribute(attn_fwd_t5_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdCfg<128>::SMEM) != cudaSuccess) return false;
  g_once.done(dev);
  return true;
}

}  // namespace

bool attention_t5_supported(int dt, int T, int H, int d) {
  return dt == DT_BF16 && H > 0 && d % H == 0 && d / H == 64 && T >= BQ && T % BQ == 0 && T / BQ <= 64;
}

// The forward kernel also exists for heads of width 128 (the backward kernels do not).
bool attention_fwd_t5_supported(int dt, int T, int H, int d) {
  return dt == DT_BF16 && H > 0 && d % H == 0 && (d / H == 64 || d / H == 128) && T >= BQ && T % BQ == 0 && T / BQ <= 64;
}

cudaError_t attention_fwd_t5(const void* qkv, int nseq, int T, int H, int d, void* o, float* lse, int* status,
                             cudaStream_t st) {
  if (!attention_fwd_t5_supported(DT_BF16, T, H, d)) return cudaErrorInvalidValue;
  if (d / H == 64) return attention_fwd_t5_h64(qkv, nseq, T, H, d, o, lse, status, st);   // its own kernel
  if (!init_device()) return cudaErrorInitializationError;
  const int sms = num_sms();
  if (!status) status = library_status_word();
  if (!status || sms < 1) return cudaErrorInitializationError;
  CUtensorMap mQKV, mO;
  if (!make_map(&mQKV, qkv, (uint64_t)nseq * T, (uint64_t)3 * d, BQ)) return cudaErrorInvalidValue;
  if (!make_map(&mO, o, (uint64_t)nseq * T, (uint64_t)d, BQ)) return cudaErrorInvalidValue;
  const int dh = d / H;
  T5Params p;
  p.T = T; p.H = H; p.d = d; p.scale_log2 = LOG2E / sqrtf((float)dh); p.lse = lse;
  p.status = status;
  p.nitems = nseq * H;
  const int cap = FwdCfg<128>::CTAS_PER_SM * sms;                                  // persistent CTAs
  attn_fwd_t5_kernel<128><<<p.nitems < cap ? p.nitems : cap, T5_THREADS, FwdCfg<128>::SMEM, st>>>(mQKV, mO, p);
  return cudaGetLastError();
}

}  // namespace sl
