// Adapter gradients G_A, G_B (Eq. 4-7) on the tensor cores.  The reduction over tokens
//   out[j][c] = sum_m Wt[m, w0 + j] * Z[m, z0 + c]
// is a product whose contraction index is the row index of BOTH operands, so both are fed to
// tcgen05.mma as MN-major tiles straight from their row-major layout (no transposed copies):
//   D[c, j] (128 x 64, fp32 in tensor memory) += Z_tile^T (128 c x 64 tokens) * Wt_tile (64 tokens x 64 j)
// One CTA owns 128 feature columns and one chunk of the token range; TMA streams 64-token blocks
// through a 4-stage ring, one thread issues the products, four warps read the accumulator back and
// write the wanted columns to scratch; a second kernel adds the chunks in a fixed order (no float
// atomics).  HBM-bound: every Z element is read once, the 64-column weight tile is re-read per
// column tile (from L2).
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"
#include "host_common.h"
#include "tc_common.cuh"

namespace sl {
namespace {

using namespace tc;

constexpr int LT_C = 128;           // feature columns per CTA = accumulator lanes
constexpr int LT_K = 64;             // tokens per pipeline stage
constexpr int LT_N = 64;             // weight columns per product (one 128-byte swizzle row)
constexpr int LT_STAGES = 4;
constexpr int LT_ZBOX = LT_K * 64 * 2;                 // one [64 tokens][64 columns] box
constexpr int LT_STAGE = 2 * LT_ZBOX + LT_K * LT_N * 2;
constexpr int LT_THREADS = 192;      // warp 0: TMA, warp 1: MMA, warps 2-5: accumulator read-back
constexpr int LT_OFF_BAR = LT_STAGES * LT_STAGE;
constexpr int LT_SMEM = LT_OFF_BAR + 128 + 1024;
constexpr int LT_TMEM_COLS = 64;
// fp32 accumulate, bf16 x bf16, A and B both MN-major
constexpr uint32_t LT_IDESC = make_idesc(LT_C, LT_N) | (1u << 15) | (1u << 16);

struct LgParams {
  int C, rows_per_chunk, R, r, rp, wsel0;
  float* partial;
  int* status;
};
// Up to LT_MAX_JOBS reductions over the same token rows in one launch (blockIdx.z picks the job): the
// adapter gradients of one layer, e.g. G_A of all targets from u and G_B of each target from its slice
// of dy.  One launch instead of one per job: the jobs are short (tens of microseconds), so their start-up,
// tail and launch gaps weigh as much as their traffic.
constexpr int LT_MAX_JOBS = 4;
struct LgBatch {
  CUtensorMap mapZ[LT_MAX_JOBS];
  CUtensorMap mapW[LT_MAX_JOBS];
  LgParams p[LT_MAX_JOBS];
  int wx0[LT_MAX_JOBS];
};

// MN-major operand stored as [k rows][64 elements] boxes (128-byte rows, 128-byte swizzle): groups
// of 8 k-rows are 1024 bytes apart; `mn_stride` is the distance between consecutive 64-element
// blocks along the MN dimension (unused when the operand is one block wide).
__device__ __forceinline__ uint64_t desc_mn(uint32_t addr, uint32_t mn_stride) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((mn_stride >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

__global__ void __launch_bounds__(LT_THREADS, 2)
lora_grad_tc_kernel(const __grid_constant__ LgBatch bt) {
  const CUtensorMap& mapZ = bt.mapZ[blockIdx.z];
  const CUtensorMap& mapW = bt.mapW[blockIdx.z];
  const LgParams& p = bt.p[blockIdx.z];
  const int wx0 = bt.wx0[blockIdx.z];
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t bar = base + LT_OFF_BAR;
  auto FULL = [&](int s) { return bar + 8u * s; };
  auto EMPTY = [&](int s) { return bar + 8u * (LT_STAGES + s); };
  const uint32_t ACC = bar + 8u * (2 * LT_STAGES);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + LT_OFF_BAR + 8 * (2 * LT_STAGES + 1));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + LT_OFF_BAR + 8 * (2 * LT_STAGES + 1) + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int c0 = blockIdx.x * LT_C, chunk = blockIdx.y;
  const int row0 = chunk * p.rows_per_chunk;
  const int kblocks = p.rows_per_chunk / LT_K;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2 * LT_STAGES + 1; ++i) mbar_init(bar + 8u * i, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)LT_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < kblocks; ++kb) {
        const int s = kb % LT_STAGES;
        if (!mbar_wait(EMPTY(s), (((uint32_t)(kb / LT_STAGES)) & 1u) ^ 1u, abort_flag, p.status, 40)) break;
        mbar_expect_tx(FULL(s), LT_STAGE);
        const uint32_t dst = base + s * LT_STAGE;
        const int row = row0 + kb * LT_K;
        tma_load_2d(dst, &mapZ, FULL(s), c0, row);
        tma_load_2d(dst + LT_ZBOX, &mapZ, FULL(s), c0 + 64, row);      // past the last column: zero fill
        tma_load_2d(dst + 2 * LT_ZBOX, &mapW, FULL(s), wx0, row);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      bool ok = true;
      for (int kb = 0; kb < kblocks && ok; ++kb) {
        const int s = kb % LT_STAGES;
        if (!mbar_wait(FULL(s), ((uint32_t)(kb / LT_STAGES)) & 1u, abort_flag, p.status, 41)) { ok = false; break; }
        tc_fence_after();
        const uint32_t a = base + s * LT_STAGE, b = a + 2 * LT_ZBOX;
#pragma unroll
        for (int k = 0; k < LT_K / UMMA_K; ++k)     // 16 tokens = two 8-row groups = 2048 bytes
          tc_mma_bf16(tmem_base, desc_mn(a + k * 2048, LT_ZBOX), desc_mn(b + k * 2048, 16), LT_IDESC,
                      (kb | k) != 0 ? 1u : 0u);
        tc_commit(EMPTY(s));
      }
      if (ok) tc_commit(ACC);
    }
  } else {
    // accumulator read-back: lane group (warp % 4) of tensor memory, one feature column per thread
    const int q = warp & 3;
    if (mbar_wait(ACC, 0u, abort_flag, p.status, 42)) {
      tc_fence_after();
      float v[LT_N];
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
      tc_ld32(t_row, v);
      tc_ld32(t_row + 32u, v + 32);
      tc_wait_ld();
      const int c = c0 + q * 32 + lane;
      if (c < p.C) {
        float* out = p.partial + (size_t)chunk * p.R * p.C + c;
        const int sh = p.rp == 16 ? 4 : (p.rp == 32 ? 5 : 6);
#pragma unroll
        for (int col = 0; col < LT_N; ++col) {
          const int rel = col - p.wsel0;
          const int t = rel >> sh, jj = rel & (p.rp - 1);
          const int j = t * p.r + jj;
          if (rel >= 0 && jj < p.r && j < p.R) out[(size_t)j * p.C] = v[col];
        }
      }
    }
  }

  __syncwarp();
  if (*abort_flag) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);     // let copies in flight land before the CTA exits
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)LT_TMEM_COLS) : "memory");
  }
}

PerDeviceOnce g_once;

// bf16 [rows, cols] with leading dimension ld; box = 64 columns x 64 rows, 128-byte swizzle
bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld) {
  return cached_map_2d(m, ptr, rows, cols, ld, 64, (uint32_t)LT_K, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

bool init_device() {
  const int dev = current_device();
  if (dev < 0 || !tensor_map_encoder()) return false;
  if (!g_once.needed(dev)) return true;
  if (cudaFuncSetAttribute(lora_grad_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, LT_SMEM) != cudaSuccess)
    return false;
  g_once.done(dev);
  return true;
}

bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

bool lora_grad_tc_supported(int dt, const void* Z, int64_t ldz, int zcol0, int C, const void* Wt, int64_t ldwt,
                            int wcol0, int r, int rp, int nt, int M, int rows_per_group) {
  if (dt != DT_BF16 || !(rp == 16 || rp == 32 || rp == 64) || r < 1 || r > rp || nt < 1) return false;
  if (M % 128 != 0 || (rows_per_group > 0 && (rows_per_group % 128 != 0 || M % rows_per_group != 0))) return false;
  if (C % 8 != 0 || ldz % 8 != 0 || zcol0 % 8 != 0 || ldwt % 64 != 0 || !al16(Z) || !al16(Wt)) return false;
  const int wsel0 = wcol0 % LT_N;
  if (wsel0 + (nt - 1) * rp + r > LT_N || wcol0 - wsel0 + LT_N > ldwt) return false;
  return true;
}

// Chunks per group for a grid of `ctas_per_chunk_set` CTAs per chunk: the choice that minimises
// (waves of 296 resident CTAs) x (rows per chunk), every chunk a whole number of 128-row blocks.
static int pick_chunks(int ctas_per_chunk_set, int rpg) {
  int best = 1;
  double best_cost = 1e300;
  for (int s = 1; s <= rpg / 128; ++s) {
    if (rpg % (s * 128) != 0) continue;
    const int ctas = ctas_per_chunk_set * s;
    const double cost = (double)((ctas + 295) / 296) * ((double)rpg / s + 256.0);   // + a chunk's start-up, in rows
    if (cost < best_cost) { best_cost = cost; best = s; }
  }
  return best;
}

// Chunk partials of job j go to partial + offset_j as [chunk][R_j][C] (R_j = nt*r); *chunks_per_group
// receives the number of chunks per group (the same for every job) so that the caller's second kernel
// can add them, offsets[j] the start of job j's partials (floats).  All jobs share M, rows_per_group and C.
cudaError_t lora_grad_tc_partial_batch(const LoraGradJob* jobs, int njobs, int M, int rows_per_group, float* partial,
                                       size_t partial_floats, int* status, int* chunks_per_group, size_t* offsets,
                                       cudaStream_t st) {
  if (njobs < 1 || njobs > LT_MAX_JOBS) return cudaErrorInvalidValue;
  if (!init_device()) return cudaErrorNotSupported;
  if (!status) status = library_status_word();
  if (!status) return cudaErrorNotSupported;
  const int rpg = rows_per_group > 0 ? rows_per_group : M;
  const int groups = M / rpg;
  const int C = jobs[0].C;
  const int ctiles = (C + LT_C - 1) / LT_C;
  const int s = pick_chunks(ctiles * groups * njobs, rpg);
  LgBatch bt;
  size_t off = 0;
  for (int j = 0; j < njobs; ++j) {
    const LoraGradJob& jb = jobs[j];
    if (jb.C != C) return cudaErrorInvalidValue;
    if (!make_map(&bt.mapZ[j], (const bf16*)jb.Z + jb.zcol0, (uint64_t)M, (uint64_t)C, (uint64_t)jb.ldz)) return cudaErrorInvalidValue;
    if (!make_map(&bt.mapW[j], jb.Wt, (uint64_t)M, (uint64_t)jb.ldwt, (uint64_t)jb.ldwt)) return cudaErrorInvalidValue;
    LgParams& p = bt.p[j];
    p.C = C; p.rows_per_chunk = rpg / s; p.R = jb.nt * jb.r; p.r = jb.r; p.rp = jb.rp; p.wsel0 = jb.wcol0 % LT_N;
    p.partial = partial + off; p.status = status;
    bt.wx0[j] = jb.wcol0 - p.wsel0;
    offsets[j] = off;
    off += (size_t)groups * s * p.R * C;
  }
  if (off > partial_floats) return cudaErrorInvalidValue;
  for (int j = njobs; j < LT_MAX_JOBS; ++j) { bt.mapZ[j] = bt.mapZ[0]; bt.mapW[j] = bt.mapW[0]; bt.p[j] = bt.p[0]; bt.wx0[j] = bt.wx0[0]; }
  dim3 grid(ctiles, groups * s, njobs);
  lora_grad_tc_kernel<<<grid, LT_THREADS, LT_SMEM, st>>>(bt);
  *chunks_per_group = s;
  return cudaGetLastError();
}

cudaError_t lora_grad_tc_partial(const void* Z, int64_t ldz, int zcol0, int C, const void* Wt, int64_t ldwt, int wcol0,
                                 int r, int rp, int nt, int M, int rows_per_group, float* partial, int* status,
                                 int* chunks_per_group, cudaStream_t st) {
  LoraGradJob jb;
  jb.Z = Z; jb.ldz = ldz; jb.zcol0 = zcol0; jb.C = C; jb.Wt = Wt; jb.ldwt = ldwt; jb.wcol0 = wcol0; jb.r = r; jb.rp = rp; jb.nt = nt;
  size_t off;
  return lora_grad_tc_partial_batch(&jb, 1, M, rows_per_group, partial, (size_t)-1, status, chunks_per_group, &off, st);
}

}  // namespace sl
