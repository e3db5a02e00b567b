// Linear-layer kernel for sm_100a: bf16 operands staged in shared memory by TMA, products issued
// with tcgen05.mma from one thread, fp32 accumulators in tensor memory, epilogue read back with
// tcgen05.ld.  Persistent CTAs (one per SM) walk the output tiles; the accumulator is double
// buffered in tensor memory so that the epilogue of one tile overlaps the products of the next.
//
//   Y[M,N] = epilogue( X[M,K] W[N,K]^T  +  Xe[M,Ke] We[N,Ke]^T )
//
// The second term is the rank-r LoRA path: it enters as extra blocks of the contraction, read
// through a second pair of tensor maps whose rows are selected by the row group (client) of the
// tile, so K clients with their own adapters share one pass over the frozen W.
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = tensor-memory owner + MMA issuer,
// warps 2..9 = epilogue (a warp reads the 32 accumulator lanes its warp id modulo 4 selects; the
// two warps of a lane quarter take one half of the tile's columns each).
// Every wait on an mbarrier is bounded: when it expires the kernel records a code in `status`,
// stops issuing work, waits briefly for copies in flight, frees its tensor memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"

namespace sl {
namespace {

constexpr int BM = 128;
constexpr int BK = 64;            // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 320;
constexpr int GROUP_M = 16;       // output tiles are walked in bands of GROUP_M tile rows
constexpr unsigned long long WAIT_LIMIT_NS = 4000000000ull;

struct TcParams {
  int M, N, K;                    // K counts the main contraction only
  int num_kb;                     // K / 64
  int ext_blocks;                 // blocks of 64 in the extension
  int ext_last_mmas;              // MMAs (of 16) in the last extension block
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

// ---- PTX wrappers --------------------------------------------------------------------------
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
// Bounded wait.  Returns false when the limit expired or another role already gave up.
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
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
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

template <int BN> struct Cfg {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (196608 / STAGE_BYTES) > 8 ? 8 : (196608 / STAGE_BYTES);
  static constexpr int TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
  // kind::f16, fp32 accumulate, bf16 x bf16, both operands K-major, N = BN, M = 128
  static constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
};

template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW,
               const __grid_constant__ CUtensorMap mapXe, const __grid_constant__ CUtensorMap mapWe, TcParams p) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t bar_base = base + C::STAGES * C::STAGE_BYTES;
  // barrier slots: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + C::STAGES * C::STAGE_BYTES + 8 * (2 * C::STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + C::STAGES * C::STAGE_BYTES + 8 * (2 * C::STAGES + 4) + 8);

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
  const int band_tiles = GROUP_M * p.tiles_n;

  auto tile_coords = [&](int tile, int& tm, int& tn) {
    int band = tile / band_tiles, in = tile % band_tiles;
    int m_first = band * GROUP_M;
    int rows = min(GROUP_M, p.tiles_m - m_first);
    tm = m_first + in % rows;
    tn = in / rows;
  };

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int tm, tn; tile_coords(tile, tm, tn);
        const int m0 = tm * BM, n0 = tn * BN;
        const int g = p.rows_per_group > 0 ? m0 / p.rows_per_group : 0;
        const int w_row = g * p.w_group_rows + n0;
        const int we_row = g * p.we_group_rows + n0;
        for (int kb = 0; kb < kb_total; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 1)) { ok = false; break; }
          mbar_expect_tx(full_bar(stage), C::STAGE_BYTES);
          const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
          if (kb < p.num_kb) {
            tma_load_2d(sa, &mapX, full_bar(stage), kb * BK, m0);
            tma_load_2d(sb, &mapW, full_bar(stage), kb * BK, w_row);
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
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        if (!mbar_wait(tempty_bar(as), aphase ^ 1u, abort_flag, p.status, 2)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * BN);
        for (int kb = 0; kb < kb_total; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 3)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
          const uint64_t adesc = make_smem_desc(sa), bdesc = make_smem_desc(sb);
          int nmma = BK / UMMA_K;
          if (kb >= p.num_kb && kb == kb_total - 1) nmma = p.ext_last_mmas;
#pragma unroll 1
          for (int k = 0; k < nmma; ++k) {
            // advancing 16 elements along K inside the swizzled row = +32 bytes = +2 in descriptor units
            tc_mma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), C::IDESC, (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));          // frees the stage once these products have read it
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
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      int tm, tn; tile_coords(tile, tm, tn);
      const int m = tm * BM + q * 32 + lane;
      const int n0 = tn * BN;
      if (!mbar_wait(tfull_bar(as), aphase, abort_flag, p.status, 4)) { ok = false; break; }
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BN);
#pragma unroll 1
      for (int c = c_begin; c < c_end; c += 32) {
        const int n = n0 + c;
        if (n >= p.N) break;                    // warp-uniform
        float v[32];
        tc_ld32(t_row + (uint32_t)c, v);
        tc_wait_ld();
        if (p.bias && p.epi != EPI_MUL_GELUGRAD) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (n + 8 * j < p.N) {
              uint4 bw = __ldg(reinterpret_cast<const uint4*>(p.bias + n + 8 * j));
              const bf16* bp = reinterpret_cast<const bf16*>(&bw);
#pragma unroll
              for (int i = 0; i < 8; ++i) v[8 * j + i] += __bfloat162float(bp[i]);
            }
          }
        }
        if (p.epi == EPI_BIAS_GELU) {
          bf16* zrow = p.Z + (size_t)m * p.ldz + n;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (n + 8 * j < p.N) {
              uint4 zw; bf16* zp = reinterpret_cast<bf16*>(&zw);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                zp[i] = __float2bfloat16_rn(v[8 * j + i]);
                v[8 * j + i] = gelu_tc(__bfloat162float(zp[i]), tanh_form);
              }
              *reinterpret_cast<uint4*>(zrow + 8 * j) = zw;
            }
          }
        } else if (p.epi == EPI_BIAS_RESID || p.epi == EPI_MUL_GELUGRAD) {
          const bf16* rrow = p.R + (size_t)m * p.ldr + n;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (n + 8 * j < p.N) {
              uint4 rw = *reinterpret_cast<const uint4*>(rrow + 8 * j);
              const bf16* rp = reinterpret_cast<const bf16*>(&rw);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                float rv = __bfloat162float(rp[i]);
                if (p.epi == EPI_BIAS_RESID) v[8 * j + i] += rv;
                else v[8 * j + i] *= gelu_grad_tc(rv, tanh_form);
              }
            }
          }
        }
        bf16* yrow = p.Y + (size_t)m * p.ldy + n;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (n + 8 * j < p.N) {
            uint4 yw; __nv_bfloat162* yp = reinterpret_cast<__nv_bfloat162*>(&yw);
#pragma unroll
            for (int i = 0; i < 4; ++i) yp[i] = __floats2bfloat162_rn(v[8 * j + 2 * i], v[8 * j + 2 * i + 1]);
            *reinterpret_cast<uint4*>(yrow + 8 * j) = yw;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(as));
      if (++as == 2) { as = 0; aphase ^= 1u; }
    }
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

// ---- host side -----------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
int g_num_sms = 0;

// 2-D bf16 tensor [rows, cols] with leading dimension ld (elements); box = 64 columns x box_rows rows.
bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

int pick_bn(const GemmArgs& a) {
  if (a.N % 256 == 0) return 256;
  if (a.N % 128 == 0) return 128;
  if (a.N <= 64) return 64;
  if (a.N <= 128) return 128;
  return 256;
}

template <int BN>
cudaError_t launch(const GemmArgs& a, int* status, cudaStream_t st) {
  using C = Cfg<BN>;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int G = a.rows_per_group > 0 ? a.M / a.rows_per_group : 1;
  const int w_rows = a.w_rows > 0 ? a.w_rows : a.N;
  CUtensorMap mX, mW, mXe, mWe;
  if (!make_map(&mX, a.X, a.M, a.K, a.ldx, BM)) return cudaErrorInvalidValue;
  if (!make_map(&mW, a.W, a.w_grouped ? (uint64_t)G * a.N : (uint64_t)w_rows, a.K, a.ldw, BN)) return cudaErrorInvalidValue;
  TcParams p;
  p.M = a.M; p.N = a.N; p.K = a.K; p.num_kb = a.K / BK;
  if (a.Ke > 0) {
    const uint64_t ke_cols = (uint64_t)((a.Ke + BK - 1) / BK) * BK;
    if (!make_map(&mXe, a.Xe, a.M, ke_cols, a.ldxe, BM)) return cudaErrorInvalidValue;
    if (!make_map(&mWe, a.We, a.we_grouped ? (uint64_t)G * a.N : (uint64_t)a.N, ke_cols, a.ldwe, BN)) return cudaErrorInvalidValue;
    p.ext_blocks = (a.Ke + BK - 1) / BK;
    p.ext_last_mmas = (a.Ke - (p.ext_blocks - 1) * BK) / UMMA_K;
  } else {
    mXe = mX; mWe = mW;
    p.ext_blocks = 0; p.ext_last_mmas = 0;
  }
  p.rows_per_group = a.rows_per_group;
  p.w_group_rows = a.w_grouped ? a.N : 0;
  p.we_group_rows = a.we_grouped ? a.N : 0;
  p.tiles_m = a.M / BM; p.tiles_n = (a.N + BN - 1) / BN;
  p.epi = a.epi; p.gelu_tanh = a.gelu_tanh;
  p.bias = (const bf16*)a.bias; p.R = (const bf16*)a.R; p.ldr = a.ldr;
  p.Y = (bf16*)a.Y; p.ldy = a.ldy; p.Z = (bf16*)a.Z; p.ldz = a.ldz;
  p.status = status;
  const int tiles = p.tiles_m * p.tiles_n;
  const int grid = tiles < g_num_sms ? tiles : g_num_sms;
  gemm_tc_kernel<BN><<<grid, NUM_THREADS, C::SMEM_BYTES, st>>>(mX, mW, mXe, mWe, p);
  return cudaGetLastError();
}

}  // namespace

int gemm_tc_init() {
  if (g_encode) return 0;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn ||
      q != cudaDriverEntryPointSuccess)
    return -1;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return -1;
  if (cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || g_num_sms < 1) return -1;
  g_encode = (EncodeTiledFn)fn;
  return 0;
}

bool gemm_tc_supported(const GemmArgs& a) {
  auto al16 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
  if (!g_encode || a.dtype != DT_BF16) return false;
  if (a.M < BM || a.M % BM != 0 || a.K < BK || a.K % BK != 0 || a.N < 8 || a.N % 8 != 0) return false;
  if (a.rows_per_group > 0 && (a.rows_per_group % BM != 0 || a.M % a.rows_per_group != 0)) return false;
  if (a.ldx % 8 || a.ldw % 8 || a.ldy % 8) return false;
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
  switch (pick_bn(a)) {
    case 256: return launch<256>(a, status, st);
    case 128: return launch<128>(a, status, st);
    default: return launch<64>(a, status, st);
  }
}

}  // namespace sl
