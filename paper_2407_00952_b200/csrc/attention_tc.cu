// Causal multi-head attention on tensor cores (bf16 operands, fp32 softmax and accumulation),
// head width 64 or 128, sequence length a multiple of 64.  Flash-style: scores are never written to
// memory; the forward keeps only the log-sum-exp per row, the backward recomputes probabilities.
//   forward : one CTA per (sequence, head, 64-row query tile), 4 warps x 16 rows, K/V tiles double
//             buffered in shared memory with cp.async, online softmax in registers.
//   backward: rowdot = sum(dO*O); a dQ kernel per query tile (loops over key tiles) and a dK/dV
//             kernel per key tile (loops over query tiles).  No atomics: results are bit-reproducible.
// Products use mma.sync m16n8k16 with ldmatrix-fed fragments from XOR-swizzled shared tiles.

#include "common.cuh"
#include "host_common.h"
#include "kernels.h"

namespace sl {
namespace {

constexpr int BT = 64;            // rows of a query tile and of a key tile
constexpr int NT = 128;           // threads per CTA
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

template <int DH> struct Sizes {
  static constexpr int TILE = BT * DH * 2;     // bytes of one [64][DH] bf16 tile
  static constexpr int FWD = 5 * TILE, DQ = 6 * TILE, DKV = 6 * TILE + 4 * BT * 4;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// byte offset of element (r, c) in a [64][DH] bf16 tile; the 16-byte chunks of every 128-byte
// segment of a row are XOR-swizzled by the row index
template <int DH> __device__ __forceinline__ uint32_t swz(int r, int c) {
  int ch = c >> 3;
  return (uint32_t)(r * (DH * 2) + ((((ch & ~7) | ((ch & 7) ^ (r & 7))) << 4) | ((c & 7) << 1)));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// 64 x DH bf16 tile, global rows `ld` elements apart -> swizzled shared tile
template <int DH> __device__ __forceinline__ void load_tile(uint32_t sbase, const bf16* g, int64_t ld) {
  constexpr int CH = DH / 8;
#pragma unroll
  for (int i = threadIdx.x; i < BT * CH; i += NT) {
    int r = i / CH, ch = i % CH;
    cp_async16(sbase + swz<DH>(r, ch * 8), g + (size_t)r * ld + ch * 8);
  }
}

__device__ __forceinline__ void ldsm4(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// A fragment (16 x 16) of a row-major [rows][DH] tile at (row0, k0)
template <int DH> __device__ __forceinline__ void load_a(uint32_t* a, uint32_t sbase, int row0, int k0) {
  int l = threadIdx.x & 31;
  ldsm4(a, sbase + swz<DH>(row0 + (l & 7) + ((l >> 3) & 1) * 8, k0 + (l >> 4) * 8));
}
// B fragments for two n-tiles (n0, n0+8) x k16 from a tile stored [n][k]: b[0],b[1] -> n0 ; b[2],b[3] -> n0+8
template <int DH> __device__ __forceinline__ void load_b_nk(uint32_t* b, uint32_t sbase, int n0, int k0) {
  int l = threadIdx.x & 31;
  ldsm4(b, sbase + swz<DH>(n0 + (l & 7) + (l >> 4) * 8, k0 + ((l >> 3) & 1) * 8));
}
// B fragments for two n-tiles (n0, n0+8) x k16 from a tile stored [k][n]
template <int DH> __device__ __forceinline__ void load_b_kn(uint32_t* b, uint32_t sbase, int k0, int n0) {
  int l = threadIdx.x & 31;
  ldsm4t(b, sbase + swz<DH>(k0 + (l & 7) + ((l >> 3) & 1) * 8, n0 + (l >> 4) * 8));
}

// acc[8][4] (16 x 64) += A(16 x DH from `a_tile` rows row0..) * B^T where the B tile is stored [64][DH]
template <int DH>
__device__ __forceinline__ void mma_a_smem_b_nk(float (*acc)[4], uint32_t a_tile, int row0, uint32_t b_tile) {
#pragma unroll
  for (int ks = 0; ks < DH / 16; ++ks) {
    uint32_t a[4];
    load_a<DH>(a, a_tile, row0, ks * 16);
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      uint32_t b[4];
      load_b_nk<DH>(b, b_tile, np * 16, ks * 16);
      mma16816(acc[2 * np], a, b[0], b[1]);
      mma16816(acc[2 * np + 1], a, b[2], b[3]);
    }
  }
}
// acc[DH/8][4] (16 x DH) += P(16 x 64, fp32 accumulator layout, converted to bf16) * B, B tile stored [64][DH]
template <int DH>
__device__ __forceinline__ void mma_p_regs_b_kn(float (*acc)[4], const float (*p)[4], uint32_t b_tile) {
#pragma unroll
  for (int ks = 0; ks < 4; ++ks) {
    uint32_t a[4];
    a[0] = pack2(p[2 * ks][0], p[2 * ks][1]);
    a[1] = pack2(p[2 * ks][2], p[2 * ks][3]);
    a[2] = pack2(p[2 * ks + 1][0], p[2 * ks + 1][1]);
    a[3] = pack2(p[2 * ks + 1][2], p[2 * ks + 1][3]);
#pragma unroll
    for (int np = 0; np < DH / 16; ++np) {
      uint32_t b[4];
      load_b_kn<DH>(b, b_tile, ks * 16, np * 16);
      mma16816(acc[2 * np], a, b[0], b[1]);
      mma16816(acc[2 * np + 1], a, b[2], b[3]);
    }
  }
}

template <int N> __device__ __forceinline__ void zero_acc(float (*a)[4]) {
#pragma unroll
  for (int i = 0; i < N; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) a[i][j] = 0.f;
}

// ------------------------------------------------------------------------------------------
// forward
// ------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(NT) attn_fwd_tc_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ o,
                                                         float* __restrict__ lse, int T, int H, int d, float scale_log2) {
  constexpr int TILE_BYTES = Sizes<DH>::TILE;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sQ = smem_u32(smem), sK0 = sQ + TILE_BYTES, sV0 = sQ + 3 * TILE_BYTES;
  const int qt = gridDim.x - 1 - blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int64_t ld = 3 * (int64_t)d;
  const bf16* qbase = qkv + ((size_t)b * T + (size_t)qt * BT) * ld + (size_t)h * DH;
  const bf16* kbase = qkv + (size_t)b * T * ld + d + (size_t)h * DH;
  const bf16* vbase = kbase + d;
  load_tile<DH>(sQ, qbase, ld);
  load_tile<DH>(sK0, kbase, ld);
  load_tile<DH>(sV0, vbase, ld);
  cp_commit();
  float oacc[DH / 8][4];
  zero_acc<DH / 8>(oacc);
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  const int r0 = warp * 16 + g, r1 = r0 + 8;
  for (int j = 0; j <= qt; ++j) {
    const uint32_t sK = sK0 + (j & 1) * TILE_BYTES, sV = sV0 + (j & 1) * TILE_BYTES;
    if (j < qt) {
      load_tile<DH>(sK0 + ((j + 1) & 1) * TILE_BYTES, kbase + (size_t)(j + 1) * BT * ld, ld);
      load_tile<DH>(sV0 + ((j + 1) & 1) * TILE_BYTES, vbase + (size_t)(j + 1) * BT * ld, ld);
      cp_commit();
      cp_wait<1>();
    } else {
      cp_wait<0>();
    }
    __syncthreads();
    float s[8][4];
    zero_acc<8>(s);
    mma_a_smem_b_nk<DH>(s, sQ, warp * 16, sK);
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int n = 0; n < 8; ++n) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int col = n * 8 + 2 * t + (e & 1);
        int row = (e < 2) ? r0 : r1;
        float v = s[n][e] * scale_log2;
        if (j == qt && col > row) v = -INFINITY;
        s[n][e] = v;
        if (e < 2) mx0 = fmaxf(mx0, v); else mx1 = fmaxf(mx1, v);
      }
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float nm0 = fmaxf(m0, mx0), nm1 = fmaxf(m1, mx1);   // finite: column 0 is never masked
    const float c0 = exp2f(m0 - nm0), c1 = exp2f(m1 - nm1);
    float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      s[n][0] = exp2f(s[n][0] - nm0); s[n][1] = exp2f(s[n][1] - nm0);
      s[n][2] = exp2f(s[n][2] - nm1); s[n][3] = exp2f(s[n][3] - nm1);
      ps0 += s[n][0] + s[n][1]; ps1 += s[n][2] + s[n][3];
    }
#pragma unroll
    for (int n = 0; n < DH / 8; ++n) { oacc[n][0] *= c0; oacc[n][1] *= c0; oacc[n][2] *= c1; oacc[n][3] *= c1; }
    l0 = l0 * c0 + ps0; l1 = l1 * c1 + ps1;
    m0 = nm0; m1 = nm1;
    mma_p_regs_b_kn<DH>(oacc, s, sV);
    __syncthreads();
  }
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float i0 = 1.f / l0, i1 = 1.f / l1;
  bf16* o0 = o + ((size_t)b * T + (size_t)qt * BT + r0) * d + (size_t)h * DH;
  bf16* o1 = o + ((size_t)b * T + (size_t)qt * BT + r1) * d + (size_t)h * DH;
#pragma unroll
  for (int n = 0; n < DH / 8; ++n) {
    *reinterpret_cast<uint32_t*>(o0 + n * 8 + 2 * t) = pack2(oacc[n][0] * i0, oacc[n][1] * i0);
    *reinterpret_cast<uint32_t*>(o1 + n * 8 + 2 * t) = pack2(oacc[n][2] * i1, oacc[n][3] * i1);
  }
  if (t == 0) {
    float* lrow = lse + ((size_t)b * H + h) * T + (size_t)qt * BT;
    lrow[r0] = (m0 + log2f(l0)) * LN2;
    lrow[r1] = (m1 + log2f(l1)) * LN2;
  }
}

// rowdot[b, h, i] = sum_c dO[i, c] O[i, c] over the head's DH columns; DH/8 lanes per row
template <int DH>
__global__ void attn_rowdot_tc_kernel(const bf16* __restrict__ o, const bf16* __restrict__ d_o, int nseq, int T, int H,
                                      int d, float* __restrict__ rowdot) {
  constexpr int LPR = DH / 8;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t rowhead = idx / LPR;
  int part = (int)(idx % LPR);
  if (rowhead >= (int64_t)nseq * T * H) return;
  int h = (int)(rowhead % H);
  int64_t row = rowhead / H;
  size_t off = (size_t)row * d + (size_t)h * DH + part * 8;
  uint4 a = *reinterpret_cast<const uint4*>(o + off), bb = *reinterpret_cast<const uint4*>(d_o + off);
  const bf16* ap = reinterpret_cast<const bf16*>(&a);
  const bf16* bp = reinterpret_cast<const bf16*>(&bb);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) s = fmaf(__bfloat162float(ap[i]), __bfloat162float(bp[i]), s);
#pragma unroll
  for (int m = 1; m < LPR; m <<= 1) s += __shfl_xor_sync(0xffffffffu, s, m);
  if (part == 0) {
    int bq = (int)(row / T), i = (int)(row % T);
    rowdot[((size_t)bq * H + h) * T + i] = s;
  }
}

// ------------------------------------------------------------------------------------------
// backward, dQ: one CTA per query tile, loops over key tiles j <= qt
// ------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(NT) attn_bwd_dq_tc_kernel(const bf16* __restrict__ qkv, const bf16* __restrict__ d_o,
                                                            const float* __restrict__ lse, const float* __restrict__ rowdot,
                                                            bf16* __restrict__ dqkv, int T, int H, int d, float scale) {
  constexpr int TILE_BYTES = Sizes<DH>::TILE;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sQ = smem_u32(smem), sdO = sQ + TILE_BYTES, sK0 = sQ + 2 * TILE_BYTES, sV0 = sQ + 4 * TILE_BYTES;
  const int qt = gridDim.x - 1 - blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int64_t ld = 3 * (int64_t)d;
  const bf16* qbase = qkv + ((size_t)b * T + (size_t)qt * BT) * ld + (size_t)h * DH;
  const bf16* kbase = qkv + (size_t)b * T * ld + d + (size_t)h * DH;
  const bf16* vbase = kbase + d;
  const bf16* dobase = d_o + ((size_t)b * T + (size_t)qt * BT) * d + (size_t)h * DH;
  load_tile<DH>(sQ, qbase, ld);
  load_tile<DH>(sdO, dobase, d);
  load_tile<DH>(sK0, kbase, ld);
  load_tile<DH>(sV0, vbase, ld);
  cp_commit();
  const int r0 = warp * 16 + g, r1 = r0 + 8;
  const size_t stat = ((size_t)b * H + h) * T + (size_t)qt * BT;
  const float L0 = lse[stat + r0] * LOG2E, L1 = lse[stat + r1] * LOG2E;
  const float D0 = rowdot[stat + r0], D1 = rowdot[stat + r1];
  const float scale_log2 = scale * LOG2E;
  float dq[DH / 8][4];
  zero_acc<DH / 8>(dq);
  for (int j = 0; j <= qt; ++j) {
    const uint32_t sK = sK0 + (j & 1) * TILE_BYTES, sV = sV0 + (j & 1) * TILE_BYTES;
    if (j < qt) {
      load_tile<DH>(sK0 + ((j + 1) & 1) * TILE_BYTES, kbase + (size_t)(j + 1) * BT * ld, ld);
      load_tile<DH>(sV0 + ((j + 1) & 1) * TILE_BYTES, vbase + (size_t)(j + 1) * BT * ld, ld);
      cp_commit();
      cp_wait<1>();
    } else {
      cp_wait<0>();
    }
    __syncthreads();
    float s[8][4], dp[8][4];
    zero_acc<8>(s);
    mma_a_smem_b_nk<DH>(s, sQ, warp * 16, sK);       // S = Q K^T
    zero_acc<8>(dp);
    mma_a_smem_b_nk<DH>(dp, sdO, warp * 16, sV);     // dP = dO V^T
#pragma unroll
    for (int n = 0; n < 8; ++n) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int col = n * 8 + 2 * t + (e & 1);
        int row = (e < 2) ? r0 : r1;
        float p = exp2f(s[n][e] * scale_log2 - ((e < 2) ? L0 : L1));
        if (j == qt && col > row) p = 0.f;
        s[n][e] = p * (dp[n][e] - ((e < 2) ? D0 : D1));    // dS (without the 1/sqrt(dh) factor)
      }
    }
    mma_p_regs_b_kn<DH>(dq, s, sK);                  // dQ += dS K
    __syncthreads();
  }
  bf16* q0 = dqkv + ((size_t)b * T + (size_t)qt * BT + r0) * ld + (size_t)h * DH;
  bf16* q1 = dqkv + ((size_t)b * T + (size_t)qt * BT + r1) * ld + (size_t)h * DH;
#pragma unroll
  for (int n = 0; n < DH / 8; ++n) {
    *reinterpret_cast<uint32_t*>(q0 + n * 8 + 2 * t) = pack2(dq[n][0] * scale, dq[n][1] * scale);
    *reinterpret_cast<uint32_t*>(q1 + n * 8 + 2 * t) = pack2(dq[n][2] * scale, dq[n][3] * scale);
  }
}

// ------------------------------------------------------------------------------------------
// backward, dK and dV: one CTA per key tile, loops over query tiles i >= kt.
// Works on the transposed score tile S^T = K Q^T so that P^T and dS^T land in the register layout
// the next product needs as its left operand.
// ------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(NT) attn_bwd_dkv_tc_kernel(const bf16* __restrict__ qkv, const bf16* __restrict__ d_o,
                                                             const float* __restrict__ lse, const float* __restrict__ rowdot,
                                                             bf16* __restrict__ dqkv, int T, int H, int d, float scale) {
  constexpr int TILE_BYTES = Sizes<DH>::TILE;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sK = smem_u32(smem), sV = sK + TILE_BYTES, sQ0 = sK + 2 * TILE_BYTES, sdO0 = sK + 4 * TILE_BYTES;
  float* sL = reinterpret_cast<float*>(smem + 6 * TILE_BYTES);     // [2][64] lse * log2e
  float* sD = sL + 2 * BT;                                         // [2][64] rowdot
  const int kt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int nT = T / BT;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int64_t ld = 3 * (int64_t)d;
  const bf16* qhead = qkv + (size_t)b * T * ld + (size_t)h * DH;
  const bf16* kbase = qhead + (size_t)kt * BT * ld + d;
  const bf16* dohead = d_o + (size_t)b * T * d + (size_t)h * DH;
  const size_t stat = ((size_t)b * H + h) * T;
  load_tile<DH>(sK, kbase, ld);
  load_tile<DH>(sV, kbase + d, ld);
  load_tile<DH>(sQ0 + (kt & 1) * TILE_BYTES, qhead + (size_t)kt * BT * ld, ld);
  load_tile<DH>(sdO0 + (kt & 1) * TILE_BYTES, dohead + (size_t)kt * BT * d, d);
  cp_commit();
  if (threadIdx.x < BT) {
    sL[(kt & 1) * BT + threadIdx.x] = lse[stat + (size_t)kt * BT + threadIdx.x] * LOG2E;
    sD[(kt & 1) * BT + threadIdx.x] = rowdot[stat + (size_t)kt * BT + threadIdx.x];
  }
  const float scale_log2 = scale * LOG2E;
  const int r0 = warp * 16 + g, r1 = r0 + 8;       // key rows of this thread inside the tile
  float dk[DH / 8][4], dv[DH / 8][4];
  zero_acc<DH / 8>(dk); zero_acc<DH / 8>(dv);
  for (int i = kt; i < nT; ++i) {
    const uint32_t sQ = sQ0 + (i & 1) * TILE_BYTES, sdO = sdO0 + (i & 1) * TILE_BYTES;
    const float* Lq = sL + (i & 1) * BT;
    const float* Dq = sD + (i & 1) * BT;
    if (i + 1 < nT) {
      load_tile<DH>(sQ0 + ((i + 1) & 1) * TILE_BYTES, qhead + (size_t)(i + 1) * BT * ld, ld);
      load_tile<DH>(sdO0 + ((i + 1) & 1) * TILE_BYTES, dohead + (size_t)(i + 1) * BT * d, d);
      cp_commit();
      if (threadIdx.x < BT) {
        sL[((i + 1) & 1) * BT + threadIdx.x] = lse[stat + (size_t)(i + 1) * BT + threadIdx.x] * LOG2E;
        sD[((i + 1) & 1) * BT + threadIdx.x] = rowdot[stat + (size_t)(i + 1) * BT + threadIdx.x];
      }
      cp_wait<1>();
    } else {
      cp_wait<0>();
    }
    __syncthreads();
    float st[8][4], dpt[8][4];
    zero_acc<8>(st);
    mma_a_smem_b_nk<DH>(st, sK, warp * 16, sQ);       // S^T = K Q^T   (rows: keys, columns: queries)
    zero_acc<8>(dpt);
    mma_a_smem_b_nk<DH>(dpt, sV, warp * 16, sdO);     // dP^T = V dO^T
#pragma unroll
    for (int n = 0; n < 8; ++n) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int qcol = n * 8 + 2 * t + (e & 1);
        int krow = (e < 2) ? r0 : r1;
        float p = exp2f(st[n][e] * scale_log2 - Lq[qcol]);
        if (i == kt && qcol < krow) p = 0.f;        // causal: query must not precede key
        st[n][e] = p;
        dpt[n][e] = p * (dpt[n][e] - Dq[qcol]);     // dS^T (without the 1/sqrt(dh) factor)
      }
    }
    mma_p_regs_b_kn<DH>(dv, st, sdO);                 // dV += P^T dO
    mma_p_regs_b_kn<DH>(dk, dpt, sQ);                 // dK += dS^T Q
    __syncthreads();
  }
  bf16* k0 = dqkv + ((size_t)b * T + (size_t)kt * BT + r0) * ld + d + (size_t)h * DH;
  bf16* k1 = dqkv + ((size_t)b * T + (size_t)kt * BT + r1) * ld + d + (size_t)h * DH;
#pragma unroll
  for (int n = 0; n < DH / 8; ++n) {
    *reinterpret_cast<uint32_t*>(k0 + n * 8 + 2 * t) = pack2(dk[n][0] * scale, dk[n][1] * scale);
    *reinterpret_cast<uint32_t*>(k1 + n * 8 + 2 * t) = pack2(dk[n][2] * scale, dk[n][3] * scale);
    *reinterpret_cast<uint32_t*>(k0 + d + n * 8 + 2 * t) = pack2(dv[n][0], dv[n][1]);
    *reinterpret_cast<uint32_t*>(k1 + d + n * 8 + 2 * t) = pack2(dv[n][2], dv[n][3]);
  }
}

template <int DH>
cudaError_t launch_fwd(const void* qkv, int nseq, int T, int H, int d, void* o, float* lse, cudaStream_t st) {
  static PerDeviceOnce once;                    // one per instantiation; attributes are per device
  const int dev = current_device();
  if (once.needed(dev)) {
    cudaError_t e = cudaFuncSetAttribute(attn_fwd_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, Sizes<DH>::FWD);
    if (e != cudaSuccess) return e;
    once.done(dev);
  }
  dim3 grid(T / BT, H, nseq);
  attn_fwd_tc_kernel<DH><<<grid, NT, Sizes<DH>::FWD, st>>>((const bf16*)qkv, (bf16*)o, lse, T, H, d,
                                                          LOG2E / sqrtf((float)DH));
  return cudaGetLastError();
}

template <int DH>
cudaError_t launch_bwd(const void* qkv, const void* o, const float* lse, const void* d_o, int nseq, int T, int H, int d,
                       void* dqkv, float* rowdot, int* status, cudaStream_t st) {
  static PerDeviceOnce once;
  const int dev = current_device();
  if (once.needed(dev)) {
    cudaError_t e = cudaFuncSetAttribute(attn_bwd_dq_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, Sizes<DH>::DQ);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_bwd_dkv_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, Sizes<DH>::DKV);
    if (e != cudaSuccess) return e;
    once.done(dev);
  }
  int64_t threads = (int64_t)nseq * T * H * (DH / 8);
  attn_rowdot_tc_kernel<DH><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>((const bf16*)o, (const bf16*)d_o, nseq, T, H, d, rowdot);
  dim3 grid(T / BT, H, nseq);
  const float scale = 1.0f / sqrtf((float)DH);
  if (DH == 128 && attention_bwd_t5_128_supported(DT_BF16, T, H, d))
    // dQ, dK, dV on the tcgen05 kernels (they read D[row] from `rowdot`, written just above)
    return attention_bwd_t5_128(qkv, lse, d_o, rowdot, nseq, T, H, d, dqkv, status, st);
  attn_bwd_dq_tc_kernel<DH><<<grid, NT, Sizes<DH>::DQ, st>>>((const bf16*)qkv, (const bf16*)d_o, lse, rowdot, (bf16*)dqkv, T, H, d, scale);
  attn_bwd_dkv_tc_kernel<DH><<<grid, NT, Sizes<DH>::DKV, st>>>((const bf16*)qkv, (const bf16*)d_o, lse, rowdot, (bf16*)dqkv, T, H, d, scale);
  return cudaGetLastError();
}

}  // namespace

bool attention_tc_supported(int dt, int T, int H, int d) {
  return dt == DT_BF16 && H > 0 && d % H == 0 && (d / H == 64 || d / H == 128) && T >= BT && T % BT == 0;
}

// status: device word that receives a code when a bounded wait inside the tcgen05 kernels expires
// (nullptr: the library's own word, see library_status_word).
cudaError_t attention_fwd_tc(const void* qkv, int nseq, int T, int H, int d, void* o, float* lse, int* status,
                             cudaStream_t st) {
  if (!attention_tc_supported(DT_BF16, T, H, d)) return cudaErrorInvalidValue;
  if (attention_fwd_t5_supported(DT_BF16, T, H, d)) return attention_fwd_t5(qkv, nseq, T, H, d, o, lse, status, st);
  return d / H == 64 ? launch_fwd<64>(qkv, nseq, T, H, d, o, lse, st) : launch_fwd<128>(qkv, nseq, T, H, d, o, lse, st);
}

cudaError_t attention_bwd_tc(const void* qkv, const void* o, const float* lse, const void* d_o, int nseq, int T, int H,
                             int d, void* dqkv, float* rowdot, int* status, cudaStream_t st) {
  if (!attention_tc_supported(DT_BF16, T, H, d)) return cudaErrorInvalidValue;
  if (attention_t5_supported(DT_BF16, T, H, d))
    return attention_bwd_t5(qkv, o, lse, d_o, nseq, T, H, d, dqkv, rowdot, status, st);
  return d / H == 64 ? launch_bwd<64>(qkv, o, lse, d_o, nseq, T, H, d, dqkv, rowdot, status, st)
                     : launch_bwd<128>(qkv, o, lse, d_o, nseq, T, H, d, dqkv, rowdot, status, st);
}

}  // namespace sl
