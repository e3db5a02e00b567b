// Causal multi-head attention with plain FMA arithmetic (fp32 or bf16 storage): the arithmetic of
// the fp32 configuration and a second opinion for the tensor-core kernels.
// One warp per (sequence, head, row).  Scores are computed one key per lane; the value / key / query
// accumulations are one feature per lane with the probability broadcast by shuffle.
#include "common.cuh"
#include "kernels.h"

namespace sl {
namespace {

constexpr int WARPS = 4;
constexpr int MAX_DH = 128;
constexpr int DPL = MAX_DH / 32;   // features per lane

template <typename T>
__device__ __forceinline__ float dot_row(const float* __restrict__ a_s, const T* __restrict__ row, int dh) {
  float s = 0.f;
  for (int c = 0; c < dh; ++c) s = fmaf(a_s[c], to_f<T>(row[c]), s);
  return s;
}

template <typename T>
__global__ void __launch_bounds__(WARPS * 32) attn_fwd_kernel(const T* __restrict__ qkv, int nseq, int Tn, int H,
                                                              int d, T* __restrict__ o, float* __restrict__ lse) {
  __shared__ float q_s[WARPS][MAX_DH];
  const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t w = (int64_t)blockIdx.x * WARPS + wib;
  if (w >= (int64_t)nseq * H * Tn) return;
  const int i = (int)(w % Tn), h = (int)((w / Tn) % H), b = (int)(w / ((int64_t)Tn * H));
  const int dh = d / H;
  const float scale = rsqrtf((float)dh);
  const size_t ld = (size_t)3 * d;
  const T* qrow = qkv + ((size_t)b * Tn + i) * ld + (size_t)h * dh;
  for (int c = lane; c < dh; c += 32) q_s[wib][c] = to_f<T>(qrow[c]);
  __syncwarp();
  float m = -INFINITY, l = 0.f, acc[DPL];
#pragma unroll
  for (int c = 0; c < DPL; ++c) acc[c] = 0.f;
  for (int j0 = 0; j0 <= i; j0 += 32) {
    int j = j0 + lane;
    float s = -INFINITY;
    if (j <= i) s = dot_row<T>(q_s[wib], qkv + ((size_t)b * Tn + j) * ld + d + (size_t)h * dh, dh) * scale;
    float nm = fmaxf(m, warp_max(s));
    float p = (j <= i) ? expf(s - nm) : 0.f;
    float corr = (m == -INFINITY) ? 0.f : expf(m - nm);
    l = l * corr + warp_sum(p);
#pragma unroll
    for (int c = 0; c < DPL; ++c) acc[c] *= corr;
    int cnt = min(32, i - j0 + 1);
    for (int jj = 0; jj < cnt; ++jj) {
      float pj = __shfl_sync(0xffffffffu, p, jj);
      const T* vrow = qkv + ((size_t)b * Tn + j0 + jj) * ld + 2 * (size_t)d + (size_t)h * dh;
#pragma unroll
      for (int c = 0; c < DPL; ++c) {
        int dim = lane + 32 * c;
        if (dim < dh) acc[c] = fmaf(pj, to_f<T>(vrow[dim]), acc[c]);
      }
    }
    m = nm;
  }
  T* orow = o + ((size_t)b * Tn + i) * d + (size_t)h * dh;
#pragma unroll
  for (int c = 0; c < DPL; ++c) {
    int dim = lane + 32 * c;
    if (dim < dh) orow[dim] = from_f<T>(acc[c] / l);
  }
  if (lane == 0) lse[((size_t)b * H + h) * Tn + i] = m + logf(l);
}

// rowdot[b, h, i] = sum_dim dO[i, dim] * O[i, dim]
template <typename T>
__global__ void attn_rowdot_kernel(const T* __restrict__ o, const T* __restrict__ d_o, int nseq, int Tn, int H,
                                   int d, float* __restrict__ rowdot) {
  const int lane = threadIdx.x & 31;
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (w >= (int64_t)nseq * H * Tn) return;
  const int i = (int)(w % Tn), h = (int)((w / Tn) % H), b = (int)(w / ((int64_t)Tn * H));
  const int dh = d / H;
  const size_t off = ((size_t)b * Tn + i) * d + (size_t)h * dh;
  float s = 0.f;
  for (int c = lane; c < dh; c += 32) s = fmaf(to_f<T>(o[off + c]), to_f<T>(d_o[off + c]), s);
  s = warp_sum(s);
  if (lane == 0) rowdot[((size_t)b * H + h) * Tn + i] = s;
}

// dQ: one warp per query row i; loops over keys j <= i.
template <typename T>
__global__ void __launch_bounds__(WARPS * 32) attn_bwd_dq_kernel(const T* __restrict__ qkv, const float* __restrict__ lse,
                                                                 const T* __restrict__ d_o, const float* __restrict__ rowdot,
                                                                 int nseq, int Tn, int H, int d, T* __restrict__ dqkv) {
  __shared__ float q_s[WARPS][MAX_DH], do_s[WARPS][MAX_DH];
  const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t w = (int64_t)blockIdx.x * WARPS + wib;
  if (w >= (int64_t)nseq * H * Tn) return;
  const int i = (int)(w % Tn), h = (int)((w / Tn) % H), b = (int)(w / ((int64_t)Tn * H));
  const int dh = d / H;
  const float scale = rsqrtf((float)dh);
  const size_t ld = (size_t)3 * d;
  const T* qrow = qkv + ((size_t)b * Tn + i) * ld + (size_t)h * dh;
  const T* dorow = d_o + ((size_t)b * Tn + i) * d + (size_t)h * dh;
  for (int c = lane; c < dh; c += 32) { q_s[wib][c] = to_f<T>(qrow[c]); do_s[wib][c] = to_f<T>(dorow[c]); }
  __syncwarp();
  const float L = lse[((size_t)b * H + h) * Tn + i], D = rowdot[((size_t)b * H + h) * Tn + i];
  float acc[DPL];
#pragma unroll
  for (int c = 0; c < DPL; ++c) acc[c] = 0.f;
  for (int j0 = 0; j0 <= i; j0 += 32) {
    int j = j0 + lane;
    float ds = 0.f;
    if (j <= i) {
      const T* krow = qkv + ((size_t)b * Tn + j) * ld + d + (size_t)h * dh;
      const T* vrow = krow + d;
      float s = dot_row<T>(q_s[wib], krow, dh) * scale;
      float p = expf(s - L);
      float dp = dot_row<T>(do_s[wib], vrow, dh);
      ds = p * (dp - D) * scale;
    }
    int cnt = min(32, i - j0 + 1);
    for (int jj = 0; jj < cnt; ++jj) {
      float dsj = __shfl_sync(0xffffffffu, ds, jj);
      const T* krow = qkv + ((size_t)b * Tn + j0 + jj) * ld + d + (size_t)h * dh;
#pragma unroll
      for (int c = 0; c < DPL; ++c) {
        int dim = lane + 32 * c;
        if (dim < dh) acc[c] = fmaf(dsj, to_f<T>(krow[dim]), acc[c]);
      }
    }
  }
  T* out = dqkv + ((size_t)b * Tn + i) * ld + (size_t)h * dh;
#pragma unroll
  for (int c = 0; c < DPL; ++c) {
    int dim = lane + 32 * c;
    if (dim < dh) out[dim] = from_f<T>(acc[c]);
  }
}

// dK, dV: one warp per key row j; loops over queries i >= j.
template <typename T>
__global__ void __launch_bounds__(WARPS * 32) attn_bwd_dkv_kernel(const T* __restrict__ qkv, const float* __restrict__ lse,
                                                                  const T* __restrict__ d_o, const float* __restrict__ rowdot,
                                                                  int nseq, int Tn, int H, int d, T* __restrict__ dqkv) {
  __shared__ float k_s[WARPS][MAX_DH], v_s[WARPS][MAX_DH];
  const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t w = (int64_t)blockIdx.x * WARPS + wib;
  if (w >= (int64_t)nseq * H * Tn) return;
  const int j = (int)(w % Tn), h = (int)((w / Tn) % H), b = (int)(w / ((int64_t)Tn * H));
  const int dh = d / H;
  const float scale = rsqrtf((float)dh);
  const size_t ld = (size_t)3 * d;
  const T* krow = qkv + ((size_t)b * Tn + j) * ld + d + (size_t)h * dh;
  for (int c = lane; c < dh; c += 32) { k_s[wib][c] = to_f<T>(krow[c]); v_s[wib][c] = to_f<T>(krow[d + c]); }
  __syncwarp();
  float dk[DPL], dv[DPL];
#pragma unroll
  for (int c = 0; c < DPL; ++c) { dk[c] = 0.f; dv[c] = 0.f; }
  for (int i0 = j; i0 < Tn; i0 += 32) {
    int i = i0 + lane;
    float p = 0.f, ds = 0.f;
    if (i < Tn) {
      const T* qrow = qkv + ((size_t)b * Tn + i) * ld + (size_t)h * dh;
      const T* dorow = d_o + ((size_t)b * Tn + i) * d + (size_t)h * dh;
      float s = dot_row<T>(k_s[wib], qrow, dh) * scale;
      p = expf(s - lse[((size_t)b * H + h) * Tn + i]);
      float dp = dot_row<T>(v_s[wib], dorow, dh);
      ds = p * (dp - rowdot[((size_t)b * H + h) * Tn + i]) * scale;
    }
    int cnt = min(32, Tn - i0);
    for (int ii = 0; ii < cnt; ++ii) {
      float pi = __shfl_sync(0xffffffffu, p, ii), dsi = __shfl_sync(0xffffffffu, ds, ii);
      const T* qrow = qkv + ((size_t)b * Tn + i0 + ii) * ld + (size_t)h * dh;
      const T* dorow = d_o + ((size_t)b * Tn + i0 + ii) * d + (size_t)h * dh;
#pragma unroll
      for (int c = 0; c < DPL; ++c) {
        int dim = lane + 32 * c;
        if (dim < dh) {
          dv[c] = fmaf(pi, to_f<T>(dorow[dim]), dv[c]);
          dk[c] = fmaf(dsi, to_f<T>(qrow[dim]), dk[c]);
        }
      }
    }
  }
  T* out = dqkv + ((size_t)b * Tn + j) * ld + (size_t)h * dh;
#pragma unroll
  for (int c = 0; c < DPL; ++c) {
    int dim = lane + 32 * c;
    if (dim < dh) { out[d + dim] = from_f<T>(dk[c]); out[2 * (size_t)d + dim] = from_f<T>(dv[c]); }
  }
}

}  // namespace

cudaError_t attention_fwd_simt(int dt, const void* qkv, int nseq, int T, int H, int d, void* o, float* lse,
                               cudaStream_t st) {
  if (d % H != 0 || d / H > MAX_DH) return cudaErrorInvalidValue;
  int64_t warps = (int64_t)nseq * H * T;
  unsigned blocks = (unsigned)((warps + WARPS - 1) / WARPS);
  if (dt == DT_BF16) attn_fwd_kernel<bf16><<<blocks, WARPS * 32, 0, st>>>((const bf16*)qkv, nseq, T, H, d, (bf16*)o, lse);
  else attn_fwd_kernel<float><<<blocks, WARPS * 32, 0, st>>>((const float*)qkv, nseq, T, H, d, (float*)o, lse);
  return cudaGetLastError();
}

cudaError_t attention_bwd_simt(int dt, const void* qkv, const void* o, const float* lse, const void* d_o,
                               int nseq, int T, int H, int d, void* dqkv, float* rowdot, cudaStream_t st) {
  if (d % H != 0 || d / H > MAX_DH) return cudaErrorInvalidValue;
  int64_t warps = (int64_t)nseq * H * T;
  unsigned blocks = (unsigned)((warps + WARPS - 1) / WARPS);
  unsigned rb = (unsigned)((warps * 32 + 255) / 256);
  if (dt == DT_BF16) {
    attn_rowdot_kernel<bf16><<<rb, 256, 0, st>>>((const bf16*)o, (const bf16*)d_o, nseq, T, H, d, rowdot);
    attn_bwd_dq_kernel<bf16><<<blocks, WARPS * 32, 0, st>>>((const bf16*)qkv, lse, (const bf16*)d_o, rowdot, nseq, T, H, d, (bf16*)dqkv);
    attn_bwd_dkv_kernel<bf16><<<blocks, WARPS * 32, 0, st>>>((const bf16*)qkv, lse, (const bf16*)d_o, rowdot, nseq, T, H, d, (bf16*)dqkv);
  } else {
    attn_rowdot_kernel<float><<<rb, 256, 0, st>>>((const float*)o, (const float*)d_o, nseq, T, H, d, rowdot);
    attn_bwd_dq_kernel<float><<<blocks, WARPS * 32, 0, st>>>((const float*)qkv, lse, (const float*)d_o, rowdot, nseq, T, H, d, (float*)dqkv);
    attn_bwd_dkv_kernel<float><<<blocks, WARPS * 32, 0, st>>>((const float*)qkv, lse, (const float*)d_o, rowdot, nseq, T, H, d, (float*)dqkv);
  }
  return cudaGetLastError();
}

}  // namespace sl
