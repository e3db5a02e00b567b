// Plain-FMA linear-layer kernel: any shape, fp32 or bf16 storage, fp32 accumulation.
// It is the arithmetic of the fp32 configuration and a second opinion for the tensor-core kernel.
#include "common.cuh"
#include "kernels.h"

namespace sl {

namespace {
constexpr int BM = 64, BN = 64, BK = 16;

template <typename T>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs a) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const int lrow = threadIdx.x / 4, lk = (threadIdx.x % 4) * 4;
  const int g = a.rows_per_group > 0 ? m0 / a.rows_per_group : 0;
  const int w_rows = a.w_rows > 0 ? a.w_rows : a.N;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int phase = 0; phase < 2; ++phase) {
    const T* X; const T* W; int64_t ldx, ldw; int Kp; int wr;
    if (phase == 0) {
      X = (const T*)a.X; ldx = a.ldx; ldw = a.ldw; Kp = a.K; wr = w_rows;
      W = (const T*)a.W + (a.w_grouped ? (size_t)g * a.N * a.ldw : 0);
    } else {
      if (a.Ke == 0) break;
      X = (const T*)a.Xe; ldx = a.ldxe; ldw = a.ldwe; Kp = a.Ke; wr = a.N;
      W = (const T*)a.We + (a.we_grouped ? (size_t)g * a.N * a.ldwe : 0);
    }
    for (int k0 = 0; k0 < Kp; k0 += BK) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        int k = k0 + lk + i;
        int m = m0 + lrow, n = n0 + lrow;
        As[lk + i][lrow] = (m < a.M && k < Kp) ? to_f<T>(X[(size_t)m * ldx + k]) : 0.f;
        Bs[lk + i][lrow] = (n < wr && k < Kp) ? to_f<T>(W[(size_t)n * ldw + k]) : 0.f;
      }
      __syncthreads();
#pragma unroll
      for (int k = 0; k < BK; ++k) {
        float av[4], bv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) av[i] = As[k][ty * 4 + i];
#pragma unroll
        for (int j = 0; j < 4; ++j) bv[j] = Bs[k][tx * 4 + j];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
      }
      __syncthreads();
    }
  }

  const T* bias = (const T*)a.bias;
  const T* R = (const T*)a.R;
  T* Y = (T*)a.Y;
  T* Z = (T*)a.Z;
  const bool tanh_form = a.gelu_tanh != 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int m = m0 + ty * 4 + i;
    if (m >= a.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int n = n0 + tx * 4 + j;
      if (n >= a.N) continue;
      float v = acc[i][j];
      if (bias && a.epi != EPI_MUL_GELUGRAD) v += to_f<T>(bias[n]);
      switch (a.epi) {
        case EPI_BIAS_GELU:
          Z[(size_t)m * a.ldz + n] = from_f<T>(v);
          // the activation is applied to the value as it is stored, so that forward and backward agree
          v = gelu_f(to_f<T>(from_f<T>(v)), tanh_form);
          break;
        case EPI_BIAS_RESID: v += to_f<T>(R[(size_t)m * a.ldr + n]); break;
        case EPI_MUL_GELUGRAD: v *= gelu_grad_f(to_f<T>(R[(size_t)m * a.ldr + n]), tanh_form); break;
        default: break;
      }
      Y[(size_t)m * a.ldy + n] = from_f<T>(v);
    }
  }
}
}  // namespace

cudaError_t gemm_simt(const GemmArgs& a, cudaStream_t st) {
  if (a.rows_per_group > 0 && (a.rows_per_group % BM) != 0 && (a.w_grouped || a.we_grouped))
    return cudaErrorInvalidValue;
  dim3 grid((a.N + BN - 1) / BN, (a.M + BM - 1) / BM);
  if (a.dtype == DT_BF16) gemm_simt_kernel<bf16><<<grid, 256, 0, st>>>(a);
  else gemm_simt_kernel<float><<<grid, 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace sl
