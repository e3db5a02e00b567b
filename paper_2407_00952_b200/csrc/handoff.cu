// Compressed cut-layer hand-off: the activations S and the activation gradients dL/dS that cross
// the cut (Sec. III-B steps a2 and a4) as 8-bit codes with one fp32 scale per token.  The paper
// names quantisation of this exchange as a direction (Sec. V, efficiency) and fixes no format;
// the format here is E4M3 (4 exponent bits, bias 7, 3 mantissa bits, largest finite value 448)
// scaled per row:
//   absmax_m = max_c |x[m,c]|,  inv_m = 448 / absmax_m,  scale_m = absmax_m / 448   (fp32 divisions)
//   code[m,c] = E4M3(x[m,c] * inv_m)       fp32 product, nearest value, ties to even, saturating
//   x^[m,c]   = value(code[m,c]) * scale_m  fp32 product, rounded once to the buffer's type
// HBM-bound: one warp per row; the row is read twice (the second time from L1 / L2), the codes are
// written once: (2 + 1) bytes per bf16 element one way, (1 + 2) the other.
#include <cuda_fp16.h>

#include "common.cuh"
#include "kernels.h"

namespace sl {
namespace {

// two fp32 values -> two E4M3 codes; the first value's code is the low byte
__device__ __forceinline__ uint32_t e4m3x2(float first, float second) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(second), "f"(first));
  return r;
}
// two E4M3 codes -> their values (exact in fp16, then widened)
__device__ __forceinline__ float2 e4m3x2_values(uint32_t two_codes) {
  uint32_t h;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h) : "h"((uint16_t)two_codes));
  return __half22float2(*reinterpret_cast<__half2*>(&h));
}

template <typename T>
__global__ void __launch_bounds__(256)
handoff_quantize_kernel(const T* __restrict__ x, int64_t M, int d, uint8_t* __restrict__ codes,
                        float* __restrict__ scales) {
  constexpr int N = Vec16<T>::N;
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  const T* xr = x + row * d;
  float amax = 0.f;
  for (int c = lane * N; c < d; c += 32 * N) {
    Vec16<T> v; v.load(xr + c);
#pragma unroll
    for (int i = 0; i < N; ++i) amax = fmaxf(amax, fabsf(v.get(i)));
  }
  amax = warp_max(amax);
  const float inv = amax > 0.f ? __fdiv_rn(448.0f, amax) : 0.f;
  if (lane == 0) scales[row] = amax > 0.f ? __fdiv_rn(amax, 448.0f) : 0.f;
  uint8_t* cr = codes + row * d;
  for (int c = lane * N; c < d; c += 32 * N) {
    Vec16<T> v; v.load(xr + c);
    uint32_t w[N / 4];
#pragma unroll
    for (int i = 0; i < N / 4; ++i)
      w[i] = e4m3x2(__fmul_rn(v.get(4 * i), inv), __fmul_rn(v.get(4 * i + 1), inv)) |
             (e4m3x2(__fmul_rn(v.get(4 * i + 2), inv), __fmul_rn(v.get(4 * i + 3), inv)) << 16);
    if (N == 8) *reinterpret_cast<uint2*>(cr + c) = make_uint2(w[0], w[N / 4 - 1]);
    else *reinterpret_cast<uint32_t*>(cr + c) = w[0];
  }
}

template <typename T>
__global__ void __launch_bounds__(256)
handoff_dequantize_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ scales, int64_t M, int d,
                          T* __restrict__ y) {
  constexpr int N = Vec16<T>::N;
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  const float sc = scales[row];
  const uint8_t* cr = codes + row * d;
  T* yr = y + row * d;
  for (int c = lane * N; c < d; c += 32 * N) {
    uint32_t w[2];
    if (N == 8) { uint2 raw = *reinterpret_cast<const uint2*>(cr + c); w[0] = raw.x; w[1] = raw.y; }
    else { w[0] = *reinterpret_cast<const uint32_t*>(cr + c); w[1] = 0u; }
    Vec16<T> o;
#pragma unroll
    for (int i = 0; i < N / 4; ++i) {
      const float2 a = e4m3x2_values(w[i] & 0xffffu), b = e4m3x2_values(w[i] >> 16);
      o.set(4 * i, __fmul_rn(a.x, sc)); o.set(4 * i + 1, __fmul_rn(a.y, sc));
      o.set(4 * i + 2, __fmul_rn(b.x, sc)); o.set(4 * i + 3, __fmul_rn(b.y, sc));
    }
    o.store(yr + c);
  }
}

}  // namespace

cudaError_t handoff_quantize(int dt, const void* x, int64_t M, int d, uint8_t* codes, float* scales, cudaStream_t st) {
  const unsigned blocks = (unsigned)((M + 7) / 8);
  if (dt == DT_BF16) handoff_quantize_kernel<bf16><<<blocks, 256, 0, st>>>((const bf16*)x, M, d, codes, scales);
  else handoff_quantize_kernel<float><<<blocks, 256, 0, st>>>((const float*)x, M, d, codes, scales);
  return cudaGetLastError();
}

cudaError_t handoff_dequantize(int dt, const uint8_t* codes, const float* scales, int64_t M, int d, void* y,
                               cudaStream_t st) {
  const unsigned blocks = (unsigned)((M + 7) / 8);
  if (dt == DT_BF16) handoff_dequantize_kernel<bf16><<<blocks, 256, 0, st>>>(codes, scales, M, d, (bf16*)y);
  else handoff_dequantize_kernel<float><<<blocks, 256, 0, st>>>(codes, scales, M, d, (float*)y);
  return cudaGetLastError();
}

}  // namespace sl
