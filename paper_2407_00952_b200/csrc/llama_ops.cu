// Memory-bound kernels of the Llama-shaped block: RMSNorm forward / backward, the rotary position
// rotation of q and k inside the fused qkv buffer, and the SwiGLU gate (forward and backward).
// The paper does not describe this block shape (it only cites Llama-2 as an LLM); the definitions
// are the usual ones: y = x * rsqrt(mean(x^2) + eps) * g; pairs (j, j + dh/2) of a head rotated by
// t * theta^(-2j/dh); act = silu(gate) * up.
#include "common.cuh"
#include "kernels.h"

namespace sl {
namespace {

constexpr int NORM_THREADS = 128;

__device__ __forceinline__ float block_sum_128(float v, float* sh) {
  v = warp_sum(v);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = sh[0] + sh[1] + sh[2] + sh[3];
  __syncthreads();
  return t;
}

// One 128-thread block per row.  NV > 0: the row (at most NV * 128 vectors) stays in registers
// between the reduction and the output.  NV == 0: any width, the row is read twice.
template <typename T, int NV>
__global__ void __launch_bounds__(NORM_THREADS) rms_fwd_kernel(const T* __restrict__ x, const T* __restrict__ g,
                                                               T* __restrict__ y, float* __restrict__ rstd, int d,
                                                               float eps) {
  constexpr int N = Vec16<T>::N;
  __shared__ float sh[4];
  const size_t off = (size_t)blockIdx.x * d;
  const int nvec = d / N;
  float q = 0.f;
  if constexpr (NV > 0) {
    Vec16<T> xv[NV];
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const int v = k * NORM_THREADS + threadIdx.x;
      if (v < nvec) {
        xv[k].load(x + off + (size_t)v * N);
#pragma unroll
        for (int i = 0; i < N; ++i) { float t = xv[k].get(i); q += t * t; }
      }
    }
    const float rs = rsqrtf(block_sum_128(q, sh) / d + eps);
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const int v = k * NORM_THREADS + threadIdx.x;
      if (v < nvec) {
        Vec16<T> gv, o;
        gv.load(g + (size_t)v * N);
#pragma unroll
        for (int i = 0; i < N; ++i) o.set(i, xv[k].get(i) * rs * gv.get(i));
        o.store(y + off + (size_t)v * N);
      }
    }
    if (threadIdx.x == 0) rstd[blockIdx.x] = rs;
  } else {
    for (int v = threadIdx.x; v < nvec; v += NORM_THREADS) {
      Vec16<T> xv; xv.load(x + off + (size_t)v * N);
#pragma unroll
      for (int i = 0; i < N; ++i) { float t = xv.get(i); q += t * t; }
    }
    const float rs = rsqrtf(block_sum_128(q, sh) / d + eps);
    for (int v = threadIdx.x; v < nvec; v += NORM_THREADS) {
      Vec16<T> xv, gv, o;
      xv.load(x + off + (size_t)v * N); gv.load(g + (size_t)v * N);
#pragma unroll
      for (int i = 0; i < N; ++i) o.set(i, xv.get(i) * rs * gv.get(i));
      o.store(y + off + (size_t)v * N);
    }
    if (threadIdx.x == 0) rstd[blockIdx.x] = rs;
  }
}

// dx = resid + (dy*g - xhat * mean(dy*g*xhat)) * rstd,   xhat = x * rstd
template <typename T, int NV>
__global__ void __launch_bounds__(NORM_THREADS) rms_bwd_kernel(const T* __restrict__ dy, const T* __restrict__ x,
                                                               const T* __restrict__ g, const float* __restrict__ rstd,
                                                               const T* __restrict__ resid, T* __restrict__ dx, int d) {
  constexpr int N = Vec16<T>::N;
  __shared__ float sh[4];
  const size_t off = (size_t)blockIdx.x * d;
  const int nvec = d / N;
  const float rs = rstd[blockIdx.x];
  float s2 = 0.f;
  if constexpr (NV > 0) {
    // everything the row needs is requested before the reduction (the residual too), so that the
    // block waits for memory once
    Vec16<T> xv[NV], dv[NV], gv[NV], rv[NV];
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const int v = k * NORM_THREADS + threadIdx.x;
      if (v < nvec) {
        xv[k].load(x + off + (size_t)v * N); dv[k].load(dy + off + (size_t)v * N); gv[k].load(g + (size_t)v * N);
        if (resid) rv[k].load(resid + off + (size_t)v * N);
      }
    }
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const int v = k * NORM_THREADS + threadIdx.x;
      if (v < nvec) {
#pragma unroll
        for (int i = 0; i < N; ++i) s2 += dv[k].get(i) * gv[k].get(i) * xv[k].get(i) * rs;
      }
    }
    const float m2 = block_sum_128(s2, sh) / d;
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const int v = k * NORM_THREADS + threadIdx.x;
      if (v < nvec) {
        Vec16<T> o;
#pragma unroll
        for (int i = 0; i < N; ++i) {
          float val = (dv[k].get(i) * gv[k].get(i) - xv[k].get(i) * rs * m2) * rs;
          if (resid) val += rv[k].get(i);
          o.set(i, val);
        }
        o.store(dx + off + (size_t)v * N);
      }
    }
  } else {
    for (int v = threadIdx.x; v < nvec; v += NORM_THREADS) {
      Vec16<T> xv, dv, gv;
      xv.load(x + off + (size_t)v * N); dv.load(dy + off + (size_t)v * N); gv.load(g + (size_t)v * N);
#pragma unroll
      for (int i = 0; i < N; ++i) s2 += dv.get(i) * gv.get(i) * xv.get(i) * rs;
    }
    const float m2 = block_sum_128(s2, sh) / d;
    for (int v = threadIdx.x; v < nvec; v += NORM_THREADS) {
      Vec16<T> xv, dv, gv, rv, o;
      xv.load(x + off + (size_t)v * N); dv.load(dy + off + (size_t)v * N); gv.load(g + (size_t)v * N);
      if (resid) rv.load(resid + off + (size_t)v * N);
#pragma unroll
      for (int i = 0; i < N; ++i) {
        float val = (dv.get(i) * gv.get(i) - xv.get(i) * rs * m2) * rs;
        if (resid) val += rv.get(i);
        o.set(i, val);
      }
      o.store(dx + off + (size_t)v * N);
    }
  }
}

template <typename T>
cudaError_t rms_fwd_t(const void* x, const void* g, void* y, float* rstd, int M, int d, float eps, cudaStream_t st) {
  const int need = (d / Vec16<T>::N + NORM_THREADS - 1) / NORM_THREADS;
  const T *xp = (const T*)x, *gp = (const T*)g; T* yp = (T*)y;
  if (need <= 1) rms_fwd_kernel<T, 1><<<M, NORM_THREADS, 0, st>>>(xp, gp, yp, rstd, d, eps);
  else if (need <= 2) rms_fwd_kernel<T, 2><<<M, NORM_THREADS, 0, st>>>(xp, gp, yp, rstd, d, eps);
  else if (need <= 4) rms_fwd_kernel<T, 4><<<M, NORM_THREADS, 0, st>>>(xp, gp, yp, rstd, d, eps);
  else rms_fwd_kernel<T, 0><<<M, NORM_THREADS, 0, st>>>(xp, gp, yp, rstd, d, eps);
  return cudaGetLastError();
}

template <typename T>
cudaError_t rms_bwd_t(const void* dy, const void* x, const void* g, const float* rstd, const void* resid, void* dx,
                      int M, int d, cudaStream_t st) {
  const int need = (d / Vec16<T>::N + NORM_THREADS - 1) / NORM_THREADS;
  const T *dyp = (const T*)dy, *xp = (const T*)x, *gp = (const T*)g, *rp = (const T*)resid; T* dxp = (T*)dx;
  if (need <= 1) rms_bwd_kernel<T, 1><<<M, NORM_THREADS, 0, st>>>(dyp, xp, gp, rstd, rp, dxp, d);
  else if (need <= 2) rms_bwd_kernel<T, 2><<<M, NORM_THREADS, 0, st>>>(dyp, xp, gp, rstd, rp, dxp, d);
  else if (need <= 4) rms_bwd_kernel<T, 4><<<M, NORM_THREADS, 0, st>>>(dyp, xp, gp, rstd, rp, dxp, d);
  else rms_bwd_kernel<T, 0><<<M, NORM_THREADS, 0, st>>>(dyp, xp, gp, rstd, rp, dxp, d);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// rotary positions, in place on the q and k slices of qkv [M, 3d].  One thread rotates one vector
// of the lower half of a head against the matching vector of the upper half.
// table [T, dh/2] holds (cos, sin) of t * theta^(-2j/dh); sign = -1 applies the inverse rotation,
// which is the gradient map.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void rope_kernel(T* __restrict__ qkv, const float2* __restrict__ table, int64_t total, int Tseq, int H,
                            int d, int half, float sign) {
  constexpr int N = Vec16<T>::N;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int cpv = half / N;                       // vectors per half head
  int c = (int)(idx % cpv); idx /= cpv;
  int h = (int)(idx % H); idx /= H;
  int part = (int)(idx & 1);                      // 0: q, 1: k
  int64_t m = idx >> 1;
  int t = (int)(m % Tseq);
  T* lo = qkv + (size_t)m * 3 * d + (size_t)part * d + (size_t)h * 2 * half + (size_t)c * N;
  T* hi = lo + half;
  Vec16<T> a, b, oa, ob;
  a.load(lo); b.load(hi);
  const float2* tr = table + (size_t)t * half + c * N;
#pragma unroll
  for (int i = 0; i < N; ++i) {
    float2 cs = tr[i];
    float sn = cs.y * sign;
    oa.set(i, a.get(i) * cs.x - b.get(i) * sn);
    ob.set(i, b.get(i) * cs.x + a.get(i) * sn);
  }
  oa.store(lo); ob.store(hi);
}

__device__ __forceinline__ float sigmoid_f(float z) { return 1.0f / (1.0f + __expf(-z)); }

// z [M, 2F]: columns [0, F) gate, [F, 2F) up.  act [M, F] = silu(gate) * up
template <typename T>
__global__ void swiglu_fwd_kernel(const T* __restrict__ z, T* __restrict__ act, int64_t total, int F) {
  constexpr int N = Vec16<T>::N;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int vpr = F / N;
  int64_t m = idx / vpr;
  int c = (int)(idx % vpr) * N;
  Vec16<T> gv, uv, o;
  gv.load(z + (size_t)m * 2 * F + c); uv.load(z + (size_t)m * 2 * F + F + c);
#pragma unroll
  for (int i = 0; i < N; ++i) { float gg = gv.get(i); o.set(i, gg * sigmoid_f(gg) * uv.get(i)); }
  o.store(act + (size_t)m * F + c);
}

// dz [M, 2F] from dact [M, F]:  d gate = dact * up * silu'(gate),  d up = dact * silu(gate)
template <typename T>
__global__ void swiglu_bwd_kernel(const T* __restrict__ dact, const T* __restrict__ z, T* __restrict__ dz,
                                  int64_t total, int F) {
  constexpr int N = Vec16<T>::N;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int vpr = F / N;
  int64_t m = idx / vpr;
  int c = (int)(idx % vpr) * N;
  Vec16<T> gv, uv, dv, og, ou;
  gv.load(z + (size_t)m * 2 * F + c); uv.load(z + (size_t)m * 2 * F + F + c); dv.load(dact + (size_t)m * F + c);
#pragma unroll
  for (int i = 0; i < N; ++i) {
    float gg = gv.get(i), sg = sigmoid_f(gg), da = dv.get(i);
    og.set(i, da * uv.get(i) * sg * (1.0f + gg * (1.0f - sg)));
    ou.set(i, da * gg * sg);
  }
  og.store(dz + (size_t)m * 2 * F + c); ou.store(dz + (size_t)m * 2 * F + F + c);
}

}  // namespace

cudaError_t rmsnorm_fwd(int dt, const void* x, const void* g, void* y, float* rstd, int M, int d, float eps,
                        cudaStream_t st) {
  return dt == DT_BF16 ? rms_fwd_t<bf16>(x, g, y, rstd, M, d, eps, st) : rms_fwd_t<float>(x, g, y, rstd, M, d, eps, st);
}

cudaError_t rmsnorm_bwd(int dt, const void* dy, const void* x, const void* g, const float* rstd, const void* resid,
                        void* dx, int M, int d, cudaStream_t st) {
  return dt == DT_BF16 ? rms_bwd_t<bf16>(dy, x, g, rstd, resid, dx, M, d, st)
                       : rms_bwd_t<float>(dy, x, g, rstd, resid, dx, M, d, st);
}

cudaError_t rope_inplace(int dt, void* qkv, const float* table, int M, int T, int H, int d, float sign, cudaStream_t st) {
  const int n = dt == DT_BF16 ? 8 : 4;
  const int half = d / H / 2;
  if (half < n || half % n != 0) return cudaErrorInvalidValue;
  const int64_t total = (int64_t)M * 2 * H * (half / n);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (dt == DT_BF16)
    rope_kernel<bf16><<<blocks, 256, 0, st>>>((bf16*)qkv, (const float2*)table, total, T, H, d, half, sign);
  else
    rope_kernel<float><<<blocks, 256, 0, st>>>((float*)qkv, (const float2*)table, total, T, H, d, half, sign);
  return cudaGetLastError();
}

cudaError_t swiglu_fwd(int dt, const void* z, void* act, int M, int F, cudaStream_t st) {
  const int n = dt == DT_BF16 ? 8 : 4;
  const int64_t total = (int64_t)M * (F / n);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (dt == DT_BF16) swiglu_fwd_kernel<bf16><<<blocks, 256, 0, st>>>((const bf16*)z, (bf16*)act, total, F);
  else swiglu_fwd_kernel<float><<<blocks, 256, 0, st>>>((const float*)z, (float*)act, total, F);
  return cudaGetLastError();
}

cudaError_t swiglu_bwd(int dt, const void* dact, const void* z, void* dz, int M, int F, cudaStream_t st) {
  const int n = dt == DT_BF16 ? 8 : 4;
  const int64_t total = (int64_t)M * (F / n);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (dt == DT_BF16) swiglu_bwd_kernel<bf16><<<blocks, 256, 0, st>>>((const bf16*)dact, (const bf16*)z, (bf16*)dz, total, F);
  else swiglu_bwd_kernel<float><<<blocks, 256, 0, st>>>((const float*)dact, (const float*)z, (float*)dz, total, F);
  return cudaGetLastError();
}

}  // namespace sl
