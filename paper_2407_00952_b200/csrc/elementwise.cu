// Memory-bound kernels of the split-LoRA round: embedding gather, LayerNorm forward/backward,
// cross-entropy, adapter gradients (skinny reductions over tokens), optimizer step, the
// client-side aggregation of Eq. 8-9, adapter compute copies and transposes.
// All global accesses are 16-byte vectors where the layout allows; reductions use warp shuffles.
#include "common.cuh"
#include "kernels.h"

namespace sl {

// ------------------------------------------------------------------------------------------
// embedding: x0[m, :] = wte[tok[m], :] + wpe[m % T, :]
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void embed_kernel(const int32_t* __restrict__ tok, const T* __restrict__ wte,
                             const T* __restrict__ wpe, T* __restrict__ out, int M, int Tseq, int d, int vocab) {
  constexpr int N = Vec16<T>::N;
  const int vec_per_row = d / N;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)M * vec_per_row) return;
  int m = (int)(idx / vec_per_row);
  int c = (int)(idx % vec_per_row) * N;
  int t = tok[m];
  t = t < 0 ? 0 : (t >= vocab ? vocab - 1 : t);
  Vec16<T> a, b, o;
  a.load(wte + (size_t)t * d + c);
  if (wpe == nullptr) {             // no learned positions (rotary models): plain gather
    a.store(out + (size_t)m * d + c);
    return;
  }
  b.load(wpe + (size_t)(m % Tseq) * d + c);
#pragma unroll
  for (int i = 0; i < N; ++i) o.set(i, a.get(i) + b.get(i));
  o.store(out + (size_t)m * d + c);
}

cudaError_t embed(int dt, const int32_t* tokens, const void* wte, const void* wpe, void* out, int M, int T,
                  int d, int vocab, cudaStream_t st) {
  int n = dt == DT_BF16 ? 8 : 4;
  int64_t total = (int64_t)M * (d / n);
  int blocks = (int)((total + 255) / 256);
  if (dt == DT_BF16)
    embed_kernel<bf16><<<blocks, 256, 0, st>>>(tokens, (const bf16*)wte, (const bf16*)wpe, (bf16*)out, M, T, d, vocab);
  else
    embed_kernel<float><<<blocks, 256, 0, st>>>(tokens, (const float*)wte, (const float*)wpe, (float*)out, M, T, d, vocab);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// LayerNorm: one warp per row, statistics in fp32.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void ln_fwd_kernel(const T* __restrict__ x, const T* __restrict__ g, const T* __restrict__ b,
                              T* __restrict__ y, float* __restrict__ mean, float* __restrict__ rstd, int M,
                              int d, float eps) {
  constexpr int N = Vec16<T>::N;
  int row = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  int lane = threadIdx.x & 31;
  if (row >= M) return;
  const T* xr = x + (size_t)row * d;
  float s = 0.f;
  for (int c = lane * N; c < d; c += 32 * N) {
    Vec16<T> v; v.load(xr + c);
#pragma unroll
    for (int i = 0; i < N; ++i) s += v.get(i);
  }
  float mu = warp_sum(s) / d;
  float q = 0.f;
  for (int c = lane * N; c < d; c += 32 * N) {
    Vec16<T> v; v.load(xr + c);
#pragma unroll
    for (int i = 0; i < N; ++i) { float t = v.get(i) - mu; q += t * t; }
  }
  float rs = rsqrtf(warp_sum(q) / d + eps);
  T* yr = y + (size_t)row * d;
  for (int c = lane * N; c < d; c += 32 * N) {
    Vec16<T> v, gv, bv, o;
    v.load(xr + c); gv.load(g + c); bv.load(b + c);
#pragma unroll
    for (int i = 0; i < N; ++i) o.set(i, (v.get(i) - mu) * rs * gv.get(i) + bv.get(i));
    o.store(yr + c);
  }
  if (lane == 0) { mean[row] = mu; rstd[row] = rs; }
}

template <typename T>
__global__ void ln_bwd_kernel(const T* __restrict__ dy, const T* __restrict__ x, const T* __restrict__ g,
                              const float* __restrict__ mean, const float* __restrict__ rstd,
                              const T* __restrict__ resid, T* __restrict__ dx, int M, int d) {
  constexpr int N = Vec16<T>::N;
  int row = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  int lane = threadIdx.x & 31;
  if (row >= M) return;
  const T* xr = x + (size_t)row * d;
  const T* dyr = dy + (size_t)row * d;
  float mu = mean[row], rs = rstd[row];
  float s1 = 0.f, s2 = 0.f;
  for (int c = lane * N; c < d; c += 32 * N) {
    Vec16<T> xv, dv, gv;
    xv.load(xr + c); dv.load(dyr + c); gv.load(g + c);
#pragma unroll
    for (int i = 0; i < N; ++i) {
      float dxh = dv.get(i) * gv.get(i);
      s1 += dxh;
      s2 += dxh * (xv.get(i) - mu) * rs;
    }
  }
  float m1 = warp_sum(s1) / d, m2 = warp_sum(s2) / d;
  T* dxr = dx + (size_t)row * d;
  for (int c = lane * N; c < d; c += 32 * N) {
    Vec16<T> xv, dv, gv, rv, o;
    xv.load(xr + c); dv.load(dyr + c); gv.load(g + c);
    if (resid) rv.load(resid + (size_t)row * d + c);
#pragma unroll
    for (int i = 0; i < N; ++i) {
      float xh = (xv.get(i) - mu) * rs;
      float v = (dv.get(i) * gv.get(i) - m1 - xh * m2) * rs;
      if (resid) v += rv.get(i);
      o.set(i, v);
    }
    o.store(dxr + c);
  }
}

// Register-resident variants for rows of exactly NV vectors per lane (d = NV * 32 * vector width):
// the row is read from memory once and kept in registers between the statistics and the output.
template <typename T, int NV>
__global__ void __launch_bounds__(256) ln_fwd_reg_kernel(const T* __restrict__ x, const T* __restrict__ g,
                                                         const T* __restrict__ b, T* __restrict__ y,
                                                         float* __restrict__ mean, float* __restrict__ rstd, int M,
                                                         int d, float eps) {
  constexpr int N = Vec16<T>::N;
  int row = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  int lane = threadIdx.x & 31;
  if (row >= M) return;
  const T* xr = x + (size_t)row * d;
  Vec16<T> xv[NV];
#pragma unroll
  for (int k = 0; k < NV; ++k) xv[k].load(xr + (k * 32 + lane) * N);
  float s = 0.f;
#pragma unroll
  for (int k = 0; k < NV; ++k)
#pragma unroll
    for (int i = 0; i < N; ++i) s += xv[k].get(i);
  const float mu = warp_sum(s) / d;
  float q = 0.f;
#pragma unroll
  for (int k = 0; k < NV; ++k)
#pragma unroll
    for (int i = 0; i < N; ++i) { float t = xv[k].get(i) - mu; q += t * t; }
  const float rs = rsqrtf(warp_sum(q) / d + eps);
  T* yr = y + (size_t)row * d;
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    const int c = (k * 32 + lane) * N;
    Vec16<T> gv, bv, o;
    gv.load(g + c); bv.load(b + c);
#pragma unroll
    for (int i = 0; i < N; ++i) o.set(i, (xv[k].get(i) - mu) * rs * gv.get(i) + bv.get(i));
    o.store(yr + c);
  }
  if (lane == 0) { mean[row] = mu; rstd[row] = rs; }
}

template <typename T, int NV>
__global__ void __launch_bounds__(256) ln_bwd_reg_kernel(const T* __restrict__ dy, const T* __restrict__ x,
                                                         const T* __restrict__ g, const float* __restrict__ mean,
                                                         const float* __restrict__ rstd, const T* __restrict__ resid,
                                                         T* __restrict__ dx, int M, int d) {
  constexpr int N = Vec16<T>::N;
  int row = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  int lane = threadIdx.x & 31;
  if (row >= M) return;
  const size_t off = (size_t)row * d;
  const float mu = mean[row], rs = rstd[row];
  // everything the row needs is requested before the reduction (gain and residual too), so that the
  // warp waits for memory once
  Vec16<T> xv[NV], dv[NV], gv[NV], rv[NV];
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    const int c = (k * 32 + lane) * N;
    xv[k].load(x + off + c); dv[k].load(dy + off + c); gv[k].load(g + c);
    if (resid) rv[k].load(resid + off + c);
  }
  float s1 = 0.f, s2 = 0.f;
#pragma unroll
  for (int k = 0; k < NV; ++k) {
#pragma unroll
    for (int i = 0; i < N; ++i) {
      float dxh = dv[k].get(i) * gv[k].get(i);
      s1 += dxh;
      s2 += dxh * (xv[k].get(i) - mu) * rs;
    }
  }
  const float m1 = warp_sum(s1) / d, m2 = warp_sum(s2) / d;
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    const int c = (k * 32 + lane) * N;
    Vec16<T> o;
#pragma unroll
    for (int i = 0; i < N; ++i) {
      float xh = (xv[k].get(i) - mu) * rs;
      float v = (dv[k].get(i) * gv[k].get(i) - m1 - xh * m2) * rs;
      if (resid) v += rv[k].get(i);
      o.set(i, v);
    }
    o.store(dx + off + c);
  }
}

cudaError_t layernorm_fwd(int dt, const void* x, const void* g, const void* b, void* y, float* mean, float* rstd,
                          int M, int d, float eps, cudaStream_t st) {
  int blocks = (M + 7) / 8;
  if (dt == DT_BF16 && d == 1024) {
    ln_fwd_reg_kernel<bf16, 4><<<blocks, 256, 0, st>>>((const bf16*)x, (const bf16*)g, (const bf16*)b, (bf16*)y, mean, rstd, M, d, eps);
    return cudaGetLastError();
  }
  if (dt == DT_BF16 && d == 768) {
    ln_fwd_reg_kernel<bf16, 3><<<blocks, 256, 0, st>>>((const bf16*)x, (const bf16*)g, (const bf16*)b, (bf16*)y, mean, rstd, M, d, eps);
    return cudaGetLastError();
  }
  if (dt == DT_BF16)
    ln_fwd_kernel<bf16><<<blocks, 256, 0, st>>>((const bf16*)x, (const bf16*)g, (const bf16*)b, (bf16*)y, mean, rstd, M, d, eps);
  else
    ln_fwd_kernel<float><<<blocks, 256, 0, st>>>((const float*)x, (const float*)g, (const float*)b, (float*)y, mean, rstd, M, d, eps);
  return cudaGetLastError();
}

cudaError_t layernorm_bwd(int dt, const void* dy, const void* x, const void* g, const float* mean,
                          const float* rstd, const void* resid, void* dx, int M, int d, cudaStream_t st) {
  int blocks = (M + 7) / 8;
  if (dt == DT_BF16 && d == 1024) {
    ln_bwd_reg_kernel<bf16, 4><<<blocks, 256, 0, st>>>((const bf16*)dy, (const bf16*)x, (const bf16*)g, mean, rstd, (const bf16*)resid, (bf16*)dx, M, d);
    return cudaGetLastError();
  }
  if (dt == DT_BF16 && d == 768) {
    ln_bwd_reg_kernel<bf16, 3><<<blocks, 256, 0, st>>>((const bf16*)dy, (const bf16*)x, (const bf16*)g, mean, rstd, (const bf16*)resid, (bf16*)dx, M, d);
    return cudaGetLastError();
  }
  if (dt == DT_BF16)
    ln_bwd_kernel<bf16><<<blocks, 256, 0, st>>>((const bf16*)dy, (const bf16*)x, (const bf16*)g, mean, rstd, (const bf16*)resid, (bf16*)dx, M, d);
  else
    ln_bwd_kernel<float><<<blocks, 256, 0, st>>>((const float*)dy, (const float*)x, (const float*)g, mean, rstd, (const float*)resid, (float*)dx, M, d);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// cross-entropy: one block per row.  Pass 1: online max / sum of exp; pass 2: overwrite the row
// with (softmax - onehot) / n_valid.  Pad columns [V, ld) are written as zero.
// ------------------------------------------------------------------------------------------
__global__ void count_valid_kernel(const int32_t* __restrict__ labels, int M, int V, int* __restrict__ n_valid,
                                   int normalizer_override) {
  if (normalizer_override > 0) {       // the batch is one shard of a larger one: use the global count
    if (threadIdx.x == 0) *n_valid = normalizer_override;
    return;
  }
  __shared__ int sh[32];
  int c = 0;
  for (int i = threadIdx.x; i < M; i += blockDim.x) c += (labels[i] >= 0 && labels[i] < V) ? 1 : 0;   // the predicate of the row kernels
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = c;
  __syncthreads();
  if (threadIdx.x == 0) {
    int t = 0;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += sh[i];
    *n_valid = t;
  }
}

template <typename T>
__global__ void ce_kernel(T* __restrict__ logits, int64_t ld, const int32_t* __restrict__ labels, int V,
                          float* __restrict__ row_loss, const int* __restrict__ n_valid) {
  constexpr int N = Vec16<T>::N;
  __shared__ float sh_m[32], sh_s[32];
  __shared__ float sh_lse;
  int row = blockIdx.x;
  T* z = logits + (size_t)row * ld;
  int y = labels[row];
  bool valid = y >= 0 && y < V;
  const int Vv = (V / N) * N;
  float mx = -INFINITY, sm = 0.f;
  for (int c = threadIdx.x * N; c < Vv; c += blockDim.x * N) {
    Vec16<T> v; v.load(z + c);
    float lm = v.get(0);
#pragma unroll
    for (int i = 1; i < N; ++i) lm = fmaxf(lm, v.get(i));
    float nm = fmaxf(mx, lm);
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < N; ++i) acc += __expf(v.get(i) - nm);
    sm = sm * __expf(mx - nm) + acc;
    mx = nm;
  }
  for (int c = Vv + threadIdx.x; c < V; c += blockDim.x) {
    float zc = to_f<T>(z[c]);
    float nm = fmaxf(mx, zc);
    sm = sm * __expf(mx - nm) + __expf(zc - nm);
    mx = nm;
  }
  // combine (max, sum) pairs across the warp, then across warps
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float om = __shfl_xor_sync(0xffffffffu, mx, o), os = __shfl_xor_sync(0xffffffffu, sm, o);
    float nm = fmaxf(mx, om);
    float a = (mx == -INFINITY) ? 0.f : sm * __expf(mx - nm);
    float b = (om == -INFINITY) ? 0.f : os * __expf(om - nm);
    sm = a + b; mx = nm;
  }
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  if (lane == 0) { sh_m[warp] = mx; sh_s[warp] = sm; }
  __syncthreads();
  if (warp == 0) {
    float m2 = lane < nw ? sh_m[lane] : -INFINITY, s2 = lane < nw ? sh_s[lane] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float om = __shfl_xor_sync(0xffffffffu, m2, o), os = __shfl_xor_sync(0xffffffffu, s2, o);
      float nm = fmaxf(m2, om);
      float a = (m2 == -INFINITY) ? 0.f : s2 * __expf(m2 - nm);
      float b = (om == -INFINITY) ? 0.f : os * __expf(om - nm);
      s2 = a + b; m2 = nm;
    }
    if (lane == 0) {
      float lse = m2 + logf(s2);
      sh_lse = lse;
      row_loss[row] = valid ? lse - to_f<T>(z[y]) : 0.f;
    }
  }
  __syncthreads();
  float lse = sh_lse;
  int nv = *n_valid;
  float inv = (valid && nv > 0) ? 1.0f / (float)nv : 0.f;
  const int ldv = (int)ld;
  for (int c = threadIdx.x * N; c < ldv; c += blockDim.x * N) {
    Vec16<T> v, o;
    v.load(z + c);
#pragma unroll
    for (int i = 0; i < N; ++i) {
      int col = c + i;
      float p = col < V ? __expf(v.get(i) - lse) : 0.f;
      if (col == y) p -= 1.0f;
      o.set(i, p * inv);
    }
    o.store(z + c);
  }
}

// bf16 rows with a 16-byte aligned stride: the same two passes with fewer instructions per element
// (the arithmetic of this kernel weighs as much as its memory traffic: about 15 instructions and 2.1
// exponentials per element in ce_kernel).  Row maximum on packed bf16 pairs, exponentials as
// ex2(fma(z, log2 e, -max log2 e)), no per-element test for the label or the pad columns: the vectors
// that hold only valid columns take the fast loop, the last few go element by element, and the
// label's entry is corrected by one thread afterwards.
__device__ __forceinline__ float ce_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__global__ void __launch_bounds__(256)
ce_bf16_kernel(bf16* __restrict__ logits, int64_t ld, const int32_t* __restrict__ labels, int V,
               float* __restrict__ row_loss, const int* __restrict__ n_valid) {
  __shared__ float sh_m[32], sh_s[32];
  __shared__ float sh_lse, sh_zy;
  const float L = 1.4426950408889634f;
  const int row = blockIdx.x;
  bf16* z = logits + (size_t)row * ld;
  uint4* zv = reinterpret_cast<uint4*>(z);
  const int y = labels[row];
  const bool valid = y >= 0 && y < V;
  const int nfull = V >> 3, nvec = (int)(ld >> 3);
  float mx = -INFINITY, sm = 0.f;
  for (int i = threadIdx.x; i < nfull; i += blockDim.x) {
    const uint4 raw = zv[i];
    const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
    const uint32_t* w = reinterpret_cast<const uint32_t*>(&raw);
    const __nv_bfloat162 m2 = __hmax2(__hmax2(h2[0], h2[1]), __hmax2(h2[2], h2[3]));
    const float nm = fmaxf(mx, fmaxf(__low2float(m2), __high2float(m2)));
    const float nml = -nm * L;
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k)
      acc += ce_ex2(fmaf(__uint_as_float(w[k] << 16), L, nml)) + ce_ex2(fmaf(__uint_as_float(w[k] & 0xffff0000u), L, nml));
    sm = sm * ce_ex2(fmaf(mx, L, nml)) + acc;      // mx = -inf the first time: the factor is 0
    mx = nm;
  }
  for (int c = 8 * nfull + threadIdx.x; c < V; c += blockDim.x) {
    const float zc = __bfloat162float(z[c]);
    const float nm = fmaxf(mx, zc);
    sm = sm * __expf(mx - nm) + __expf(zc - nm);
    mx = nm;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float om = __shfl_xor_sync(0xffffffffu, mx, o), os = __shfl_xor_sync(0xffffffffu, sm, o);
    float nm = fmaxf(mx, om);
    float a = (mx == -INFINITY) ? 0.f : sm * __expf(mx - nm);
    float b = (om == -INFINITY) ? 0.f : os * __expf(om - nm);
    sm = a + b; mx = nm;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  if (lane == 0) { sh_m[warp] = mx; sh_s[warp] = sm; }
  __syncthreads();
  if (warp == 0) {
    float m2 = lane < nw ? sh_m[lane] : -INFINITY, s2 = lane < nw ? sh_s[lane] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float om = __shfl_xor_sync(0xffffffffu, m2, o), os = __shfl_xor_sync(0xffffffffu, s2, o);
      float nm = fmaxf(m2, om);
      float a = (m2 == -INFINITY) ? 0.f : s2 * __expf(m2 - nm);
      float b = (om == -INFINITY) ? 0.f : os * __expf(om - nm);
      s2 = a + b; m2 = nm;
    }
    if (lane == 0) {
      const float lse = m2 + logf(s2);
      const float zy = valid ? __bfloat162float(z[y]) : 0.f;
      sh_lse = lse; sh_zy = zy;
      row_loss[row] = valid ? lse - zy : 0.f;
    }
  }
  __syncthreads();
  const float lse = sh_lse;
  const int nv = *n_valid;
  const float inv = (valid && nv > 0) ? 1.0f / (float)nv : 0.f;
  const float nl = -lse * L;
  for (int i = threadIdx.x; i < nfull; i += blockDim.x) {
    const uint4 raw = zv[i];
    const uint32_t* w = reinterpret_cast<const uint32_t*>(&raw);
    uint4 out;
    uint32_t* o = reinterpret_cast<uint32_t*>(&out);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float p0 = ce_ex2(fmaf(__uint_as_float(w[k] << 16), L, nl)) * inv;
      const float p1 = ce_ex2(fmaf(__uint_as_float(w[k] & 0xffff0000u), L, nl)) * inv;
      __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
      o[k] = *reinterpret_cast<uint32_t*>(&pb);
    }
    zv[i] = out;
  }
  for (int c = 8 * nfull + threadIdx.x; c < 8 * nvec; c += blockDim.x)    // last valid columns, then the pad
    z[c] = __float2bfloat16_rn(c < V ? __expf(__bfloat162float(z[c]) - lse) * inv : 0.f);
  __syncthreads();
  if (threadIdx.x == 0 && valid)                     // d/dz_y = (p_y - 1) / n_valid
    z[y] = __float2bfloat16_rn((__expf(sh_zy - lse) - 1.0f) * inv);
}

__global__ void loss_reduce_kernel(const float* __restrict__ row_loss, int M, const int* __restrict__ n_valid,
                                   float* __restrict__ loss) {
  __shared__ double sh[32];
  double s = 0.0;
  for (int i = threadIdx.x; i < M; i += blockDim.x) s += (double)row_loss[i];
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += sh[i];
    int nv = *n_valid;
    *loss = nv > 0 ? (float)(t / nv) : 0.f;
  }
}

cudaError_t cross_entropy(int dt, void* logits, int64_t ld, const int32_t* labels, int M, int V, float* row_loss,
                          int* n_valid, float* loss, int normalizer_override, cudaStream_t st) {
  count_valid_kernel<<<1, 1024, 0, st>>>(labels, M, V, n_valid, normalizer_override);
  if (dt == DT_BF16 && ld % 8 == 0 && (reinterpret_cast<uintptr_t>(logits) & 15u) == 0)
    ce_bf16_kernel<<<M, 256, 0, st>>>((bf16*)logits, ld, labels, V, row_loss, n_valid);
  else if (dt == DT_BF16) ce_kernel<bf16><<<M, 256, 0, st>>>((bf16*)logits, ld, labels, V, row_loss, n_valid);
  else ce_kernel<float><<<M, 256, 0, st>>>((float*)logits, ld, labels, V, row_loss, n_valid);
  loss_reduce_kernel<<<1, 1024, 0, st>>>(row_loss, M, n_valid, loss);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// optimizer on adapter parameters only (Eq. 4-7; AdamW as configured)
// ------------------------------------------------------------------------------------------
__global__ void optimizer_kernel(float* __restrict__ p, const float* __restrict__ g, float* __restrict__ m,
                                 float* __restrict__ v, int64_t n4, OptArgs o) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  float4 pv = reinterpret_cast<float4*>(p)[i];
  float4 gv = reinterpret_cast<const float4*>(g)[i];
  float* pp = reinterpret_cast<float*>(&pv);
  const float* gp = reinterpret_cast<const float*>(&gv);
  if (o.optimizer == 0) {
#pragma unroll
    for (int k = 0; k < 4; ++k) pp[k] = pp[k] - o.lr * gp[k];
  } else {
    float4 mv = reinterpret_cast<float4*>(m)[i];
    float4 vv = reinterpret_cast<float4*>(v)[i];
    float* mp = reinterpret_cast<float*>(&mv);
    float* vp = reinterpret_cast<float*>(&vv);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float pk = pp[k] * (1.0f - o.lr * o.wd);
      mp[k] = o.beta1 * mp[k] + (1.0f - o.beta1) * gp[k];
      vp[k] = o.beta2 * vp[k] + (1.0f - o.beta2) * gp[k] * gp[k];
      float mh = mp[k] / o.bc1, vh = vp[k] / o.bc2;
      pp[k] = pk - o.lr * mh / (sqrtf(vh) + o.eps);
    }
    reinterpret_cast<float4*>(m)[i] = mv;
    reinterpret_cast<float4*>(v)[i] = vv;
  }
  reinterpret_cast<float4*>(p)[i] = pv;
}

cudaError_t optimizer_step(float* p, const float* g, float* m, float* v, int64_t n, const OptArgs& o,
                           cudaStream_t st) {
  if (n % 4 != 0) return cudaErrorInvalidValue;
  if (n == 0) return cudaSuccess;     // a side without adapters (all blocks on the clients)
  int64_t n4 = n / 4;
  optimizer_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(p, g, m, v, n4, o);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Eq. 8-9 + write-back.  One float4 per thread: read the K client copies, write the average to
// all K.  Weights arrive by value.
// ------------------------------------------------------------------------------------------
struct AggWeights { float w[AGG_MAX_CLIENTS]; };

__global__ void __launch_bounds__(256) aggregate_kernel(float* __restrict__ params, int K, int64_t P4, int64_t S4,
                                                        AggWeights w) {
  // P4: float4s averaged per client, S4: float4s between two clients' rows (S4 >= P4)
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < P4; i += stride) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = 0; k < K; ++k) {
      float4 v = __ldcs(reinterpret_cast<const float4*>(params) + (size_t)k * S4 + i);
      acc.x = fmaf(w.w[k], v.x, acc.x);
      acc.y = fmaf(w.w[k], v.y, acc.y);
      acc.z = fmaf(w.w[k], v.z, acc.z);
      acc.w = fmaf(w.w[k], v.w, acc.w);
    }
    for (int k = 0; k < K; ++k) __stcs(reinterpret_cast<float4*>(params) + (size_t)k * S4 + i, acc);
  }
}

// The two halves of the same step for clients spread over several devices: the weighted sum of the
// local clients' rows goes to `sum` [P] (which the caller then adds up over devices), and `sum` is
// afterwards written to every local client's row (the downlink of step b3).
__global__ void __launch_bounds__(256) weighted_sum_kernel(const float* __restrict__ params, int K, int64_t P4,
                                                           AggWeights w, float* __restrict__ sum) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < P4; i += stride) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = 0; k < K; ++k) {
      float4 v = __ldcs(reinterpret_cast<const float4*>(params) + (size_t)k * P4 + i);
      acc.x = fmaf(w.w[k], v.x, acc.x);
      acc.y = fmaf(w.w[k], v.y, acc.y);
      acc.z = fmaf(w.w[k], v.z, acc.z);
      acc.w = fmaf(w.w[k], v.w, acc.w);
    }
    reinterpret_cast<float4*>(sum)[i] = acc;
  }
}
__global__ void __launch_bounds__(256) broadcast_rows_kernel(const float* __restrict__ sum, int K, int64_t P4,
                                                             float* __restrict__ params) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < P4; i += stride) {
    const float4 v = reinterpret_cast<const float4*>(sum)[i];
    for (int k = 0; k < K; ++k) __stcs(reinterpret_cast<float4*>(params) + (size_t)k * P4 + i, v);
  }
}

// Clients with different adapter ranks (Sec. V, heterogeneous configuration): every client is stored
// at the configured rank r with the components it does not have equal to zero.  The arena of client
// i is a sequence of (A [r, d], B [d, r]) pairs; this kernel zeroes rank components >= rank[i]
// (rows of A, columns of B), e.g. after the average of Eq. 8-9 has been written back to everyone.
struct ClientRanks { int r[AGG_MAX_CLIENTS]; };
__global__ void rank_mask_kernel(float* __restrict__ p, int64_t n, int64_t P, int r, int d, ClientRanks ranks) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n) return;
  const int client = (int)(e / P);
  const int64_t off = (e % P) % (2 * (int64_t)r * d);
  const int j = off < (int64_t)r * d ? (int)(off / d) : (int)((off - (int64_t)r * d) % r);
  if (j >= ranks.r[client]) p[e] = 0.f;
}

cudaError_t rank_mask(float* params, int K, int64_t P, int r, int d, const int* ranks_host, cudaStream_t st) {
  if (K < 1 || K > AGG_MAX_CLIENTS || P < 1 || r < 1 || d < 1 || P % (2 * (int64_t)r * d) != 0) return cudaErrorInvalidValue;
  ClientRanks ranks;
  for (int k = 0; k < AGG_MAX_CLIENTS; ++k) ranks.r[k] = k < K ? ranks_host[k] : r;
  const int64_t n = (int64_t)K * P;
  rank_mask_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(params, n, P, r, d, ranks);
  return cudaGetLastError();
}

cudaError_t aggregate(float* params, int K, int64_t P, const float* w_host, cudaStream_t st, int64_t row_stride) {
  if (row_stride == 0) row_stride = P;
  if (K < 1 || K > AGG_MAX_CLIENTS || P % 4 != 0 || row_stride % 4 != 0 || row_stride < P) return cudaErrorInvalidValue;
  AggWeights w;
  for (int k = 0; k < AGG_MAX_CLIENTS; ++k) w.w[k] = k < K ? w_host[k] : 0.f;
  int64_t P4 = P / 4;
  int64_t blocks = (P4 + 255) / 256;
  const int64_t cap = 148 * 8;      // a few resident blocks per SM, grid-stride beyond that
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  aggregate_kernel<<<(unsigned)blocks, 256, 0, st>>>(params, K, P4, row_stride / 4, w);
  return cudaGetLastError();
}

static unsigned agg_blocks(int64_t P4) {
  int64_t blocks = (P4 + 255) / 256;
  const int64_t cap = 148 * 8;
  if (blocks > cap) blocks = cap;
  return (unsigned)(blocks < 1 ? 1 : blocks);
}

cudaError_t aggregate_local_sum(const float* params, int K, int64_t P, const float* w_host, float* sum, cudaStream_t st) {
  if (K < 1 || K > AGG_MAX_CLIENTS || P % 4 != 0) return cudaErrorInvalidValue;
  AggWeights w;
  for (int k = 0; k < AGG_MAX_CLIENTS; ++k) w.w[k] = k < K ? w_host[k] : 0.f;
  weighted_sum_kernel<<<agg_blocks(P / 4), 256, 0, st>>>(params, K, P / 4, w, sum);
  return cudaGetLastError();
}

cudaError_t aggregate_broadcast(const float* sum, int K, int64_t P, float* params, cudaStream_t st) {
  if (K < 1 || K > AGG_MAX_CLIENTS || P % 4 != 0) return cudaErrorInvalidValue;
  broadcast_rows_kernel<<<agg_blocks(P / 4), 256, 0, st>>>(sum, K, P / 4, params);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// adapter compute copies (only live entries are written; the padding was zeroed once)
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void adapter_copy_kernel(AdapterCopyArgs a) {
  const int64_t nA = (int64_t)a.r * a.d_in, nB = (int64_t)a.r * a.d_out;
  const int64_t per_t = nA + nB;
  const int64_t total = (int64_t)a.G * a.n_targets * per_t;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int g = (int)(idx / (a.n_targets * per_t));
  int64_t rem = idx % (a.n_targets * per_t);
  const int t = (int)(rem / per_t);
  rem = rem % per_t;
  T* Acat = (T*)a.Acat; T* AcatT = (T*)a.AcatT; T* Bext = (T*)a.Bext; T* BextT = (T*)a.BextT;
  if (rem < nA) {
    const int j = (int)(rem / a.d_in), c = (int)(rem % a.d_in);
    const float av = a.A[(size_t)g * a.a_gs + (size_t)t * a.a_ts + (size_t)j * a.d_in + c];
    const int col = t * a.rp + j;
    const size_t base = (size_t)g * a.ext * a.d_in;
    if (Acat) Acat[base + (size_t)col * a.d_in + c] = from_f<T>(av);
    if (AcatT) AcatT[base + (size_t)c * a.ext + col] = from_f<T>(av);
  } else {
    rem -= nA;
    const int c = (int)(rem / a.r), j = (int)(rem % a.r);
    const float bv = a.scale * a.B[(size_t)g * a.b_gs + (size_t)t * a.b_ts + (size_t)c * a.r + j];
    const int col = t * a.rp + j;
    const int row = a.slice_off[t] + c;
    const size_t base = (size_t)g * a.n_out * a.ext;
    if (Bext) Bext[base + (size_t)row * a.ext + col] = from_f<T>(bv);
    if (BextT) BextT[base + (size_t)col * a.n_out + row] = from_f<T>(bv);
  }
}

cudaError_t refresh_adapter_copies(const AdapterCopyArgs& a, cudaStream_t st) {
  int64_t total = (int64_t)a.G * a.n_targets * a.r * ((int64_t)a.d_in + a.d_out);
  if (total == 0) return cudaSuccess;
  unsigned blocks = (unsigned)((total + 255) / 256);
  if (a.dtype == DT_BF16) adapter_copy_kernel<bf16><<<blocks, 256, 0, st>>>(a);
  else adapter_copy_kernel<float><<<blocks, 256, 0, st>>>(a);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// transpose: out[c, r] = in[r, c], out has leading dimension ldo
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void transpose_kernel(const T* __restrict__ in, int rows, int cols, T* __restrict__ out, int64_t ldo) {
  __shared__ T tile[32][33];
  int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    int r = r0 + i, c = c0 + threadIdx.x;
    if (r < rows && c < cols) tile[i][threadIdx.x] = in[(size_t)r * cols + c];
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    int c = c0 + i, r = r0 + threadIdx.x;
    if (r < rows && c < cols) out[(size_t)c * ldo + r] = tile[threadIdx.x][i];
  }
}

cudaError_t transpose(int dt, const void* in, int rows, int cols, void* out, int64_t ldo, cudaStream_t st) {
  dim3 grid((cols + 31) / 32, (rows + 31) / 32), block(32, 8);
  if (dt == DT_BF16) transpose_kernel<bf16><<<grid, block, 0, st>>>((const bf16*)in, rows, cols, (bf16*)out, ldo);
  else transpose_kernel<float><<<grid, block, 0, st>>>((const float*)in, rows, cols, (float*)out, ldo);
  return cudaGetLastError();
}

}  // namespace sl
