// Adapter gradients G_A, G_B (Eq. 4-7): skinny reductions over the tokens of each group,
//   out[g][t][jj][c] = scale * sum_{m in group g} Wt[m, wcol0 + t*rp + jj] * Z[m, zcol0 + c]
// for nt targets of rank r (R = nt*r weight columns) and C feature columns.  HBM-bound: Z is read
// once per 4 weight columns.  A block is 64 column threads (one 16-byte vector each) x 4 row lanes
// over a chunk of LG_ROWS rows, four blocks per SM so that enough loads are in flight; the row
// lanes are summed through shared memory, chunk partials go to scratch and a second kernel adds
// them in chunk order (no float atomics, so the result does not depend on scheduling).
#include "common.cuh"
#include "kernels.h"

namespace sl {
namespace {

constexpr int LG_ROWS = 128;   // rows per chunk; group sizes must be multiples of it
constexpr int LG_CT = 64;      // column threads per block
constexpr int LG_RL = 4;       // row lanes per block
constexpr int RJ = 4;          // weight columns per block

// four consecutive weights of one row
template <typename T> __device__ __forceinline__ void load4(const T* p, float* w);
template <> __device__ __forceinline__ void load4<float>(const float* p, float* w) {
  float4 v = *reinterpret_cast<const float4*>(p);
  w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
}
template <> __device__ __forceinline__ void load4<bf16>(const bf16* p, float* w) {
  uint2 v = *reinterpret_cast<const uint2*>(p);
  const bf16* b = reinterpret_cast<const bf16*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) w[i] = __bfloat162float(b[i]);
}

template <typename T, bool VEC4>
__global__ void __launch_bounds__(LG_CT * LG_RL, 4)
lora_grad_partial_kernel(const T* __restrict__ Z, int64_t ldz, int zcol0, int C, const T* __restrict__ Wt,
                         int64_t ldwt, int wcol0, int r, int rp, int R, int M, float* __restrict__ partial) {
  constexpr int N = Vec16<T>::N;
  __shared__ float red[RJ * N][LG_CT];
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int c = (blockIdx.x * LG_CT + tx) * N;
  const int chunk = blockIdx.y;
  const int j0 = blockIdx.z * RJ;
  const int m0 = chunk * LG_ROWS;
  const int m1 = min(m0 + LG_ROWS, M);
  const bool active = c < C;
  int wc[RJ];
#pragma unroll
  for (int j = 0; j < RJ; ++j) {
    int jj = j0 + j;
    wc[j] = jj < R ? wcol0 + (jj / r) * rp + (jj % r) : -1;
  }
  float acc[RJ][N];
#pragma unroll
  for (int j = 0; j < RJ; ++j)
#pragma unroll
    for (int i = 0; i < N; ++i) acc[j][i] = 0.f;
  if (active) {
#pragma unroll 4
    for (int m = m0 + ty; m < m1; m += LG_RL) {
      Vec16<T> v; v.load(Z + (size_t)m * ldz + zcol0 + c);
      float w[RJ];
      if (VEC4) {
        load4<T>(Wt + (size_t)m * ldwt + wc[0], w);     // r % 4 == 0: the four columns are adjacent
      } else {
#pragma unroll
        for (int j = 0; j < RJ; ++j) w[j] = wc[j] >= 0 ? to_f<T>(Wt[(size_t)m * ldwt + wc[j]]) : 0.f;
      }
#pragma unroll
      for (int i = 0; i < N; ++i) {
        float zv = v.get(i);
#pragma unroll
        for (int j = 0; j < RJ; ++j) acc[j][i] = fmaf(w[j], zv, acc[j][i]);
      }
    }
  }
  // add row lanes 1..3 into lane 0, one lane at a time (fixed order)
  for (int lane = 1; lane < LG_RL; ++lane) {
    if (ty == lane) {
#pragma unroll
      for (int j = 0; j < RJ; ++j)
#pragma unroll
        for (int i = 0; i < N; ++i) red[j * N + i][tx] = acc[j][i];
    }
    __syncthreads();
    if (ty == 0) {
#pragma unroll
      for (int j = 0; j < RJ; ++j)
#pragma unroll
        for (int i = 0; i < N; ++i) acc[j][i] += red[j * N + i][tx];
    }
    __syncthreads();
  }
  if (ty == 0 && active) {
    // partial layout: [chunk][R][C]
#pragma unroll
    for (int j = 0; j < RJ; ++j) {
      if (j0 + j < R) {
        float* p = partial + ((size_t)chunk * R + (j0 + j)) * C + c;
#pragma unroll
        for (int i = 0; i < N; i += 4)
          *reinterpret_cast<float4*>(p + i) = make_float4(acc[j][i], acc[j][i + 1], acc[j][i + 2], acc[j][i + 3]);
      }
    }
  }
}

// Many outputs (wide models): one output per thread; the chunk partials of a group are added in chunk order (adjacent threads
// read adjacent floats of every partial, so the reads coalesce; no shared memory, no barrier).
constexpr int RED_THREADS = 256;
__global__ void __launch_bounds__(RED_THREADS)
lora_grad_reduce_kernel(const float* __restrict__ partial, int r, int R, int C, int chunks_per_group, float scale,
                        float* __restrict__ out, int64_t out_group_stride, int64_t out_target_stride,
                        int64_t out_sj, int64_t out_sc) {
  const int idx = blockIdx.x * RED_THREADS + threadIdx.x;   // over R*C
  const int g = blockIdx.y;
  if (idx >= R * C) return;
  const size_t rc = (size_t)R * C;
  const float* p = partial + (size_t)g * chunks_per_group * rc + idx;
  float s = 0.f;
#pragma unroll 4
  for (int k = 0; k < chunks_per_group; ++k) s += p[(size_t)k * rc];
  const int j = idx / C, c = idx % C;
  out[(size_t)g * out_group_stride + (size_t)(j / r) * out_target_stride + (size_t)(j % r) * out_sj +
      (size_t)c * out_sc] = scale * s;
}

// Few outputs, many chunks (narrow models, long groups): 32 outputs per block (threadIdx.x) and
// RED_LANES chunk lanes (threadIdx.y), each adding every RED_LANES-th partial, combined in lane order.
constexpr int RED_LANES = 8;
__global__ void __launch_bounds__(32 * RED_LANES)
lora_grad_reduce_lanes_kernel(const float* __restrict__ partial, int r, int R, int C, int chunks_per_group, float scale,
                        float* __restrict__ out, int64_t out_group_stride, int64_t out_target_stride,
                        int64_t out_sj, int64_t out_sc) {
  __shared__ float red[RED_LANES][32];
  const int idx = blockIdx.x * 32 + threadIdx.x;   // over R*C
  const int g = blockIdx.y;
  const bool active = idx < R * C;
  float s = 0.f;
  if (active) {
    const float* p = partial + (size_t)g * chunks_per_group * R * C + idx;
    for (int k = threadIdx.y; k < chunks_per_group; k += RED_LANES) s += p[(size_t)k * R * C];
  }
  red[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0 && active) {
    float t = 0.f;
#pragma unroll
    for (int l = 0; l < RED_LANES; ++l) t += red[l][threadIdx.x];
    const int j = idx / C, c = idx % C;
    out[(size_t)g * out_group_stride + (size_t)(j / r) * out_target_stride + (size_t)(j % r) * out_sj +
        (size_t)c * out_sc] = scale * t;
  }
}

// The second kernel for a batch of jobs (blockIdx.z): one output per thread, chunks added in order.
struct RedJob { const float* partial; float* out; int r, R; float scale; int64_t ogs, ots, osj, osc; };
struct RedBatch { RedJob j[4]; };
__global__ void __launch_bounds__(RED_THREADS)
lora_grad_reduce_batch_kernel(RedBatch b, int C, int chunks_per_group) {
  const RedJob& jb = b.j[blockIdx.z];
  const int idx = blockIdx.x * RED_THREADS + threadIdx.x;   // over R*C
  const int g = blockIdx.y;
  if (idx >= jb.R * C) return;
  const size_t rc = (size_t)jb.R * C;
  const float* p = jb.partial + (size_t)g * chunks_per_group * rc + idx;
  float s = 0.f;
#pragma unroll 4
  for (int k = 0; k < chunks_per_group; ++k) s += p[(size_t)k * rc];
  const int j = idx / C, c = idx % C;
  jb.out[(size_t)g * jb.ogs + (size_t)(j / jb.r) * jb.ots + (size_t)(j % jb.r) * jb.osj + (size_t)c * jb.osc] = jb.scale * s;
}

// picks the second kernel by the number of outputs (both add in a fixed order)
void launch_reduce(const float* partial, int r, int R, int C, int cpg, int groups, float scale, float* out,
                   int64_t out_group_stride, int64_t out_target_stride, int64_t out_sj, int64_t out_sc, cudaStream_t st) {
  if ((int64_t)R * C >= 32768) {
    dim3 g2((R * C + RED_THREADS - 1) / RED_THREADS, groups), b2(RED_THREADS);
    lora_grad_reduce_kernel<<<g2, b2, 0, st>>>(partial, r, R, C, cpg, scale, out, out_group_stride, out_target_stride, out_sj, out_sc);
  } else {
    dim3 g2((R * C + 31) / 32, groups), b2(32, RED_LANES);
    lora_grad_reduce_lanes_kernel<<<g2, b2, 0, st>>>(partial, r, R, C, cpg, scale, out, out_group_stride, out_target_stride, out_sj, out_sc);
  }
}

template <typename T>
void launch_partial(dim3 grid, cudaStream_t st, bool vec4, const void* Z, int64_t ldz, int zcol0, int C, const void* Wt,
                    int64_t ldwt, int wcol0, int r, int rp, int R, int M, float* partial) {
  dim3 block(LG_CT, LG_RL);
  if (vec4)
    lora_grad_partial_kernel<T, true><<<grid, block, 0, st>>>((const T*)Z, ldz, zcol0, C, (const T*)Wt, ldwt, wcol0, r, rp, R, M, partial);
  else
    lora_grad_partial_kernel<T, false><<<grid, block, 0, st>>>((const T*)Z, ldz, zcol0, C, (const T*)Wt, ldwt, wcol0, r, rp, R, M, partial);
}

}  // namespace

size_t lora_grad_scratch_floats(int M, int R, int C) {
  size_t chunks = (size_t)(M + LG_ROWS - 1) / LG_ROWS;
  return chunks * (size_t)R * (size_t)C;
}

cudaError_t lora_grad(int dt, const void* Z, int64_t ldz, int zcol0, int C, const void* Wt, int64_t ldwt, int wcol0,
                      int r, int rp, int nt, int M, int rows_per_group, float scale, float* out,
                      int64_t out_group_stride, int64_t out_target_stride, int64_t out_sj, int64_t out_sc,
                      float* partial, cudaStream_t st, int* status, bool use_tc) {
  if (use_tc && status && dt == DT_BF16 && (rp == 16 || rp == 32 || rp == 64)) {
    // tensor-core path, in windows of the targets whose weight columns share one 64-column tile
    const int tw = 64 / rp;
    bool ok = true;
    for (int t0 = 0; t0 < nt && ok; t0 += tw)
      ok = lora_grad_tc_supported(dt, Z, ldz, zcol0, C, Wt, ldwt, wcol0 + t0 * rp, r, rp, min(tw, nt - t0), M,
                                  rows_per_group);
    if (ok) {
      const int groups = rows_per_group > 0 && rows_per_group < M ? M / rows_per_group : 1;
      for (int t0 = 0; t0 < nt; t0 += tw) {
        const int ntw = min(tw, nt - t0), Rw = ntw * r;
        int cpg = 0;
        cudaError_t e = lora_grad_tc_partial(Z, ldz, zcol0, C, Wt, ldwt, wcol0 + t0 * rp, r, rp, ntw, M, rows_per_group,
                                             partial, status, &cpg, st);
        if (e != cudaSuccess) return e;
        launch_reduce(partial, r, Rw, C, cpg, groups, scale, out + (size_t)t0 * out_target_stride, out_group_stride,
                      out_target_stride, out_sj, out_sc, st);
      }
      return cudaGetLastError();
    }
  }
  const int R = nt * r;
  const int rpg = rows_per_group > 0 ? rows_per_group : M;
  const int n = dt == DT_BF16 ? 8 : 4;
  const int chunks = (M + LG_ROWS - 1) / LG_ROWS;
  int chunks_per_group, groups;
  if (rpg >= M) { groups = 1; chunks_per_group = chunks; }
  else {
    if (rpg % LG_ROWS != 0 || M % rpg != 0) return cudaErrorInvalidValue;   // chunks must not straddle groups
    groups = M / rpg; chunks_per_group = rpg / LG_ROWS;
  }
  if (C % n != 0 || R < 1) return cudaErrorInvalidValue;
  // vector loads of four adjacent weights need r % 4 == 0 and aligned rows / column offsets
  const bool vec4 = (r % 4 == 0) && (wcol0 % 4 == 0) && (rp % 4 == 0) && (ldwt % 4 == 0);
  const int cvec = C / n;
  dim3 grid((cvec + LG_CT - 1) / LG_CT, chunks, (R + RJ - 1) / RJ);
  if (dt == DT_BF16) launch_partial<bf16>(grid, st, vec4, Z, ldz, zcol0, C, Wt, ldwt, wcol0, r, rp, R, M, partial);
  else launch_partial<float>(grid, st, vec4, Z, ldz, zcol0, C, Wt, ldwt, wcol0, r, rp, R, M, partial);
  launch_reduce(partial, r, R, C, chunks_per_group, groups, scale, out, out_group_stride, out_target_stride, out_sj,
                out_sc, st);
  return cudaGetLastError();
}

cudaError_t lora_grad_batch(int dt, const LoraGradJob* jobs, int njobs, int M, int rows_per_group, float* partial,
                            size_t partial_floats, cudaStream_t st, int* status, bool use_tc) {
  bool batched = use_tc && status && dt == DT_BF16 && njobs >= 1 && njobs <= 4;
  for (int j = 0; j < njobs && batched; ++j) {
    const LoraGradJob& jb = jobs[j];
    batched = jb.C == jobs[0].C && (jb.rp == 16 || jb.rp == 32 || jb.rp == 64) &&
              lora_grad_tc_supported(dt, jb.Z, jb.ldz, jb.zcol0, jb.C, jb.Wt, jb.ldwt, jb.wcol0, jb.r, jb.rp, jb.nt, M, rows_per_group);
  }
  if (batched) {
    const int groups = rows_per_group > 0 && rows_per_group < M ? M / rows_per_group : 1;
    int cpg = 0;
    size_t offs[4];
    cudaError_t e = lora_grad_tc_partial_batch(jobs, njobs, M, rows_per_group, partial, partial_floats, status, &cpg, offs, st);
    if (e == cudaSuccess) {
      RedBatch rb;
      int maxRC = 0;
      for (int j = 0; j < 4; ++j) {
        const LoraGradJob& jb = jobs[j < njobs ? j : 0];
        rb.j[j] = {partial + offs[j < njobs ? j : 0], jb.out, jb.r, jb.nt * jb.r, jb.scale, jb.out_group_stride,
                   jb.out_target_stride, jb.out_sj, jb.out_sc};
        if (j < njobs && jb.nt * jb.r * jb.C > maxRC) maxRC = jb.nt * jb.r * jb.C;
      }
      dim3 g2((maxRC + RED_THREADS - 1) / RED_THREADS, groups, njobs);
      lora_grad_reduce_batch_kernel<<<g2, RED_THREADS, 0, st>>>(rb, jobs[0].C, cpg);
      return cudaGetLastError();
    }
    if (e != cudaErrorInvalidValue) return e;      // invalid value: the scratch does not hold the batch, go one by one
  }
  for (int j = 0; j < njobs; ++j) {
    const LoraGradJob& jb = jobs[j];
    cudaError_t e = lora_grad(dt, jb.Z, jb.ldz, jb.zcol0, jb.C, jb.Wt, jb.ldwt, jb.wcol0, jb.r, jb.rp, jb.nt, M, rows_per_group,
                              jb.scale, jb.out, jb.out_group_stride, jb.out_target_stride, jb.out_sj, jb.out_sc, partial, st,
                              status, use_tc);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace sl
