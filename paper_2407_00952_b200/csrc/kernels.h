// Internal launchers of the split-LoRA kernels.  Host-callable, stream-ordered, no allocation.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace sl {

enum { DT_F32 = 0, DT_BF16 = 1 };
static inline size_t dtype_size(int dt) { return dt == DT_BF16 ? 2 : 4; }

// Epilogues of the linear-layer kernels.
enum Epilogue {
  EPI_BIAS = 0,          // Y = acc + bias
  EPI_BIAS_GELU = 1,     // Z = acc + bias ; Y = gelu(Z)
  EPI_BIAS_RESID = 2,    // Y = acc + bias + R
  EPI_MUL_GELUGRAD = 3   // Y = acc * gelu'(R)           (R holds the saved pre-activation)
};

// Width of one block of the rank-r extension of the contraction (elements).
static const int EXT_BLOCK = 64;

// Y[M,N] = epilogue( X[M,K] W[N,K]^T + Xe[M,Ke] We[N,Ke]^T )
// Rows are split into groups of rows_per_group consecutive rows (0: one group).  A grouped operand
// holds one [N, .] matrix per group, stacked along rows.  The extension term is how the rank-r LoRA
// path enters: Xe is the down-projected activation, We the (scaled) up-projection of the row's group.
struct GemmArgs {
  int dtype = DT_BF16;
  const void* X = nullptr; int64_t ldx = 0;
  const void* W = nullptr; int64_t ldw = 0;
  void* Y = nullptr;       int64_t ldy = 0;
  int M = 0, N = 0, K = 0;
  int w_rows = 0;           // number of valid rows of W (rows >= w_rows read as zero); 0 means N
  int rows_per_group = 0;
  int w_grouped = 0;        // W is [G*N, K]
  const void* bias = nullptr;
  int epi = EPI_BIAS;
  const void* R = nullptr; int64_t ldr = 0;
  void* Z = nullptr;       int64_t ldz = 0;
  int gelu_tanh = 1;
  const void* Xe = nullptr; int64_t ldxe = 0;
  const void* We = nullptr; int64_t ldwe = 0;
  int Ke = 0;               // 0: no extension; else a multiple of 16
  int we_grouped = 0;       // We is [G*N, Ke]
  // Columns [k_gap_begin, k_gap_begin + k_gap_len) of X and W are left out of the contraction (both
  // multiples of 64; K counts the contracted columns only).  Single-CTA tensor-core kernel only.
  int k_gap_begin = 0, k_gap_len = 0;
};

// Plain-FMA tiled kernel, any shape, fp32 or bf16 storage with fp32 accumulation.
cudaError_t gemm_simt(const GemmArgs& a, cudaStream_t st);
// tcgen05 / TMEM / TMA kernel (bf16 only).  Shape rules: M % 128 == 0, K % 64 == 0, N % 8 == 0,
// rows_per_group % 128 == 0, leading dimensions multiples of 8 elements, 16-byte aligned bases.
// status: device word that receives a non-zero code if a bounded wait expires.
bool gemm_tc_supported(const GemmArgs& a);
cudaError_t gemm_tc(const GemmArgs& a, int* status, cudaStream_t st);
int gemm_tc_init();   // resolves the driver entry point for tensor-map encoding; 0 on success

cudaError_t embed(int dt, const int32_t* tokens, const void* wte, const void* wpe, void* out,
                  int M, int T, int d, int vocab, cudaStream_t st);
cudaError_t layernorm_fwd(int dt, const void* x, const void* g, const void* b, void* y, float* mean,
                          float* rstd, int M, int d, float eps, cudaStream_t st);
// dx = resid + dLN(dy)  (resid may be null); gradient w.r.t. the input only.
cudaError_t layernorm_bwd(int dt, const void* dy, const void* x, const void* g, const float* mean,
                          const float* rstd, const void* resid, void* dx, int M, int d, cudaStream_t st);

// Llama-shaped block pieces.  RMSNorm: y = x * rsqrt(mean(x^2) + eps) * g, saves rstd [M];
// backward gives dx = resid + d/dx (resid may be null).
cudaError_t rmsnorm_fwd(int dt, const void* x, const void* g, void* y, float* rstd, int M, int d, float eps,
                        cudaStream_t st);
cudaError_t rmsnorm_bwd(int dt, const void* dy, const void* x, const void* g, const float* rstd, const void* resid,
                        void* dx, int M, int d, cudaStream_t st);
// Rotates the q and k slices of qkv [M, 3d] in place; table [T, d/H/2] of (cos, sin) pairs as
// float2; sign +1 forward, -1 inverse (= gradient).  Needs d/H/2 to be a multiple of the 16-byte
// vector width.
cudaError_t rope_inplace(int dt, void* qkv, const float* table, int M, int T, int H, int d, float sign,
                         cudaStream_t st);
// z [M, 2F] = (gate | up).  act [M, F] = silu(gate) * up;  dz [M, 2F] from dact [M, F].
cudaError_t swiglu_fwd(int dt, const void* z, void* act, int M, int F, cudaStream_t st);
cudaError_t swiglu_bwd(int dt, const void* dact, const void* z, void* dz, int M, int F, cudaStream_t st);

// Cross-entropy over logits [M, ld] (V valid columns): writes per-row losses, then overwrites the
// logits with d loss / d logits (zero in the pad columns) and reduces the mean loss.
// normalizer_override > 0 replaces the count of valid labels (the batch is a shard of a larger one).
cudaError_t cross_entropy(int dt, void* logits, int64_t ld, const int32_t* labels, int M, int V,
                          float* row_loss, int* n_valid, float* loss, int normalizer_override, cudaStream_t st);

// Attention, fused qkv layout [nseq*T, 3d]; heads are contiguous slices of width d/H.
cudaError_t attention_fwd_simt(int dt, const void* qkv, int nseq, int T, int H, int d, void* o, float* lse,
                               cudaStream_t st);
cudaError_t attention_bwd_simt(int dt, const void* qkv, const void* o, const float* lse, const void* d_o,
                               int nseq, int T, int H, int d, void* dqkv, float* rowdot, cudaStream_t st);
// tcgen05 / TMEM attention (bf16, head width 64, T a multiple of 128).  status: device word for the
// code of an expired bounded wait (nullptr: a word inside the library).
bool attention_t5_supported(int dt, int T, int H, int d);
bool attention_fwd_t5_supported(int dt, int T, int H, int d);
bool attention_bwd_t5_128_supported(int dt, int T, int H, int d);
cudaError_t attention_bwd_t5_128(const void* qkv, const float* lse, const void* d_o, const float* rowdot, int nseq,
                                    int T, int H, int d, void* dqkv, int* status, cudaStream_t st);
// head width 64: one softmax thread per row, half-steps of 64 keys (attention_t5_fwd64.cu)
cudaError_t attention_fwd_t5_h64(const void* qkv, int nseq, int T, int H, int d, void* o, float* lse, int* status,
                                 cudaStream_t st);
cudaError_t attention_fwd_t5(const void* qkv, int nseq, int T, int H, int d, void* o, float* lse, int* status,
                             cudaStream_t st);
cudaError_t attention_bwd_t5(const void* qkv, const void* o, const float* lse, const void* d_o, int nseq, int T, int H,
                             int d, void* dqkv, float* rowdot, int* status, cudaStream_t st);
bool attention_tc_supported(int dt, int T, int H, int d);
cudaError_t attention_fwd_tc(const void* qkv, int nseq, int T, int H, int d, void* o, float* lse, int* status,
                             cudaStream_t st);
cudaError_t attention_bwd_tc(const void* qkv, const void* o, const float* lse, const void* d_o, int nseq,
                             int T, int H, int d, void* dqkv, float* rowdot, int* status, cudaStream_t st);

// Adapter gradients: for nt targets of rank r (weight columns wcol0 + t*rp + jj of Wt),
//   out[g][t][jj][c] = scale * sum_{m in group g} Wt[m, wcol0 + t*rp + jj] * Z[m, zcol0 + c],  c < C,
// stored at out + g*out_group_stride + t*out_target_stride + jj*out_sj + c*out_sc.
// rows_per_group (0: one group) must be a multiple of 128.  partial: scratch of at least
// lora_grad_scratch_floats(M, nt*r, C) floats.
size_t lora_grad_scratch_floats(int M, int R, int C);
cudaError_t lora_grad(int dt, const void* Z, int64_t ldz, int zcol0, int C, const void* Wt, int64_t ldwt,
                      int wcol0, int r, int rp, int nt, int M, int rows_per_group, float scale, float* out,
                      int64_t out_group_stride, int64_t out_target_stride, int64_t out_sj, int64_t out_sc,
                      float* partial, cudaStream_t st, int* status = nullptr, bool use_tc = false);
// One reduction of lora_grad as a record, for lora_grad_batch: several of them over the same token rows
// (the adapter gradients of one layer) in one pair of launches.
struct LoraGradJob {
  const void* Z = nullptr; int64_t ldz = 0; int zcol0 = 0, C = 0;
  const void* Wt = nullptr; int64_t ldwt = 0; int wcol0 = 0, r = 0, rp = 0, nt = 1;
  float scale = 1.f; float* out = nullptr;
  int64_t out_group_stride = 0, out_target_stride = 0, out_sj = 0, out_sc = 0;
};
// partial: scratch of partial_floats floats.  Falls back to one lora_grad per job where the batched
// tensor-core path does not apply.
cudaError_t lora_grad_batch(int dt, const LoraGradJob* jobs, int njobs, int M, int rows_per_group, float* partial,
                            size_t partial_floats, cudaStream_t st, int* status, bool use_tc);
cudaError_t lora_grad_tc_partial_batch(const LoraGradJob* jobs, int njobs, int M, int rows_per_group, float* partial,
                                       size_t partial_floats, int* status, int* chunks_per_group, size_t* offsets,
                                       cudaStream_t st);
// The same reduction as a tcgen05 product with both operands MN-major (bf16, rp in {16, 32, 64},
// ldwt a multiple of 64, the wanted weight columns inside one 64-column tile).  Writes per-chunk
// partials [chunk][nt*r][C]; lora_grad adds them.  status: device word for an expired bounded wait.
bool lora_grad_tc_supported(int dt, const void* Z, int64_t ldz, int zcol0, int C, const void* Wt, int64_t ldwt,
                            int wcol0, int r, int rp, int nt, int M, int rows_per_group);
cudaError_t lora_grad_tc_partial(const void* Z, int64_t ldz, int zcol0, int C, const void* Wt, int64_t ldwt, int wcol0,
                                 int r, int rp, int nt, int M, int rows_per_group, float* partial, int* status,
                                 int* chunks_per_group, cudaStream_t st);

struct OptArgs {
  int optimizer; float lr, beta1, beta2, eps, wd; float bc1, bc2;   // bc = 1 - beta^step
};
cudaError_t optimizer_step(float* p, const float* g, float* m, float* v, int64_t n, const OptArgs& o,
                           cudaStream_t st);

// Eq. 8-9 and the write-back: every row of params [K, P] becomes sum_i w[i] params[i, :].
static const int AGG_MAX_CLIENTS = 64;
// zero rank components >= ranks_host[i] in client i's arena of (A [r, d], B [d, r]) pairs (P floats per client)
cudaError_t rank_mask(float* params, int K, int64_t P, int r, int d, const int* ranks_host, cudaStream_t st);
// row_stride: floats between two clients' rows (0: P), so that a column range of a wider arena can be averaged
cudaError_t aggregate(float* params, int K, int64_t P, const float* w_host, cudaStream_t st, int64_t row_stride = 0);
// The same step in two halves, for clients spread over devices: sum [P] = sum_i w[i] params[i, :], and
// (after the caller has added the sums of all devices) every row of params [K, P] = sum.
cudaError_t aggregate_local_sum(const float* params, int K, int64_t P, const float* w_host, float* sum, cudaStream_t st);
cudaError_t aggregate_broadcast(const float* sum, int K, int64_t P, float* params, cudaStream_t st);

// Compute copies of the adapters of one layer (G groups), built from fp32 masters.
// Target t of group g has A_t [r, d_in] at A + g*a_gs + t*a_ts and B_t [d_out, r] at B + g*b_gs + t*b_ts.
// With col = t*rp + j the copies are
//   Acat  [G][ext, d_in]  : Acat[col, c]  = A_t[j, c]          AcatT [G][d_in, ext] : its transpose
//   Bext  [G][n_out, ext] : Bext[slice_off[t] + c, col] = scale * B_t[c, j]
//   BextT [G][ext, n_out] : its transpose
// Only live entries are written; the padding must have been zeroed once.
struct AdapterCopyArgs {
  int dtype;
  const float* A; int64_t a_gs, a_ts;
  const float* B; int64_t b_gs, b_ts;
  int G, n_targets, r, rp, d_in, d_out, n_out, ext;
  int slice_off[4];
  float scale;
  void *Acat, *AcatT, *Bext, *BextT;   // any of them may be null (skipped)
};
cudaError_t refresh_adapter_copies(const AdapterCopyArgs& a, cudaStream_t st);

cudaError_t transpose(int dt, const void* in, int rows, int cols, void* out, int64_t ldo, cudaStream_t st);
// compressed hand-off (handoff.cu): rows of d values <-> d E4M3 codes + one fp32 scale
cudaError_t handoff_quantize(int dt, const void* x, int64_t M, int d, uint8_t* codes, float* scales, cudaStream_t st);
cudaError_t handoff_dequantize(int dt, const uint8_t* codes, const float* scales, int64_t M, int d, void* y,
                               cudaStream_t st);

}  // namespace sl
