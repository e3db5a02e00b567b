// Stand-alone operator entry points of the C ABI: the grouped LoRA linear layer (forward and
// backward), transposes, raw-buffer aggregation and attention.  Used by kernel-level parity tests
// and by the micro-benchmark sweeps.  Host code only.
#include <cuda_runtime.h>

#include "../../include/splitlora.h"
#include "host_common.h"
#include "kernels.h"

using namespace sl;

namespace {
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct LinearPlan {
  int rp, ext;
  size_t off_acat, off_acatT, off_bext, off_bextT, off_h, off_dh, off_scratch, off_status, total;
};

LinearPlan plan_linear(int dtype, int M, int n_in, int n_out, int r, int G) {
  LinearPlan p;
  const size_t es = dtype_size(dtype);
  p.rp = (int)align_up((size_t)r, 16);
  p.ext = (int)align_up((size_t)p.rp, EXT_BLOCK);
  size_t off = 0;
  auto take = [&](size_t bytes) { off = align_up(off, 256); size_t o = off; off += bytes; return o; };
  p.off_status = take(256);
  p.off_acat = take((size_t)G * p.ext * n_in * es);
  p.off_acatT = take((size_t)G * n_in * p.ext * es);
  p.off_bext = take((size_t)G * n_out * p.ext * es);
  p.off_bextT = take((size_t)G * p.ext * n_out * es);
  p.off_h = take((size_t)M * p.ext * es);
  p.off_dh = take((size_t)M * p.ext * es);
  size_t sc = lora_grad_scratch_floats(M, r, n_in > n_out ? n_in : n_out);
  p.off_scratch = take(sc * 4);
  p.total = align_up(off, 256);
  return p;
}

int check_linear(int dtype, int M, int n_in, int n_out, int r, int G) {
  if (dtype != DT_F32 && dtype != DT_BF16) return SPLITLORA_ERR_ARG;
  if (M < 1 || n_in < 8 || n_out < 8 || r < 1 || r > 64 || G < 1 || M % G != 0) return SPLITLORA_ERR_ARG;
  if (n_in % 8 != 0 || n_out % 8 != 0) return SPLITLORA_ERR_ARG;
  if (G > 1 && (M / G) % 128 != 0) return SPLITLORA_ERR_ARG;
  return SPLITLORA_OK;
}

cudaError_t run_gemm(int use_tc, const GemmArgs& a, int* status, cudaStream_t st) {
  if (use_tc && a.dtype == DT_BF16 && gemm_tc_supported(a)) return gemm_tc(a, status, st);
  return gemm_simt(a, st);
}
}  // namespace

extern "C" {

int splitlora_lora_linear_workspace_bytes(int dtype, int M, int n_in, int n_out, int r, int G, size_t* bytes) {
  if (!bytes) return SPLITLORA_ERR_ARG;
  int rc = check_linear(dtype, M, n_in, n_out, r, G);
  if (rc) return rc;
  *bytes = plan_linear(dtype, M, n_in, n_out, r, G).total;
  return SPLITLORA_OK;
}

static int make_copies(int dtype, const LinearPlan& p, const float* A, const float* B, float alpha, int n_in,
                       int n_out, int r, int G, char* ws, bool fwd, cudaStream_t st) {
  const size_t es = dtype_size(dtype);
  AdapterCopyArgs a;
  a.dtype = dtype;
  a.A = A; a.a_gs = (int64_t)r * n_in; a.a_ts = 0;
  a.B = B; a.b_gs = (int64_t)n_out * r; a.b_ts = 0;
  a.G = G; a.n_targets = 1; a.r = r; a.rp = p.rp; a.d_in = n_in; a.d_out = n_out; a.n_out = n_out; a.ext = p.ext;
  for (int t = 0; t < 4; ++t) a.slice_off[t] = 0;
  a.scale = alpha / (float)r;
  a.Acat = ws + p.off_acat; a.AcatT = fwd ? nullptr : ws + p.off_acatT;
  a.Bext = fwd ? ws + p.off_bext : nullptr; a.BextT = fwd ? nullptr : ws + p.off_bextT;
  // the padding of the copies must be zero: clear the ones this call uses
  if (cudaMemsetAsync(ws + p.off_acat, 0, (size_t)G * p.ext * n_in * es, st) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  if (fwd) {
    if (cudaMemsetAsync(ws + p.off_bext, 0, (size_t)G * n_out * p.ext * es, st) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  } else {
    if (cudaMemsetAsync(ws + p.off_acatT, 0, (size_t)G * p.ext * n_in * es, st) != cudaSuccess) return SPLITLORA_ERR_CUDA;
    if (cudaMemsetAsync(ws + p.off_bextT, 0, (size_t)G * n_out * p.ext * es, st) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  }
  if (cudaMemsetAsync(ws + p.off_status, 0, 256, st) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  return refresh_adapter_copies(a, st) == cudaSuccess ? SPLITLORA_OK : SPLITLORA_ERR_CUDA;
}

int splitlora_lora_linear_fwd(int dtype, int use_tc, const void* x, const void* W, const void* bias, const float* A,
                              const float* B, float alpha, int M, int n_in, int n_out, int r, int G, void* y,
                              void* workspace, size_t workspace_bytes, void* stream) {
  return splitlora_lora_linear_fwd_parts(dtype, use_tc, x, W, bias, A, B, alpha, M, n_in, n_out, r, G, y, workspace,
                                         workspace_bytes, stream, 3);
}

int splitlora_lora_linear_fwd_parts(int dtype, int use_tc, const void* x, const void* W, const void* bias, const float* A,
                                    const float* B, float alpha, int M, int n_in, int n_out, int r, int G, void* y,
                                    void* workspace, size_t workspace_bytes, void* stream, int parts) {
  int rc = check_linear(dtype, M, n_in, n_out, r, G);
  if (rc) return rc;
  if (parts < 1 || parts > 3) return SPLITLORA_ERR_ARG;
  if (!x || !W || !A || !B || !y || !workspace) return SPLITLORA_ERR_ARG;
  if (!aligned16(x) || !aligned16(W) || !aligned16(y) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return SPLITLORA_ERR_ALIGN;
  LinearPlan p = plan_linear(dtype, M, n_in, n_out, r, G);
  if (workspace_bytes < p.total) return SPLITLORA_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  if (gemm_tc_init() != 0) return SPLITLORA_ERR_CUDA;
  const int rpg = G > 1 ? M / G : 0;
  int* status = (int*)(ws + p.off_status);
  if (parts & 1) {
    if ((rc = make_copies(dtype, p, A, B, alpha, n_in, n_out, r, G, ws, true, st))) return rc;
    GemmArgs h;
    h.dtype = dtype; h.X = x; h.ldx = n_in; h.W = ws + p.off_acat; h.ldw = n_in; h.Y = ws + p.off_h; h.ldy = p.ext;
    h.M = M; h.N = p.ext; h.K = n_in; h.rows_per_group = rpg; h.w_grouped = G > 1;
    if (run_gemm(use_tc, h, status, st) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  }
  if (!(parts & 2)) return SPLITLORA_OK;
  GemmArgs a;
  a.dtype = dtype; a.X = x; a.ldx = n_in; a.W = W; a.ldw = n_in; a.Y = y; a.ldy = n_out;
  a.M = M; a.N = n_out; a.K = n_in; a.bias = bias; a.rows_per_group = rpg;
  a.Xe = ws + p.off_h; a.ldxe = p.ext; a.We = ws + p.off_bext; a.ldwe = p.ext; a.Ke = p.rp; a.we_grouped = G > 1;
  if (run_gemm(use_tc, a, status, st) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  return SPLITLORA_OK;
}

int splitlora_lora_linear_bwd(int dtype, int use_tc, const void* x, const void* Wt, const void* dy, const float* A,
                              const float* B, float alpha, int M, int n_in, int n_out, int r, int G, void* dx,
                              float* dA, float* dB, void* workspace, size_t workspace_bytes, void* stream) {
  return splitlora_lora_linear_bwd_parts(dtype, use_tc, x, Wt, dy, A, B, alpha, M, n_in, n_out, r, G, dx, dA, dB, workspace,
                                         workspace_bytes, stream, 7);
}

int splitlora_lora_linear_bwd_parts(int dtype, int use_tc, const void* x, const void* Wt, const void* dy, const float* A,
                                    const float* B, float alpha, int M, int n_in, int n_out, int r, int G, void* dx,
                                    float* dA, float* dB, void* workspace, size_t workspace_bytes, void* stream, int parts) {
  int rc = check_linear(dtype, M, n_in, n_out, r, G);
  if (rc) return rc;
  if (parts < 1 || parts > 7) return SPLITLORA_ERR_ARG;
  if (!x || !Wt || !dy || !A || !B || !dx || !dA || !dB || !workspace) return SPLITLORA_ERR_ARG;
  if (!aligned16(x) || !aligned16(Wt) || !aligned16(dy) || !aligned16(dx) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return SPLITLORA_ERR_ALIGN;
  LinearPlan p = plan_linear(dtype, M, n_in, n_out, r, G);
  if (workspace_bytes < p.total) return SPLITLORA_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  if (gemm_tc_init() != 0) return SPLITLORA_ERR_CUDA;
  if ((rc = make_copies(dtype, p, A, B, alpha, n_in, n_out, r, G, ws, false, st))) return rc;
  const int rpg = G > 1 ? M / G : 0;
  int* status = (int*)(ws + p.off_status);
  const float s = alpha / (float)r;
  if (parts & 1) {
    // h = x A_g^T (recomputed here; the training runtime keeps it from the forward pass)
    GemmArgs h;
    h.dtype = dtype; h.X = x; h.ldx = n_in; h.W = ws + p.off_acat; h.ldw = n_in; h.Y = ws + p.off_h; h.ldy = p.ext;
    h.M = M; h.N = p.ext; h.K = n_in; h.rows_per_group = rpg; h.w_grouped = G > 1;
    if (run_gemm(use_tc, h, status, st) != cudaSuccess) return SPLITLORA_ERR_CUDA;
    // dh = s dy B_g
    GemmArgs g;
    g.dtype = dtype; g.X = dy; g.ldx = n_out; g.W = ws + p.off_bextT; g.ldw = n_out; g.Y = ws + p.off_dh; g.ldy = p.ext;
    g.M = M; g.N = p.ext; g.K = n_out; g.rows_per_group = rpg; g.w_grouped = G > 1;
    if (run_gemm(use_tc, g, status, st) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  }
  if (parts & 2) {
    // dx = dy W + dh A_g
    GemmArgs a;
    a.dtype = dtype; a.X = dy; a.ldx = n_out; a.W = Wt; a.ldw = n_out; a.Y = dx; a.ldy = n_in;
    a.M = M; a.N = n_in; a.K = n_out; a.rows_per_group = rpg;
    a.Xe = ws + p.off_dh; a.ldxe = p.ext; a.We = ws + p.off_acatT; a.ldwe = p.ext; a.Ke = p.rp; a.we_grouped = G > 1;
    if (run_gemm(use_tc, a, status, st) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  }
  if (!(parts & 4)) return SPLITLORA_OK;
  float* scratch = (float*)(ws + p.off_scratch);
  if (lora_grad(dtype, x, n_in, 0, n_in, ws + p.off_dh, p.ext, 0, r, p.rp, 1, M, rpg, 1.0f, dA, (int64_t)r * n_in, 0, n_in, 1,
                scratch, st, status, use_tc != 0) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  if (lora_grad(dtype, dy, n_out, 0, n_out, ws + p.off_h, p.ext, 0, r, p.rp, 1, M, rpg, s, dB, (int64_t)n_out * r, 0, 1, r,
                scratch, st, status, use_tc != 0) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  return SPLITLORA_OK;
}

int splitlora_library_status(int32_t* code) {
  if (!code) return SPLITLORA_ERR_ARG;
  int* word = library_status_word();
  if (!word) return SPLITLORA_ERR_CUDA;
  if (cudaDeviceSynchronize() != cudaSuccess) return SPLITLORA_ERR_CUDA;
  if (cudaMemcpy(code, word, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return SPLITLORA_ERR_CUDA;
  return *code ? SPLITLORA_ERR_TIMEOUT : SPLITLORA_OK;
}

int splitlora_transpose(int dtype, const void* in, int rows, int cols, void* out, void* stream) {
  if (!in || !out || rows < 1 || cols < 1 || (dtype != DT_F32 && dtype != DT_BF16)) return SPLITLORA_ERR_ARG;
  return transpose(dtype, in, rows, cols, out, rows, (cudaStream_t)stream) == cudaSuccess ? SPLITLORA_OK : SPLITLORA_ERR_CUDA;
}

int splitlora_handoff_quantize(int dtype, const void* x, int64_t M, int d, uint8_t* codes, float* scales, void* stream) {
  const int n = dtype == DT_BF16 ? 8 : 4;
  if (!x || !codes || !scales || M < 1 || d < n || d % n != 0 || (dtype != DT_F32 && dtype != DT_BF16)) return SPLITLORA_ERR_ARG;
  if (!aligned16(x) || !aligned16(codes)) return SPLITLORA_ERR_ALIGN;
  return handoff_quantize(dtype, x, M, d, codes, scales, (cudaStream_t)stream) == cudaSuccess ? SPLITLORA_OK : SPLITLORA_ERR_CUDA;
}

int splitlora_handoff_dequantize(int dtype, const uint8_t* codes, const float* scales, int64_t M, int d, void* y,
                                 void* stream) {
  const int n = dtype == DT_BF16 ? 8 : 4;
  if (!y || !codes || !scales || M < 1 || d < n || d % n != 0 || (dtype != DT_F32 && dtype != DT_BF16)) return SPLITLORA_ERR_ARG;
  if (!aligned16(y) || !aligned16(codes)) return SPLITLORA_ERR_ALIGN;
  return handoff_dequantize(dtype, codes, scales, M, d, y, (cudaStream_t)stream) == cudaSuccess ? SPLITLORA_OK : SPLITLORA_ERR_CUDA;
}

int splitlora_aggregate_buffers(float* params, int K, int64_t P, const double* weights, void* stream) {
  if (!params || !weights || K < 1 || K > AGG_MAX_CLIENTS || P < 4 || P % 4 != 0) return SPLITLORA_ERR_ARG;
  if (!aligned16(params)) return SPLITLORA_ERR_ALIGN;
  float w[AGG_MAX_CLIENTS];
  for (int i = 0; i < K; ++i) w[i] = (float)weights[i];
  return aggregate(params, K, P, w, (cudaStream_t)stream) == cudaSuccess ? SPLITLORA_OK : SPLITLORA_ERR_CUDA;
}

int splitlora_attention_fwd(int dtype, int use_tc, const void* qkv, int nseq, int T, int n_head, int d_model, void* o,
                            float* lse, void* stream) {
  if (!qkv || !o || !lse || nseq < 1 || T < 1 || n_head < 1 || d_model % n_head != 0 || d_model / n_head > 128 ||
      (dtype != DT_F32 && dtype != DT_BF16))
    return SPLITLORA_ERR_ARG;
  cudaError_t e;
  if (use_tc && attention_tc_supported(dtype, T, n_head, d_model))
    e = attention_fwd_tc(qkv, nseq, T, n_head, d_model, o, lse, nullptr, (cudaStream_t)stream);
  else
    e = attention_fwd_simt(dtype, qkv, nseq, T, n_head, d_model, o, lse, (cudaStream_t)stream);
  return e == cudaSuccess ? SPLITLORA_OK : SPLITLORA_ERR_CUDA;
}

int splitlora_attention_bwd(int dtype, int use_tc, const void* qkv, const void* o, const float* lse, const void* d_o,
                            int nseq, int T, int n_head, int d_model, void* dqkv, float* rowdot, void* stream) {
  if (!qkv || !o || !lse || !d_o || !dqkv || !rowdot || nseq < 1 || T < 1 || n_head < 1 || d_model % n_head != 0 ||
      d_model / n_head > 128 || (dtype != DT_F32 && dtype != DT_BF16))
    return SPLITLORA_ERR_ARG;
  cudaError_t e;
  if (use_tc && attention_tc_supported(dtype, T, n_head, d_model))
    e = attention_bwd_tc(qkv, o, lse, d_o, nseq, T, n_head, d_model, dqkv, rowdot, nullptr, (cudaStream_t)stream);
  else
    e = attention_bwd_simt(dtype, qkv, o, lse, d_o, nseq, T, n_head, d_model, dqkv, rowdot, (cudaStream_t)stream);
  return e == cudaSuccess ? SPLITLORA_OK : SPLITLORA_ERR_CUDA;
}

}  // extern "C"

// Frozen linear layer with a fused epilogue (steps a4 / a11), stand-alone.
extern "C" int splitlora_linear(int dtype, int use_tc, const void* x, const void* W, const void* bias, int epilogue,
                                const void* r, void* z, int gelu_tanh, int M, int n_in, int n_out, void* y,
                                int* status_word, void* stream) {
  if (!x || !W || !y || M < 1 || n_in < 8 || n_out < 8 || n_in % 8 || n_out % 8 || (dtype != DT_F32 && dtype != DT_BF16))
    return SPLITLORA_ERR_ARG;
  if (epilogue < EPI_BIAS || epilogue > EPI_MUL_GELUGRAD) return SPLITLORA_ERR_ARG;
  if ((epilogue == EPI_BIAS_RESID || epilogue == EPI_MUL_GELUGRAD) && !r) return SPLITLORA_ERR_ARG;
  if (epilogue == EPI_BIAS_GELU && !z) return SPLITLORA_ERR_ARG;
  if (use_tc && dtype == DT_BF16 && !status_word) return SPLITLORA_ERR_ARG;
  if (gemm_tc_init() != 0) return SPLITLORA_ERR_CUDA;
  GemmArgs a;
  a.dtype = dtype; a.X = x; a.ldx = n_in; a.W = W; a.ldw = n_in; a.Y = y; a.ldy = n_out;
  a.M = M; a.N = n_out; a.K = n_in; a.bias = bias; a.epi = epilogue; a.R = r; a.ldr = n_out; a.Z = z; a.ldz = n_out;
  a.gelu_tanh = gelu_tanh;
  return run_gemm(use_tc, a, status_word, (cudaStream_t)stream) == cudaSuccess ? SPLITLORA_OK : SPLITLORA_ERR_CUDA;
}
