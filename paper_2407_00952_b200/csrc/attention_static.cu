// Attention backward for callers that cannot provide scratch memory.
//
// splitlora_attention_bwd needs one float per (sequence, head, position) of scratch for the
// row-wise products sum(dO * O) that the dQ and dK/dV kernels read.  Here that scratch is a fixed
// array inside the library image, so the call neither takes a scratch pointer nor allocates.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/splitlora.h"
#include "kernels.h"

using namespace sl;

namespace {

// One float per (sequence, head, position).  Lives in every CUDA context that loads the library,
// from load until exit (4 MiB per device).
static __device__ __align__(256) float g_rowdot_scratch[SPLITLORA_STATIC_ATTENTION_ROWS];

constexpr int kMaxDevices = 64;
float* g_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_scratch_mutex;

// In host code `g_rowdot_scratch` is only a handle for the runtime, not an address a kernel may
// use; the device address is looked up once per device (with that device current) and cached.
int scratch_address(float** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPLITLORA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_rowdot_scratch) != cudaSuccess || !p) return SPLITLORA_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return SPLITLORA_OK;
}

}  // namespace

extern "C" int splitlora_attention_bwd_static(int dtype, int use_tc, const void* qkv, const void* o, const float* lse,
                                              const void* d_o, int nseq, int T, int n_head, int d_model, void* dqkv,
                                              void* stream) {
  if (!qkv || !o || !lse || !d_o || !dqkv || nseq < 1 || T < 1 || n_head < 1 || d_model % n_head != 0 ||
      d_model / n_head > 128 || (dtype != DT_F32 && dtype != DT_BF16))
    return SPLITLORA_ERR_ARG;
  if ((int64_t)nseq * T * n_head > (int64_t)SPLITLORA_STATIC_ATTENTION_ROWS) return SPLITLORA_ERR_TOO_LARGE;
  float* rowdot = nullptr;
  int rc = scratch_address(&rowdot);
  if (rc) return rc;
  // Every element of the scratch that the dQ / dK,dV kernels read is written first by the row-product
  // kernel of this same call, so nothing has to be cleared between calls.
  cudaError_t e;
  if (use_tc && attention_tc_supported(dtype, T, n_head, d_model))
    e = attention_bwd_tc(qkv, o, lse, d_o, nseq, T, n_head, d_model, dqkv, rowdot, nullptr, (cudaStream_t)stream);
  else
    e = attention_bwd_simt(dtype, qkv, o, lse, d_o, nseq, T, n_head, d_model, dqkv, rowdot, (cudaStream_t)stream);
  return e == cudaSuccess ? SPLITLORA_OK : SPLITLORA_ERR_CUDA;
}
