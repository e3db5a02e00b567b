// Tensor-core causal attention (bf16).  Placeholder until the kernels land: reports "unsupported"
// so that callers use the plain-FMA kernels.
#include "common.cuh"
#include "kernels.h"

namespace sl {
bool attention_tc_supported(int, int, int, int) { return false; }
cudaError_t attention_fwd_tc(const void*, int, int, int, int, void*, float*, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t attention_bwd_tc(const void*, const void*, const float*, const void*, int, int, int, int, void*, float*,
                             cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace sl
