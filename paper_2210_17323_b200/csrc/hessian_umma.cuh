// Tensor-core (tcgen05 / TMEM / TMA) path of the Hessian accumulation; see hessian_umma.cu.
#pragma once
#include "common.cuh"

namespace gptq {
bool hessian_umma_supported(int C, int64_t n_tokens);
// mirror: copy the upper triangle onto the lower one afterwards (false: the strictly lower triangle is left as it is)
gptq_status_t hessian_umma(float* H, const __nv_bfloat16* X, int64_t n_tokens, int C, int* dev_info,
                           cudaStream_t stream, bool mirror = true);

cudaError_t launch_mirror_upper_to_lower(float* H, int C, cudaStream_t stream);
}  // namespace gptq
