#include "hessian_umma.cuh"
namespace gptq {
bool hessian_umma_supported(int, int64_t) { return false; }
gptq_status_t hessian_umma(float*, const __nv_bfloat16*, int64_t, int, cudaStream_t) { return GPTQ_ERR_UNSUPPORTED; }
}  // namespace gptq
