// Status strings and diagnostics of the C ABI.
#include <atomic>

#include "common.cuh"

namespace gptq {
static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
}  // namespace gptq

namespace gptq {
cudaError_t hessian_set_wait_test_knobs(unsigned long long limit_ns, int skip_item);
cudaError_t hinv_set_wait_test_knobs(unsigned long long limit_ns, int skip_item);
cudaError_t quantize_set_wait_test_knobs(unsigned long long limit_ns, int skip_item);
}  // namespace gptq

extern "C" gptq_status_t gptq_debug_wait_test(uint64_t wait_limit_ns, int skip_loads_of_item) {
  const unsigned long long lim = wait_limit_ns ? wait_limit_ns : 4000000000ull;
  if (gptq::hessian_set_wait_test_knobs(lim, skip_loads_of_item) != cudaSuccess ||
      gptq::hinv_set_wait_test_knobs(lim, skip_loads_of_item) != cudaSuccess ||
      gptq::quantize_set_wait_test_knobs(lim, skip_loads_of_item) != cudaSuccess)
    return GPTQ_ERR_CUDA;
  return GPTQ_OK;
}

extern "C" uint64_t gptq_launch_count(void) { return gptq::g_launches.load(std::memory_order_relaxed); }

extern "C" const char* gptq_status_string(gptq_status_t status) {
  switch (status) {
    case GPTQ_OK: return "GPTQ_OK";
    case GPTQ_ERR_INVALID_ARG: return "GPTQ_ERR_INVALID_ARG";
    case GPTQ_ERR_UNSUPPORTED: return "GPTQ_ERR_UNSUPPORTED";
    case GPTQ_ERR_NOT_PD: return "GPTQ_ERR_NOT_PD";
    case GPTQ_ERR_WORKSPACE: return "GPTQ_ERR_WORKSPACE";
    case GPTQ_ERR_CUDA: return "GPTQ_ERR_CUDA";
    case GPTQ_ERR_TIMEOUT: return "GPTQ_ERR_TIMEOUT";
    case GPTQ_ERR_NONFINITE: return "GPTQ_ERR_NONFINITE";
  }
  return "GPTQ_ERR_UNKNOWN";
}
