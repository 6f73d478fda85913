// Shared host/device helpers of the GPTQ B200 library (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/gptq_b200.h"

namespace gptq {

constexpr size_t kAlign = 256;

inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

// Carves 256-byte aligned pieces out of the caller's workspace; with base == nullptr it only measures.
struct WsCarver {
  char* base;
  size_t off = 0;
  explicit WsCarver(void* b) : base(static_cast<char*>(b)) {}
  template <class T>
  T* take(size_t count) {
    size_t o = off;
    off = align_up(off + count * sizeof(T));
    return base ? reinterpret_cast<T*>(base + o) : nullptr;
  }
};

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

#define GPTQ_CUDA_TRY(expr)                           \
  do {                                                \
    cudaError_t _e = (expr);                          \
    if (_e != cudaSuccess) return GPTQ_ERR_CUDA;      \
  } while (0)

// Number of kernels this library has launched in this process (diagnostic, see gptq_launch_count()).
void count_launch(int n = 1);

// Placed after every kernel launch: counts it and surfaces launch-configuration errors.
#define GPTQ_LAUNCH_CHECK()                 \
  do {                                      \
    ::gptq::count_launch();                 \
    GPTQ_CUDA_TRY(cudaGetLastError());      \
  } while (0)

// dev_info word layout: [0] status, [1] detail (pivot index, ...).  First error wins.
__device__ __forceinline__ void report_error(int* dev_info, int status, int detail) {
  if (dev_info && atomicCAS(dev_info, 0, status) == 0) dev_info[1] = detail;
}

// largest power of two <= x (x > 0, finite); 1 for anything else
__device__ __forceinline__ float pow2_floor(float x) {
  if (!(x > 0.f) || !isfinite(x)) return 1.f;
  int e;
  frexpf(x, &e);                       // x = m 2^e, m in [0.5, 1)
  e = max(-100, min(100, e - 1));
  return ldexpf(1.f, e);
}
// power of two s with s * x in [2^(top-1), 2^top) (x > 0, finite); 1 for anything else
__device__ __forceinline__ float pow2_scale_to(float x, int top) {
  if (!(x > 0.f) || !isfinite(x)) return 1.f;
  int e;
  frexpf(x, &e);
  e = max(-100, min(100, top - e));
  return ldexpf(1.f, e);
}
__device__ __forceinline__ int ceil_div_d(int a, int b) { return (a + b - 1) / b; }
inline int ceil_div(int64_t a, int64_t b) { return static_cast<int>((a + b - 1) / b); }

}  // namespace gptq
