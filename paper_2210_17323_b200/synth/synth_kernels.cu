// Device-side filler for the seeded synthetic inputs.  It reproduces, bit for bit, the
// host generator in generator.py: a splitmix64 counter hash picks a cell of the same fp32
// normal-quantile table and interpolates with separately rounded fp32 sub / mul / add.
// No step of the quantization method lives here.
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__device__ __forceinline__ float std_normal(uint64_t seed, uint64_t idx, const float* __restrict__ table) {
  uint64_t h = mix64(seed ^ (idx * 0x9E3779B97F4A7C15ull));
  uint32_t k = (uint32_t)(h >> 48);
  float frac = __fmul_rn((float)(uint32_t)((h >> 24) & 0xFFFFFFull), 5.9604644775390625e-08f);
  float t0 = table[k];
  float d = __fsub_rn(table[k + 1], t0);
  return __fadd_rn(t0, __fmul_rn(d, frac));
}

__global__ void fill_x_kernel(__nv_bfloat16* __restrict__ X, int64_t n_tokens, int C, int64_t t0,
                              uint64_t seed, const float* __restrict__ table, const float* __restrict__ scales) {
  int64_t total = n_tokens * C;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    int c = (int)(e % C);
    float z = std_normal(seed, (uint64_t)(t0 * C + e), table);
    X[e] = __float2bfloat16_rn(__fmul_rn(z, scales[c]));
  }
}

__global__ void fill_w_kernel(__half* __restrict__ W, int64_t total, int64_t e0, uint64_t seed,
                              const float* __restrict__ table) {
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x)
    W[e] = __float2half_rn(__fmul_rn(std_normal(seed, (uint64_t)(e0 + e), table), 0.02f));
}

}  // namespace

// X[t0 : t0 + n_tokens, :] (device, bf16) of the stream `seed`; table = 65537 floats, scales = C floats (device).
extern "C" int synth_fill_x_bf16(void* X, int64_t n_tokens, int C, int64_t t0, uint64_t seed,
                                 const float* table, const float* scales, void* stream) {
  if (n_tokens <= 0) return 0;
  fill_x_kernel<<<148 * 16, 256, 0, (cudaStream_t)stream>>>((__nv_bfloat16*)X, n_tokens, C, t0, seed, table, scales);
  return (int)cudaGetLastError();
}

// W flat elements [e0, e0 + total) (device, fp16) of the stream `seed`.
extern "C" int synth_fill_w_fp16(void* W, int64_t total, int64_t e0, uint64_t seed, const float* table, void* stream) {
  if (total <= 0) return 0;
  fill_w_kernel<<<148 * 16, 256, 0, (cudaStream_t)stream>>>((__half*)W, total, e0, seed, table);
  return (int)cudaGetLastError();
}
