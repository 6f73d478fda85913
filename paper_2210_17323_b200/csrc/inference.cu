// Inference-side kernels for the packed format the solver writes (Section 5, "Practical Speedups" and the
// appendix on kernels: a quantized-matrix x fp16-vector product with on-the-fly dequantization, and a
// whole-matrix dequantization).  Both are bound by HBM bandwidth: the matvec reads f bits per weight.
//
// Dequantized value of code q in group gi of row r:  scales[r][gi] * (q - zeros[r][gi]), formed in fp32.
#include "common.cuh"

namespace gptq {
namespace {

// Codes of 32 consecutive columns occupy exactly f consecutive words.  Extracts code i (0..31).
template <int F>
__device__ __forceinline__ uint32_t code_at(const uint32_t (&w)[F], int i) {
  const int bit = i * F, k = bit >> 5, o = bit & 31;
  uint32_t v = w[k] >> o;
  if (o + F > 32 && k + 1 < F) v |= w[k + 1] << (32 - o);
  return v & ((1u << F) - 1u);
}

// ---- whole-matrix dequantization: one thread per 32 columns ------------------------------------
template <int F>
__global__ void dequantize_kernel(const uint32_t* __restrict__ qweight, const float* __restrict__ scales,
                                  const float* __restrict__ zeros, int R, int C, int g, int G,
                                  __half* __restrict__ out) {
  const int chunks = C / 32;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)R * chunks) return;
  const int r = (int)(idx / chunks), ch = (int)(idx % chunks);
  uint32_t w[F];
  const uint32_t* p = qweight + ((int64_t)r * chunks + ch) * F;
#pragma unroll
  for (int k = 0; k < F; ++k) w[k] = p[k];
  __align__(16) __half h[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    const int gi = (ch * 32 + i) / g;
    const float s = scales[(int64_t)r * G + gi], z = zeros[(int64_t)r * G + gi];
    h[i] = __float2half_rn(__fmul_rn(s, (float)code_at<F>(w, i) - z));
  }
  uint4* o = reinterpret_cast<uint4*>(out + (int64_t)r * C + ch * 32);
  const uint4* hv = reinterpret_cast<const uint4*>(h);
#pragma unroll
  for (int k = 0; k < 4; ++k) o[k] = hv[k];
}

// ---- y = dequant(Q) x for one fp16 vector x: one warp per row -------------------------------------
// Lanes take 32-column chunks round-robin.  Per chunk: sq = sum_i q_i x_i, combined with the group's
// scale and zero as  s * (sq - z * sum_i x_i);  the per-chunk sums of x are computed once per CTA.
// x is staged in shared memory as fp32, in 16-byte slots XOR-swizzled by chunk so that the lanes of a
// quarter warp (eight different chunks, same slot) hit eight different bank groups.
// Codes become floats without an integer-to-float conversion: (code | 0x4B000000) is 2^23 + code.
constexpr int kMatvecThreads = 1024;

template <int F>
__global__ void __launch_bounds__(kMatvecThreads)
matvec_kernel(const uint32_t* __restrict__ qweight, const float* __restrict__ scales, const float* __restrict__ zeros,
              const __half* __restrict__ x, int R, int C, int g, int G, float* __restrict__ y) {
  extern __shared__ float4 xs4[];                       // [C/32][8] swizzled
  const int chunks = C / 32;
  float* csum = reinterpret_cast<float*>(xs4 + (size_t)chunks * 8);   // [C/32] sum of x over the chunk
  for (int i = threadIdx.x; i < C / 4; i += blockDim.x) {
    const int ch = i >> 3, j = i & 7;
    const __half2* xp = reinterpret_cast<const __half2*>(x + 4 * i);
    const float2 a = __half22float2(xp[0]), b = __half22float2(xp[1]);
    xs4[ch * 8 + (j ^ (ch & 7))] = make_float4(a.x, a.y, b.x, b.y);
  }
  __syncthreads();
  for (int ch = threadIdx.x; ch < chunks; ch += blockDim.x) {
    float t = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) { const float4 v = xs4[ch * 8 + (j ^ (ch & 7))]; t += (v.x + v.y) + (v.z + v.w); }
    csum[ch] = t;
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
  for (int r = blockIdx.x * wpb + warp; r < R; r += gridDim.x * wpb) {
    const uint32_t* rowp = qweight + (int64_t)r * chunks * F;
    const float* srow = scales + (int64_t)r * G;
    const float* zrow = zeros + (int64_t)r * G;
    float acc = 0.f;
#pragma unroll 2
    for (int ch = lane; ch < chunks; ch += 32) {
      uint32_t w[F];
#pragma unroll
      for (int k = 0; k < F; ++k) w[k] = __ldg(rowp + (int64_t)ch * F + k);
      if (g >= 32) {            // one group covers the chunk
        float sq = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float4 xv = xs4[ch * 8 + (j ^ (ch & 7))];
          sq = fmaf(__uint_as_float(code_at<F>(w, 4 * j) | 0x4B000000u) - 8388608.f, xv.x, sq);
          sq = fmaf(__uint_as_float(code_at<F>(w, 4 * j + 1) | 0x4B000000u) - 8388608.f, xv.y, sq);
          sq = fmaf(__uint_as_float(code_at<F>(w, 4 * j + 2) | 0x4B000000u) - 8388608.f, xv.z, sq);
          sq = fmaf(__uint_as_float(code_at<F>(w, 4 * j + 3) | 0x4B000000u) - 8388608.f, xv.w, sq);
        }
        const int gi = (ch * 32) / g;
        acc = fmaf(srow[gi], sq - zrow[gi] * csum[ch], acc);
      } else {                  // several small groups (4, 8, 16 columns) inside the chunk
        const float* xc = reinterpret_cast<const float*>(xs4 + ch * 8);
#pragma unroll 1
        for (int i0 = 0; i0 < 32; i0 += g) {
          float sq = 0.f, sx = 0.f;
          for (int i = i0; i < i0 + g; ++i) {
            const float xv = xc[(((i >> 2) ^ (ch & 7)) << 2) + (i & 3)];
            sq = fmaf((float)code_at<F>(w, i), xv, sq); sx += xv;
          }
          const int gi = (ch * 32 + i0) / g;
          acc = fmaf(srow[gi], sq - zrow[gi] * sx, acc);
        }
      }
    }
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) y[r] = acc;
  }
}

inline bool group_ok(int C, int g) { return g > 0 && C % g == 0 && (g % 32 == 0 || 32 % g == 0); }

}  // namespace
}  // namespace gptq

template <int F>
gptq_status_t launch_dequantize(const uint32_t* qweight, const float* scales, const float* zeros, int R, int C, int g,
                                int G, __half* out, cudaStream_t s) {
  const int64_t total = (int64_t)R * (C / 32);
  gptq::dequantize_kernel<F><<<(unsigned)((total + 127) / 128), 128, 0, s>>>(qweight, scales, zeros, R, C, g, G, out);
  GPTQ_LAUNCH_CHECK();
  return GPTQ_OK;
}

template <int F>
gptq_status_t launch_matvec(const uint32_t* qweight, const float* scales, const float* zeros, const __half* x, int R,
                            int C, int g, int G, float* y, cudaStream_t s) {
  const size_t smem = (size_t)C * sizeof(float) + (size_t)(C / 32) * sizeof(float);
  const int wpb = gptq::kMatvecThreads / 32;
  int grid = (R + wpb - 1) / wpb;
  if (grid > 148) grid = 148;
  GPTQ_CUDA_TRY(cudaFuncSetAttribute(gptq::matvec_kernel<F>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  gptq::matvec_kernel<F><<<grid, wpb * 32, smem, s>>>(qweight, scales, zeros, x, R, C, g, G, y);
  GPTQ_LAUNCH_CHECK();
  return GPTQ_OK;
}

extern "C" gptq_status_t gptq_dequantize(const uint32_t* qweight, const float* scales, const float* zeros,
                                         int R, int C, int bits, int group_size, void* W_out_fp16, void* stream) {
  using namespace gptq;
  if (!qweight || !scales || !zeros || !W_out_fp16 || R <= 0 || C <= 0 || C % 32 != 0) return GPTQ_ERR_INVALID_ARG;
  const int g = group_size > 0 ? group_size : C;
  if (!group_ok(C, g)) return GPTQ_ERR_UNSUPPORTED;
  const int f = bits == GPTQ_BITS_TERNARY ? 2 : bits, G = C / g;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  __half* out = static_cast<__half*>(W_out_fp16);
  switch (f) {
    case 2: return launch_dequantize<2>(qweight, scales, zeros, R, C, g, G, out, s);
    case 3: return launch_dequantize<3>(qweight, scales, zeros, R, C, g, G, out, s);
    case 4: return launch_dequantize<4>(qweight, scales, zeros, R, C, g, G, out, s);
    case 8: return launch_dequantize<8>(qweight, scales, zeros, R, C, g, G, out, s);
  }
  return GPTQ_ERR_UNSUPPORTED;
}

extern "C" gptq_status_t gptq_matvec(const uint32_t* qweight, const float* scales, const float* zeros,
                                     const void* x_fp16, int R, int C, int bits, int group_size, float* y,
                                     void* stream) {
  using namespace gptq;
  if (!qweight || !scales || !zeros || !x_fp16 || !y || R <= 0 || C <= 0 || C % 32 != 0) return GPTQ_ERR_INVALID_ARG;
  const int g = group_size > 0 ? group_size : C;
  if (!group_ok(C, g)) return GPTQ_ERR_UNSUPPORTED;
  if (C > 51200) return GPTQ_ERR_UNSUPPORTED;   // x is staged in shared memory (4 bytes per column)
  const int f = bits == GPTQ_BITS_TERNARY ? 2 : bits, G = C / g;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half* x = static_cast<const __half*>(x_fp16);
  switch (f) {
    case 2: return launch_matvec<2>(qweight, scales, zeros, x, R, C, g, G, y, s);
    case 3: return launch_matvec<3>(qweight, scales, zeros, x, R, C, g, G, y, s);
    case 4: return launch_matvec<4>(qweight, scales, zeros, x, R, C, g, G, y, s);
    case 8: return launch_matvec<8>(qweight, scales, zeros, x, R, C, g, G, y, s);
  }
  return GPTQ_ERR_UNSUPPORTED;
}
