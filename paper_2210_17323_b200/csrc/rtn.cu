// Round-to-nearest baseline (Section 5, "Baselines"): every weight rounded to the nearest value of
// exactly the grid the solver would use for untouched weights -- per-row or per-group min-max,
// asymmetric with an integer zero-point (or symmetric / ternary) -- with no error feedback.
// Output layout is that of gptq_quantize_layer.  Two bandwidth-bound passes over W.
#include "common.cuh"

namespace gptq {
namespace {

struct RtnGrid { int maxq; int symmetric; int f16scale; };

__device__ __forceinline__ float storage_rounded(float scale, int f16scale) {
  if (!f16scale) return scale;
  const float s16 = __half2float(__float2half_rn(scale));
  return (s16 > 0.f && isfinite(s16)) ? s16 : scale;
}

// One warp per (row, group): min / max of the group -> scale (rounded to fp32), integer zero-point.
__global__ void rtn_params_kernel(const __half* __restrict__ W, int R, int C, int g, int G, RtnGrid grid,
                                  float* __restrict__ scales, float* __restrict__ zeros) {
  const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (wid >= (int64_t)R * G) return;
  const int row = (int)(wid / G), gi = (int)(wid % G);
  const __half* p = W + (int64_t)row * C + (int64_t)gi * g;
  float mn = INFINITY, mx = -INFINITY;
  for (int i = lane; i < g; i += 32) { const float v = __half2float(p[i]); mn = fminf(mn, v); mx = fmaxf(mx, v); }
  for (int o = 16; o > 0; o >>= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  if (lane == 0) {
    double xmin = fmin((double)mn, 0.0), xmax = fmax((double)mx, 0.0);
    if (xmin == 0.0 && xmax == 0.0) { xmin = -1.0; xmax = 1.0; }
    float scale, zero;
    if (grid.symmetric) {
      scale = storage_rounded((float)(2.0 * fmax(fabs(xmin), xmax) / (double)grid.maxq), grid.f16scale);
      zero = (float)((grid.maxq + 1) / 2);
    } else {
      scale = storage_rounded((float)((xmax - xmin) / (double)grid.maxq), grid.f16scale);
      zero = (float)rint(-xmin / (double)scale);
    }
    scales[wid] = scale; zeros[wid] = zero;
  }
}

// One thread per packed word: quantizes the codes that overlap the word and assembles it.
__global__ void rtn_pack_kernel(const __half* __restrict__ W, int R, int C, int g, int G, int f, int maxq,
                                const float* __restrict__ scales, const float* __restrict__ zeros,
                                uint32_t* __restrict__ qweight) {
  const int nwords = C * f / 32;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)R * nwords) return;
  const int r = (int)(idx / nwords), k = (int)(idx % nwords);
  const __half* w = W + (int64_t)r * C;
  const int lo = 32 * k / f, hi = (32 * k + 31) / f;
  uint32_t word = 0;
  for (int col = lo; col <= hi; ++col) {
    const int gi = col / g;
    const double scale = (double)scales[(int64_t)r * G + gi], zero = (double)zeros[(int64_t)r * G + gi];
    double q = rint((double)__half2float(w[col]) / scale) + zero;
    q = fmin(fmax(q, 0.0), (double)maxq);
    const uint32_t v = (uint32_t)q;
    const int sh = col * f - 32 * k;
    word |= sh >= 0 ? (v << sh) : (v >> (-sh));
  }
  qweight[idx] = word;
}

}  // namespace
}  // namespace gptq

extern "C" gptq_status_t gptq_rtn_layer(const void* W_fp16, int R, int C, int bits, int group_size, int sym,
                                        uint32_t* qweight, float* scales, float* zeros, void* stream) {
  using namespace gptq;
  if (!W_fp16 || !qweight || !scales || !zeros || R <= 0 || C <= 0 || C % 32 != 0) return GPTQ_ERR_INVALID_ARG;
  if (!(bits == 2 || bits == 3 || bits == 4 || bits == 8 || bits == GPTQ_BITS_TERNARY)) return GPTQ_ERR_UNSUPPORTED;
  const int g = group_size > 0 ? group_size : C;
  if (C % g != 0) return GPTQ_ERR_INVALID_ARG;
  const int G = C / g, f = bits == GPTQ_BITS_TERNARY ? 2 : bits;
  if (sym & ~(GPTQ_GRID_SYMMETRIC | GPTQ_GRID_FP16_SCALES)) return GPTQ_ERR_INVALID_ARG;
  RtnGrid grid{bits == GPTQ_BITS_TERNARY ? 2 : (1 << bits) - 1, ((sym & GPTQ_GRID_SYMMETRIC) != 0 || bits == GPTQ_BITS_TERNARY) ? 1 : 0,
               (sym & GPTQ_GRID_FP16_SCALES) ? 1 : 0};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half* W = static_cast<const __half*>(W_fp16);
  {
    const int64_t warps = (int64_t)R * G;
    rtn_params_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, s>>>(W, R, C, g, G, grid, scales, zeros);
    GPTQ_LAUNCH_CHECK();
  }
  {
    const int64_t total = (int64_t)R * (C * f / 32);
    rtn_pack_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(W, R, C, g, G, f, grid.maxq, scales, zeros, qweight);
    GPTQ_LAUNCH_CHECK();
  }
  return GPTQ_OK;
}
