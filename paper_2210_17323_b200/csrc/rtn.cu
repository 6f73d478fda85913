// Round-to-nearest baseline (Section 5, "Baselines"): every weight rounded to the nearest value of
// exactly the grid the solver would use for untouched weights -- per-row or per-group min-max,
// asymmetric with an integer zero-point (or symmetric / ternary) -- with no error feedback.
// Output layout is that of gptq_quantize_layer.  One pass over W for groups that are multiples of 32 columns and per-row
// grids (rtn_span_kernel, rtn_fused_kernel), two plain passes for the small groups (4, 8, 16).
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

// ---- one pass for groups that are multiples of 32 columns (and per-row grids) -----------------------------------
// The code is rne(w / scale) + zero, clamped.  w * (1 / scale) in fp32 is within 5e-5 of the quotient (|quotient| <= 256),
// so its rounding is the quotient's unless it lies within 1e-3 of a tie; only then is the fp64 division done, which is
// the operation the oracle performs.
__device__ __forceinline__ void rtn_grid_of(float mn, float mx, RtnGrid grid, float& scale, float& zero) {
  double xmin = fmin((double)mn, 0.0), xmax = fmax((double)mx, 0.0);
  if (xmin == 0.0 && xmax == 0.0) { xmin = -1.0; xmax = 1.0; }
  if (grid.symmetric) {
    scale = storage_rounded((float)(2.0 * fmax(fabs(xmin), xmax) / (double)grid.maxq), grid.f16scale);
    zero = (float)((grid.maxq + 1) / 2);
  } else {
    scale = storage_rounded((float)((xmax - xmin) / (double)grid.maxq), grid.f16scale);
    zero = (float)rint(-xmin / (double)scale);
  }
}
__device__ __forceinline__ void rtn_minmax8(const uint4& v, float& mn, float& mx) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float2 f2 = __half22float2(h[k]);
    mn = fminf(mn, fminf(f2.x, f2.y));
    mx = fmaxf(mx, fmaxf(f2.x, f2.y));
  }
}
// eight codes of one 16-byte piece as 8 F bits.  t = w / scale + zero is clamped to [-1/4, maxq + 1/4] first (which
// rounds to the same code as clamping afterwards) and rounded by adding 1.5 * 2^23, whose sum holds rne(t) in its low
// mantissa bits: no rounding or conversion instruction per code.
template <int F>
__device__ __forceinline__ uint64_t rtn_codes8(const uint4& v, float scale, float rs, float zero, float fmaxq) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
  constexpr float kRound = 12582912.f;
  uint64_t bits = 0;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const float2 w2 = __half22float2(h[k >> 1]);
    const float w = (k & 1) ? w2.y : w2.x;
    const float t = fminf(fmaxf(fmaf(w, rs, zero), -0.25f), fmaxq + 0.25f);
    const float tm = __fadd_rn(t, kRound);
    uint32_t code = __float_as_uint(tm) & 0xFFu;
    if (fabsf(t - __fadd_rn(tm, -kRound)) > 0.499f) {       // within 1e-3 of a tie: the oracle's own operation decides
      const double q = fmin(fmax(rint((double)w / (double)scale) + (double)zero, 0.0), (double)fmaxq);
      code = (uint32_t)q;
    }
    bits |= (uint64_t)code << (k * F);
  }
  return bits;
}
// The lanes of a warp hold consecutive pieces (piece index i, `on` = the piece exists); their 8 F bits become whole words
// of the row with at most one shuffle.  Every lane of the warp must call this.
template <int F>
__device__ __forceinline__ void rtn_store_words(uint32_t* qrow, int i, bool on, uint64_t bits, int lane) {
  if constexpr (F == 4) {
    if (on) qrow[i] = (uint32_t)bits;
  } else if constexpr (F == 8) {
    if (on) reinterpret_cast<uint2*>(qrow)[i] = make_uint2((uint32_t)bits, (uint32_t)(bits >> 32));
  } else if constexpr (F == 2) {
    const uint32_t mine = (uint32_t)bits, next = __shfl_down_sync(0xffffffffu, mine, 1);
    if ((lane & 1) == 0 && on) qrow[i >> 1] = mine | (next << 16);
  } else {                                                  // F == 3: four lanes' 24-bit runs make three words
    const uint32_t mine = (uint32_t)bits, next = __shfl_down_sync(0xffffffffu, mine, 1);
    const int k = lane & 3;
    const uint32_t word = k == 0 ? (mine | (next << 24)) : k == 1 ? ((mine >> 8) | (next << 16)) : ((mine >> 16) | (next << 8));
    if (k != 3 && on) qrow[3 * (i >> 2) + k] = word;
  }
}

// One warp per (row, group), any group that is a multiple of 32 columns.  Phase A: the group's minimum and maximum from
// 16-byte loads (a lane takes the 8-column pieces lane, lane + 32, ...).  Phase B: the same pieces again (now from L1 /
// L2: the group was just read), eight codes per lane, stored as whole words.  W comes from memory once.
template <int F>
__global__ void __launch_bounds__(256)
rtn_fused_kernel(const __half* __restrict__ W, int R, int C, int g, int G, RtnGrid grid,
                 float* __restrict__ scales, float* __restrict__ zeros, uint32_t* __restrict__ qweight) {
  const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (wid >= (int64_t)R * G) return;
  const int row = (int)(wid / G), gi = (int)(wid % G);
  const uint4* p = reinterpret_cast<const uint4*>(W + (int64_t)row * C + (int64_t)gi * g);
  const int pieces = g / 8;
  float mn = INFINITY, mx = -INFINITY;
  int i0 = lane;
  for (; i0 + 96 < pieces; i0 += 128) {                     // four loads in flight per lane
    const uint4 a = __ldg(p + i0), b = __ldg(p + i0 + 32), c = __ldg(p + i0 + 64), d = __ldg(p + i0 + 96);
    rtn_minmax8(a, mn, mx); rtn_minmax8(b, mn, mx); rtn_minmax8(c, mn, mx); rtn_minmax8(d, mn, mx);
  }
  for (; i0 < pieces; i0 += 32) { const uint4 a = __ldg(p + i0); rtn_minmax8(a, mn, mx); }
  for (int o = 16; o > 0; o >>= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  float scale = 0.f, zero = 0.f;
  if (lane == 0) {
    rtn_grid_of(mn, mx, grid, scale, zero);
    scales[wid] = scale; zeros[wid] = zero;
  }
  scale = __shfl_sync(0xffffffffu, scale, 0);
  zero = __shfl_sync(0xffffffffu, zero, 0);
  const float rs = 1.0f / scale, fmaxq = (float)grid.maxq;
  // words of this group inside the row: the group starts at bit gi * g * F, a multiple of 32 F bits
  uint32_t* qrow = qweight + (int64_t)row * (C / 32 * F) + (int64_t)gi * (g / 32 * F);
  for (int base = 0; base < pieces; base += 32) {           // uniform trip count: every lane joins the shuffles
    const int i = base + lane;
    const bool on = i < pieces;
    uint64_t bits = 0;
    if (on) { const uint4 v = __ldg(p + i); bits = rtn_codes8<F>(v, scale, rs, zero, fmaxq); }
    rtn_store_words<F>(qrow, i, on, bits, lane);
  }
}

// Groups of 32, 64, 128 or 256 columns: one warp per run of 32 groups of a row (32 g columns), a group on g / 8
// neighbouring lanes of one 256-column span.  First pass over the run's spans: the group's lanes reduce minimum and
// maximum among themselves and hand them to the lane that owns the group (group t of the run belongs to lane t), so that
// the 32 grids of the run are derived in one go, one per lane.  Second pass: the spans again (from L1 / L2: at most 8 KB
// per warp, just read), quantized with their groups' grids fetched by shuffles.  Both loops stay rolled: the code is
// small enough for the instruction cache.
template <int F, int kLanes>                                // kLanes = g / 8 = lanes per group = spans of one run
__global__ void __launch_bounds__(256)
rtn_span_kernel(const __half* __restrict__ W, int R, int C, int G, RtnGrid grid,
                float* __restrict__ scales, float* __restrict__ zeros, uint32_t* __restrict__ qweight) {
  constexpr int kGroupsPerSpan = 32 / kLanes;
  const int runs = (G + 31) / 32;
  const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (wid >= (int64_t)R * runs) return;
  const int row = (int)(wid / runs), run = (int)(wid % runs);
  const int piece0 = run * 32 * kLanes;                     // first piece of the run inside the row
  const int row_pieces = C / 8;
  const uint4* p = reinterpret_cast<const uint4*>(W + (int64_t)row * C);
  float my_mn = INFINITY, my_mx = -INFINITY;                // of the group this lane owns (group `lane` of the run)
#pragma unroll 4
  for (int sp = 0; sp < kLanes; ++sp) {
    const int i = piece0 + sp * 32 + lane;
    float mn = INFINITY, mx = -INFINITY;
    if (i < row_pieces) { const uint4 v = __ldg(p + i); rtn_minmax8(v, mn, mx); }
#pragma unroll
    for (int o = 1; o < kLanes; o <<= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    // group t = sp * kGroupsPerSpan + j of the run sits on lanes j * kLanes ..; its owner is lane t
    const int j = lane - sp * kGroupsPerSpan;               // which group of this span this lane owns, if any
    const float gmn = __shfl_sync(0xffffffffu, mn, (j & (kGroupsPerSpan - 1)) * kLanes);
    const float gmx = __shfl_sync(0xffffffffu, mx, (j & (kGroupsPerSpan - 1)) * kLanes);
    if (j >= 0 && j < kGroupsPerSpan) { my_mn = gmn; my_mx = gmx; }
  }
  float my_scale = 1.f, my_zero = 0.f;
  const int my_group = run * 32 + lane;
  if (my_group < G) {
    rtn_grid_of(my_mn, my_mx, grid, my_scale, my_zero);
    scales[(int64_t)row * G + my_group] = my_scale;
    zeros[(int64_t)row * G + my_group] = my_zero;
  }
  const float my_rs = 1.0f / my_scale, fmaxq = (float)grid.maxq;
  uint32_t* qrow = qweight + (int64_t)row * (C / 32 * F);
#pragma unroll 1
  for (int sp = 0; sp < kLanes; ++sp) {
    const int i = piece0 + sp * 32 + lane;
    const int owner = sp * kGroupsPerSpan + lane / kLanes;  // lane that owns this lane's group in span sp
    const float scale = __shfl_sync(0xffffffffu, my_scale, owner), rs = __shfl_sync(0xffffffffu, my_rs, owner);
    const float zero = __shfl_sync(0xffffffffu, my_zero, owner);
    const bool on = i < row_pieces;
    uint64_t bits = 0;
    if (on) { const uint4 v = __ldg(p + i); bits = rtn_codes8<F>(v, scale, rs, zero, fmaxq); }
    rtn_store_words<F>(qrow, i, on, bits, lane);
  }
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
  if (g % 32 == 0 && aligned_to(W_fp16, 16)) {              // one pass; (row, group) starts are then 16-byte aligned too
    const bool span = g == 32 || g == 64 || g == 128 || g == 256;
    const int64_t warps = span ? (int64_t)R * ((G + 31) / 32) : (int64_t)R * G;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
#define GPTQ_RTN_LAUNCH(FF)                                                                                               \
    if (g == 32) rtn_span_kernel<FF, 4><<<blocks, 256, 0, s>>>(W, R, C, G, grid, scales, zeros, qweight);                 \
    else if (g == 64) rtn_span_kernel<FF, 8><<<blocks, 256, 0, s>>>(W, R, C, G, grid, scales, zeros, qweight);            \
    else if (g == 128) rtn_span_kernel<FF, 16><<<blocks, 256, 0, s>>>(W, R, C, G, grid, scales, zeros, qweight);          \
    else if (g == 256) rtn_span_kernel<FF, 32><<<blocks, 256, 0, s>>>(W, R, C, G, grid, scales, zeros, qweight);          \
    else rtn_fused_kernel<FF><<<blocks, 256, 0, s>>>(W, R, C, g, G, grid, scales, zeros, qweight)
    switch (f) {
      case 2: GPTQ_RTN_LAUNCH(2); break;
      case 3: GPTQ_RTN_LAUNCH(3); break;
      case 4: GPTQ_RTN_LAUNCH(4); break;
      default: GPTQ_RTN_LAUNCH(8); break;
    }
#undef GPTQ_RTN_LAUNCH
    GPTQ_LAUNCH_CHECK();
    return GPTQ_OK;
  }
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
