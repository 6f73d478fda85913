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

// ---- y = dequant(Q) x on the warp-level tensor path (mma.sync m16n8k16, f16 x f16 -> f32) ---------
// For per-row grids and group sizes that are multiples of 128.  The CUDA-core kernel above spends about
// four instructions per weight (extract, convert, multiply-add), which bounds it well below the HBM rate;
// here two codes become one half2 register with a single logic instruction,
//     (w >> s) & mask | 0x6400_6400  =  (1024 + k c_i, 1024 + k c_j)   in fp16,   k a power of two,
// one half2 multiply-add removes the offset exactly (codes are small integers, exact in fp16), and the
// multiply-adds themselves run on the tensor cores: A = 16 rows x 16 codes, B = the matching 16 entries
// of x replicated over the 8 columns, fp32 accumulators.  Products of two fp16 values are exact in fp32;
// the accumulator is drained into an fp32 sum after every 128 columns (8 MMAs).
//
// Which code meets which x is free as long as A and B agree, so x is staged in shared memory (fp16,
// once per CTA) in exactly the order the unpacking produces: position p of a 32-column chunk holds
// x[chunk * 32 + perm<F>(p)].  A task is 16 consecutive rows; the 16 warps of a CTA take the 128-column
// blocks of those rows round-robin and their partial sums meet in shared memory.
// Per 128-column block b of group gi:  y_r += s[r][gi] * (sum_{c in b} q_c x_c - z[r][gi] * sum_{c in b} x_c).
constexpr int kMvThreads = 512, kMvWarps = kMvThreads / 32;

__device__ __forceinline__ uint32_t h2_sub(uint32_t a, uint32_t b) {
  __half2 r = __hsub2(*reinterpret_cast<__half2*>(&a), *reinterpret_cast<__half2*>(&b));
  return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ uint32_t h2_fma(uint32_t a, uint32_t b, uint32_t c) {
  __half2 r = __hfma2(*reinterpret_cast<__half2*>(&a), *reinterpret_cast<__half2*>(&b), *reinterpret_cast<__half2*>(&c));
  return *reinterpret_cast<uint32_t*>(&r);
}
constexpr uint32_t kH1024 = 0x64006400u;                       // (1024, 1024)
// (1024 + k c) * (1 / k) - 1024 / k = c for k = 4, 16, 64, 256: multiplier and addend as half2 bit patterns
constexpr uint32_t kInv4 = 0x34003400u, kNeg256 = 0xDC00DC00u, kInv16 = 0x2C002C00u, kNeg64 = 0xD400D400u;
constexpr uint32_t kInv64 = 0x24002400u, kNeg16 = 0xCC00CC00u, kInv256 = 0x1C001C00u, kNeg4 = 0xC400C400u;

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Code index (0..31 inside a 32-column chunk) whose x value sits at position p of the staged chunk.
template <int F>
__host__ __device__ constexpr int mv_perm(int p) {
  if (F == 4) { return (p & ~7) + ((p & 1) ? 4 : 0) + ((p & 7) >> 1); }          // word of 8: 0 4 1 5 2 6 3 7
  if (F == 2) { return (p & ~15) + ((p & 1) ? 8 : 0) + ((p & 15) >> 1); }        // word of 16: 0 8 1 9 ... 7 15
  if (F == 8) { return (p & ~3) + ((p & 1) ? 2 : 0) + ((p & 3) >> 1); }          // word of 4: 0 2 1 3
  return p;                                                                        // 3-bit: natural order
}

// One 32-column chunk of two rows (A fragment rows g and g + 8) against the staged x: 8 MMAs.
template <int F>
__device__ __forceinline__ void mv_chunk(const uint32_t (&wa)[F], const uint32_t (&wb)[F], const uint4* xs, float (&c)[4]);

template <>
__device__ __forceinline__ void mv_chunk<4>(const uint32_t (&wa)[4], const uint32_t (&wb)[4], const uint4* xs, float (&c)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 x = xs[i];
    const uint32_t a = wa[i], b = wb[i], a8 = a >> 8, b8 = b >> 8;
    const uint32_t a0 = h2_sub((a & 0x000F000Fu) | kH1024, kH1024), a1 = h2_fma((a & 0x00F000F0u) | kH1024, kInv16, kNeg64);
    const uint32_t b0 = h2_sub((b & 0x000F000Fu) | kH1024, kH1024), b1 = h2_fma((b & 0x00F000F0u) | kH1024, kInv16, kNeg64);
    mma_16816(c, a0, b0, a1, b1, x.x, x.y);
    const uint32_t a2 = h2_sub((a8 & 0x000F000Fu) | kH1024, kH1024), a3 = h2_fma((a8 & 0x00F000F0u) | kH1024, kInv16, kNeg64);
    const uint32_t b2 = h2_sub((b8 & 0x000F000Fu) | kH1024, kH1024), b3 = h2_fma((b8 & 0x00F000F0u) | kH1024, kInv16, kNeg64);
    mma_16816(c, a2, b2, a3, b3, x.z, x.w);
  }
}

// eight half2 (c_j, c_{j+8}), j = 0..7, from one word of sixteen 2-bit codes
__device__ __forceinline__ void unpack2(uint32_t w, uint32_t (&h)[8]) {
  const uint32_t v = w >> 10;
  h[0] = h2_sub((w & 0x00030003u) | kH1024, kH1024);
  h[1] = h2_fma((w & 0x000C000Cu) | kH1024, kInv4, kNeg256);
  h[2] = h2_fma((w & 0x00300030u) | kH1024, kInv16, kNeg64);
  h[3] = h2_fma((w & 0x00C000C0u) | kH1024, kInv64, kNeg16);
  h[4] = h2_fma((w & 0x03000300u) | kH1024, kInv256, kNeg4);
  h[5] = h2_sub((v & 0x00030003u) | kH1024, kH1024);
  h[6] = h2_fma((v & 0x000C000Cu) | kH1024, kInv4, kNeg256);
  h[7] = h2_fma((v & 0x00300030u) | kH1024, kInv16, kNeg64);
}
template <>
__device__ __forceinline__ void mv_chunk<2>(const uint32_t (&wa)[2], const uint32_t (&wb)[2], const uint4* xs, float (&c)[4]) {
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    uint32_t ha[8], hb[8];
    unpack2(wa[i], ha); unpack2(wb[i], hb);
    const uint4 x0 = xs[2 * i], x1 = xs[2 * i + 1];
    mma_16816(c, ha[0], hb[0], ha[1], hb[1], x0.x, x0.y);
    mma_16816(c, ha[2], hb[2], ha[3], hb[3], x0.z, x0.w);
    mma_16816(c, ha[4], hb[4], ha[5], hb[5], x1.x, x1.y);
    mma_16816(c, ha[6], hb[6], ha[7], hb[7], x1.z, x1.w);
  }
}

template <>
__device__ __forceinline__ void mv_chunk<8>(const uint32_t (&wa)[8], const uint32_t (&wb)[8], const uint4* xs, float (&c)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 x = xs[i];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const uint32_t a = wa[2 * i + u], b = wb[2 * i + u];
      const uint32_t a0 = h2_sub((a & 0x00FF00FFu) | kH1024, kH1024), a1 = h2_sub(((a >> 8) & 0x00FF00FFu) | kH1024, kH1024);
      const uint32_t b0 = h2_sub((b & 0x00FF00FFu) | kH1024, kH1024), b1 = h2_sub(((b >> 8) & 0x00FF00FFu) | kH1024, kH1024);
      mma_16816(c, a0, b0, a1, b1, u ? x.z : x.x, u ? x.w : x.y);
    }
  }
}

// 3-bit: codes 2m and 2m + 1 sit next to each other at stream bit 6m; (v & 63) * 0x2001 copies the second
// one to bit 16, and the mask keeps one code per half.
__device__ __forceinline__ uint32_t pair3(const uint32_t (&w)[3], int m) {
  const int bit = 6 * m, k = bit >> 5, o = bit & 31;
  uint32_t v = w[k] >> o;
  if (o + 6 > 32 && k + 1 < 3) v |= w[k + 1] << (32 - o);
  return h2_sub((((v & 63u) * 0x2001u) & 0x00070007u) | kH1024, kH1024);
}
template <>
__device__ __forceinline__ void mv_chunk<3>(const uint32_t (&wa)[3], const uint32_t (&wb)[3], const uint4* xs, float (&c)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 x = xs[i];
    mma_16816(c, pair3(wa, 4 * i), pair3(wb, 4 * i), pair3(wa, 4 * i + 1), pair3(wb, 4 * i + 1), x.x, x.y);
    mma_16816(c, pair3(wa, 4 * i + 2), pair3(wb, 4 * i + 2), pair3(wa, 4 * i + 3), pair3(wb, 4 * i + 3), x.z, x.w);
  }
}

template <int F>
__device__ __forceinline__ void mv_load(const uint32_t* p, bool valid, uint32_t (&w)[F]) {
#pragma unroll
  for (int k = 0; k < F; ++k) w[k] = 0u;
  if (!valid) return;
  if constexpr (F == 4) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
    w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
  } else if constexpr (F == 2) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    w[0] = v.x; w[1] = v.y;
  } else if constexpr (F == 8) {
    const uint4 v0 = __ldg(reinterpret_cast<const uint4*>(p)), v1 = __ldg(reinterpret_cast<const uint4*>(p) + 1);
    w[0] = v0.x; w[1] = v0.y; w[2] = v0.z; w[3] = v0.w; w[4] = v1.x; w[5] = v1.y; w[6] = v1.z; w[7] = v1.w;
  } else {
#pragma unroll
    for (int k = 0; k < F; ++k) w[k] = __ldg(p + k);
  }
}

// grid: min(tasks, 2 x SMs) CTAs of 512 threads; dynamic shared memory: staged x (fp16, C rounded up to 128),
// per-128-column sums of x (fp32), and two buffers of 16 warps x 16 rows partial sums.
template <int F>
__global__ void __launch_bounds__(kMvThreads, 2)
matvec_mma_kernel(const uint32_t* __restrict__ qweight, const float* __restrict__ scales, const float* __restrict__ zeros,
                  const __half* __restrict__ x, int R, int C, int g, int G, float* __restrict__ y) {
  extern __shared__ uint4 mv_smem[];
  const int chunks = C / 32, n_blk = (C + 127) / 128, Cpad = n_blk * 128;
  __half* xs = reinterpret_cast<__half*>(mv_smem);                       // [Cpad], permuted inside every 32-column chunk
  float* sx = reinterpret_cast<float*>(xs + Cpad);                       // [n_blk] sum of x over a 128-column block
  float* red = sx + ((n_blk + 3) & ~3);                                  // [2][kMvWarps][16]
  for (int ch = threadIdx.x; ch < Cpad / 32; ch += blockDim.x) {          // one 32-column chunk (64 bytes) per thread
    __align__(16) __half in[32], out[32];
#pragma unroll
    for (int q = 0; q < 4; ++q)
      reinterpret_cast<uint4*>(in)[q] = ch < chunks ? __ldg(reinterpret_cast<const uint4*>(x + ch * 32) + q) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int p = 0; p < 32; ++p) out[p] = in[mv_perm<F>(p)];
#pragma unroll
    for (int q = 0; q < 4; ++q) reinterpret_cast<uint4*>(xs + ch * 32)[q] = reinterpret_cast<const uint4*>(out)[q];
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int b = warp; b < n_blk; b += kMvWarps) {
    float t = 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) t += __half2float(xs[b * 128 + lane + 32 * j]);
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (lane == 0) sx[b] = t;
  }
  __syncthreads();

  const int gq = lane >> 2, t4 = lane & 3;                               // fragment row and k-quarter of this lane
  const int n_tasks = (R + 15) / 16;
  const bool per_block = g < C;                                          // grouped: scale and zero change along the row
  int par = 0;
  for (int task = blockIdx.x; task < n_tasks; task += gridDim.x, par ^= 1) {
    const int ra = min(task * 16 + gq, R - 1), rb = min(task * 16 + gq + 8, R - 1);   // clamped: loads stay in range
    const uint32_t* pa = qweight + (int64_t)ra * chunks * F;
    const uint32_t* pb = qweight + (int64_t)rb * chunks * F;
    const float* sa = scales + (int64_t)ra * G; const float* za = zeros + (int64_t)ra * G;
    const float* sb = scales + (int64_t)rb * G; const float* zb = zeros + (int64_t)rb * G;
    float ya = 0.f, yb = 0.f;                                            // grouped: finished sums; per-row: sum of q x
    float xsum = 0.f;                                                    // per-row: sum of x over this warp's blocks
    // software pipeline: the codes of the next block are in flight while this block is unpacked and multiplied
    uint32_t wa[F], wb[F];
    {
      const int ch = warp * 4 + t4;
      mv_load<F>(pa + (int64_t)ch * F, warp < n_blk && ch < chunks, wa);
      mv_load<F>(pb + (int64_t)ch * F, warp < n_blk && ch < chunks, wb);
    }
    for (int blk = warp; blk < n_blk; blk += kMvWarps) {
      const int ch = blk * 4 + t4, chn = ch + 4 * kMvWarps;
      uint32_t na[F], nb[F];
      mv_load<F>(pa + (int64_t)chn * F, blk + kMvWarps < n_blk && chn < chunks, na);
      mv_load<F>(pb + (int64_t)chn * F, blk + kMvWarps < n_blk && chn < chunks, nb);
      float c[4] = {0.f, 0.f, 0.f, 0.f};
      mv_chunk<F>(wa, wb, reinterpret_cast<const uint4*>(xs + ch * 32), c);
      if (per_block) {
        const int gi = (blk * 128) / g;
        const float bx = sx[blk];
        ya = fmaf(__ldg(sa + gi), c[0] - __ldg(za + gi) * bx, ya);
        yb = fmaf(__ldg(sb + gi), c[2] - __ldg(zb + gi) * bx, yb);
      } else {
        ya += c[0]; yb += c[2]; xsum += sx[blk];
      }
#pragma unroll
      for (int k = 0; k < F; ++k) { wa[k] = na[k]; wb[k] = nb[k]; }
    }
    if (!per_block) {
      ya = __ldg(sa) * (ya - __ldg(za) * xsum);
      yb = __ldg(sb) * (yb - __ldg(zb) * xsum);
    }
    float* rp = red + (par * kMvWarps + warp) * 16;
    if (t4 == 0) { rp[gq] = ya; rp[gq + 8] = yb; }
    __syncthreads();
    if (threadIdx.x < 16) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < kMvWarps; ++w) t += red[(par * kMvWarps + w) * 16 + threadIdx.x];
      const int r = task * 16 + threadIdx.x;
      if (r < R) y[r] = t;
    }
  }
}

inline bool group_ok(int C, int g) { return g > 0 && C % g == 0 && (g % 32 == 0 || 32 % g == 0); }

inline int device_sm_count_inference() {
  int dev = 0, n = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  return n > 0 ? n : 148;
}

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
  if (g == C || g % 128 == 0) {
    // tensor path: x staged as fp16
    const int n_blk = (C + 127) / 128;
    const size_t smem = (size_t)n_blk * 128 * sizeof(__half) + (size_t)((n_blk + 3) & ~3) * sizeof(float) +
                        (size_t)2 * gptq::kMvWarps * 16 * sizeof(float);
    if (smem > 110 * 1024) return GPTQ_ERR_UNSUPPORTED;               // two CTAs per SM
    const int tasks = (R + 15) / 16;
    int grid = 2 * gptq::device_sm_count_inference();
    if (grid > tasks) grid = tasks;
    GPTQ_CUDA_TRY(cudaFuncSetAttribute(gptq::matvec_mma_kernel<F>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    gptq::matvec_mma_kernel<F><<<grid, gptq::kMvThreads, smem, s>>>(qweight, scales, zeros, x, R, C, g, G, y);
    GPTQ_LAUNCH_CHECK();
    return GPTQ_OK;
  }
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
