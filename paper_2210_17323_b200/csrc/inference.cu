// Inference-side kernels for the packed format the solver writes (Section 5, "Practical Speedups" and the
// appendix on kernels: a quantized-matrix x fp16-vector product with on-the-fly dequantization, and a
// whole-matrix dequantization).  Both are bound by HBM bandwidth: the matvec reads f bits per weight.
//
// Dequantized value of code q in group gi of row r:  scales[r][gi] * (q - zeros[r][gi]), formed in fp32.
#include "common.cuh"

#include <type_traits>

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

// ---- whole-matrix dequantization: one thread per 8 columns --------------------------------------
// A warp reads 32 F consecutive bytes of codes and writes 512 consecutive bytes of fp16 with one 16-byte
// streaming store per lane.  A thread keeps its 8 columns and walks down the rows (blockIdx.y, grid-stride), so
// the bit offset, the word index and the group index are computed once.
template <int F>
__global__ void __launch_bounds__(256)
dequantize_kernel(const uint32_t* __restrict__ qweight, const float* __restrict__ scales,
                  const float* __restrict__ zeros, int R, int C, int g, int G, __half* __restrict__ out) {
  const int c0 = (blockIdx.x * blockDim.x + threadIdx.x) * 8;
  if (c0 >= C) return;
  // the 8 codes are 8 F bits of the row's bit stream, starting at bit c0 * F (a multiple of 8)
  const int bit = c0 * F, k = bit >> 5, o = bit & 31;
  const bool two = o + 8 * F > 32;
  const int gi0 = c0 / g;
  const int64_t wpr = (int64_t)(C / 32) * F;                  // words per row
  // four rows per trip: their loads are issued together, so that a thread has four independent round trips to
  // memory in flight instead of one
  constexpr int kRows = 4;
  const int stride = gridDim.y;
  for (int r0 = blockIdx.y; r0 < R; r0 += kRows * stride) {
    uint64_t v[kRows];
    float s[kRows], z[kRows];
    // 3-bit (two load instructions per row for half of the lanes): the next trip's codes are asked into L2 now, one
    // request per 24 bytes of a row, so that its loads return sooner -- the kernel's traffic is mostly writes and loads
    // queue behind them.  (Measured: 63 % -> 74 % of the copy bandwidth; the other widths lose 1-8 % with it.)
    if constexpr (F == 3) {
      if ((threadIdx.x & 7) == 0) {
#pragma unroll
        for (int u = 0; u < kRows; ++u) {
          const int r = r0 + (kRows + u) * stride;
          if (r < R) asm volatile("prefetch.global.L2 [%0];" ::"l"(qweight + r * wpr + k));
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
      const int r = r0 + u * stride;
      v[u] = 0; s[u] = 0.f; z[u] = 0.f;
      if (r < R) {
        const uint32_t* rowp = qweight + r * wpr;
        v[u] = __ldg(rowp + k);
        if (two) v[u] |= (uint64_t)__ldg(rowp + k + 1) << 32;
        if (g >= 8) { s[u] = __ldg(scales + (int64_t)r * G + gi0); z[u] = __ldg(zeros + (int64_t)r * G + gi0); }
      }
    }
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
      const int r = r0 + u * stride;
      if (r >= R) break;
      const uint64_t w64 = v[u] >> o;
      const uint32_t w32 = (uint32_t)w64;            // the 8 F bits of the eight codes fit one word unless F = 8
      // code -> float without an integer conversion: the bit pattern (code | 0x4B000000) is 2^23 + code exactly
      auto code_f = [&](int i) -> float {
        const uint32_t q = (F < 8 ? (w32 >> (i * F)) : (uint32_t)(w64 >> (i * F))) & ((1u << F) - 1u);
        return __fsub_rn(__uint_as_float(q | 0x4B000000u), 8388608.f);
      };
      __align__(16) __half h[8];
      if (g >= 8) {
#pragma unroll
        for (int i = 0; i < 8; ++i) h[i] = __float2half_rn(__fmul_rn(s[u], __fsub_rn(code_f(i), z[u])));
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int gi = (c0 + i) / g;
          const float sc = __ldg(scales + (int64_t)r * G + gi), zz = __ldg(zeros + (int64_t)r * G + gi);
          h[i] = __float2half_rn(__fmul_rn(sc, __fsub_rn(code_f(i), zz)));
        }
      }
      __stcs(reinterpret_cast<uint4*>(out + (int64_t)r * C + c0), *reinterpret_cast<const uint4*>(h));
    }
  }
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
// here two codes become one half2 operand with a single AND (see mma_16816 below), and the multiply-adds
// themselves run on the tensor cores: A = 16 rows x 16 codes, B = the matching 16 entries
// of x replicated over the 8 columns, fp32 accumulators.  Products of two fp16 values are exact in fp32;
// the accumulator is drained into an fp32 sum after every 128 columns (8 MMAs).
//
// Which code meets which x is free as long as A and B agree, so x is staged in shared memory (fp16,
// once per CTA) in exactly the order the unpacking produces: position p of a 32-column chunk holds
// x[chunk * 32 + perm<F>(p)].  A task is 16 consecutive rows; the 16 warps of a CTA take the 128-column
// blocks of those rows round-robin and their partial sums meet in shared memory.
// Per 128-column block b of group gi:  y_r += s[r][gi] * (sum_{c in b} q_c x_c - z[r][gi] * sum_{c in b} x_c).
constexpr int kMvThreads = 512, kMvWarps = kMvThreads / 32, kMvDepth = 2, kMvCtasPerSm = 2;

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// A masked field IS an fp16 number: the bit pattern 0x000c is the subnormal c * 2^-24, and a field that
// starts at bit s (< 10) is c * 2^(s-24).  So one AND turns two codes into a half2 operand with no offset
// to remove; fields that sit at different bit positions carry different power-of-two factors and go to
// separate accumulators (c1 for factor 1, c2 for the factor kMvScale2<F>), combined once per 128 columns:
//     sum q x = 2^24 * (c1 + c2 / kMvScale2).
// Code index (0..31 inside a 32-column chunk) whose x value sits at position p of the staged chunk.
template <int F>
__host__ __device__ constexpr int mv_perm(int p) {
  if (F == 4) { constexpr int o[8] = {0, 4, 2, 6, 1, 5, 3, 7}; return (p & ~7) + o[p & 7]; }
  if (F == 2) { constexpr int o[16] = {0, 8, 4, 12, 1, 9, 5, 13, 2, 10, 6, 14, 3, 11, 7, 15}; return (p & ~15) + o[p & 15]; }
  if (F == 8) { constexpr int o[4] = {0, 2, 1, 3}; return (p & ~3) + o[p & 3]; }
  { constexpr int o[8] = {0, 1, 4, 5, 2, 3, 6, 7}; return (p & ~7) + o[p & 7]; }            // 3-bit
}
template <int F> struct MvScale2 { static constexpr float inv = 0.f; };            // 1 / factor of the second accumulator
template <> struct MvScale2<4> { static constexpr float inv = 1.f / 16.f; };
template <> struct MvScale2<2> { static constexpr float inv = 1.f / 4.f; };
template <> struct MvScale2<3> { static constexpr float inv = 1.f / 64.f; };

// One 32-column chunk of two rows (A fragment rows g and g + 8) against the staged x: 8 MMAs.
template <int F>
__device__ __forceinline__ void mv_chunk(const uint32_t (&wa)[F], const uint32_t (&wb)[F], const uint4* xs,
                                         float (&c1)[4], float (&c2)[4]);

template <>
__device__ __forceinline__ void mv_chunk<4>(const uint32_t (&wa)[4], const uint32_t (&wb)[4], const uint4* xs,
                                            float (&c1)[4], float (&c2)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {          // word i: codes (0,4) (2,6) at factor 1, (1,5) (3,7) at factor 16
    const uint4 x = xs[i];
    const uint32_t a = wa[i], b = wb[i], a8 = a >> 8, b8 = b >> 8;
    mma_16816(c1, a & 0x000F000Fu, b & 0x000F000Fu, a8 & 0x000F000Fu, b8 & 0x000F000Fu, x.x, x.y);
    mma_16816(c2, a & 0x00F000F0u, b & 0x00F000F0u, a8 & 0x00F000F0u, b8 & 0x00F000F0u, x.z, x.w);
  }
}

template <>
__device__ __forceinline__ void mv_chunk<2>(const uint32_t (&wa)[2], const uint32_t (&wb)[2], const uint4* xs,
                                            float (&c1)[4], float (&c2)[4]) {
  // a 2-bit field may start at bit 0, 2, 4 or 6 of a half and still be an fp16 subnormal: four factors (1, 4, 16, 64), one
  // shift per word.  The factors 16 and 64 are summed apart and folded into the first two accumulators at the end.
  float c3[4] = {0.f, 0.f, 0.f, 0.f}, c4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int i = 0; i < 2; ++i) {          // word i, v in {w, w >> 8}: field s of v holds codes (s / 2 [+ 4], 8 + s / 2 [+ 4])
    const uint4 x0 = xs[2 * i], x1 = xs[2 * i + 1];
    const uint32_t a = wa[i], b = wb[i], a8 = a >> 8, b8 = b >> 8;
    mma_16816(c1, a & 0x00030003u, b & 0x00030003u, a8 & 0x00030003u, b8 & 0x00030003u, x0.x, x0.y);
    mma_16816(c2, a & 0x000C000Cu, b & 0x000C000Cu, a8 & 0x000C000Cu, b8 & 0x000C000Cu, x0.z, x0.w);
    mma_16816(c3, a & 0x00300030u, b & 0x00300030u, a8 & 0x00300030u, b8 & 0x00300030u, x1.x, x1.y);
    mma_16816(c4, a & 0x00C000C0u, b & 0x00C000C0u, a8 & 0x00C000C0u, b8 & 0x00C000C0u, x1.z, x1.w);
  }
  c1[0] = fmaf(c3[0], 1.f / 16.f, c1[0]); c1[2] = fmaf(c3[2], 1.f / 16.f, c1[2]);
  c2[0] = fmaf(c4[0], 1.f / 16.f, c2[0]); c2[2] = fmaf(c4[2], 1.f / 16.f, c2[2]);
}

template <>
__device__ __forceinline__ void mv_chunk<8>(const uint32_t (&wa)[8], const uint32_t (&wb)[8], const uint4* xs,
                                            float (&c1)[4], float (&)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {          // word: codes (0,2) and (1,3); 255 * 2^-24 is still subnormal
    const uint4 x = xs[i];
    mma_16816(c1, wa[2 * i] & 0x00FF00FFu, wb[2 * i] & 0x00FF00FFu,
              (wa[2 * i] >> 8) & 0x00FF00FFu, (wb[2 * i] >> 8) & 0x00FF00FFu, x.x, x.y);
    mma_16816(c1, wa[2 * i + 1] & 0x00FF00FFu, wb[2 * i + 1] & 0x00FF00FFu,
              (wa[2 * i + 1] >> 8) & 0x00FF00FFu, (wb[2 * i + 1] >> 8) & 0x00FF00FFu, x.z, x.w);
  }
}

// 3-bit: four consecutive codes are 12 bits of the stream.  With those 12 bits alone in a register (v),
// v * 0x2001 = v | v << 13 holds code 0 at bit 0 and code 1 at bit 16 (one half2 operand under the mask 0x00070007,
// factor 1), and code 2 at bit 6 and code 3 at bit 22 (a second operand under 0x01C001C0, factor 64, which goes to
// the second accumulator): shift, mask, multiply and two ANDs for four codes.  Returns v * 0x2001 for run j (0..7)
// of the chunk's three words.
__device__ __forceinline__ uint32_t quad3(const uint32_t (&w)[3], int j) {
  const int bit = 12 * j, k = bit >> 5, o = bit & 31;
  uint32_t v;
  if (o + 12 < 32) v = (w[k] >> o) & 0xFFFu;
  else if (o + 12 == 32) v = w[k] >> 20;
  else v = __funnelshift_r(w[k], w[k + 1 < 3 ? k + 1 : k], o) & 0xFFFu;
  return v * 0x2001u;
}
template <>
__device__ __forceinline__ void mv_chunk<3>(const uint32_t (&wa)[3], const uint32_t (&wb)[3], const uint4* xs,
                                            float (&c1)[4], float (&c2)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {          // runs 2i and 2i + 1: codes 8i .. 8i + 7
    const uint4 x = xs[i];
    const uint32_t a0 = quad3(wa, 2 * i), a1 = quad3(wa, 2 * i + 1), b0 = quad3(wb, 2 * i), b1 = quad3(wb, 2 * i + 1);
    mma_16816(c1, a0 & 0x00070007u, b0 & 0x00070007u, a1 & 0x00070007u, b1 & 0x00070007u, x.x, x.y);
    mma_16816(c2, a0 & 0x01C001C0u, b0 & 0x01C001C0u, a1 & 0x01C001C0u, b1 & 0x01C001C0u, x.z, x.w);
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

// grid: min(tasks, kMvCtasPerSm x SMs) CTAs of 512 threads; dynamic shared memory: staged x (fp16, C rounded up to 128),
// per-128-column sums of x (fp32), and two buffers of 16 warps x 16 rows partial sums.
template <int F>
__global__ void __launch_bounds__(kMvThreads, kMvCtasPerSm)
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
  const int my_tasks = blockIdx.x < n_tasks ? (n_tasks - 1 - blockIdx.x) / gridDim.x + 1 : 0;
  const int per_task = (n_blk + kMvWarps - 1) / kMvWarps;                // blocks per warp and task (the same for all warps)
  const bool per_block = g < C;                                          // grouped: scale and zero change along the row
  const int chunk_bytes_w = F;                                           // words per chunk

  // The (task, block) pairs of this warp form one stream; the codes of the next kMvDepth pairs are in flight in
  // a register ring (indexed by compile-time constants only) while one block is unpacked and multiplied, also
  // across task boundaries.
  uint32_t wa[kMvDepth][F], wb[kMvDepth][F];
  int lk = 0, lj = 0;                                                    // load cursor: task number, block number
  auto issue = [&](uint32_t (&ua)[F], uint32_t (&ub)[F]) {
    const int task = blockIdx.x + lk * gridDim.x, blk = warp + lj * kMvWarps, ch = blk * 4 + t4;
    const bool ok = lk < my_tasks && ch < chunks;
    const int ra = min(task * 16 + gq, R - 1), rb = min(task * 16 + gq + 8, R - 1);   // clamped: loads stay in range
    mv_load<F>(qweight + ((int64_t)ra * chunks + ch) * chunk_bytes_w, ok, ua);
    mv_load<F>(qweight + ((int64_t)rb * chunks + ch) * chunk_bytes_w, ok, ub);
    if (++lj == per_task) { lj = 0; ++lk; }
  };
#pragma unroll
  for (int d = 0; d < kMvDepth; ++d) issue(wa[d], wb[d]);

  int k = 0, j = 0, par = 0;
  float ya = 0.f, yb = 0.f, xsum = 0.f;                                  // grouped: finished sums; per-row: sums of q x and of x
  const int total = my_tasks * per_task;
  for (int it0 = 0; it0 < total; it0 += kMvDepth) {
#pragma unroll
    for (int d = 0; d < kMvDepth; ++d) {
      if (it0 + d < total) {                                             // uniform over the CTA
        const int task = blockIdx.x + k * gridDim.x, blk = warp + j * kMvWarps, ch = blk * 4 + t4;
        const int ra = min(task * 16 + gq, R - 1), rb = min(task * 16 + gq + 8, R - 1);
        float c1[4] = {0.f, 0.f, 0.f, 0.f}, c2[4] = {0.f, 0.f, 0.f, 0.f};
        if (blk < n_blk) mv_chunk<F>(wa[d], wb[d], reinterpret_cast<const uint4*>(xs + ch * 32), c1, c2);
        issue(wa[d], wb[d]);
        if (blk < n_blk) {
          const float da = (c1[0] + c2[0] * MvScale2<F>::inv) * 16777216.f;  // sum of q x over the block, rows a and b
          const float db = (c1[2] + c2[2] * MvScale2<F>::inv) * 16777216.f;
          const float bx = sx[blk];
          if (per_block) {
            const int gi = (blk * 128) / g;
            ya = fmaf(__ldg(scales + (int64_t)ra * G + gi), da - __ldg(zeros + (int64_t)ra * G + gi) * bx, ya);
            yb = fmaf(__ldg(scales + (int64_t)rb * G + gi), db - __ldg(zeros + (int64_t)rb * G + gi) * bx, yb);
          } else {
            ya += da; yb += db; xsum += bx;
          }
        }
        if (++j == per_task) {                                           // the task is complete: combine the warps' partial sums
          if (!per_block) {
            ya = __ldg(scales + ra) * (ya - __ldg(zeros + ra) * xsum);
            yb = __ldg(scales + rb) * (yb - __ldg(zeros + rb) * xsum);
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
          j = 0; ++k; par ^= 1; ya = yb = xsum = 0.f;
        }
      }
    }
  }
}

// ---- y = dequant(Q) x, tensor path with the codes staged through shared memory --------------------------------
// Same arithmetic as matvec_mma_kernel; what differs is how the codes travel.  There a lane loads its own fragment
// words from global memory (16 row segments of 64 bytes per warp instruction, held in registers while in flight).
// Here every warp owns a ring of kDepth stages in shared memory and fills it with asynchronous 16-byte copies
// (cp.async.cg: global -> shared, no register, no L1 allocation) whose lanes cover whole consecutive pieces of a row;
// the lanes then read their fragments from the stage.  Waiting is cp.async.wait_group + __syncwarp only: no
// barrier object and no spin.  A stage is 16 rows x up to kSB blocks of 128 columns; a row of a stage is padded so
// that the fragment reads of a warp fall on distinct banks.
// A task is 16 consecutive rows; warp w of the CTA takes the blocks [w bpw, (w + 1) bpw) of every task in `nsub`
// stages of `sbk` blocks, and the warps' partial sums meet in shared memory as before.
// x is staged once per CTA, permuted as the unpacking wants it and interleaved inside a block: the 16-byte piece i
// (0..3) of chunk t (0..3) sits at piece 4 i + t of the block, so that a warp's four lane groups read 64 consecutive
// bytes.
// Every warp waits on its own chain copy -> fragment read -> mask -> MMA, so the kernel lives on independent work inside a
// warp (blocks per stage, all unrolled) and on warps per SM, and both cost ring memory.  Measured at C = 12288 (49152
// rows): 4-bit 14 warps x 2 stages of 7 blocks 63 us; 12 x 3 x 4 blocks 67; 16 x 4 x 3 blocks 75; 8 x 4 x 4 blocks 71;
// 3-bit 12 x 2 x 8 blocks 82; 12 x 4 x 4 blocks 85; 10 x 2 x 10 blocks 87; 16 x 2 x 6 blocks 83.  A long x leaves less
// room: the launcher takes the first geometry of a short list that fits.
// smallest pitch >= the row's bytes that keeps a warp's fragment reads on distinct banks: 4-bit (one 16-byte read per
// lane, two rows per quarter warp) wants the rows 64 bytes apart modulo 128, 2-bit (8-byte reads, four rows per half
// warp) 32 modulo 128, 3-bit (4-byte reads, eight rows per warp) and 8-bit (two 16-byte reads) 16 modulo 32.
constexpr int mp_pitch(int F, int row_bytes) {
  const int m = F == 4 ? 128 : F == 2 ? 128 : 32, want = F == 4 ? 64 : F == 2 ? 32 : 16;
  int p = (row_bytes + 15) / 16 * 16;
  while (p % m != want) p += 16;
  return p;
}
// W warps per CTA (one CTA per SM), stages of at most SB blocks.
template <int F_, int W, int SB> struct MpGeom {
  static constexpr int F = F_;
  static constexpr int kWarps = W;
  static constexpr int kThreads = kWarps * 32;
  static constexpr int kSB = SB;
  static constexpr int kPiecesPerRow = kSB * F;                               // 16-byte pieces of one row of a stage (<= 32)
  static constexpr int kRowsPerCopy = 32 / kPiecesPerRow;                     // rows one warp-wide copy instruction covers
  static constexpr int kPitch = mp_pitch(F, kSB * 16 * F);                    // bytes between rows of a stage
  static constexpr int kStageBytes = 16 * kPitch;
  static_assert(kPiecesPerRow <= 32 && kSB <= 10, "a row of a stage is copied by one warp instruction");
};

__device__ __forceinline__ void cp_async_16(uint32_t sdst, const void* gsrc, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(sdst), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int F>
__device__ __forceinline__ void mp_read(const unsigned char* p, uint32_t (&w)[F]) {
  if constexpr (F == 4) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
  } else if constexpr (F == 2) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    w[0] = v.x; w[1] = v.y;
  } else if constexpr (F == 8) {
    const uint4 v0 = *reinterpret_cast<const uint4*>(p), v1 = *(reinterpret_cast<const uint4*>(p) + 1);
    w[0] = v0.x; w[1] = v0.y; w[2] = v0.z; w[3] = v0.w; w[4] = v1.x; w[5] = v1.y; w[6] = v1.z; w[7] = v1.w;
  } else {
#pragma unroll
    for (int k = 0; k < F; ++k) w[k] = reinterpret_cast<const uint32_t*>(p)[k];
  }
}

// The eight MMAs of one block for fragment rows a and b, x read in the interleaved order.
template <int F>
__device__ __forceinline__ void mp_block(const uint32_t (&wa)[F], const uint32_t (&wb)[F], const uint4* xb, int t4,
                                         float (&c1)[4], float (&c2)[4]) {
  uint4 xs[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) xs[i] = xb[4 * i + t4];
  mv_chunk<F>(wa, wb, xs, c1, c2);
}

// grid: min(tasks, SMs) CTAs of Geo::kThreads threads.  dynamic shared memory: x (fp16, C rounded up to 128), the block
// sums of x (fp32), two buffers of partial sums, then one ring of kDepth stages per warp.
template <class Geo, int kDepth>
__global__ void __launch_bounds__(Geo::kThreads, 1)
matvec_staged_kernel(const uint32_t* __restrict__ qweight, const float* __restrict__ scales, const float* __restrict__ zeros,
                     const __half* __restrict__ x, int R, int C, int g, int G, int bpw, int nsub, int sbk,
                     float* __restrict__ y) {
  constexpr int F = Geo::F;
  constexpr int kMpWarps = Geo::kWarps;
  extern __shared__ uint4 mv_smem[];
  const int chunks = C / 32, n_blk = (C + 127) / 128, Cpad = n_blk * 128;
  uint4* xs = mv_smem;                                                    // [n_blk][16] pieces
  float* sx = reinterpret_cast<float*>(xs + (size_t)n_blk * 16);          // [n_blk]
  float* red = sx + ((n_blk + 3) & ~3);                                   // [2][kMpWarps][16]
  unsigned char* rings = reinterpret_cast<unsigned char*>(red + 2 * kMpWarps * 16);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gq = lane >> 2, t4 = lane & 3;
  const int n_tasks = (R + 15) / 16;
  const int my_tasks = blockIdx.x < n_tasks ? (n_tasks - 1 - blockIdx.x) / gridDim.x + 1 : 0;
  const bool per_block = g < C;
  const int64_t row_bytes = (int64_t)chunks * F * 4;
  const int blk_lo = warp * bpw, blk_hi = min(blk_lo + bpw, n_blk);        // this warp's blocks of every task
  const int valid_pieces_row = (int)(row_bytes / 16);                     // pieces of a row that exist in memory
  unsigned char* ring = rings + (size_t)warp * kDepth * Geo::kStageBytes;
  const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);
  const unsigned char* qbytes = reinterpret_cast<const unsigned char*>(qweight);

  // copy side: lane -> (row within the copy instruction, piece within the row)
  const int c_row = lane / Geo::kPiecesPerRow, c_piece = lane % Geo::kPiecesPerRow;
  const bool c_lane = lane < Geo::kRowsPerCopy * Geo::kPiecesPerRow;
  int lk = 0, lj = 0, ls = 0;                                             // load cursor: task number, stage of the task, ring slot
  auto issue = [&]() {
    if (lk < my_tasks) {
      const int task = blockIdx.x + lk * gridDim.x;
      const int b0 = blk_lo + lj * sbk, nb = min(sbk, blk_hi - b0);       // blocks of this stage (nb may be <= 0)
      const int piece0 = b0 * F;                                          // first piece of the stage inside the row
      if (c_lane && c_piece < nb * F) {
        const uint32_t fill = piece0 + c_piece < valid_pieces_row ? 16u : 0u;   // past the row's end: zeros
        const int64_t col_off = fill ? (int64_t)(piece0 + c_piece) * 16 : 0;
        uint32_t dst = ring_s + ls * Geo::kStageBytes + c_row * Geo::kPitch + c_piece * 16;
        if (task * 16 + 16 <= R) {
          const unsigned char* src = qbytes + (int64_t)(task * 16 + c_row) * row_bytes + col_off;
#pragma unroll
          for (int r = 0; r < 16; r += Geo::kRowsPerCopy) {
            if (16 % Geo::kRowsPerCopy == 0 || r + c_row < 16) cp_async_16(dst, src, fill);
            src += Geo::kRowsPerCopy * row_bytes;
            dst += Geo::kRowsPerCopy * Geo::kPitch;
          }
        } else {                                                          // ragged last task: rows clamped, copies stay in range
#pragma unroll
          for (int r = 0; r < 16; r += Geo::kRowsPerCopy) {
            const int row = min(task * 16 + r + c_row, R - 1);
            if (16 % Geo::kRowsPerCopy == 0 || r + c_row < 16) cp_async_16(dst, qbytes + row * row_bytes + col_off, fill);
            dst += Geo::kRowsPerCopy * Geo::kPitch;
          }
        }
      }
      if (++lj == nsub) { lj = 0; ++lk; }
    }
    cp_async_commit();                                                    // one group per slot, empty or not
    if (++ls == kDepth) ls = 0;
  };
#pragma unroll
  for (int d = 0; d < kDepth - 1; ++d) issue();            // the first stages are on their way while x is staged

  // x: one 32-column chunk (64 bytes) per thread, permuted, written interleaved; the four threads of a block add up
  // their chunks' sums
  for (int base = warp * 32; base < Cpad / 32; base += blockDim.x) {
    const int ch = base + lane;
    float t = 0.f;
    if (ch < Cpad / 32) {
      __align__(16) __half in[32], out[32];
#pragma unroll
      for (int q = 0; q < 4; ++q)
        reinterpret_cast<uint4*>(in)[q] = ch < chunks ? __ldg(reinterpret_cast<const uint4*>(x + ch * 32) + q) : make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int p = 0; p < 32; ++p) { out[p] = in[mv_perm<F>(p)]; t += __half2float(in[p]); }
#pragma unroll
      for (int q = 0; q < 4; ++q) xs[(ch >> 2) * 16 + 4 * q + (ch & 3)] = reinterpret_cast<const uint4*>(out)[q];
    }
    t += __shfl_xor_sync(0xffffffffu, t, 1);
    t += __shfl_xor_sync(0xffffffffu, t, 2);
    if ((lane & 3) == 0 && ch < Cpad / 32) sx[ch >> 2] = t;
  }
  __syncthreads();

  int k = 0, j = 0, cs = 0, par = 0;
  float ya = 0.f, yb = 0.f, ya2 = 0.f, yb2 = 0.f;
  float rsa = 0.f, rza = 0.f, rsb = 0.f, rzb = 0.f;                       // per-row grids: this task's scale and zero, rows a and b
  float xsum_w = 0.f;                                                     // sum of x over this warp's blocks (the same for every task)
  for (int b = blk_lo; b < blk_hi; ++b) xsum_w += sx[b];
  const int total = my_tasks * nsub;
  for (int it = 0; it < total; ++it) {
    const int task = blockIdx.x + k * gridDim.x;
    const int ra = min(task * 16 + gq, R - 1), rb = min(task * 16 + gq + 8, R - 1);
    const int b0 = blk_lo + j * sbk, nb = min(sbk, blk_hi - b0);
    // grouped grids: the stage's scales and zero-points are requested before the wait for its codes
    float gsa[Geo::kSB], gza[Geo::kSB], gsb[Geo::kSB], gzb[Geo::kSB];
    if (!per_block && j == 0) {                                           // one grid per row: asked for when the task begins,
      rsa = __ldg(scales + ra); rza = __ldg(zeros + ra);                  // used when it ends
      rsb = __ldg(scales + rb); rzb = __ldg(zeros + rb);
    }
    if (per_block) {
#pragma unroll
      for (int b = 0; b < Geo::kSB; ++b) {
        if (b < nb) {
          const int gi = ((b0 + b) * 128) / g;
          gsa[b] = __ldg(scales + (int64_t)ra * G + gi); gza[b] = __ldg(zeros + (int64_t)ra * G + gi);
          gsb[b] = __ldg(scales + (int64_t)rb * G + gi); gzb[b] = __ldg(zeros + (int64_t)rb * G + gi);
        }
      }
    }
    cp_async_wait<kDepth - 2>();                                          // this stage's copies have landed (this lane's)
    __syncwarp();                                                         // ... and every lane's; the previous stage is read
    issue();                                                              // refill the slot read in the previous iteration
    const unsigned char* st = ring + (size_t)cs * Geo::kStageBytes + gq * Geo::kPitch + t4 * (4 * F);
    // one instance per block count, without per-block branches, so that the blocks' loads and MMA chains interleave
    auto run_stage = [&](auto count) {
#pragma unroll
    for (int b = 0; b < Geo::kSB; ++b) {
      if (b < decltype(count)::value) {
        const int blk = b0 + b;
        uint32_t wa[F], wb[F];
        mp_read<F>(st + b * 16 * F, wa);
        mp_read<F>(st + b * 16 * F + 8 * Geo::kPitch, wb);
        float c1[4] = {0.f, 0.f, 0.f, 0.f}, c2[4] = {0.f, 0.f, 0.f, 0.f};
        mp_block<F>(wa, wb, xs + (size_t)blk * 16, t4, c1, c2);
        if (per_block) {
          const float da = (c1[0] + c2[0] * MvScale2<F>::inv) * 16777216.f;
          const float db = (c1[2] + c2[2] * MvScale2<F>::inv) * 16777216.f;
          const float bx = sx[blk];
          ya = fmaf(gsa[b], da - gza[b] * bx, ya);
          yb = fmaf(gsb[b], db - gzb[b] * bx, yb);
        } else {                                                          // one grid per row: the two factors' sums stay apart
          ya += c1[0]; yb += c1[2]; ya2 += c2[0]; yb2 += c2[2];           // until the task ends
        }
      }
    }
    };
    switch (nb) {                                                         // (uniform over the warp)
      case 10: if constexpr (Geo::kSB >= 10) run_stage(std::integral_constant<int, 10>{}); break;
      case 9: if constexpr (Geo::kSB >= 9) run_stage(std::integral_constant<int, 9>{}); break;
      case 8: if constexpr (Geo::kSB >= 8) run_stage(std::integral_constant<int, 8>{}); break;
      case 7: if constexpr (Geo::kSB >= 7) run_stage(std::integral_constant<int, 7>{}); break;
      case 6: if constexpr (Geo::kSB >= 6) run_stage(std::integral_constant<int, 6>{}); break;
      case 5: if constexpr (Geo::kSB >= 5) run_stage(std::integral_constant<int, 5>{}); break;
      case 4: if constexpr (Geo::kSB >= 4) run_stage(std::integral_constant<int, 4>{}); break;
      case 3: if constexpr (Geo::kSB >= 3) run_stage(std::integral_constant<int, 3>{}); break;
      case 2: if constexpr (Geo::kSB >= 2) run_stage(std::integral_constant<int, 2>{}); break;
      case 1: run_stage(std::integral_constant<int, 1>{}); break;
      default: break;
    }
    if (++cs == kDepth) cs = 0;
    if (++j == nsub) {                                                    // the task is complete: combine the warps' partial sums
      if (!per_block) {
        ya = rsa * ((ya + ya2 * MvScale2<F>::inv) * 16777216.f - rza * xsum_w);
        yb = rsb * ((yb + yb2 * MvScale2<F>::inv) * 16777216.f - rzb * xsum_w);
      }
      float* rp = red + (par * kMpWarps + warp) * 16;
      if (t4 == 0) { rp[gq] = ya; rp[gq + 8] = yb; }
      __syncthreads();
      if (threadIdx.x < 16) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < kMpWarps; ++w) t += red[(par * kMpWarps + w) * 16 + threadIdx.x];
        const int r = task * 16 + threadIdx.x;
        if (r < R) y[r] = t;
      }
      j = 0; ++k; par ^= 1; ya = yb = ya2 = yb2 = 0.f;
    }
  }
  cp_async_wait<0>();
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
  const int gx = (C / 8 + 255) / 256;
  int gy = gptq::device_sm_count_inference() * 32 / gx;                  // about 32 CTAs per SM in total
  if (gy < 1) gy = 1;
  if (gy > R) gy = R;
  if (gy > 65535) gy = 65535;
  gptq::dequantize_kernel<F><<<dim3(gx, gy), 256, 0, s>>>(qweight, scales, zeros, R, C, g, G, out);
  GPTQ_LAUNCH_CHECK();
  return GPTQ_OK;
}

template <int F>
gptq_status_t launch_matvec(const uint32_t* qweight, const float* scales, const float* zeros, const __half* x, int R,
                            int C, int g, int G, float* y, cudaStream_t s) {
  if (g == C || g % 128 == 0) {
    // tensor path: x staged as fp16
    const int n_blk = (C + 127) / 128;
    // codes staged through shared memory when a row is a whole number of 16-byte pieces and rings of at least two stages
    // fit beside x: the first geometry that fits, from the one measured best at C = 12288 to smaller rings
    if (((int64_t)(C / 32) * F * 4) % 16 == 0) {
      bool launched = false;
      auto attempt = [&](auto geo) -> gptq_status_t {
        using Geo = decltype(geo);
        const size_t fixed = (size_t)n_blk * 256 + (size_t)((n_blk + 3) & ~3) * sizeof(float) +
                             (size_t)2 * Geo::kWarps * 16 * sizeof(float);
        const size_t ring1 = (size_t)Geo::kWarps * Geo::kStageBytes, budget = 227 * 1024;
        if (fixed + 2 * ring1 > budget) return GPTQ_OK;                   // does not fit: the caller tries the next one
        const int depth = fixed + 4 * ring1 <= budget ? 4 : fixed + 3 * ring1 <= budget ? 3 : 2;
        const int bpw = (n_blk + Geo::kWarps - 1) / Geo::kWarps, nsub = (bpw + Geo::kSB - 1) / Geo::kSB,
                  sbk = (bpw + nsub - 1) / nsub;
        const int tasks = (R + 15) / 16;
        int grid = gptq::device_sm_count_inference();
        if (grid > tasks) grid = tasks;
        const size_t smem = fixed + depth * ring1;
        auto go = [&](auto kern) -> gptq_status_t {
          GPTQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
          kern<<<grid, Geo::kThreads, smem, s>>>(qweight, scales, zeros, x, R, C, g, G, bpw, nsub, sbk, y);
          GPTQ_LAUNCH_CHECK();
          launched = true;
          return GPTQ_OK;
        };
        if (depth == 4) return go(gptq::matvec_staged_kernel<Geo, 4>);
        if (depth == 3) return go(gptq::matvec_staged_kernel<Geo, 3>);
        return go(gptq::matvec_staged_kernel<Geo, 2>);
      };
      gptq_status_t st = GPTQ_OK;
      if constexpr (F == 4) {
        st = attempt(gptq::MpGeom<4, 14, 7>{});
        if (st == GPTQ_OK && !launched) st = attempt(gptq::MpGeom<4, 12, 4>{});
      } else if constexpr (F == 8) {
        st = attempt(gptq::MpGeom<8, 12, 2>{});
      } else {
        st = attempt(gptq::MpGeom<F, 12, 8>{});
        if (st == GPTQ_OK && !launched) st = attempt(gptq::MpGeom<F, 12, 4>{});
      }
      if (st != GPTQ_OK || launched) return st;
    }
    const size_t smem = (size_t)n_blk * 128 * sizeof(__half) + (size_t)((n_blk + 3) & ~3) * sizeof(float) +
                        (size_t)2 * gptq::kMvWarps * 16 * sizeof(float);
    if (smem > 220 * 1024 / gptq::kMvCtasPerSm) return GPTQ_ERR_UNSUPPORTED;
    const int tasks = (R + 15) / 16;
    int grid = gptq::kMvCtasPerSm * gptq::device_sm_count_inference();
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
  if (!aligned_to(W_out_fp16, 16) || !aligned_to(qweight, 4)) return GPTQ_ERR_INVALID_ARG;   // 16-byte stores, 4-byte loads
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
  if (!aligned_to(x_fp16, 16) || !aligned_to(qweight, 16)) return GPTQ_ERR_INVALID_ARG;   // both are read in 16-byte pieces
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
