// Small fp32 CUDA-core GEMM for the latency-bound products inside a 1024-column panel of the
// factorisation (M, N <= 1024, K a few hundred): what matters there is the time of ONE launch, not
// throughput.  64 x BN output tiles (many CTAs even for small outputs), the whole K extent of a
// 128-wide chunk staged in shared memory with one round of wide loads, then 128 uninterrupted
// FFMA steps.
//
//   acc[m][n] = sum_{k in [k0,k1)} A[m][k] * Bop[k][n],   epi(m, n, acc)
//
// A is row-major [M][K] (K contiguous).  B is either row-major [N][K] (kBisNK: the product is
// A * B^T) or row-major [K][N].  All leading dimensions and offsets are multiples of 4 floats and
// the bases 16-byte aligned.  Range functor: bool operator()(m0, n0, int& k0, int& k1) -- false
// skips the tile; k0 a multiple of 4.  Epilogue functor: void operator()(m, n, acc).
#pragma once
#include "common.cuh"

namespace gptq {
namespace small {

constexpr int BM = 64, KC = 128, kThreads = 256;

template <int BN>
constexpr size_t smem_bytes() { return (size_t)KC * (BM + 4) * 4 + (size_t)KC * (BN + 4) * 4; }

template <int BN, bool kBisNK, class RangeF, class EpiF>
__global__ void __launch_bounds__(kThreads)
gemm_small_kernel(const float* __restrict__ A, int64_t lda, const float* __restrict__ B, int64_t ldb,
                  int M, int N, RangeF range, EpiF epi) {
  static_assert(BN == 64 || BN == 128, "tile width");
  constexpr int TN = BN / 16;                       // output columns per thread (4 or 8)
  extern __shared__ __align__(16) float smem_f[];
  float (*As)[BM + 4] = reinterpret_cast<float (*)[BM + 4]>(smem_f);
  float (*Bs)[BN + 4] = reinterpret_cast<float (*)[BN + 4]>(smem_f + KC * (BM + 4));
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  int k0, k1;
  if (!range(m0, n0, k0, k1)) return;
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  float acc[4][TN];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  for (int kc = k0; kc < k1; kc += KC) {
    const int kw = min(KC, k1 - kc);
    // A chunk: lanes along m (each lane one row, 16 bytes of k), stored transposed As[k][m]
#pragma unroll
    for (int i = 0; i < (BM * KC / 4) / kThreads; ++i) {
      const int idx = t + kThreads * i, m = idx & (BM - 1), kq = idx / BM;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (m0 + m < M && 4 * kq < kw) v = *reinterpret_cast<const float4*>(A + (int64_t)(m0 + m) * lda + kc + 4 * kq);
      As[4 * kq][m] = v.x; As[4 * kq + 1][m] = v.y; As[4 * kq + 2][m] = v.z; As[4 * kq + 3][m] = v.w;
    }
    if (kBisNK) {
#pragma unroll
      for (int i = 0; i < (BN * KC / 4) / kThreads; ++i) {
        const int idx = t + kThreads * i, n = idx & (BN - 1), kq = idx / BN;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (n0 + n < N && 4 * kq < kw) v = *reinterpret_cast<const float4*>(B + (int64_t)(n0 + n) * ldb + kc + 4 * kq);
        Bs[4 * kq][n] = v.x; Bs[4 * kq + 1][n] = v.y; Bs[4 * kq + 2][n] = v.z; Bs[4 * kq + 3][n] = v.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < (BN * KC / 4) / kThreads; ++i) {
        const int idx = t + kThreads * i, nq = idx % (BN / 4), k = idx / (BN / 4);
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (k < kw && n0 + 4 * nq < N) v = *reinterpret_cast<const float4*>(B + (int64_t)(kc + k) * ldb + n0 + 4 * nq);
        *reinterpret_cast<float4*>(&Bs[k][4 * nq]) = v;
      }
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < kw; ++k) {
      const float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      const float af[4] = {a.x, a.y, a.z, a.w};
      float bf[TN];
#pragma unroll
      for (int h = 0; h < TN / 4; ++h) {
        const float4 b = *reinterpret_cast<const float4*>(&Bs[k][h * 64 + tx * 4]);
        bf[4 * h] = b.x; bf[4 * h + 1] = b.y; bf[4 * h + 2] = b.z; bf[4 * h + 3] = b.w;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(af[i], bf[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int n = n0 + (j >> 2) * 64 + tx * 4 + (j & 3);
      if (n < N) epi(m, n, acc[i][j]);
    }
  }
}

template <int BN, bool kBisNK, class RangeF, class EpiF>
inline cudaError_t launch(const float* A, int64_t lda, const float* B, int64_t ldb, int M, int N, RangeF range,
                          EpiF epi, cudaStream_t stream) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  auto kern = gemm_small_kernel<BN, kBisNK, RangeF, EpiF>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes<BN>());
  if (e != cudaSuccess) return e;
  dim3 grid((N + BN - 1) / BN, (M + BM - 1) / BM);
  kern<<<grid, kThreads, smem_bytes<BN>(), stream>>>(A, lda, B, ldb, M, N, range, epi);
  count_launch();
  return cudaGetLastError();
}

// ---- range functors ---------------------------------------------------------------------------
struct AllK {                      // every tile, k in [0, K)
  int K;
  __device__ __forceinline__ bool operator()(int, int, int& k0, int& k1) const { k0 = 0; k1 = K; return K > 0; }
};
template <int BN>
struct UpperTiles {                // only tiles that reach the part on or above the diagonal, k in [0, K)
  int K;
  __device__ __forceinline__ bool operator()(int m0, int n0, int& k0, int& k1) const {
    k0 = 0; k1 = K;
    return m0 <= n0 + BN - 1;
  }
};
template <int BN>
struct UpperRightFactor {          // B[k][n] upper triangular (zero for k > n): k in [0, min(K, n0 + BN))
  int K;
  __device__ __forceinline__ bool operator()(int, int n0, int& k0, int& k1) const {
    k0 = 0; k1 = min(K, n0 + BN);
    return k1 > 0;
  }
};

}  // namespace small
}  // namespace gptq
