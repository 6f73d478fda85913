// Generic CUDA-core (FFMA) tile GEMM used for the parts of the solver that are not on the
// tensor pipe: small / triangular products of the factorisation and as the plain-fp32
// contraction for shapes the tensor-core kernels do not cover.
//
//   for every tile (m0, n0):   acc[m][n] = sum_{k in [k0,k1)} A(m,k) * B(k,n)   (fp32 FMA)
//                              epi(m, n, acc[m][n])
//
// A, B: functors `float operator()(int m_or_k, int k_or_n) const` (do their own dtype
//       conversion and addressing; only called with in-range indices).
//       `static constexpr bool kInnerContig` says whether the SECOND index is the one that
//       is contiguous in memory (used to choose a coalesced tile-load pattern).
// Range: functor `bool operator()(int m0, int n0, int z, int nz, int& k0, int& k1) const`;
//       returns false to skip the tile (e.g. below the diagonal), sets the K range of this
//       tile / split (z of nz = blockIdx.z of gridDim.z).
// Epi:  functor `void operator()(int m, int n, float acc) const`.
#pragma once
#include "common.cuh"

namespace gptq {

constexpr int kSimtBM = 128, kSimtBN = 128, kSimtBK = 16, kSimtThreads = 256;

template <class AF, class BF, class RangeF, class EpiF>
__global__ void __launch_bounds__(kSimtThreads)
gemm_simt_kernel(int M, int N, AF a, BF b, RangeF range, EpiF epi) {
  constexpr int BM = kSimtBM, BN = kSimtBN, BK = kSimtBK;
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  int k0, k1;
  if (!range(m0, n0, (int)blockIdx.z, (int)gridDim.z, k0, k1)) return;
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;  // thread tile: rows ty*8.., cols tx*8..
  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  for (int kt = k0; kt < k1; kt += BK) {
#pragma unroll
    for (int i = 0; i < (BM * BK) / kSimtThreads; ++i) {
      int e = tid + i * kSimtThreads, m, k;
      if (AF::kInnerContig) { k = e % BK; m = e / BK; } else { m = e % BM; k = e / BM; }
      As[k][m] = (m0 + m < M && kt + k < k1) ? a(m0 + m, kt + k) : 0.f;
    }
#pragma unroll
    for (int i = 0; i < (BN * BK) / kSimtThreads; ++i) {
      int e = tid + i * kSimtThreads, n, k;
      if (BF::kInnerContig) { n = e % BN; k = e / BN; } else { k = e % BK; n = e / BK; }
      Bs[k][n] = (n0 + n < N && kt + k < k1) ? b(kt + k, n0 + n) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float af[8], bf[8];
      *reinterpret_cast<float4*>(&af[0]) = *reinterpret_cast<const float4*>(&As[k][ty * 8]);
      *reinterpret_cast<float4*>(&af[4]) = *reinterpret_cast<const float4*>(&As[k][ty * 8 + 4]);
      *reinterpret_cast<float4*>(&bf[0]) = *reinterpret_cast<const float4*>(&Bs[k][tx * 8]);
      *reinterpret_cast<float4*>(&bf[4]) = *reinterpret_cast<const float4*>(&Bs[k][tx * 8 + 4]);
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(af[i], bf[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    int m = m0 + ty * 8 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      int n = n0 + tx * 8 + j;
      if (n < N) epi(m, n, acc[i][j]);
    }
  }
}

template <class AF, class BF, class RangeF, class EpiF>
inline cudaError_t launch_gemm_simt(int M, int N, int nz, AF a, BF b, RangeF range, EpiF epi,
                                    cudaStream_t stream) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  dim3 grid((N + kSimtBN - 1) / kSimtBN, (M + kSimtBM - 1) / kSimtBM, nz);
  gemm_simt_kernel<<<grid, kSimtThreads, 0, stream>>>(M, N, a, b, range, epi);
  count_launch();
  return cudaGetLastError();
}

// ---- common functors --------------------------------------------------------------------
// Row-major fp32 matrix element (row, col); second index contiguous.
struct RowMajorF32 {
  static constexpr bool kInnerContig = true;
  const float* p; int64_t ld;
  __device__ __forceinline__ float operator()(int r, int c) const { return p[(int64_t)r * ld + c]; }
};
// Transposed view of a row-major fp32 matrix: element (i, j) = p[j][i]; first index contiguous.
struct RowMajorF32T {
  static constexpr bool kInnerContig = false;
  const float* p; int64_t ld;
  __device__ __forceinline__ float operator()(int i, int j) const { return p[(int64_t)j * ld + i]; }
};
// Full K range, no tile skipped, optional split over blockIdx.z in multiples of the K tile.
struct FullRange {
  int K;
  __device__ __forceinline__ bool operator()(int, int, int z, int nz, int& k0, int& k1) const {
    int per = ((K + nz - 1) / nz + kSimtBK - 1) / kSimtBK * kSimtBK;
    k0 = z * per; k1 = min(K, k0 + per);
    return k0 < k1;
  }
};

}  // namespace gptq
