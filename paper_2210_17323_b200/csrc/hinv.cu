// Stage 2: dampening and U = Cholesky((H + lambda I)^-1)^T   (Section 3, Step 3; Algorithm 1 line 3).
//
// Route: factor H~ = U~ U~^T with U~ UPPER triangular (a Cholesky factorisation that runs from
// the last row/column backwards), then U = U~^-1.  U is upper triangular with positive diagonal
// and U^T U = U~^-T U~^-1 = H~^-1, so by uniqueness it is the matrix Algorithm 1 asks for, at
// 2 C^3 / 3 flops and without ever forming H~^-1.
//
// Blocked with 128-wide panels: diagonal blocks are factored and inverted in fp64 in shared
// memory by one CTA; panel and trailing products are fp32 tile GEMMs.
#include "common.cuh"
#include "gemm_simt.cuh"

namespace gptq {
namespace {

constexpr int kNB = 128;

__global__ void lambda_kernel(const float* __restrict__ H, int C, float damp, double* __restrict__ lam) {
  __shared__ double red[32];
  double s = 0.0;
  for (int i = threadIdx.x; i < C; i += blockDim.x) s += (double)H[(int64_t)i * C + i];
  for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x < 32) {
    s = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.0;
    for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
    if (threadIdx.x == 0) *lam = (double)damp * (s / (double)C);
  }
}

// U <- upper triangle of (H + lambda I); strict lower triangle <- 0.
__global__ void init_upper_damped_kernel(const float* __restrict__ H, float* __restrict__ U, int C,
                                         const double* __restrict__ lam) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t total = (int64_t)C * C / 4;
  if (idx >= total) return;
  int r = (int)(idx * 4 / C), c = (int)(idx * 4 % C);
  float4 v = reinterpret_cast<const float4*>(H)[idx];
  float o[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int cc = c + i;
    o[i] = cc < r ? 0.f : (cc == r ? (float)((double)o[i] + *lam) : o[i]);
  }
  reinterpret_cast<float4*>(U)[idx] = make_float4(o[0], o[1], o[2], o[3]);
}

// One CTA: factor the nb x nb diagonal block at (k0, k0) as A = T T^T with T upper (backwards
// Cholesky), store T in place (fp32) and its inverse V = T^-1 (upper) to Dinv (fp32, ld = kNB).
// A non-positive pivot is reported and replaced by 1 so everything downstream stays finite.
__global__ void __launch_bounds__(256)
rchol_diag_kernel(float* __restrict__ U, int C, int k0, int nb, float* __restrict__ Dinv, int* dev_info) {
  extern __shared__ double sm[];
  const int LD = kNB + 1;
  double* S = sm;               // [nb][LD]: T in the upper triangle; V^T (strictly upper part of V) in the lower
  double* vd = sm + kNB * LD;   // [nb]: diagonal of V
  const int tid = threadIdx.x, nt = blockDim.x;
  for (int e = tid; e < nb * nb; e += nt) {
    int i = e / nb, j = e % nb;
    S[i * LD + j] = j >= i ? (double)U[(int64_t)(k0 + i) * C + k0 + j] : 0.0;
  }
  __syncthreads();
  for (int j = nb - 1; j >= 0; --j) {
    double d = S[j * LD + j];
    __syncthreads();
    if (!(d > 0.0)) {
      if (tid == 0) report_error(dev_info, GPTQ_ERR_NOT_PD, k0 + j);
      d = 1.0;
    }
    double piv = sqrt(d), rp = 1.0 / piv;
    for (int i = tid; i < j; i += nt) S[i * LD + j] *= rp;
    if (tid == 0) S[j * LD + j] = piv;
    __syncthreads();
    // trailing update of the leading j x j upper part: A[i][i2] -= T[i][j] T[i2][j], i <= i2 < j
    for (int e = tid; e < j * j; e += nt) {
      int i = e / j, i2 = e % j;
      if (i <= i2) S[i * LD + i2] -= S[i * LD + j] * S[i2 * LD + j];
    }
    __syncthreads();
  }
  // V = T^-1, one column c per thread (back substitution up the column); V[i][c], i < c, is kept
  // at S[c][i] (the unused lower triangle), V[c][c] in vd[c].
  for (int c = tid; c < nb; c += nt) {
    const double vcc = 1.0 / S[c * LD + c];
    vd[c] = vcc;
    for (int i = c - 1; i >= 0; --i) {
      double s = S[i * LD + c] * vcc;
      for (int k = i + 1; k < c; ++k) s += S[i * LD + k] * S[c * LD + k];
      S[c * LD + i] = -s / S[i * LD + i];
    }
  }
  __syncthreads();
  for (int e = tid; e < nb * nb; e += nt) {
    int i = e / nb, j = e % nb;
    if (j >= i) U[(int64_t)(k0 + i) * C + k0 + j] = (float)S[i * LD + j];
    Dinv[i * kNB + j] = j > i ? (float)S[j * LD + i] : (j == i ? (float)vd[i] : 0.f);
  }
}

__global__ void store_diag_block_kernel(float* __restrict__ U, int C, int k0, int nb,
                                        const float* __restrict__ Dinv) {
  for (int e = threadIdx.x + blockIdx.x * blockDim.x; e < nb * nb; e += blockDim.x * gridDim.x) {
    int i = e / nb, j = e % nb;
    U[(int64_t)(k0 + i) * C + k0 + j] = Dinv[i * kNB + j];
  }
}

struct UpperTiles {
  int K;
  __device__ __forceinline__ bool operator()(int m0, int n0, int, int, int& k0, int& k1) const {
    k0 = 0; k1 = K;
    return m0 <= n0 + kSimtBN - 1;
  }
};
// K starts at the tile's first row: the left factor is upper triangular.
struct UpperLeftFactorRange {
  int K;
  __device__ __forceinline__ bool operator()(int m0, int, int, int, int& k0, int& k1) const {
    k0 = m0; k1 = K;
    return k0 < k1;
  }
};
struct StoreF32 {
  float* p; int64_t ld;
  __device__ __forceinline__ void operator()(int m, int n, float acc) const { p[(int64_t)m * ld + n] = acc; }
};
struct StoreNegF32 {
  float* p; int64_t ld;
  __device__ __forceinline__ void operator()(int m, int n, float acc) const { p[(int64_t)m * ld + n] = -acc; }
};
struct SubUpperF32 {
  float* p; int64_t ld;
  __device__ __forceinline__ void operator()(int m, int n, float acc) const {
    if (m <= n) p[(int64_t)m * ld + n] -= acc;
  }
};

}  // namespace
}  // namespace gptq

extern "C" size_t gptq_prepare_hinv_workspace_bytes(int C) {
  using namespace gptq;
  if (C <= 0) return 0;
  WsCarver w(nullptr);
  w.take<double>(1);                                        // lambda
  w.take<float>((size_t)ceil_div(C, kNB) * kNB * kNB);      // inverses of the diagonal blocks
  w.take<float>((size_t)C * kNB);                           // panel temporary
  return w.off;
}

extern "C" gptq_status_t gptq_prepare_hinv(const float* H, float damp, int C, float* U,
                                           void* ws, size_t ws_bytes, int* dev_info, void* stream) {
  using namespace gptq;
  if (!H || !U || !dev_info || C <= 0 || C % 32 != 0 || H == U || !(damp >= 0.f)) return GPTQ_ERR_INVALID_ARG;
  if (!aligned_to(H, 16) || !aligned_to(U, 16)) return GPTQ_ERR_INVALID_ARG;
  if (!ws || !aligned_to(ws, kAlign) || ws_bytes < gptq_prepare_hinv_workspace_bytes(C)) return GPTQ_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  WsCarver w(ws);
  const int nbk = ceil_div(C, kNB);
  double* lam = w.take<double>(1);
  float* Dinv = w.take<float>((size_t)nbk * kNB * kNB);
  float* T = w.take<float>((size_t)C * kNB);

  const int diag_smem = (kNB * (kNB + 1) + kNB) * (int)sizeof(double);
  GPTQ_CUDA_TRY(cudaFuncSetAttribute(rchol_diag_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, diag_smem));
  GPTQ_CUDA_TRY(cudaMemsetAsync(dev_info, 0, 2 * sizeof(int), s));
  lambda_kernel<<<1, 1024, 0, s>>>(H, C, damp, lam);
  GPTQ_LAUNCH_CHECK();
  {
    int64_t total = (int64_t)C * C / 4;
    init_upper_damped_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(H, U, C, lam);
    GPTQ_LAUNCH_CHECK();
  }
  // Phase 1: backwards blocked Cholesky, H~ = U~ U~^T, in place in U's upper triangle.
  for (int kb = nbk - 1; kb >= 0; --kb) {
    const int k0 = kb * kNB, nb = (C - k0 < kNB) ? C - k0 : kNB;
    float* Dk = Dinv + (size_t)kb * kNB * kNB;
    rchol_diag_kernel<<<1, 256, diag_smem, s>>>(U, C, k0, nb, Dk, dev_info);
    GPTQ_LAUNCH_CHECK();
    if (k0 == 0) break;
    // panel: U~[0:k0, blk] = A[0:k0, blk] * T_kk^-T      (out[m][n] = sum_k A[m][k0+k] V[n][k])
    GPTQ_CUDA_TRY(launch_gemm_simt(k0, nb, 1, RowMajorF32{U + k0, C}, RowMajorF32T{Dk, kNB},
                                   FullRange{nb}, StoreF32{U + k0, C}, s));
    // trailing: A[0:k0, 0:k0] -= P P^T on upper tiles     (P = U~[0:k0, blk])
    GPTQ_CUDA_TRY(launch_gemm_simt(k0, k0, 1, RowMajorF32{U + k0, C}, RowMajorF32T{U + k0, C},
                                   UpperTiles{nb}, SubUpperF32{U, C}, s));
  }
  // Phase 2: U = U~^-1, column block by column block, in place.
  for (int kb = 0; kb < nbk; ++kb) {
    const int k0 = kb * kNB, nb = (C - k0 < kNB) ? C - k0 : kNB;
    float* Dk = Dinv + (size_t)kb * kNB * kNB;
    if (k0 > 0) {
      // T = U~[0:k0, blk] * V_kk
      GPTQ_CUDA_TRY(launch_gemm_simt(k0, nb, 1, RowMajorF32{U + k0, C}, RowMajorF32{Dk, kNB},
                                     FullRange{nb}, StoreF32{T, kNB}, s));
      // U[0:k0, blk] = -U[0:k0, 0:k0] * T   (left factor already inverted, upper triangular)
      GPTQ_CUDA_TRY(launch_gemm_simt(k0, nb, 1, RowMajorF32{U, C}, RowMajorF32{T, kNB},
                                     UpperLeftFactorRange{k0}, StoreNegF32{U + k0, C}, s));
    }
    store_diag_block_kernel<<<8, 256, 0, s>>>(U, C, k0, nb, Dk);
    GPTQ_LAUNCH_CHECK();
  }
  return GPTQ_OK;
}
