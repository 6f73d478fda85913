// Stage 1: H += 2 * sum_t x_t x_t^T  (Section 2, "Optimal Brain Quantization": H = 2 X X^T;
// Algorithm 1 caption).  X arrives token-major (n_tokens x C, bf16).
//
// Only tiles that touch the upper triangle are computed; a mirror pass copies the strict
// upper triangle onto the lower one so both are valid (and exactly symmetric) on return.
#include "common.cuh"
#include "gemm_simt.cuh"
#include "hessian_umma.cuh"

namespace gptq {

namespace {

// A(m, k) = X[k][m]  (the paper's X is C x tokens; memory holds its transpose)
struct XtAsA {
  static constexpr bool kInnerContig = false;
  const __nv_bfloat16* x; int64_t C;
  __device__ __forceinline__ float operator()(int m, int k) const {
    return __bfloat162float(x[(int64_t)k * C + m]);
  }
};
struct XtAsB {
  static constexpr bool kInnerContig = true;
  const __nv_bfloat16* x; int64_t C;
  __device__ __forceinline__ float operator()(int k, int n) const {
    return __bfloat162float(x[(int64_t)k * C + n]);
  }
};
// Tiles strictly below the diagonal are skipped; tokens are split over blockIdx.z.
struct UpperTilesSplitK {
  int64_t n_tokens;
  __device__ __forceinline__ bool operator()(int m0, int n0, int z, int nz, int& k0, int& k1) const {
    if (m0 > n0 + kSimtBN - 1) return false;
    int64_t per = ((n_tokens + nz - 1) / nz + kSimtBK - 1) / kSimtBK * kSimtBK;
    int64_t a = (int64_t)z * per, b = a + per < n_tokens ? a + per : n_tokens;
    k0 = (int)a; k1 = (int)b;
    return a < b;
  }
};
struct AddTwiceUpper {
  float* H; int64_t C;
  __device__ __forceinline__ void operator()(int m, int n, float acc) const {
    if (m <= n) atomicAdd(&H[(int64_t)m * C + n], 2.f * acc);
  }
};

__global__ void mirror_upper_to_lower_kernel(float* __restrict__ H, int C) {
  // 32x32 tiles through shared memory so both the read and the write are coalesced
  __shared__ float t[32][33];
  int bi = blockIdx.y, bj = blockIdx.x;
  if (bi > bj) return;
  int r = bi * 32 + threadIdx.y, c = bj * 32 + threadIdx.x;
  t[threadIdx.y][threadIdx.x] = H[(int64_t)r * C + c];
  __syncthreads();
  int rr = bj * 32 + threadIdx.y, cc = bi * 32 + threadIdx.x;  // transposed position
  if (rr > cc) H[(int64_t)rr * C + cc] = t[threadIdx.x][threadIdx.y];
}

}  // namespace

cudaError_t launch_mirror_upper_to_lower(float* H, int C, cudaStream_t stream) {
  dim3 grid(C / 32, C / 32), block(32, 32);
  mirror_upper_to_lower_kernel<<<grid, block, 0, stream>>>(H, C);
  count_launch();
  return cudaGetLastError();
}

static gptq_status_t hessian_simt(float* H, const __nv_bfloat16* X, int64_t n_tokens, int C,
                                  cudaStream_t stream, bool mirror) {
  const int64_t kMaxTokensPerLaunch = 1 << 30;  // K indices are 32-bit inside the tile kernel
  for (int64_t t0 = 0; t0 < n_tokens; t0 += kMaxTokensPerLaunch) {
    int64_t nt = n_tokens - t0 < kMaxTokensPerLaunch ? n_tokens - t0 : kMaxTokensPerLaunch;
    const __nv_bfloat16* x = X + t0 * C;
    int tiles = ceil_div(C, kSimtBM);
    int upper = tiles * (tiles + 1) / 2;
    int nz = 1;
    while (upper * nz < 2 * 148 && nz * 2 * 512 <= nt) nz *= 2;
    GPTQ_CUDA_TRY(launch_gemm_simt(C, C, nz, XtAsA{x, C}, XtAsB{x, C}, UpperTilesSplitK{nt},
                                   AddTwiceUpper{H, C}, stream));
  }
  if (mirror) GPTQ_CUDA_TRY(launch_mirror_upper_to_lower(H, C, stream));
  return GPTQ_OK;
}

}  // namespace gptq

extern "C" size_t gptq_hessian_workspace_bytes(int C, int64_t n_tokens) {
  (void)C; (void)n_tokens;
  return 0;
}

static gptq_status_t hessian_accumulate_impl(float* H, const void* X_bf16, int64_t n_tokens, int C, int* dev_info,
                                             void* stream, bool mirror) {
  using namespace gptq;
  if (!H || C <= 0 || C % 32 != 0 || n_tokens < 0) return GPTQ_ERR_INVALID_ARG;
  if (n_tokens == 0) return GPTQ_OK;
  if (!X_bf16 || !aligned_to(X_bf16, 16) || !aligned_to(H, 16)) return GPTQ_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16* X = static_cast<const __nv_bfloat16*>(X_bf16);
  if (dev_info) GPTQ_CUDA_TRY(cudaMemsetAsync(dev_info, 0, 2 * sizeof(int), s));
  if (hessian_umma_supported(C, n_tokens)) return hessian_umma(H, X, n_tokens, C, dev_info, s, mirror);
  return hessian_simt(H, X, n_tokens, C, s, mirror);
}

extern "C" gptq_status_t gptq_hessian_accumulate(float* H, const void* X_bf16, int64_t n_tokens, int C,
                                                 void* ws, size_t ws_bytes, int* dev_info, void* stream) {
  (void)ws; (void)ws_bytes;
  return hessian_accumulate_impl(H, X_bf16, n_tokens, C, dev_info, stream, true);
}

extern "C" gptq_status_t gptq_hessian_accumulate_upper(float* H, const void* X_bf16, int64_t n_tokens, int C,
                                                       void* ws, size_t ws_bytes, int* dev_info, void* stream) {
  (void)ws; (void)ws_bytes;
  return hessian_accumulate_impl(H, X_bf16, n_tokens, C, dev_info, stream, false);
}

extern "C" gptq_status_t gptq_hessian_symmetrize(float* H, int C, void* stream) {
  using namespace gptq;
  if (!H || C <= 0 || C % 32 != 0 || !aligned_to(H, 16)) return GPTQ_ERR_INVALID_ARG;
  GPTQ_CUDA_TRY(launch_mirror_upper_to_lower(H, C, static_cast<cudaStream_t>(stream)));
  return GPTQ_OK;
}
