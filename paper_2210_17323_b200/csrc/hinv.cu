// Stage 2: dampening and U = Cholesky((H + lambda I)^-1)^T   (Section 3, Step 3; Algorithm 1 line 3).
//
// Route: factor H~ = U~ U~^T with U~ UPPER triangular (a Cholesky factorisation that runs from
// the last row/column backwards), then U = U~^-1.  U is upper triangular with positive diagonal
// and U^T U = U~^-T U~^-1 = H~^-1, so by uniqueness it is the matrix Algorithm 1 asks for, at
// 2 C^3 / 3 flops and without ever forming H~^-1.
//
// Two-level blocking.  128 x 128 diagonal blocks are factored and inverted in fp64 (registers) by
// one CTA; products inside a 1024-column outer panel are small fp32 CUDA-core GEMMs
// (gemm_small.cuh); everything that reaches across outer panels (almost all of the flops for
// large C) is a left-looking fp32-accurate tensor-core contraction over fp16 hi / lo copies of the
// factor (three kind::f16 products per term, gemm_umma_f16.cuh) that are written as each panel is
// finalised.  fp16's narrow exponent range is met with exact power-of-two scalings (below).  The launches of one
// call go to three streams (dependency chain, wide contractions, diagonal-block inverses): see
// gptq_prepare_hinv below.
#include "common.cuh"
#include "gemm_small.cuh"
#include "gemm_umma_f16.cuh"

#include <mutex>

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
__global__ void init_upper_damped_kernel(const float* H, float* U, int C,
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
// Both run in fp64, fused in one sweep over the columns j = nb-1 .. 0: column j of T and row j of V
// (solving T V = I from the bottom row up) are finished together, and both trailing updates,
//   A[i][c] -= T[i][j] T[c][j]   (i <= c < j)      and      B[c][i] -= T[c][j] V[j][i]   (c < j <= i),
// where B is the running right-hand side of the solve, are the same formula on one working matrix M
// whose upper triangle holds A / T and whose strictly lower triangle holds B / V transposed:
//   M[i][c] -= x_j[i] * T[c][j]   for c < j and (c >= i or i >= j),   x_j[i] = T[i][j] (i < j), V[j][i] (i >= j).
// M lives in REGISTERS (32 doubles per thread, element (i, c) with i = tx + 32 a, c = ty + 16 b,
// ty = warp), so a column belongs to ONE warp.  Updates are batched lazily, four columns at a time
// (the same idea as Algorithm 1's Step 2, one level down): inside a batch only the owning warp of
// the next column applies the pending updates to that column, takes the pivot, scales and
// publishes it through shared memory; after the batch every warp applies the four rank-1 updates
// to its other elements in one pass.  Register arrays are indexed by compile-time constants only
// (thread coordinates are compared, never loop indices).
// A non-positive pivot is reported and replaced by 1 so everything downstream stays finite.
constexpr int kDiagThreads = 512;
constexpr int kDiagBatch = 4;
// Owner warp, column j = slots M[.][B] (rows i = tx + 32 a): apply the batch's pending updates to the
// column, take the pivot, scale the column and publish it as colv[q][.] (colv[q][j] = 1 / pivot).
template <int B>
__device__ __forceinline__ void diag_owner_step(double (&M)[4][8], double (*colv)[kNB], double* pd, int q, int j, int jt,
                                                int tx, int k0, int* dev_info) {
  double piv_c = 0.0;
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    const int i = tx + 32 * a;
    for (int qq = 0; qq < q; ++qq)
      if (i >= jt - qq || j >= i) M[a][B] -= colv[qq][i] * colv[qq][j];
    if (i == j) piv_c = M[a][B];
  }
  double d = __shfl_sync(0xffffffffu, piv_c, j & 31);
  if (!(d > 0.0)) {
    if (tx == 0) report_error(dev_info, GPTQ_ERR_NOT_PD, k0 + j);
    d = 1.0;
  }
  const double rp = rsqrt(d), piv = d * rp;
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    const int i = tx + 32 * a;
    if (i == j) { pd[j] = piv; colv[q][i] = rp; }
    else { M[a][B] *= rp; colv[q][i] = M[a][B]; }
  }
}
__global__ void __launch_bounds__(kDiagThreads)
rchol_diag_kernel(float* __restrict__ U, int C, int k0, int nb, float* __restrict__ Dinv, int* dev_info) {
  __shared__ double colv[kDiagBatch][kNB];   // published columns of the current batch: colv[q][i] = x_{jt-q}[i]
  __shared__ double pd[kNB];                 // diagonal of T
  const int tid = threadIdx.x, tx = tid & 31, ty = tid >> 5;
  double M[4][8];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      const int i = tx + 32 * a, c = ty + 16 * b;
      M[a][b] = (i < nb && c < nb && c >= i) ? (double)U[(int64_t)(k0 + i) * C + k0 + c] : 0.0;
    }
  for (int jt = nb - 1; jt >= 0; jt -= kDiagBatch) {
#pragma unroll
    for (int q = 0; q < kDiagBatch; ++q) {
      const int j = jt - q;
      if (ty == (j & 15)) {
        // owner warp of column j (its slots have b == j >> 4).  Inside a batch a column is handed from its owner to
        // the next column's owner alone (a two-warp named barrier; consecutive columns have different owners): the
        // other fourteen warps have nothing to do until the batch is complete and wait for the full barrier below.
        if (q > 0) asm volatile("bar.sync %0, 64;" ::"r"(q) : "memory");
        // dispatch once on b so that the four slots are addressed with compile-time indices
        switch (j >> 4) {
          case 0: diag_owner_step<0>(M, colv, pd, q, j, jt, tx, k0, dev_info); break;
          case 1: diag_owner_step<1>(M, colv, pd, q, j, jt, tx, k0, dev_info); break;
          case 2: diag_owner_step<2>(M, colv, pd, q, j, jt, tx, k0, dev_info); break;
          case 3: diag_owner_step<3>(M, colv, pd, q, j, jt, tx, k0, dev_info); break;
          case 4: diag_owner_step<4>(M, colv, pd, q, j, jt, tx, k0, dev_info); break;
          case 5: diag_owner_step<5>(M, colv, pd, q, j, jt, tx, k0, dev_info); break;
          case 6: diag_owner_step<6>(M, colv, pd, q, j, jt, tx, k0, dev_info); break;
          default: diag_owner_step<7>(M, colv, pd, q, j, jt, tx, k0, dev_info); break;
        }
        if (q + 1 < kDiagBatch) asm volatile("bar.arrive %0, 64;" ::"r"(q + 1) : "memory");
      }
    }
    __syncthreads();
    // the batch's four rank-1 updates on every element left of the batch
    const int jlow = jt - (kDiagBatch - 1);
    double x[kDiagBatch][4];
    bool below[kDiagBatch][4];
#pragma unroll
    for (int q = 0; q < kDiagBatch; ++q)
#pragma unroll
      for (int a = 0; a < 4; ++a) { const int i = tx + 32 * a; x[q][a] = colv[q][i]; below[q][a] = i >= jt - q; }
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      const int c = ty + 16 * b;
      if (c < jlow) {                                // warp-uniform
        double tc[kDiagBatch];
#pragma unroll
        for (int q = 0; q < kDiagBatch; ++q) tc[q] = colv[q][c];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          const bool upper = c >= tx + 32 * a;
#pragma unroll
          for (int q = 0; q < kDiagBatch; ++q)
            if (upper || below[q][a]) M[a][b] -= x[q][a] * tc[q];
        }
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      const int i = tx + 32 * a, c = ty + 16 * b;
      if (i < nb && c < nb) {
        if (c > i) U[(int64_t)(k0 + i) * C + k0 + c] = (float)M[a][b];
        else if (c == i) { U[(int64_t)(k0 + i) * C + k0 + c] = (float)pd[i]; Dinv[i * kNB + i] = (float)(1.0 / pd[i]); }
        // V[c][i] (c < i) sits in M[i][c]; the strictly lower part of V is zero
        if (c < i) { Dinv[c * kNB + i] = (float)M[a][b]; Dinv[i * kNB + c] = 0.f; }
      }
    }
}

__global__ void store_diag_block_kernel(float* __restrict__ U, int C, int k0, int nb,
                                        const float* __restrict__ Dinv) {
  for (int e = threadIdx.x + blockIdx.x * blockDim.x; e < nb * nb; e += blockDim.x * gridDim.x) {
    int i = e / nb, j = e % nb;
    U[(int64_t)(k0 + i) * C + k0 + j] = Dinv[i * kNB + j];
  }
}

struct StoreF32 {
  float* p; int64_t ld;
  __device__ __forceinline__ void operator()(int m, int n, float acc) const { p[(int64_t)m * ld + n] = acc; }
};
struct StoreNegF32 {
  float* p; int64_t ld;
  __device__ __forceinline__ void operator()(int m, int n, float acc) const { p[(int64_t)m * ld + n] = -acc; }
};
struct SubUpperOfsF32 {   // p[m][nofs + n] -= acc where that element is on or above the diagonal
  float* p; int64_t ld; int nofs;
  __device__ __forceinline__ void operator()(int m, int n, float acc) const {
    if (m <= nofs + n) p[(int64_t)m * ld + nofs + n] -= acc;
  }
};

// ---- power-of-two scalings of the fp16 operand pairs ------------------------------------------------
// With d_i = sqrt(H~_ii) (the norm of row i of the factor U~, H~ = U~ U~^T) and r_i the power of two with
// r_i d_i in [0.5, 1), every operand is brought into fp16's range by exact scalings that the epilogues undo:
//   rows of the factor          F'[i][k]  = U~[i][k] * r_i 2^12                          (|.| < 2^12: an entry is at most its row's norm)
//   Schur-complement blocks     A'[i][j]  = A[i][j] * r_i 2^12 * r_j                     (|A_ij| <= d_i d_j)
//   inverse of a diagonal block V'[j'][j] = V[j'][j] / r_j * g_j'                        (g_j' from the row's actual maximum, < 2^15)
//   its transpose (phase 2)     VT'[j'][j] = V[j][j'] * gam_j'                           (gam_j' from the column's actual maximum, < 2^15)
//   T = V^T U~^T (phase 2)      T'[j'][i] = T[j'][i] * r_i * gam_j' 2^-5                 (|.| < 2^15 by Cauchy-Schwarz)
//   rows of the inverse         U'[i][k]  = U[i][k] / r_k * u_i                          (u_i brings the diagonal entry to ~2^9; saturated and
//                                                                                         reported if an entry still leaves the range)
// r_i 2^12 is called rs_i below.
__global__ void factor_scales_kernel(const float* __restrict__ U, int C, float* __restrict__ r, float* __restrict__ rinv,
                                     float* __restrict__ rs, float* __restrict__ rsinv) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= C) return;
  const float ri = pow2_scale_to(sqrtf(U[(int64_t)i * C + i]), 0);
  r[i] = ri; rinv[i] = 1.f / ri; rs[i] = ri * 4096.f; rsinv[i] = 1.f / (ri * 4096.f);
}
// One CTA per row / column index b of the w x w block V at D (leading dimension ld):
//   g[b]   brings max_j |V[b][j]| / r[j] just below 2^15,  ginv = 1 / g
//   gam[b] brings max_j |V[j][b]|        just below 2^15,  gam2inv = 2^5 / gam
__global__ void panel_scales_kernel(const float* __restrict__ D, int64_t ld, int w, const float* __restrict__ rinv,
                                    float* __restrict__ g, float* __restrict__ ginv, float* __restrict__ gam, float* __restrict__ gam2inv) {
  __shared__ float red[2][32];
  const int b = blockIdx.x;
  float mr = 0.f, mc = 0.f;
  for (int j = threadIdx.x; j < w; j += blockDim.x) {
    mr = fmaxf(mr, fabsf(D[(int64_t)b * ld + j]) * rinv[j]);
    mc = fmaxf(mc, fabsf(D[(int64_t)j * ld + b]));
  }
  for (int o = 16; o > 0; o >>= 1) { mr = fmaxf(mr, __shfl_xor_sync(0xffffffffu, mr, o)); mc = fmaxf(mc, __shfl_xor_sync(0xffffffffu, mc, o)); }
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = mr; red[1][threadIdx.x >> 5] = mc; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int k = 1; k < (int)(blockDim.x >> 5); ++k) { mr = fmaxf(mr, red[0][k]); mc = fmaxf(mc, red[1][k]); }
    const float gg = pow2_scale_to(mr, 15), cc = pow2_scale_to(mc, 15);
    g[b] = gg; ginv[b] = 1.f / gg; gam[b] = cc; gam2inv[b] = 32.f / cc;
  }
}
// u[i] brings the diagonal entry of row i of the inverse, U_ii / r_i, to about 2^9;  uinv = 1 / u
__global__ void inverse_row_scales_kernel(const float* __restrict__ U, int C, const float* __restrict__ rinv,
                                          float* __restrict__ u, float* __restrict__ uinv) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= C) return;
  const float ui = pow2_scale_to(fabsf(U[(int64_t)i * C + i]) * rinv[i], 9);
  u[i] = ui; uinv[i] = 1.f / ui;
}

// ---- tensor-core epilogues: one thread, one row, 32 consecutive columns of a partial sum ---------------
// Every epilogue multiplies the partial sum by sa[row] * sb[col] (powers of two: the operands' scalings undone).
// dst[row][cofs + col] -= partial for elements on or above the diagonal (fp32 reductions).
struct EpiSubUpperRed {
  float* p; int64_t ld; int cofs; int M, N;
  const float* sa; const float* sb;
  __device__ __forceinline__ void operator()(int row, int col0, const float (&v)[32]) const {
    if (row >= M || col0 >= N) return;
    float* d = p + (int64_t)row * ld + cofs + col0;
    const float a = -sa[row];
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      const int c = cofs + col0 + 4 * g;            // global column of the group's first element
      const float4 b = *reinterpret_cast<const float4*>(sb + col0 + 4 * g);
      const float x0 = v[4 * g] * a * b.x, x1 = v[4 * g + 1] * a * b.y, x2 = v[4 * g + 2] * a * b.z, x3 = v[4 * g + 3] * a * b.w;
      if (c >= row) umma::red_add_v4(d + 4 * g, x0, x1, x2, x3);
      else if (c + 3 >= row) {
        if (c + 1 >= row) atomicAdd(d + 4 * g + 1, x1);
        if (c + 2 >= row) atomicAdd(d + 4 * g + 2, x2);
        atomicAdd(d + 4 * g + 3, x3);
      }
    }
  }
};
// dst[row][col] = partial * sa[row] * sb[col] * factor (fp32).  Only valid when the contraction is a single super-chunk.
struct EpiStoreScaledF32 {
  float* p; int64_t ld; int M, N;
  const float* sa; const float* sb; float factor;
  __device__ __forceinline__ void operator()(int row, int col0, const float (&v)[32]) const {
    if (row >= M || col0 >= N) return;
    float4* d = reinterpret_cast<float4*>(p + (int64_t)row * ld + col0);
    const float a = sa[row] * factor;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      const float4 b = *reinterpret_cast<const float4*>(sb + col0 + 4 * g);
      d[g] = make_float4(v[4 * g] * a * b.x, v[4 * g + 1] * a * b.y, v[4 * g + 2] * a * b.z, v[4 * g + 3] * a * b.w);
    }
  }
};
// Stores partial * factor as an fp16 hi / lo pair.  Only valid when the contraction is a single super-chunk
// (K <= f16x3::kSuperK), so that the partial sum IS the result.
struct EpiStoreSplit {
  __half* hi; __half* lo; int64_t ld; int M, N; float factor; int* dev_info;
  __device__ __forceinline__ void operator()(int row, int col0, const float (&v)[32]) const {
    if (row >= M || col0 >= N) return;
    uint4* h = reinterpret_cast<uint4*>(hi + (int64_t)row * ld + col0);
    uint4* l = reinterpret_cast<uint4*>(lo + (int64_t)row * ld + col0);
    bool sat = false;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      uint32_t hw[4], lw[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        __half h0, l0, h1, l1;
        f16x3::split_f16(v[8 * g + 2 * u] * factor, h0, l0, sat);
        f16x3::split_f16(v[8 * g + 2 * u + 1] * factor, h1, l1, sat);
        hw[u] = (uint32_t)__half_as_ushort(h0) | ((uint32_t)__half_as_ushort(h1) << 16);
        lw[u] = (uint32_t)__half_as_ushort(l0) | ((uint32_t)__half_as_ushort(l1) << 16);
      }
      h[g] = make_uint4(hw[0], hw[1], hw[2], hw[3]); l[g] = make_uint4(lw[0], lw[1], lw[2], lw[3]);
    }
    if (sat) report_error(dev_info, GPTQ_ERR_NONFINITE, row);
  }
};

// Stores partial * sa[row] * sb[col] as fp32 into the factor AND partial * sb[col] (= that value * rs[row], the scaling of
// the factor's rows) as an fp16 hi / lo pair into its split copies (same offsets, leading dimension ldf).
// Single super-chunk contractions only, like EpiStoreSplit.
struct EpiStoreF32AndSplit {
  float* u; int64_t ldu; __half* hi; __half* lo; int64_t ldf; int M, N;
  const float* sa; const float* sb; int* dev_info;
  __device__ __forceinline__ void operator()(int row, int col0, const float (&v)[32]) const {
    if (row >= M || col0 >= N) return;
    float4* d = reinterpret_cast<float4*>(u + (int64_t)row * ldu + col0);
    uint4* h = reinterpret_cast<uint4*>(hi + (int64_t)row * ldf + col0);
    uint4* l = reinterpret_cast<uint4*>(lo + (int64_t)row * ldf + col0);
    const float a = sa[row];
    bool sat = false;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      uint32_t hw[4], lw[4];
      float x[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) x[e] = v[8 * g + e] * sb[col0 + 8 * g + e];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        __half h0, l0, h1, l1;
        f16x3::split_f16(x[2 * e], h0, l0, sat);
        f16x3::split_f16(x[2 * e + 1], h1, l1, sat);
        hw[e] = (uint32_t)__half_as_ushort(h0) | ((uint32_t)__half_as_ushort(h1) << 16);
        lw[e] = (uint32_t)__half_as_ushort(l0) | ((uint32_t)__half_as_ushort(l1) << 16);
      }
      d[2 * g] = make_float4(x[0] * a, x[1] * a, x[2] * a, x[3] * a);
      d[2 * g + 1] = make_float4(x[4] * a, x[5] * a, x[6] * a, x[7] * a);
      h[g] = make_uint4(hw[0], hw[1], hw[2], hw[3]); l[g] = make_uint4(lw[0], lw[1], lw[2], lw[3]);
    }
    if (sat) report_error(dev_info, GPTQ_ERR_NONFINITE, row);
  }
};

// dst{hi,lo}[r][c] = split(src[r][c] * sr[r] * sc[c]) for r < rows, c < w (w a multiple of 4; 16-byte aligned rows).
__global__ void split_scaled_kernel(const float* __restrict__ src, int64_t ld_src, int rows, int w,
                                    const float* __restrict__ sr, const float* __restrict__ sc,
                                    __half* __restrict__ dhi, __half* __restrict__ dlo, int64_t ld_dst, int* dev_info) {
  const int q = w / 4;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)rows * q) return;
  const int r = (int)(idx / q), c = (int)(idx % q) * 4;
  const float4 v = *reinterpret_cast<const float4*>(src + (int64_t)r * ld_src + c);
  const float4 b = *reinterpret_cast<const float4*>(sc + c);
  const float a = sr[r];
  __half h[4], l[4];
  bool sat = false;
  f16x3::split_f16(v.x * a * b.x, h[0], l[0], sat); f16x3::split_f16(v.y * a * b.y, h[1], l[1], sat);
  f16x3::split_f16(v.z * a * b.z, h[2], l[2], sat); f16x3::split_f16(v.w * a * b.w, h[3], l[3], sat);
  *reinterpret_cast<uint2*>(dhi + (int64_t)r * ld_dst + c) =
      make_uint2((uint32_t)__half_as_ushort(h[0]) | ((uint32_t)__half_as_ushort(h[1]) << 16),
                 (uint32_t)__half_as_ushort(h[2]) | ((uint32_t)__half_as_ushort(h[3]) << 16));
  *reinterpret_cast<uint2*>(dlo + (int64_t)r * ld_dst + c) =
      make_uint2((uint32_t)__half_as_ushort(l[0]) | ((uint32_t)__half_as_ushort(l[1]) << 16),
                 (uint32_t)__half_as_ushort(l[2]) | ((uint32_t)__half_as_ushort(l[3]) << 16));
  if (sat) report_error(dev_info, GPTQ_ERR_NONFINITE, r);
}
// VT{hi,lo}[c][r] = split(U[j0 + r][j0 + c] * gam[c]) for r, c < w  (transpose of a diagonal block, ld = ldv).
__global__ void split_diag_t_kernel(const float* __restrict__ U, int C, int j0, const float* __restrict__ gam,
                                    __half* __restrict__ Vhi, __half* __restrict__ Vlo, int ldv) {
  __shared__ float t[32][33];
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
  t[threadIdx.y][threadIdx.x] = U[(int64_t)(j0 + r0 + threadIdx.y) * C + j0 + c0 + threadIdx.x];
  __syncthreads();
  __half h, l;
  bool sat = false;
  f16x3::split_f16(t[threadIdx.x][threadIdx.y] * gam[c0 + threadIdx.y], h, l, sat);
  const int64_t o = (int64_t)(c0 + threadIdx.y) * ldv + r0 + threadIdx.x;
  Vhi[o] = h; Vlo[o] = l;
}

constexpr int kNB2 = 1024;   // outer panel width: contractions over everything outside it run on the tensor cores

struct HinvWs {
  double* lam; float* Dinv; float* T; __half* Fhi; __half* Flo; __half* VThi; __half* VTlo; __half* TThi; __half* TTlo;
  __half* Vhi[2]; __half* Vlo[2]; __half* TAhi; __half* TAlo;
  float* r; float* rinv; float* rs; float* rsinv; float* u; float* uinv;      // [C] each
  float* g[2]; float* ginv[2]; float* gam; float* gam2inv;                     // [kNB2] each
  size_t bytes;
};
HinvWs carve_hinv(void* ws, int C) {
  WsCarver w(ws);
  HinvWs o;
  o.lam = w.take<double>(1);
  o.Dinv = w.take<float>((size_t)ceil_div(C, kNB) * kNB * kNB);   // inverses of the 128 x 128 diagonal blocks
  o.T = w.take<float>((size_t)C * kNB);                           // panel temporary (CUDA-core path)
  const bool outer = C > kNB2;
  o.Fhi = w.take<__half>(outer ? (size_t)C * C : 0);              // scaled fp16 hi / lo of the factor as it is finalised
  o.Flo = w.take<__half>(outer ? (size_t)C * C : 0);
  o.VThi = w.take<__half>(outer ? (size_t)kNB2 * kNB2 : 0);       // transposed inverse of an outer diagonal block
  o.VTlo = w.take<__half>(outer ? (size_t)kNB2 * kNB2 : 0);
  o.TThi = w.take<__half>(outer ? (size_t)kNB2 * C : 0);          // (U~[0:j0, J] V_JJ)^T
  o.TTlo = w.take<__half>(outer ? (size_t)kNB2 * C : 0);
  for (int i = 0; i < 2; ++i) {                                   // inverse of an outer diagonal block, two in flight
    o.Vhi[i] = w.take<__half>(outer ? (size_t)kNB2 * kNB2 : 0);
    o.Vlo[i] = w.take<__half>(outer ? (size_t)kNB2 * kNB2 : 0);
  }
  o.TAhi = w.take<__half>(outer ? (size_t)kNB2 * kNB2 : 0);       // split copy of the row block above a diagonal block
  o.TAlo = w.take<__half>(outer ? (size_t)kNB2 * kNB2 : 0);
  const size_t nc = outer ? (size_t)C : 0, np = outer ? (size_t)kNB2 : 0;
  o.r = w.take<float>(nc); o.rinv = w.take<float>(nc); o.rs = w.take<float>(nc); o.rsinv = w.take<float>(nc);
  o.u = w.take<float>(nc); o.uinv = w.take<float>(nc);
  for (int i = 0; i < 2; ++i) { o.g[i] = w.take<float>(np); o.ginv[i] = w.take<float>(np); }
  o.gam = w.take<float>(np); o.gam2inv = w.take<float>(np);
  o.bytes = w.off;
  return o;
}

}  // namespace
}  // namespace gptq

extern "C" size_t gptq_prepare_hinv_workspace_bytes(int C) {
  using namespace gptq;
  if (C <= 0) return 0;
  return carve_hinv(nullptr, C).bytes;
}

// ---- second stream and events for the look-ahead schedule -----------------------------------------
// Phase 1 is issued on two streams: the caller's stream carries the dependency chain (diagonal blocks),
// an internal stream carries the wide contractions that only later panels wait for.  The internal
// stream and the events are created once per device, on the first call for that device, and never
// destroyed; they hold no device memory.  Both streams are joined before the call returns, so the
// caller sees ordinary stream semantics (the call is also capturable into a CUDA graph, where the
// two streams become two branches).
namespace gptq {
namespace {
constexpr int kMaxOuter = 64;          // C <= 65536
struct HinvAsync {
  cudaStream_t bulk = nullptr, side = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr, side_done = nullptr;
  cudaEvent_t step[8];
  cudaEvent_t c3[kMaxOuter], c4[kMaxOuter], b1[kMaxOuter], b2[kMaxOuter];
  bool ready = false;
};
constexpr int kMaxAsyncDevices = 64;
HinvAsync g_async[kMaxAsyncDevices];
std::mutex g_async_mutex;

gptq_status_t get_async(HinvAsync** out) {
  int dev = -1;
  GPTQ_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxAsyncDevices) return GPTQ_ERR_UNSUPPORTED;
  HinvAsync& a = g_async[dev];
  if (!a.ready) {
    GPTQ_CUDA_TRY(cudaStreamCreateWithFlags(&a.bulk, cudaStreamNonBlocking));
    GPTQ_CUDA_TRY(cudaStreamCreateWithFlags(&a.side, cudaStreamNonBlocking));
    GPTQ_CUDA_TRY(cudaEventCreateWithFlags(&a.side_done, cudaEventDisableTiming));
    for (int i = 0; i < 8; ++i) GPTQ_CUDA_TRY(cudaEventCreateWithFlags(&a.step[i], cudaEventDisableTiming));
    GPTQ_CUDA_TRY(cudaEventCreateWithFlags(&a.fork, cudaEventDisableTiming));
    GPTQ_CUDA_TRY(cudaEventCreateWithFlags(&a.join, cudaEventDisableTiming));
    for (int i = 0; i < kMaxOuter; ++i) {
      GPTQ_CUDA_TRY(cudaEventCreateWithFlags(&a.c3[i], cudaEventDisableTiming));
      GPTQ_CUDA_TRY(cudaEventCreateWithFlags(&a.c4[i], cudaEventDisableTiming));
      GPTQ_CUDA_TRY(cudaEventCreateWithFlags(&a.b1[i], cudaEventDisableTiming));
      GPTQ_CUDA_TRY(cudaEventCreateWithFlags(&a.b2[i], cudaEventDisableTiming));
    }
    a.ready = true;
  }
  *out = &a;
  return GPTQ_OK;
}

gptq_status_t launch_split_scaled(const float* src, int64_t ld_src, int rows, int w, const float* sr, const float* sc,
                                  __half* dhi, __half* dlo, int64_t ld_dst, int* dev_info, cudaStream_t s) {
  if (rows <= 0 || w <= 0) return GPTQ_OK;
  const int64_t total = (int64_t)rows * (w / 4);
  split_scaled_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(src, ld_src, rows, w, sr, sc, dhi, dlo, ld_dst, dev_info);
  GPTQ_LAUNCH_CHECK();
  return GPTQ_OK;
}
}  // namespace
}  // namespace gptq

namespace gptq {
namespace {
// Both forms of stage 2: the whole of it (U = U~^-1), or phase 1 alone (factor_only: U~ above the diagonal blocks of
// 1024 columns, the inverses of U~'s diagonal blocks -- which are U's diagonal blocks -- on them).
gptq_status_t prepare_impl(const float* H, float damp, int C, float* U, void* ws, size_t ws_bytes, int* dev_info,
                           void* stream, bool factor_only) {
  if (!H || !U || !dev_info || C <= 0 || C % 32 != 0 || !(damp >= 0.f)) return GPTQ_ERR_INVALID_ARG;
  // U == H is allowed: lambda is taken from H's diagonal first, then every element of U is written from the element
  // of H at the same position by the same thread.
  if (!aligned_to(H, 16) || !aligned_to(U, 16)) return GPTQ_ERR_INVALID_ARG;
  if (!ws || !aligned_to(ws, kAlign) || ws_bytes < gptq_prepare_hinv_workspace_bytes(C)) return GPTQ_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  HinvWs w = carve_hinv(ws, C);
  gptq_status_t st;
  const bool outer = C > kNB2;
  const int n_outer = ceil_div(C, kNB2);
  if (n_outer > kMaxOuter) return GPTQ_ERR_UNSUPPORTED;
  const int reserve = 16;   // SMs the wide stream's contractions leave free for the chain stream's kernels

  // enqueueing is serialised per process: the events below are shared by all calls on a device
  std::lock_guard<std::mutex> lock(g_async_mutex);
  HinvAsync* as = nullptr;
  cudaStream_t sb = s, ss = s;                      // a single panel (C <= 1024) stays on the caller's stream
  if (outer) {
    if ((st = get_async(&as)) != GPTQ_OK) return st;
    sb = as->bulk; ss = as->side;
  }

  GPTQ_CUDA_TRY(cudaMemsetAsync(dev_info, 0, 2 * sizeof(int), s));
  lambda_kernel<<<1, 1024, 0, s>>>(H, C, damp, w.lam);
  GPTQ_LAUNCH_CHECK();
  {
    int64_t total = (int64_t)C * C / 4;
    init_upper_damped_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(H, U, C, w.lam);
    GPTQ_LAUNCH_CHECK();
  }
  if (outer) {
    // scalings of the fp16 operand pairs that follow from the damped diagonal alone
    factor_scales_kernel<<<ceil_div(C, 256), 256, 0, s>>>(U, C, w.r, w.rinv, w.rs, w.rsinv);
    GPTQ_LAUNCH_CHECK();
    GPTQ_CUDA_TRY(cudaEventRecord(as->fork, s));
    GPTQ_CUDA_TRY(cudaStreamWaitEvent(sb, as->fork, 0));
    GPTQ_CUDA_TRY(cudaStreamWaitEvent(ss, as->fork, 0));
  }

  // Phase 1: backwards blocked Cholesky H~ = U~ U~^T in U's upper triangle, outer panels of kNB2 columns
  // from the last to the first, left-looking: a panel receives the contributions of all later columns in
  // one contraction over the tf32 hi / lo copies F of the finished factor.  Per panel J (rows j0..rows_p
  // are its diagonal block D, "row block J-1" are the kNB2 rows above D):
  //   chain stream                                         wide stream
  //   C1  D -= F[J rows, later] F[J rows, later]^T         B1  A[0:j0, J] -= F[0:j0, later] F[J rows, later]^T
  //   C2  factor D (128-wide steps inside D)               B2  U~[0:j0-kNB2, J] = A[..] V^T -> U and F   (after C3)
  //   C3  V = D^-1 in place (final U block), split copy
  //   C4  U~[row block J-1, J] = A[..] V^T -> U and F      (after B1)
  // C1 of panel J needs row block J of every later panel: panel J+1's comes from its C4 (same stream),
  // the others from B2 of panels >= J+2, which had the whole chain of panel J+1 to finish.
  auto phase1 = [&]() -> gptq_status_t {
  for (int J = n_outer - 1; J >= 0; --J) {
    const int j0 = J * kNB2, wj = (C - j0 < kNB2) ? C - j0 : kNB2, rows_p = j0 + wj;
    const int K = C - rows_p;                       // later columns
    float* D = U + (int64_t)j0 * C + j0;
    if (K > 0) {
      if (J + 2 < n_outer) GPTQ_CUDA_TRY(cudaStreamWaitEvent(s, as->b2[J + 2], 0));
      // C1
      f16x3::Operand A{w.Fhi + (int64_t)j0 * C + rows_p, w.Flo + (int64_t)j0 * C + rows_p, wj, K, C};
      st = f16x3::launch<false, true>(A, A, wj, wj, EpiSubUpperRed{D, C, 0, wj, wj, w.rsinv + j0, w.rsinv + j0}, dev_info, s);
      if (st != GPTQ_OK) return st;
      if (j0 > 0) {
        // B1
        GPTQ_CUDA_TRY(cudaStreamWaitEvent(sb, as->c4[J + 1], 0));
        f16x3::Operand A1{w.Fhi + rows_p, w.Flo + rows_p, j0, K, C};
        CUtensorMap out;
        if ((st = f16x3::make_out_map_f32(&out, U + j0, j0, wj, C)) != GPTQ_OK) return st;
        st = f16x3::launch<false, false>(A1, A, j0, wj, f16x3::EpiTileAddF32{j0, wj, -1.f, w.rsinv, w.rsinv + j0}, dev_info, sb,
                                         reserve, &out);
        if (st != GPTQ_OK) return st;
        GPTQ_CUDA_TRY(cudaEventRecord(as->b1[J], sb));
      }
    }
    // C2: 128-wide steps inside D (rows j0 .. k0 of the panel only).  C3 runs beside it on a side stream:
    // as soon as block k is factored, row block k of V = D^-1 follows from the rows below it,
    //   V[k, after] = -V_kk (U~[k, after] V[after, after]),
    // in place (row block k of the factor is not read again by the factorisation).
    float* Ub = U + (int64_t)j0 * C;                // first row of D
    const int ldt = wj;                             // leading dimension of the side stream's 128 x rem temporary
    for (int k0 = j0 + (wj - 1) / kNB * kNB; k0 >= j0; k0 -= kNB) {
      const int nb = (rows_p - k0 < kNB) ? rows_p - k0 : kNB;
      float* Dk = w.Dinv + (size_t)(k0 / kNB) * kNB * kNB;
      rchol_diag_kernel<<<1, kDiagThreads, 0, s>>>(U, C, k0, nb, Dk, dev_info);
      GPTQ_LAUNCH_CHECK();
      if (outer) {
        cudaEvent_t ev = as->step[(k0 - j0) / kNB];
        GPTQ_CUDA_TRY(cudaEventRecord(ev, s));
        GPTQ_CUDA_TRY(cudaStreamWaitEvent(ss, ev, 0));
      }
      const int after = k0 + nb, rem = rows_p - after;
      if (rem > 0) {
        float* Vaa = U + (int64_t)after * C + after;
        float* Rk = U + (int64_t)k0 * C + after;    // row block k, columns after it
        GPTQ_CUDA_TRY((small::launch<64, false>(Rk, C, Vaa, C, nb, rem, small::UpperRightFactor<64>{rem},
                                                StoreF32{w.T, ldt}, ss)));
        GPTQ_CUDA_TRY((small::launch<64, false>(Dk, kNB, w.T, ldt, nb, rem, small::AllK{nb}, StoreNegF32{Rk, C}, ss)));
      }
      store_diag_block_kernel<<<8, 256, 0, ss>>>(U, C, k0, nb, Dk);
      GPTQ_LAUNCH_CHECK();
      const int m = k0 - j0;                        // rows of D above this block
      if (m == 0) break;
      // P = A[j0:k0, blk] * T_kk^-T, in place (one tile spans the block's columns)
      GPTQ_CUDA_TRY((small::launch<128, true>(Ub + k0, C, Dk, kNB, m, nb, small::AllK{nb}, StoreF32{Ub + k0, C}, s)));
      // A[j0:k0, j0:k0] -= P P^T on upper tiles
      GPTQ_CUDA_TRY((small::launch<64, true>(Ub + k0, C, Ub + k0, C, m, m, small::UpperTiles<64>{nb},
                                             SubUpperOfsF32{Ub + j0, C, 0}, s)));
    }
    if (outer) {
      GPTQ_CUDA_TRY(cudaEventRecord(as->side_done, ss));
      GPTQ_CUDA_TRY(cudaStreamWaitEvent(s, as->side_done, 0));
    }
    if (!outer || j0 == 0) continue;
    __half* Vhi = w.Vhi[J & 1]; __half* Vlo = w.Vlo[J & 1];
    float* gJ = w.g[J & 1]; float* ginvJ = w.ginv[J & 1];
    // V' = V / r (columns) * g (rows, from the rows' actual maxima); gam of this panel is recomputed in phase 2
    panel_scales_kernel<<<wj, 256, 0, s>>>(D, C, wj, w.rinv + j0, gJ, ginvJ, w.gam, w.gam2inv);
    GPTQ_LAUNCH_CHECK();
    if ((st = launch_split_scaled(D, C, wj, wj, gJ, w.rinv + j0, Vhi, Vlo, kNB2, dev_info, s)) != GPTQ_OK) return st;
    GPTQ_CUDA_TRY(cudaEventRecord(as->c3[J], s));
    f16x3::Operand V{Vhi, Vlo, wj, wj, kNB2};
    const int r1 = j0 - kNB2;                       // first row of row block J-1
    // B2 (rows above row block J-1)
    if (r1 > 0) {
      GPTQ_CUDA_TRY(cudaStreamWaitEvent(sb, as->c3[J], 0));
      if ((st = launch_split_scaled(U + j0, C, r1, wj, w.rs, w.r + j0, w.TThi, w.TTlo, kNB2, dev_info, sb)) != GPTQ_OK) return st;
      f16x3::Operand A2{w.TThi, w.TTlo, r1, wj, kNB2};
      st = f16x3::launch<false, false>(A2, V, r1, wj,
                                       EpiStoreF32AndSplit{U + j0, C, w.Fhi + j0, w.Flo + j0, C, r1, wj, w.rsinv, ginvJ, dev_info},
                                       dev_info, sb, reserve);
      if (st != GPTQ_OK) return st;
    }
    GPTQ_CUDA_TRY(cudaEventRecord(as->b2[J], sb));
    // C4 (row block J-1)
    if (K > 0) GPTQ_CUDA_TRY(cudaStreamWaitEvent(s, as->b1[J], 0));
    {
      const int64_t o = (int64_t)r1 * C + j0;
      if ((st = launch_split_scaled(U + o, C, kNB2, wj, w.rs + r1, w.r + j0, w.TAhi, w.TAlo, kNB2, dev_info, s)) != GPTQ_OK) return st;
      f16x3::Operand A4{w.TAhi, w.TAlo, kNB2, wj, kNB2};
      st = f16x3::launch<false, false>(A4, V, kNB2, wj,
                                       EpiStoreF32AndSplit{U + o, C, w.Fhi + o, w.Flo + o, C, kNB2, wj, w.rsinv + r1, ginvJ, dev_info},
                                       dev_info, s);
      if (st != GPTQ_OK) return st;
    }
    GPTQ_CUDA_TRY(cudaEventRecord(as->c4[J], s));
  }
  return GPTQ_OK;
  };
  st = phase1();
  if (outer) {
    // Join the internal streams into the caller's stream whether or not phase 1 was enqueued completely:
    // an error return must not leave work on them that the caller's stream does not wait for (inside a
    // stream capture that would invalidate the capture; outside, later calls share these streams).
    const cudaError_t j1 = cudaEventRecord(as->join, sb), j2 = cudaStreamWaitEvent(s, as->join, 0);
    const cudaError_t j3 = cudaEventRecord(as->side_done, ss), j4 = cudaStreamWaitEvent(s, as->side_done, 0);
    if (st == GPTQ_OK && (j1 != cudaSuccess || j2 != cudaSuccess || j3 != cudaSuccess || j4 != cudaSuccess)) st = GPTQ_ERR_CUDA;
  }
  if (st != GPTQ_OK) return st;
  if (factor_only) {
    // The factor form's consumer multiplies residuals by U~[before, J] U_JJ (see gptq_prepare_factor): form that product
    // once here, panel by panel, from the fp16 copies of the factor's rows and the transposed diagonal block -- the first
    // of phase 2's two contractions per panel, written out in fp32 over U~[0:j0, J]; the second one (the inverse's rows,
    // K up to C) is what this form leaves out.
    for (int J = 1; J < n_outer; ++J) {
      const int j0 = J * kNB2, wj = (C - j0 < kNB2) ? C - j0 : kNB2;
      panel_scales_kernel<<<wj, 256, 0, s>>>(U + (int64_t)j0 * C + j0, C, wj, w.rinv + j0, w.g[0], w.ginv[0], w.gam, w.gam2inv);
      GPTQ_LAUNCH_CHECK();
      dim3 grid(ceil_div(wj, 32), ceil_div(wj, 32)), blk(32, 32);
      split_diag_t_kernel<<<grid, blk, 0, s>>>(U, C, j0, w.gam, w.VThi, w.VTlo, kNB2);
      GPTQ_LAUNCH_CHECK();
      f16x3::Operand A{w.Fhi + j0, w.Flo + j0, j0, wj, C};          // U~[0:j0, J] rs_i
      f16x3::Operand B{w.VThi, w.VTlo, wj, wj, kNB2};               // V_JJ[k][n] gam_n, as [n][k]
      // partial = rs_i gam_n (U~ V)[i][n];  1 / gam_n = gam2inv_n / 32
      st = f16x3::launch<false, false>(A, B, j0, wj, EpiStoreScaledF32{U + j0, C, j0, wj, w.rsinv, w.gam2inv, 1.f / 32.f}, dev_info, s);
      if (st != GPTQ_OK) return st;
    }
    return GPTQ_OK;
  }

  // Phase 2: U = U~^-1, outer panel by outer panel, in place.  The diagonal blocks are already inverted;
  // rows above them: U[0:j0, J] = -U[0:j0, 0:j0] * (U~[0:j0, J] * V_JJ).
  for (int J = 1; J < n_outer; ++J) {
    const int j0 = J * kNB2, wj = (C - j0 < kNB2) ? C - j0 : kNB2, rows_p = j0 + wj;
    if (J == 1) {                                   // row scales of the inverse; split copy of its first panel
      inverse_row_scales_kernel<<<ceil_div(C, 256), 256, 0, s>>>(U, C, w.rinv, w.u, w.uinv);
      GPTQ_LAUNCH_CHECK();
      if ((st = launch_split_scaled(U, C, kNB2, kNB2, w.u, w.rinv, w.Fhi, w.Flo, C, dev_info, s)) != GPTQ_OK) return st;
    }
    panel_scales_kernel<<<wj, 256, 0, s>>>(U + (int64_t)j0 * C + j0, C, wj, w.rinv + j0, w.g[0], w.ginv[0], w.gam, w.gam2inv);
    GPTQ_LAUNCH_CHECK();
    dim3 grid(ceil_div(wj, 32), ceil_div(wj, 32)), blk(32, 32);
    split_diag_t_kernel<<<grid, blk, 0, s>>>(U, C, j0, w.gam, w.VThi, w.VTlo, kNB2);
    GPTQ_LAUNCH_CHECK();
    // TT = V_JJ^T * U~[0:j0, J]^T   (wj x j0), written as a hi / lo pair (single super-chunk: K = wj)
    {
      f16x3::Operand A{w.VThi, w.VTlo, wj, wj, kNB2};
      f16x3::Operand B{w.Fhi + j0, w.Flo + j0, j0, wj, C};
      // partial = gam_j' rs_i T; stored as T r_i gam_j' 2^-5 = partial 2^-17
      st = f16x3::launch<false, false>(A, B, wj, j0, EpiStoreSplit{w.TThi, w.TTlo, C, wj, j0, 1.f / 131072.f, dev_info}, dev_info, s);
      if (st != GPTQ_OK) return st;
    }
    GPTQ_CUDA_TRY(cudaMemset2DAsync(U + j0, (size_t)C * 4, 0, (size_t)wj * 4, j0, s));
    {
      f16x3::Operand A{w.Fhi, w.Flo, j0, j0, C};
      f16x3::Operand B{w.TThi, w.TTlo, wj, j0, C};
      // partial = u_i gam_j' 2^-5 (sum_k U[i][k] T[j'][k])
      CUtensorMap out;
      if ((st = f16x3::make_out_map_f32(&out, U + j0, j0, wj, C)) != GPTQ_OK) return st;
      st = f16x3::launch<true, false>(A, B, j0, wj, f16x3::EpiTileAddF32{j0, wj, -1.f, w.uinv, w.gam2inv}, dev_info, s, 0, &out);
      if (st != GPTQ_OK) return st;
    }
    if (J + 1 < n_outer) {
      if ((st = launch_split_scaled(U + j0, C, rows_p, wj, w.u, w.rinv + j0, w.Fhi + j0, w.Flo + j0, C, dev_info, s)) != GPTQ_OK) return st;
    }
  }
  return GPTQ_OK;
}
}  // namespace
}  // namespace gptq

extern "C" gptq_status_t gptq_prepare_hinv(const float* H, float damp, int C, float* U,
                                           void* ws, size_t ws_bytes, int* dev_info, void* stream) {
  return gptq::prepare_impl(H, damp, C, U, ws, ws_bytes, dev_info, stream, false);
}

extern "C" gptq_status_t gptq_prepare_factor(const float* H, float damp, int C, float* F,
                                             void* ws, size_t ws_bytes, int* dev_info, void* stream) {
  return gptq::prepare_impl(H, damp, C, F, ws, ws_bytes, dev_info, stream, true);
}

// ------------------------------------------------------------------------------------------------
// Workspace-free variant of gptq_prepare_hinv for callers that cannot allocate device memory.
//
// Some callers have no way to hand this library a workspace: code that runs under a framework whose
// memory pool owns every byte of the device and forbids cudaMalloc from plug-ins, code on a
// latency-critical path where an allocation would synchronise the device, or a process that was
// given a fixed memory budget up front.  For them the scratch lives in the library itself, in a
// fixed array in device global memory.  The price: the array is sized for a stated maximum, every
// GPU that loads the library keeps it until the process exits, and all calls share it.
//
// `hinv_static_scratch` below is that array.  In host code its name is only a stand-in for the
// device object, not an address a kernel may be given; the device address is obtained once per
// device with cudaGetSymbolAddress (with that device current) and cached.
namespace gptq {
namespace {
constexpr int kStaticMaxC = GPTQ_PREPARE_HINV_STATIC_MAX_C;
// workspace of gptq_prepare_hinv at C = 1024: lambda (256 B) + eight 128 x 128 diagonal inverses
// (512 KiB) + a 1024 x 128 panel temporary (512 KiB)
constexpr size_t kStaticScratchBytes = 256 + (size_t)(kStaticMaxC / kNB) * kNB * kNB * 4 + (size_t)kStaticMaxC * kNB * 4;
static __device__ __align__(256) unsigned char hinv_static_scratch[kStaticScratchBytes];
constexpr int kMaxDevices = 64;
}  // namespace
}  // namespace gptq

extern "C" gptq_status_t gptq_prepare_hinv_static(const float* H, float damp, int C, float* U,
                                                  int* dev_info, void* stream) {
  using namespace gptq;
  if (C > kStaticMaxC) return GPTQ_ERR_UNSUPPORTED;   // larger problems need the caller-workspace entry point
  if (C <= 0) return GPTQ_ERR_INVALID_ARG;
  if (carve_hinv(nullptr, C).bytes > kStaticScratchBytes) return GPTQ_ERR_UNSUPPORTED;
  static void* scratch_of_device[kMaxDevices] = {};
  int dev = -1;
  GPTQ_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return GPTQ_ERR_UNSUPPORTED;
  void* scratch = __atomic_load_n(&scratch_of_device[dev], __ATOMIC_ACQUIRE);
  if (!scratch) {
    // one-time set-up on this device (the current one): resolve the device address of the array
    GPTQ_CUDA_TRY(cudaGetSymbolAddress(&scratch, hinv_static_scratch));
    if (!scratch) return GPTQ_ERR_CUDA;
    __atomic_store_n(&scratch_of_device[dev], scratch, __ATOMIC_RELEASE);
  }
  // Nothing in the scratch has to start at zero: lambda, every used diagonal inverse and the panel
  // temporary are all written by this call before they are read, so stale contents are harmless.
  return gptq_prepare_hinv(H, damp, C, U, scratch, kStaticScratchBytes, dev_info, stream);
}

namespace gptq {
cudaError_t hinv_set_wait_test_knobs(unsigned long long limit_ns, int skip_item) { return set_wait_test_knobs(limit_ns, skip_item); }
}  // namespace gptq
