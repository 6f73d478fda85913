// Stage 3: Algorithm 1's two loops -- column-by-column quantization with error feedback inside a
// block of B columns, and lazy batched updates of the later columns (Section 3, Steps 1-3).
//
// Organisation on the GPU (an exact regrouping of Algorithm 1's updates; Section 3, Step 2 notes
// that the rounding decisions of a column depend only on the updates that reached that column):
//   * Columns are processed in OUTER blocks of B2 (about 1024) columns.  When an outer block
//     starts, its working weights are produced in one contraction from the ORIGINAL weights and
//     all errors so far:  Wblk = W[:, blk] - E[:, :i2] * U[:i2, blk]  ("left-looking" form of the
//     lazy update W[:, (i+B):] -= E * U[i:(i+B), (i+B):] accumulated over all earlier blocks).
//   * Inside an outer block the paper's loop runs with the caller's block size B: the in-block
//     kernel quantizes B columns with immediate error feedback, then the block's errors are
//     pushed onto the remaining columns of the outer block.
//   * Working weights of the current outer block are fp64; E is kept at fp32 level (as an fp16 hi/lo
//     pair of a power-of-two-scaled copy); update sums come from the tensor cores with fp32 accuracy
//     (three fp16 products per term, gemm_umma_f16.cuh).  Each weight therefore meets one rounding at
//     fp32 level (its update sum) instead of one per preceding block.
//   * Scaling for the fp16 pairs (all factors are powers of two, so scaling is exact):
//       E'[r][k] = E[r][k] * sK[k] * sE[r],   U'[k][c] = U[k][c] / sK[k] * sC[c],   sum_k E U = (sum_k E' U') / (sE[r] sC[c])
//     sK[k] ~ U_kk (then E * sK = (w - q) / mantissa(U_kk) has the size of a weight), sE[r] ~ 2^11 / max|W[r][:]|,
//     sC[c] ~ 2^13 / max_k |U[k][c] / sK[k]|.  An E' beyond fp16's range (an error thousands of times the
//     row's largest weight) is saturated and reported as GPTQ_ERR_NONFINITE.
#include <atomic>

#include "common.cuh"
#include "gemm_umma_f16.cuh"

namespace gptq {
namespace {

constexpr int kSB = 32;  // columns held in registers at a time by the in-block kernel

struct GridSpec {
  int maxq;        // largest code
  int symmetric;   // symmetric (or ternary) grid
  int f16scale;    // scales rounded to fp16 (the stored model's precision, Section 5) before anything uses them
};

// The scale in the precision it will be stored in: fp16 when asked for (unless that would be 0 or infinite).
__device__ __forceinline__ float storage_rounded(float scale, int f16scale) {
  if (!f16scale) return scale;
  const float s16 = __half2float(__float2half_rn(scale));
  return (s16 > 0.f && isfinite(s16)) ? s16 : scale;
}

// Min-max grid of a set of weights with minimum mn and maximum mx (Section 5, Setup).  The range
// is widened to contain 0 so the zero-point is an integer code; an all-zero set gets [-1, 1].
// The scale is rounded to fp32, the precision it is returned in, and used as that value.
__device__ __forceinline__ void find_params(double mn, double mx, GridSpec g, float& scale, float& zero) {
  double xmin = fmin(mn, 0.0), xmax = fmax(mx, 0.0);
  if (xmin == 0.0 && xmax == 0.0) { xmin = -1.0; xmax = 1.0; }
  if (g.symmetric) {
    double a = fmax(fabs(xmin), xmax);
    scale = storage_rounded((float)(2.0 * a / (double)g.maxq), g.f16scale);
    zero = (float)((g.maxq + 1) / 2);
  } else {
    scale = storage_rounded((float)((xmax - xmin) / (double)g.maxq), g.f16scale);
    zero = (float)rint(-xmin / (double)scale);
  }
}

// ---- per-row static grid from the original fp16 weights: one warp per row ----------------------
__global__ void rowgrid_kernel(const __half* __restrict__ W, int R, int C, GridSpec g,
                               float* __restrict__ scales, float* __restrict__ zeros) {
  int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= R) return;
  const uint4* p = reinterpret_cast<const uint4*>(W + (int64_t)row * C);
  float mn = INFINITY, mx = -INFINITY;
  for (int i = lane; i < C / 8; i += 32) {
    uint4 v = p[i];
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float2 f = __half22float2(h[k]);
      mn = fminf(mn, fminf(f.x, f.y));
      mx = fmaxf(mx, fmaxf(f.x, f.y));
    }
  }
  for (int o = 16; o > 0; o >>= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  if (lane == 0) find_params((double)mn, (double)mx, g, scales[row], zeros[row]);
}

// ---- grid of a group wider than the block: one warp per row over the working weights ----------
__global__ void groupgrid_kernel(const double* __restrict__ Wblk, int64_t ldw, int col0, int g, int R,
                                 GridSpec gs, float* __restrict__ scales, float* __restrict__ zeros,
                                 int G, int gi) {
  int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= R) return;
  const double* p = Wblk + (int64_t)row * ldw + col0;
  double mn = INFINITY, mx = -INFINITY;
  for (int i = lane; i < g; i += 32) { mn = fmin(mn, p[i]); mx = fmax(mx, p[i]); }
  for (int o = 16; o > 0; o >>= 1) {
    mn = fmin(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  if (lane == 0) find_params(mn, mx, gs, scales[(int64_t)row * G + gi], zeros[(int64_t)row * G + gi]);
}

// ---- working weights of an outer block start as the original weights ---------------------------
// stripe_major: the layout the row-stripe kernel wants (128-row stripes, each column of a stripe contiguous);
// otherwise plain row-major [R][ldw].
__global__ void wblk_from_w16_kernel(const __half* __restrict__ W, int R, int C, int i2, int nb,
                                     double* __restrict__ Wblk, int64_t ldw, int stripe_major) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)R * nb) return;
  int r = (int)(idx / nb), c = (int)(idx % nb);
  const int64_t o = stripe_major ? ((int64_t)(r >> 7) * ldw + c) * 128 + (r & 127) : (int64_t)r * ldw + c;
  Wblk[o] = (double)__half2float(W[(int64_t)r * C + i2 + c]);
}
// The same for the stripe-major layout through a shared-memory tile of one stripe's 128 rows x 32 columns, so that both
// the reads (along rows of W and D) and the writes (along a column of the stripe: 1 KB of consecutive doubles) are
// coalesced and a thread has sixteen loads in flight; and with the lazy update folded in:
//   Wblk = W[:, blk] - D / (sE[row] sC[col]),   D = E'[:, :i2] U'[:i2, blk] (scaled fp32 sums of the tensor-core contraction)
// formed in fp64.  D == nullptr for the first outer block.  grid (nb / 32, ceil(R / 128)), block (32, 8).
__global__ void __launch_bounds__(256)
wblk_stripe_major_kernel(const __half* __restrict__ W, int R, int C, int i2,
                         const float* __restrict__ D, int64_t ldd,
                         const float* __restrict__ sEinv, const float* __restrict__ sCinv, double sign,
                         double* __restrict__ Wblk, int64_t ldw) {
  __shared__ float t[128][33];
  __shared__ float d[128][33];
  const int r0 = blockIdx.y * 128, c0 = blockIdx.x * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    const int rr = ty + 8 * k, r = r0 + rr;
    t[rr][tx] = r < R ? __half2float(W[(int64_t)r * C + i2 + c0 + tx]) : 0.f;
    d[rr][tx] = (D != nullptr && r < R) ? D[(int64_t)r * ldd + c0 + tx] : 0.f;
  }
  __syncthreads();
  double* out = Wblk + ((int64_t)blockIdx.y * ldw + c0) * 128;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int cc = ty + 8 * k;
    const double sc = D != nullptr ? (double)sCinv[i2 + c0 + cc] : 0.0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int rr = tx + 32 * q, r = r0 + rr;
      if (r < R) {
        double w = (double)t[rr][cc];
        if (D != nullptr) w += sign * ((double)d[rr][cc] * (double)sEinv[r] * sc);
        out[(int64_t)cc * 128 + rr] = w;
      }
    }
  }
}

// ---- the in-block loop (Algorithm 1, inner FOR) -------------------------------------------------
struct InblockArgs {
  const double* Wblk; int64_t ldw; int col0;  // working weights; col0 = first column of this block in Wblk
  const float* U; int C; int i; int B;         // global first column i, width B (multiple of 32, <= 256)
  int R; GridSpec grid;
  int group;        // group size (<= 0: one grid per row)
  int grid_inside;  // 1: grids of groups that start in this block are computed here (group <= B)
  float* scales; float* zeros; int G;
  __half* Ehi; __half* Elo;             // scaled errors E' = E * sK[column] * sE[row] as an fp16 hi / lo pair
  const float* sK; const float* sE;
  uint8_t* codes; double* loss; int* dev_info;
};

// Four lanes per row, 32 rows per CTA.  The block's working weights sit in shared memory,
// column-major; a lane owns every fourth column.  32 columns at a time are held in registers
// (8 per lane) and quantized one after the other: the owner's current weight is broadcast to its
// quad with a warp shuffle, all four lanes take the (identical) rounding decision and error, and
// each applies the immediate feedback W[:, j:blockend] -= E_j U[j, j:blockend] to the columns it
// owns -- first inside the registers, then, 32 errors at a time, to the rest of the block in
// shared memory.  Min/max for group grids are quad-wide shuffle reductions.
constexpr int kRPB = 32;                 // rows per CTA
constexpr int kInblockThreads = 4 * kRPB;
constexpr int kLDS = kRPB + 4;           // slab row stride (doubles): 36 % 16 == 4 keeps quad accesses conflict-free

__device__ __forceinline__ double quad_min(double v) {
  v = fmin(v, __shfl_xor_sync(0xffffffffu, v, 1));
  return fmin(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ double quad_max(double v) {
  v = fmax(v, __shfl_xor_sync(0xffffffffu, v, 1));
  return fmax(v, __shfl_xor_sync(0xffffffffu, v, 2));
}

__global__ void __launch_bounds__(kInblockThreads) inblock_kernel(InblockArgs a) {
  extern __shared__ double smem[];
  const int B = a.B;
  double* slab = smem;                    // [B][kLDS]
  double* Us = smem + (size_t)B * kLDS;   // [kSB][B]   rows j0..j0+31 of the B x B block of U
  double* rdiag = Us + (size_t)kSB * B;   // [kSB]       1 / U_jj of the current sub-block
  float* esm = reinterpret_cast<float*>(rdiag + kSB);   // [kSB][kRPB] errors of the current sub-block, per row (fp32:
                                                        // the precision E leaves the kernel in)
  float* sks = esm + kSB * kRPB;          // [kSB]       column scales sK of the current sub-block
  const int t = threadIdx.x, l = t & 3, rl = t >> 2;
  const int r0 = blockIdx.x * kRPB, row = r0 + rl;
  const bool live = row < a.R;

  // stage the slab: coalesced 16-byte loads along columns, transposed into shared memory
  {
    const int half = B >> 1;
#pragma unroll 8
    for (int e = t; e < kRPB * half; e += kInblockThreads) {
      const int rr = e / half, c2 = e - rr * half;
      double2 v = make_double2(0.0, 0.0);
      if (r0 + rr < a.R) v = *reinterpret_cast<const double2*>(a.Wblk + (int64_t)(r0 + rr) * a.ldw + a.col0 + 2 * c2);
      slab[(2 * c2) * kLDS + rr] = v.x;
      slab[(2 * c2 + 1) * kLDS + rr] = v.y;
    }
  }
  const int G = a.G, g = a.group;
  const float se_row = live ? a.sE[row] : 1.f;
  float scale_f = 1.f, zero_f = 0.f;
  if (live && !a.grid_inside) {
    const int gi = g > 0 ? a.i / g : 0;
    scale_f = a.scales[(int64_t)row * G + gi];
    zero_f = a.zeros[(int64_t)row * G + gi];
  }
  double scale = (double)scale_f, zero = (double)zero_f, rscale = 1.0 / scale;
  const double maxq = (double)a.grid.maxq;
  double loss = 0.0;
  bool bad = false;

  for (int j0 = 0; j0 < B; j0 += kSB) {
    __syncthreads();  // slab staged / previous sub-block's Us no longer read
    if (t < kSB) sks[t] = a.sK[a.i + j0 + t];
    {
      const int q4 = B >> 2;
#pragma unroll 8
      for (int e = t; e < kSB * q4; e += kInblockThreads) {
        const int jj = e / q4, c = (e - jj * q4) * 4;
        if (c + 3 >= j0) {
          const float4 u = *reinterpret_cast<const float4*>(a.U + (int64_t)(a.i + j0 + jj) * a.C + a.i + c);
          double* d = Us + jj * B + c;
          d[0] = (double)u.x; d[1] = (double)u.y; d[2] = (double)u.z; d[3] = (double)u.w;
          const int dj = j0 + jj - c;                  // the diagonal entry U_jj, if it is in this quad of columns
          if (dj >= 0 && dj < 4) rdiag[jj] = 1.0 / (double)(dj == 0 ? u.x : (dj == 1 ? u.y : (dj == 2 ? u.z : u.w)));
        }
      }
    }
    __syncthreads();
    // w[g]: this lane's column of group g (columns j0 + 4 g + l), rotated so that w[0] is always the group
    // being quantized -- the loop over groups stays a real loop (small code, no instruction-cache thrash)
    double w[kSB / 4];
#pragma unroll
    for (int m = 0; m < kSB / 4; ++m) w[m] = slab[(j0 + 4 * m + l) * kLDS + rl];
    uint32_t c0 = 0, c1 = 0;

    // grid of a group that starts at this sub-block (group a multiple of 32, inside the block)
    if (a.grid_inside && g >= kSB && ((a.i + j0) % g) == 0) {
      double mn = INFINITY, mx = -INFINITY;
      for (int c = j0 + l; c < j0 + g; c += 4) { const double v = slab[c * kLDS + rl]; mn = fmin(mn, v); mx = fmax(mx, v); }
      find_params(quad_min(mn), quad_max(mx), a.grid, scale_f, zero_f);
      scale = (double)scale_f; zero = (double)zero_f; rscale = 1.0 / scale;
      if (live && l == 0) {
        const int gi = (a.i + j0) / g;
        a.scales[(int64_t)row * G + gi] = scale_f; a.zeros[(int64_t)row * G + gi] = zero_f;
      }
    }
#pragma unroll 1
    for (int m = 0; m < kSB / 4; ++m) {
      if (a.grid_inside && g < kSB && ((4 * m) % g) == 0) {   // small groups (4, 8, 16) live inside the registers
        double mn = INFINITY, mx = -INFINITY;
#pragma unroll
        for (int mm = 0; mm < 4; ++mm)
          if (4 * mm < g) { mn = fmin(mn, w[mm]); mx = fmax(mx, w[mm]); }
        find_params(quad_min(mn), quad_max(mx), a.grid, scale_f, zero_f);
        scale = (double)scale_f; zero = (double)zero_f; rscale = 1.0 / scale;
        if (live && l == 0) {
          const int gi = (a.i + j0 + 4 * m) / g;
          a.scales[(int64_t)row * G + gi] = scale_f; a.zeros[(int64_t)row * G + gi] = zero_f;
        }
      }
      uint32_t packed = 0;
#pragma unroll
      for (int o = 0; o < 4; ++o) {
        const int jj = 4 * m + o;
        const double wj = __shfl_sync(0xffffffffu, w[0], o, 4);
        // code of this weight: rne(w / scale).  The quotient is formed with the reciprocal; only when it lands within
        // 1e-6 of a tie (where the reciprocal's last-bit error could change the rounding) is the division done.
        const double tq = wj * rscale;
        double q = rint(tq);
        if (fabs(fabs(tq - q) - 0.5) < 1e-6) q = rint(wj / scale);
        q += zero;
        q = fmin(fmax(q, 0.0), maxq);
        const double wq = scale * (q - zero);
        const double e = (wj - wq) * rdiag[jj];                // scaled error (w - q) / U_jj
        if (l == o) esm[jj * kRPB + rl] = (float)e;
        loss += e * e;
        bad |= !isfinite(e);
        packed |= (uint32_t)q << (8 * o);
        const double* urow = Us + jj * B + j0 + 4 * m + l;
#pragma unroll
        for (int mm = 0; mm < kSB / 4; ++mm)                   // immediate feedback onto own columns > jj
          if (mm < kSB / 4 - m && (mm > 0 || l > o)) w[mm] -= e * urow[4 * mm];
      }
      if ((m >> 1) == l) { if (m & 1) c1 = packed; else c0 = packed; }
#pragma unroll
      for (int mm = 0; mm + 1 < kSB / 4; ++mm) w[mm] = w[mm + 1];
    }
    __syncwarp();                                              // esm rows of this warp are complete
    double err[kSB];
#pragma unroll
    for (int jj = 0; jj < kSB; ++jj) err[jj] = (double)esm[jj * kRPB + rl];
    // remaining columns of the block: apply the 32 errors of this sub-block to the columns this lane owns
    for (int c = j0 + kSB + l; c < B; c += 4) {
      double x = slab[c * kLDS + rl];
#pragma unroll
      for (int jj = 0; jj < kSB; ++jj) x -= err[jj] * Us[jj * B + c];
      slab[c * kLDS + rl] = x;
    }
    if (live) {
      // lane l stores columns [8 l, 8 l + 8) of this sub-block: scaled errors as an fp16 hi / lo pair, codes as bytes
      uint32_t hw[4], lw[4];
      bool sat = false;
#pragma unroll
      for (int u = 0; u < 8; u += 2) {
        __half h0, l0, h1, l1;
        const double e0 = l == 0 ? err[u] : (l == 1 ? err[8 + u] : (l == 2 ? err[16 + u] : err[24 + u]));
        const double e1 = l == 0 ? err[u + 1] : (l == 1 ? err[9 + u] : (l == 2 ? err[17 + u] : err[25 + u]));
        f16x3::split_f16((float)e0 * sks[8 * l + u] * se_row, h0, l0, sat);
        f16x3::split_f16((float)e1 * sks[8 * l + u + 1] * se_row, h1, l1, sat);
        hw[u >> 1] = (uint32_t)__half_as_ushort(h0) | ((uint32_t)__half_as_ushort(h1) << 16);
        lw[u >> 1] = (uint32_t)__half_as_ushort(l0) | ((uint32_t)__half_as_ushort(l1) << 16);
      }
      bad |= sat;
      const int64_t o = (int64_t)row * a.C + a.i + j0 + 8 * l;
      *reinterpret_cast<uint4*>(a.Ehi + o) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
      *reinterpret_cast<uint4*>(a.Elo + o) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
      *reinterpret_cast<uint2*>(a.codes + o) = make_uint2(c0, c1);
    }
  }
  if (!live || l != 0) loss = 0.0;
  for (int o = 16; o > 0; o >>= 1) loss += __shfl_down_sync(0xffffffffu, loss, o);
  if ((t & 31) == 0 && loss != 0.0) atomicAdd(a.loss, loss);
  if (live && l == 0 && bad) report_error(a.dev_info, GPTQ_ERR_NONFINITE, row);
}

// ---- pack codes: little-endian bit stream per row, field width f --------------------------------
__global__ void pack_kernel(const uint8_t* __restrict__ codes, int R, int C, int f,
                            uint32_t* __restrict__ qweight) {
  const int nwords = C * f / 32;
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)R * nwords) return;
  int r = (int)(idx / nwords), k = (int)(idx % nwords);
  const uint8_t* c = codes + (int64_t)r * C;
  int lo = 32 * k / f, hi = (32 * k + 31) / f;
  uint32_t word = 0;
  for (int col = lo; col <= hi; ++col) {
    int sh = col * f - 32 * k;
    uint32_t v = c[col];
    word |= sh >= 0 ? (v << sh) : (v >> (-sh));
  }
  qweight[idx] = word;
}

// ---- power-of-two scales for the fp16 operand pairs ------------------------------------------------
// sK[k] = largest power of two <= U_kk; colmax[c] = 0
__global__ void kscale_kernel(const float* __restrict__ U, int C, float* __restrict__ sK, uint32_t* __restrict__ colmax) {
  int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= C) return;
  sK[k] = pow2_floor(U[(int64_t)k * C + k]);
  colmax[k] = 0u;
}
// colmax[c] = max over rows k <= c of |U[k][c]| / sK[k]   (bit pattern of a non-negative float: ordered as integers).
// Factor form (fblock > 0; U then holds U on its diagonal blocks of fblock columns and the factor U~ above them):
// colmax covers the rows of c's own diagonal block only, and colmax2[c] = max over the rows above that block of |U~[k][c]|.
__global__ void colmax_kernel(const float* __restrict__ U, int C, const float* __restrict__ sK, uint32_t* __restrict__ colmax,
                              int fblock, uint32_t* __restrict__ colmax2) {
  __shared__ float red[8][33];
  const int c = blockIdx.x * 32 + threadIdx.x, r0 = blockIdx.y * 256;
  if (r0 > blockIdx.x * 32 + 31) return;               // block wholly below the diagonal
  const bool above = fblock > 0 && r0 < (blockIdx.x * 32) / fblock * fblock;   // (256 divides fblock: uniform over the CTA)
  float m = 0.f;
  for (int r = r0 + threadIdx.y; r < min(C, r0 + 256); r += 8)
    if (r <= c) m = fmaxf(m, above ? fabsf(U[(int64_t)r * C + c]) : fabsf(U[(int64_t)r * C + c]) / sK[r]);
  red[threadIdx.y][threadIdx.x] = m;
  __syncthreads();
  if (threadIdx.y == 0) {
#pragma unroll
    for (int y = 1; y < 8; ++y) m = fmaxf(m, red[y][threadIdx.x]);
    if (m > 0.f && isfinite(m)) atomicMax((above ? colmax2 : colmax) + c, __float_as_uint(m));
  }
}
// sC[c] = power of two that brings the column's largest scaled entry just below 2^13; sCinv = 1 / sC
__global__ void cscale_kernel(const uint32_t* __restrict__ colmax, int C, float* __restrict__ sC, float* __restrict__ sCinv) {
  int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  const float s = pow2_scale_to(__uint_as_float(colmax[c]), 13);
  sC[c] = s; sCinv[c] = 1.f / s;
}
// sE[r] = power of two that brings the row's largest |weight| just below 2^11; sEinv = 1 / sE.  One warp per row.
__global__ void rowscale_kernel(const __half* __restrict__ W, int R, int C, float* __restrict__ sE, float* __restrict__ sEinv) {
  int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= R) return;
  const uint4* p = reinterpret_cast<const uint4*>(W + (int64_t)row * C);
  float mx = 0.f;
  for (int i = lane; i < C / 8; i += 32) {
    uint4 v = p[i];
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float2 f = __half22float2(h[k]);
      mx = fmaxf(mx, fmaxf(fabsf(f.x), fabsf(f.y)));
    }
  }
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) { const float s = pow2_scale_to(mx, 11); sE[row] = s; sEinv[row] = 1.f / s; }
}

// ---- U panel -> transposed, scaled fp16 hi / lo pair ------------------------------------------------
// Pt[c][r] = U[r][i2 + c] / sK[r] * sC[i2 + c] for r < rows, c < nb2 (row stride ldp): the right factor of the
// lazy updates, transposed so the contraction index is contiguous, split so that hi + lo ~ value to 2^-22.
// A CTA transposes 128 rows x 32 columns through shared memory: sixteen coalesced loads in flight per thread, and per
// column 256 consecutive bytes of each output written as half2 pairs.  grid (nb2 / 32, rows / 128 rounded up), block (32, 8).
__global__ void __launch_bounds__(256)
split_panel_t_kernel(const float* __restrict__ U, int C, int i2, int rows,
                     const float* __restrict__ sK, const float* __restrict__ sC, const float* __restrict__ sC2,
                     __half* __restrict__ Phi, __half* __restrict__ Plo, int64_t ldp) {
  __shared__ float t[128][33];
  const int r0 = blockIdx.y * 128, c0 = blockIdx.x * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    const int rr = ty + 8 * k, r = r0 + rr;
    // factor form (sC2 != nullptr): the rows above the outer block hold the factor U~, scaled per column only
    const bool above = sC2 != nullptr && r < i2;
    t[rr][tx] = r < rows ? (above ? U[(int64_t)r * C + i2 + c0 + tx] : U[(int64_t)r * C + i2 + c0 + tx] / sK[r]) : 0.f;
  }
  __syncthreads();
  const bool above_blk = sC2 != nullptr && r0 < i2;          // (i2 is a multiple of 128: uniform over the CTA)
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int cc = ty + 8 * k;
    const float sc = above_blk ? sC2[i2 + c0 + cc] : sC[i2 + c0 + cc];
    const int64_t o = (int64_t)(c0 + cc) * ldp + r0;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int rr = 64 * q + 2 * tx;
      if (r0 + rr >= rows) continue;               // (rows is a multiple of 32)
      __half h0, l0, h1, l1;
      bool sat = false;
      f16x3::split_f16(t[rr][cc] * sc, h0, l0, sat);
      f16x3::split_f16(t[rr + 1][cc] * sc, h1, l1, sat);
      *reinterpret_cast<__half2*>(Phi + o + rr) = __halves2half2(h0, h1);
      *reinterpret_cast<__half2*>(Plo + o + rr) = __halves2half2(l0, l1);
    }
  }
}

// Factor form: R'[r][c] = (w[r][c] - scale (code - zero)) sE[r] for the columns [i2, i2 + nb2) of every row, as an fp16
// hi / lo pair in Ehi / Elo: the plain residuals, formed in fp64 from the original weights and the codes, scales and
// zero-points the block's solve has just written.  One thread: 8 consecutive columns.
__global__ void residual_pair_kernel(const __half* __restrict__ W, const uint8_t* __restrict__ codes,
                                     const float* __restrict__ scales, const float* __restrict__ zeros, int G, int g,
                                     const float* __restrict__ sE, int R, int C, int i2, int nb2,
                                     __half* __restrict__ Ehi, __half* __restrict__ Elo, int* dev_info) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int per_row = nb2 / 8;
  if (idx >= (int64_t)R * per_row) return;
  const int r = (int)(idx / per_row), c = i2 + (int)(idx % per_row) * 8;
  const int64_t o = (int64_t)r * C + c;
  const uint4 wv = *reinterpret_cast<const uint4*>(W + o);
  const uint2 cv = *reinterpret_cast<const uint2*>(codes + o);
  const __half* wh = reinterpret_cast<const __half*>(&wv);
  const uint8_t* cb = reinterpret_cast<const uint8_t*>(&cv);
  const float se = sE[r];
  uint32_t hw[4], lw[4];
  bool sat = false;
#pragma unroll
  for (int u = 0; u < 8; u += 2) {
    float rr[2];
#pragma unroll
    for (int v = 0; v < 2; ++v) {
      const int gi = g > 0 ? (c + u + v) / g : 0;
      const double sc = (double)scales[(int64_t)r * G + gi], ze = (double)zeros[(int64_t)r * G + gi];
      rr[v] = (float)((double)__half2float(wh[u + v]) - sc * ((double)cb[u + v] - ze));
    }
    __half h0, l0, h1, l1;
    f16x3::split_f16(rr[0] * se, h0, l0, sat);
    f16x3::split_f16(rr[1] * se, h1, l1, sat);
    hw[u >> 1] = (uint32_t)__half_as_ushort(h0) | ((uint32_t)__half_as_ushort(h1) << 16);
    lw[u >> 1] = (uint32_t)__half_as_ushort(l0) | ((uint32_t)__half_as_ushort(l1) << 16);
  }
  *reinterpret_cast<uint4*>(Ehi + o) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
  *reinterpret_cast<uint4*>(Elo + o) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
  if (sat) report_error(dev_info, GPTQ_ERR_NONFINITE, r);
}

// ---- contraction epilogue (one thread: one row, 32 consecutive columns of a partial sum) --------
// Wblk[row][nofs + col ..) -= partial / (sE[row] sC[column]), as fp64 reductions: partial sums of one tile
// come from several CTA pairs (one per super-chunk of the contraction).
struct EpiSubWblk {
  double* Wblk; int64_t ldw; int nofs; int R, N;
  const float* sEinv; const float* sCinv;     // sCinv already offset to the first column of this contraction
  int stripe_major;                           // layout of Wblk (see wblk_from_w16_kernel)
  __device__ __forceinline__ void operator()(int row, int col0, const float (&v)[32]) const {
    if (row >= R || col0 >= N) return;
    const double ir = -(double)sEinv[row];
    double* p = stripe_major ? Wblk + ((int64_t)(row >> 7) * ldw + nofs + col0) * 128 + (row & 127)
                             : Wblk + (int64_t)row * ldw + nofs + col0;
    const int64_t step = stripe_major ? 128 : 1;
#pragma unroll
    for (int j = 0; j < 32; ++j)
      asm volatile("red.global.add.f64 [%0], %1;" ::"l"(p + j * step), "d"((double)v[j] * ir * (double)sCinv[col0 + j]) : "memory");
  }
};

#include "quantize_stripe.cuh"

// Which form runs inside an outer block: 1 = row-stripe kernel (one launch per outer block), 0 = one in-block
// kernel plus one small tensor-core contraction per inner block.  Process-wide; see gptq_set_stage3_variant.
std::atomic<int> g_stage3_variant{1};

gptq_status_t launch_stripe(const StripeArgs& a, const __half* Phi, const __half* Plo, cudaStream_t s) {
  StripeMaps maps;
  gptq_status_t st;
  // Pt[c - i2][k]: rows = columns of the outer block, inner dimension = contraction index (rows of U so far)
  if ((st = make_tmap_2d(&maps.p_hi, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, Phi, (uint64_t)(a.i2 + a.nb2), (uint64_t)a.nb2,
                         (uint64_t)a.C * 2, 64, kStripeNT)) != GPTQ_OK) return st;
  if ((st = make_tmap_2d(&maps.p_lo, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, Plo, (uint64_t)(a.i2 + a.nb2), (uint64_t)a.nb2,
                         (uint64_t)a.C * 2, 64, kStripeNT)) != GPTQ_OK) return st;
  GPTQ_CUDA_TRY(cudaFuncSetAttribute(stripe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stripe_smem(kStripeMaxB)));
  stripe_kernel<<<ceil_div(a.R, kStripeRows), kStripeThreads, stripe_smem(a.B), s>>>(maps, a);
  GPTQ_LAUNCH_CHECK();
  return GPTQ_OK;
}

inline int field_bits(int bits) { return bits == GPTQ_BITS_TERNARY ? 2 : bits; }
inline bool bits_ok(int bits) { return bits == 2 || bits == 3 || bits == 4 || bits == 8 || bits == GPTQ_BITS_TERNARY; }

// Outer (lazy) block width: a multiple of both the block and any group wider than it, about 1024.
inline int outer_block(int C, int group, int block) {
  int unit = (group > block) ? group : block;
  int b2 = unit * (1024 / unit > 0 ? 1024 / unit : 1);
  return b2 < C ? b2 : C;
}

}  // namespace
}  // namespace gptq

extern "C" size_t gptq_quantize_workspace_bytes(int R, int C, int bits, int group_size, int block) {
  using namespace gptq;
  if (R <= 0 || C <= 0 || block <= 0 || !bits_ok(bits)) return 0;
  WsCarver w(nullptr);
  w.take<double>((size_t)ceil_div(R, 128) * 128 * outer_block(C, group_size, block));  // working weights of the outer block
  w.take<__half>((size_t)R * C);                                  // scaled E (fp16 high parts), all columns
  w.take<__half>((size_t)R * C);                                  // scaled E (fp16 remainders)
  w.take<uint8_t>((size_t)R * C);                                 // unpacked codes
  w.take<__half>((size_t)C * outer_block(C, group_size, block));  // transposed scaled panel of U, high parts
  w.take<__half>((size_t)C * outer_block(C, group_size, block));  // panel of U, remainders
  w.take<float>((size_t)C);                                       // sK
  w.take<float>((size_t)C);                                       // sC
  w.take<float>((size_t)C);                                       // 1 / sC
  w.take<uint32_t>((size_t)C);                                    // column maxima of the scaled U
  w.take<float>((size_t)R);                                       // sE
  w.take<float>((size_t)R);                                       // 1 / sE
  w.take<float>((size_t)R * outer_block(C, group_size, block));   // scaled fp32 sums of the lazy update of the outer block
  w.take<uint32_t>((size_t)C);                                    // factor form: column maxima above the diagonal blocks,
  w.take<float>((size_t)C);                                       //   sC2,
  w.take<float>((size_t)C);                                       //   1 / sC2
  return w.off;
}

namespace gptq {
namespace {
// factor: U holds gptq_prepare_factor's output (U on the diagonal blocks of 1024 columns, the factor U~ above them)
gptq_status_t quantize_impl(const void* W_fp16, const float* U, int R, int C,
                            int bits, int group_size, int sym, int block,
                            uint32_t* qweight, float* scales, float* zeros, double* loss,
                            void* ws, size_t ws_bytes, int* dev_info, void* stream, bool factor) {
  if (!W_fp16 || !U || !qweight || !scales || !zeros || !loss || !dev_info || R <= 0 || C <= 0 || C % 32 != 0)
    return GPTQ_ERR_INVALID_ARG;
  if (!aligned_to(W_fp16, 16) || !aligned_to(U, 16)) return GPTQ_ERR_INVALID_ARG;
  if (!bits_ok(bits)) return GPTQ_ERR_UNSUPPORTED;
  if (block <= 0) return GPTQ_ERR_INVALID_ARG;
  if (block % 32 != 0 || block > 256) return GPTQ_ERR_UNSUPPORTED;
  const int g = group_size > 0 ? group_size : 0;
  if (g > 0) {
    if (C % g != 0) return GPTQ_ERR_INVALID_ARG;
    if (g % block != 0 && block % g != 0) return GPTQ_ERR_INVALID_ARG;   // groups and blocks must nest
    if (g % kSB != 0 && (kSB % g != 0 || g < 4)) return GPTQ_ERR_UNSUPPORTED;   // 4, 8, 16 or a multiple of 32
  }
  if (!ws || !aligned_to(ws, kAlign) || ws_bytes < gptq_quantize_workspace_bytes(R, C, bits, group_size, block))
    return GPTQ_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half* W = static_cast<const __half*>(W_fp16);
  const int B2 = outer_block(C, g, block);
  const int G = g > 0 ? C / g : 1;
  WsCarver w(ws);
  double* Wblk = w.take<double>((size_t)ceil_div(R, 128) * 128 * B2);
  __half* Ehi = w.take<__half>((size_t)R * C);
  __half* Elo = w.take<__half>((size_t)R * C);
  uint8_t* codes = w.take<uint8_t>((size_t)R * C);
  __half* Phi = w.take<__half>((size_t)C * B2);
  __half* Plo = w.take<__half>((size_t)C * B2);
  float* sK = w.take<float>((size_t)C);
  float* sC = w.take<float>((size_t)C);
  float* sCinv = w.take<float>((size_t)C);
  uint32_t* colmax = w.take<uint32_t>((size_t)C);
  float* sE = w.take<float>((size_t)R);
  float* sEinv = w.take<float>((size_t)R);
  float* Dsum = w.take<float>((size_t)R * B2);
  uint32_t* colmax2 = w.take<uint32_t>((size_t)C);
  float* sC2 = w.take<float>((size_t)C);
  float* sC2inv = w.take<float>((size_t)C);
  const int64_t ldw = B2;
  GridSpec gs{bits == GPTQ_BITS_TERNARY ? 2 : (1 << bits) - 1, ((sym & GPTQ_GRID_SYMMETRIC) != 0 || bits == GPTQ_BITS_TERNARY) ? 1 : 0,
              (sym & GPTQ_GRID_FP16_SCALES) ? 1 : 0};
  if (sym & ~(GPTQ_GRID_SYMMETRIC | GPTQ_GRID_FP16_SCALES)) return GPTQ_ERR_INVALID_ARG;

  GPTQ_CUDA_TRY(cudaMemsetAsync(dev_info, 0, 2 * sizeof(int), s));
  GPTQ_CUDA_TRY(cudaMemsetAsync(loss, 0, sizeof(double), s));
  if (g == 0) {
    rowgrid_kernel<<<ceil_div(R, 8), 256, 0, s>>>(W, R, C, gs, scales, zeros);
    GPTQ_LAUNCH_CHECK();
  }
  // power-of-two scales of the fp16 operand pairs: per contraction index (from U's diagonal), per column of U, per row of W
  kscale_kernel<<<ceil_div(C, 256), 256, 0, s>>>(U, C, sK, colmax);
  GPTQ_LAUNCH_CHECK();
  if (factor) GPTQ_CUDA_TRY(cudaMemsetAsync(colmax2, 0, (size_t)C * sizeof(uint32_t), s));
  {
    dim3 grid(C / 32, ceil_div(C, 256)), blk(32, 8);
    colmax_kernel<<<grid, blk, 0, s>>>(U, C, sK, colmax, factor ? GPTQ_FACTOR_BLOCK : 0, colmax2);
    GPTQ_LAUNCH_CHECK();
  }
  cscale_kernel<<<ceil_div(C, 256), 256, 0, s>>>(colmax, C, sC, sCinv);
  GPTQ_LAUNCH_CHECK();
  if (factor) {
    cscale_kernel<<<ceil_div(C, 256), 256, 0, s>>>(colmax2, C, sC2, sC2inv);
    GPTQ_LAUNCH_CHECK();
  }
  rowscale_kernel<<<ceil_div(R, 8), 256, 0, s>>>(W, R, C, sE, sEinv);
  GPTQ_LAUNCH_CHECK();
  auto inblock_smem = [&](int B) { return (size_t)((size_t)B * kLDS + (size_t)kSB * B + kSB) * sizeof(double) + (size_t)(kSB * kRPB + kSB) * sizeof(float); };
  GPTQ_CUDA_TRY(cudaFuncSetAttribute(inblock_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)inblock_smem(256)));

  // form of the loops inside an outer block (see gptq_set_stage3_variant)
  // A block wider than the row-stripe kernel's 128 columns (256) is run there as 128-column inner blocks: the same updates
  // in the same column order, regrouped (Section 3, Step 2) -- groups still nest with 128 whenever they nest with 256.
  const bool stripe = (g_stage3_variant.load(std::memory_order_relaxed) == 1 || factor) && B2 <= kStripeMaxNb2 &&
                      (block <= kStripeMaxB || block % kStripeMaxB == 0);
  const int stripe_block = block <= kStripeMaxB ? block : kStripeMaxB;
  // the factor form rests on the outer blocks being the factorisation's diagonal blocks, and runs in the row-stripe form only
  if (factor && C > GPTQ_FACTOR_BLOCK && (!stripe || B2 != GPTQ_FACTOR_BLOCK)) return GPTQ_ERR_UNSUPPORTED;
  for (int i2 = 0; i2 < C; i2 += B2) {
    const int nb2 = (C - i2 < B2) ? C - i2 : B2;
    {  // transposed tf32 hi/lo pair of U[0 : i2 + nb2, i2 : i2 + nb2] for the contractions of this outer block
      dim3 grid(nb2 / 32, ceil_div(i2 + nb2, 128)), blk(32, 8);
      split_panel_t_kernel<<<grid, blk, 0, s>>>(U, C, i2, i2 + nb2, sK, sC, factor ? sC2 : nullptr, Phi, Plo, (int64_t)C);
      GPTQ_LAUNCH_CHECK();
    }
    // working weights of the outer block: original weights minus all updates from columns < i2
    if (stripe) {
      // lazy update of the outer block: scaled fp32 sums from the tensor cores (added up in L2 by TMA reductions), then
      // the fp64 working weights of the block in stripe-major order
      if (i2 > 0) {
        GPTQ_CUDA_TRY(cudaMemsetAsync(Dsum, 0, (size_t)R * B2 * sizeof(float), s));
        f16x3::Operand A{Ehi, Elo, R, i2, C}, Bop{Phi, Plo, nb2, i2, C};
        CUtensorMap out;
        gptq_status_t st = f16x3::make_out_map_f32(&out, Dsum, R, nb2, B2);
        if (st != GPTQ_OK) return st;
        st = f16x3::launch<false, false>(A, Bop, R, nb2, f16x3::EpiTileAddF32{R, nb2, 1.f, nullptr, nullptr}, dev_info, s, 0, &out);
        if (st != GPTQ_OK) return st;
      }
      // (factor form: A holds the plain residuals and the panel rows above the block hold U~[before, blk] U_blk, scaled per
      // column by sC2: the sums ARE the block's correction, with the opposite sign)
      dim3 grid(nb2 / 32, ceil_div(R, 128)), blk(32, 8);
      wblk_stripe_major_kernel<<<grid, blk, 0, s>>>(W, R, C, i2, i2 > 0 ? Dsum : nullptr, B2, sEinv, factor ? sC2inv : sCinv,
                                                    factor ? 1.0 : -1.0, Wblk, ldw);
      GPTQ_LAUNCH_CHECK();
    } else {
      int64_t total = (int64_t)R * nb2;
      wblk_from_w16_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(W, R, C, i2, nb2, Wblk, ldw, 0);
      GPTQ_LAUNCH_CHECK();
      if (i2 > 0) {
        f16x3::Operand A{Ehi, Elo, R, i2, C}, Bop{Phi, Plo, nb2, i2, C};
        gptq_status_t st = f16x3::launch<false, false>(A, Bop, R, nb2, EpiSubWblk{Wblk, ldw, 0, R, nb2, sEinv, sCinv + i2, 0}, dev_info, s);
        if (st != GPTQ_OK) return st;
      }
    }
    if (stripe) {
      // row-stripe form: every inner block of this outer block in one launch
      StripeArgs a{Wblk, ldw, nb2, U, C, i2, stripe_block, R, gs, g, scales, zeros, G, Ehi, Elo, Phi, Plo, (int64_t)C,
                   sK, sE, sEinv, sCinv, codes, loss, dev_info, factor ? 0 : 1};
      gptq_status_t st = launch_stripe(a, Phi, Plo, s);
      if (st != GPTQ_OK) return st;
      if (factor && i2 + nb2 < C) {
        // factor form: what later outer blocks contract with is the plain residual of this block's columns
        const int64_t n8 = (int64_t)R * (nb2 / 8);
        residual_pair_kernel<<<(unsigned)((n8 + 255) / 256), 256, 0, s>>>(W, codes, scales, zeros, G, g, sE, R, C, i2, nb2, Ehi, Elo,
                                                                          dev_info);
        GPTQ_LAUNCH_CHECK();
      }
      continue;
    }
    for (int i = i2; i < i2 + nb2; i += block) {
      const int B = (i2 + nb2 - i < block) ? i2 + nb2 - i : block;
      if (g > B && i % g == 0) {   // a group wider than the block starts here
        groupgrid_kernel<<<ceil_div(R, 8), 256, 0, s>>>(Wblk, ldw, i - i2, g, R, gs, scales, zeros, G, i / g);
        GPTQ_LAUNCH_CHECK();
      }
      InblockArgs a{Wblk, ldw, i - i2, U, C, i, B, R, gs, g, (g > 0 && g <= B) ? 1 : 0,
                    scales, zeros, G, Ehi, Elo, sK, sE, codes, loss, dev_info};
      inblock_kernel<<<ceil_div(R, kRPB), kInblockThreads, inblock_smem(B), s>>>(a);
      GPTQ_LAUNCH_CHECK();
      // push this block's errors onto the remaining columns of the outer block
      const int rest = i2 + nb2 - (i + B);
      if (rest > 0) {
        const int64_t po = (int64_t)(i + B - i2) * C + i;     // U[i][i + B] inside the transposed panel
        f16x3::Operand A{Ehi + i, Elo + i, R, B, C}, Bop{Phi + po, Plo + po, rest, B, C};
        gptq_status_t st = f16x3::launch<false, false>(A, Bop, R, rest, EpiSubWblk{Wblk, ldw, i + B - i2, R, rest, sEinv, sCinv + i + B, 0},
                                                       dev_info, s);
        if (st != GPTQ_OK) return st;
      }
    }
  }
  {
    const int f = field_bits(bits);
    int64_t total = (int64_t)R * (C * f / 32);
    pack_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(codes, R, C, f, qweight);
    GPTQ_LAUNCH_CHECK();
  }
  return GPTQ_OK;
}
}  // namespace
}  // namespace gptq

extern "C" gptq_status_t gptq_quantize_layer(const void* W_fp16, const float* U, int R, int C,
                                             int bits, int group_size, int sym, int block,
                                             uint32_t* qweight, float* scales, float* zeros, double* loss,
                                             void* ws, size_t ws_bytes, int* dev_info, void* stream) {
  return gptq::quantize_impl(W_fp16, U, R, C, bits, group_size, sym, block, qweight, scales, zeros, loss, ws, ws_bytes,
                             dev_info, stream, false);
}

extern "C" gptq_status_t gptq_quantize_layer_factor(const void* W_fp16, const float* F, int R, int C,
                                                    int bits, int group_size, int sym, int block,
                                                    uint32_t* qweight, float* scales, float* zeros, double* loss,
                                                    void* ws, size_t ws_bytes, int* dev_info, void* stream) {
  return gptq::quantize_impl(W_fp16, F, R, C, bits, group_size, sym, block, qweight, scales, zeros, loss, ws, ws_bytes,
                             dev_info, stream, true);
}

namespace gptq {
cudaError_t quantize_set_wait_test_knobs(unsigned long long limit_ns, int skip_item) { return set_wait_test_knobs(limit_ns, skip_item); }
}  // namespace gptq

extern "C" int gptq_set_stage3_variant(int variant) {
  if (variant != 0 && variant != 1) return gptq::g_stage3_variant.load();
  return gptq::g_stage3_variant.exchange(variant);
}

#ifdef GPTQ_EXP_TIMING
extern "C" int gptq_dbg_stripe_timing(unsigned long long* out32, int reset) {
  if (reset) { unsigned long long z[32] = {}; return (int)cudaMemcpyToSymbol(gptq::g_stripe_dbg, z, sizeof(z)); }
  return (int)cudaMemcpyFromSymbol(out32, gptq::g_stripe_dbg, 32 * sizeof(unsigned long long));
}
#endif
