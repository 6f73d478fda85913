// fp32-accurate tensor-core contraction ("3xTF32") on tcgen05 / TMEM / TMA.
//
//   acc[m][n] = sum_{k in [k0(tile), k1(tile))} A[m][k] * B[k][n]
//             ~ Ahi*Bhi + Ahi*Blo + Alo*Bhi       (hi = tf32(x), lo = tf32(x - hi))
//
// Each fp32 operand is supplied as TWO fp32 arrays holding its tf32-representable high part
// and the tf32-rounded remainder; the dropped lo*lo term and the rounding of lo are of relative
// size 2^-22, i.e. fp32 level.  Three tcgen05.mma (kind::tf32) per 8-wide K step accumulate
// into one fp32 TMEM accumulator.
//
// Operand layouts (all through TMA with 128-byte swizzle, 32 fp32 per 128-byte row):
//   A: row-major [M][K], K contiguous.
//   B: supplied TRANSPOSED, row-major [N][K], K contiguous (so both operands are K-major; callers
//      whose right factor is stored [K][N] write its transpose when they split it into hi / lo).
// Tiles: 128 x 256, K block 32, two shared-memory stages (96 KB each), two TMEM accumulators so
// the epilogue of one tile overlaps the MMAs of the next.  Persistent: one CTA per SM.
//
// Epi functor (device): void operator()(int row, int col0, const float (&v)[32]) const
//   called by one thread per row for 32 consecutive columns starting at col0 (col0 % 32 == 0);
//   the functor does its own bounds checks against the true M, N.
// Range functor (device): bool operator()(int m0, int n0, int& k0, int& k1) const
//   false skips the tile; k0 must be a multiple of 32 (k1 may be ragged: TMA zero-fills past K).
#pragma once
#include "umma.cuh"

namespace gptq {
namespace tf32x3 {

constexpr int BM = 128, BN = 256, BK = 32, STAGES = 2;
constexpr int OP_A_BYTES = BM * BK * 4;       // 16 KB (one of hi / lo)
constexpr int OP_B_BYTES = BN * BK * 4;       // 32 KB
constexpr int STAGE_BYTES = 2 * (OP_A_BYTES + OP_B_BYTES);   // 96 KB
constexpr int kThreads = 192;
constexpr size_t kSmemBytes = (size_t)STAGES * STAGE_BYTES + 1024 + 256;

struct Maps { CUtensorMap a_hi, a_lo, b_hi, b_lo; };

struct Geometry {
  int M, N;           // output extent (tiles are enumerated over it)
  int tiles_m, tiles_n;
  int* dev_info;
};

template <class RangeF, class EpiF>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tf32x3_kernel(const __grid_constant__ Maps maps, const Geometry g, const RangeF range, const EpiF epi) {
  using namespace umma;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + (size_t)STAGES * STAGE_BYTES);
  uint64_t* full = bars;
  uint64_t* empty = bars + STAGES;
  uint64_t* acc_full = bars + 2 * STAGES;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tiles = g.tiles_m * g.tiles_n;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 128); }
    fence_barrier_init();
    fence_proxy_async();
    prefetch_tmap(&maps.a_hi); prefetch_tmap(&maps.a_lo); prefetch_tmap(&maps.b_hi); prefetch_tmap(&maps.b_lo);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  fence_before_thread_sync();
  __syncthreads();
  fence_after_thread_sync();
  const uint32_t tmem_base = *tmem_slot;

  // tile index -> (m0, n0): column-major inside bands of 8 tile rows (operand reuse in L2)
  auto tile_origin = [&](int t, int& m0, int& n0) {
    const int band = 8;
    int per_band = band * g.tiles_n;
    int b = t / per_band, r = t % per_band;
    int rows = min(band, g.tiles_m - b * band);
    m0 = (b * band + r % rows) * BM;
    n0 = (r / rows) * BN;
  };

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
        int m0, n0, k0, k1;
        tile_origin(t, m0, n0);
        if (!range(m0, n0, k0, k1)) continue;
        for (int k = k0; k < k1; k += BK) {
          if (!mbar_wait(&empty[stage], phase ^ 1)) { report_error(g.dev_info, GPTQ_ERR_TIMEOUT, 11); ok = false; break; }
          uint8_t* s = tiles + (size_t)stage * STAGE_BYTES;
          uint8_t *ahi = s, *alo = s + OP_A_BYTES, *bhi = s + 2 * OP_A_BYTES, *blo = bhi + OP_B_BYTES;
          mbar_arrive_expect_tx(&full[stage], STAGE_BYTES);
          tma_load_2d(ahi, &maps.a_hi, k, m0, &full[stage]);
          tma_load_2d(alo, &maps.a_lo, k, m0, &full[stage]);
          tma_load_2d(bhi, &maps.b_hi, k, n0, &full[stage]);
          tma_load_2d(blo, &maps.b_lo, k, n0, &full[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(kFmtTF32, false, false, BM, BN);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
        int m0, n0, k0, k1;
        tile_origin(t, m0, n0);
        if (!range(m0, n0, k0, k1)) continue;
        if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1)) { report_error(g.dev_info, GPTQ_ERR_TIMEOUT, 12); break; }
        fence_after_thread_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
        for (int k = k0; k < k1; k += BK) {
          if (!mbar_wait(&full[stage], phase)) { report_error(g.dev_info, GPTQ_ERR_TIMEOUT, 13); ok = false; break; }
          fence_after_thread_sync();
          const uint32_t s = smem_u32(tiles + (size_t)stage * STAGE_BYTES);
          const uint32_t ahi = s, alo = s + OP_A_BYTES, bhi = s + 2 * OP_A_BYTES, blo = bhi + OP_B_BYTES;
#pragma unroll
          for (int ks = 0; ks < BK / 8; ++ks) {
            // K-major tiles: 8 fp32 = 32 bytes further along the swizzled row; 8-row groups 1024 B apart
            const uint64_t dah = make_desc_sw128(ahi + ks * 32, 0, 1024), dal = make_desc_sw128(alo + ks * 32, 0, 1024);
            const uint64_t dbh = make_desc_sw128(bhi + ks * 32, 0, 1024), dbl = make_desc_sw128(blo + ks * 32, 0, 1024);
            mma_tf32(d_tmem, dal, dbh, idesc, (k > k0 || ks > 0) ? 1u : 0u);   // small terms first
            mma_tf32(d_tmem, dah, dbl, idesc, 1u);
            mma_tf32(d_tmem, dah, dbh, idesc, 1u);
          }
          mma_commit(&empty[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        mma_commit(&acc_full[acc]);
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
  } else {
    const int q = warp & 3;
    int acc = 0; uint32_t acc_phase = 0;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
      int m0, n0, k0, k1;
      tile_origin(t, m0, n0);
      if (!range(m0, n0, k0, k1)) continue;
      if (!mbar_wait(&acc_full[acc], acc_phase)) { if (lane == 0) report_error(g.dev_info, GPTQ_ERR_TIMEOUT, 14); break; }
      fence_after_thread_sync();
      const int row = m0 + q * 32 + lane;
#pragma unroll 1
      for (int cc = 0; cc < BN; cc += 32) {
        float v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + cc), v);
        tmem_ld_wait();
        if (row < g.M && n0 + cc < g.N) epi(row, n0 + cc, v);
      }
      fence_before_thread_sync();
      mbar_arrive(&acc_empty[acc]);
      if (++acc == 2) { acc = 0; acc_phase ^= 1; }
    }
  }
  fence_before_thread_sync();
  __syncthreads();
  if (warp == 1) { fence_after_thread_sync(); tmem_dealloc(tmem_base, 512); }
}

// Host-side description of one fp32 operand pair (hi, lo share the geometry).
struct Operand {
  const float* hi; const float* lo;
  int64_t rows, cols, ld;       // row-major [rows][cols], leading dimension ld (elements)
};

template <class RangeF, class EpiF>
gptq_status_t launch(const Operand& A /*[M][K]*/, const Operand& B /*[N][K]*/, int M, int N,
                     RangeF range, EpiF epi, int* dev_info, cudaStream_t stream) {
  if (M <= 0 || N <= 0) return GPTQ_OK;
  Maps maps;
  gptq_status_t st;
  auto mk = [&](CUtensorMap* m, const float* p, const Operand& o, uint32_t box_in, uint32_t box_out) {
    return make_tmap_2d(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, p, (uint64_t)o.cols, (uint64_t)o.rows,
                        (uint64_t)o.ld * 4, box_in, box_out);
  };
  if ((st = mk(&maps.a_hi, A.hi, A, BK, BM)) != GPTQ_OK) return st;
  if ((st = mk(&maps.a_lo, A.lo, A, BK, BM)) != GPTQ_OK) return st;
  if ((st = mk(&maps.b_hi, B.hi, B, BK, BN)) != GPTQ_OK) return st;
  if ((st = mk(&maps.b_lo, B.lo, B, BK, BN)) != GPTQ_OK) return st;
  Geometry g{M, N, (M + BM - 1) / BM, (N + BN - 1) / BN, dev_info};
  const int n_tiles = g.tiles_m * g.tiles_n;
  const int sms = device_sm_count();
  auto kern = gemm_tf32x3_kernel<RangeF, EpiF>;
  GPTQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
  kern<<<n_tiles < sms ? n_tiles : sms, kThreads, kSmemBytes, stream>>>(maps, g, range, epi);
  GPTQ_LAUNCH_CHECK();
  return GPTQ_OK;
}

// ---- splitting fp32 into tf32 hi / lo -----------------------------------------------------------
__device__ __forceinline__ void split_tf32(float x, float& hi, float& lo) {
  uint32_t h, l;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(h) : "f"(x));
  hi = __uint_as_float(h);
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(l) : "f"(x - hi));
  lo = __uint_as_float(l);
}

}  // namespace tf32x3
}  // namespace gptq
