// fp32-accurate tensor-core contraction ("3xTF32") on tcgen05 / TMEM / TMA.
//
//   acc[m][n] = sum_k A[m][k] * B[n][k]  ~  Ahi*Bhi + Ahi*Blo + Alo*Bhi     (hi = tf32(x), lo = tf32(x - hi))
//
// Each fp32 operand is supplied as TWO fp32 arrays holding its tf32-representable high part and
// the tf32-rounded remainder; the dropped lo*lo term and the rounding of lo are of relative size
// 2^-22, i.e. fp32 level.  Three tcgen05.mma (kind::tf32) per 8-wide K step go into one TMEM
// accumulator, which is drained into register running sums after every 32-wide K block (see
// umma_pipe.cuh for why).
//
// Operand layouts: both row-major with K contiguous -- A is [M][K], B is supplied TRANSPOSED as
// [N][K] (callers whose right factor is stored [K][N] write its transpose when they split it into
// hi / lo).  TMA boxes of 32 fp32 x rows with 128-byte swizzle give the canonical K-major tiles.
//
// The contraction of one 128 x 256 output tile is cut into super-chunks of kSuperK; each
// (tile, super-chunk) is an independent work item whose partial sum reaches the epilogue functor,
// which must therefore ACCUMULATE into memory (a reduction), not store.
#pragma once
#include "umma_pipe.cuh"

namespace gptq {
namespace tf32x3 {

constexpr int BM = pipe::BM, BN = pipe::BN, BK = 32;
constexpr int kSuperK = 2048;                 // K per work item: 64 register adds of 32-wide chunk sums

struct Traits {
  static constexpr int STAGES = 2;
  static constexpr int OP_A_BYTES = BM * BK * 4;       // 16 KB (one of hi / lo)
  static constexpr int OP_B_BYTES = BN * BK * 4;       // 32 KB
  static constexpr int STAGE_BYTES = 2 * (OP_A_BYTES + OP_B_BYTES);   // 96 KB
  static constexpr int CHUNK_KB = 1;
  struct Maps { CUtensorMap a_hi, a_lo, b_hi, b_lo; };

  static __device__ __forceinline__ void prefetch(const Maps& m) {
    umma::prefetch_tmap(&m.a_hi); umma::prefetch_tmap(&m.a_lo); umma::prefetch_tmap(&m.b_hi); umma::prefetch_tmap(&m.b_lo);
  }
  static __device__ __forceinline__ void load(uint8_t* s, const Maps& m, int m0, int n0, int kb, uint64_t* bar) {
    const int k = kb * BK;
    umma::tma_load_2d(s, &m.a_hi, k, m0, bar);
    umma::tma_load_2d(s + OP_A_BYTES, &m.a_lo, k, m0, bar);
    umma::tma_load_2d(s + 2 * OP_A_BYTES, &m.b_hi, k, n0, bar);
    umma::tma_load_2d(s + 2 * OP_A_BYTES + OP_B_BYTES, &m.b_lo, k, n0, bar);
  }
  static __device__ __forceinline__ void mma(uint32_t d_tmem, uint32_t s, bool fresh) {
    using namespace umma;
    constexpr uint32_t idesc = make_idesc(kFmtTF32, false, false, BM, BN);
    const uint32_t ahi = s, alo = s + OP_A_BYTES, bhi = s + 2 * OP_A_BYTES, blo = bhi + OP_B_BYTES;
#pragma unroll
    for (int ks = 0; ks < BK / 8; ++ks) {
      // K-major tiles: 8 fp32 = 32 bytes further along the swizzled row; 8-row groups 1024 B apart
      const uint64_t dah = make_desc_sw128(ahi + ks * 32, 0, 1024), dal = make_desc_sw128(alo + ks * 32, 0, 1024);
      const uint64_t dbh = make_desc_sw128(bhi + ks * 32, 0, 1024), dbl = make_desc_sw128(blo + ks * 32, 0, 1024);
      mma_tf32(d_tmem, dal, dbh, idesc, (fresh && ks == 0) ? 0u : 1u);   // small terms first
      mma_tf32(d_tmem, dah, dbl, idesc, 1u);
      mma_tf32(d_tmem, dah, dbh, idesc, 1u);
    }
  }
};

// Work items: tiles x super-chunks of K, chunk-major so concurrent CTAs work on different tiles of
// the same K range.  kTriLeft: A is upper triangular (A[m][k] = 0 for k < m), so K starts at the
// tile's first row.  kUpperOut: only tiles that touch the upper triangle of the output are computed.
template <bool kTriLeft, bool kUpperOut>
struct TileItems {
  int tiles_m, tiles_n, kb_total, sc_kb;
  __device__ __forceinline__ bool operator()(int idx, int& m0, int& n0, int& kb0, int& kb1) const {
    const int n_tiles = tiles_m * tiles_n;
    const int sc = idx / n_tiles, t = idx % n_tiles;
    // tiles column-major inside bands of 8 tile rows (operand reuse in L2)
    const int band = 8, per_band = band * tiles_n;
    const int b = t / per_band, r = t % per_band;
    const int rows = min(band, tiles_m - b * band);
    m0 = (b * band + r % rows) * BM;
    n0 = (r / rows) * BN;
    if (kUpperOut && m0 > n0 + BN - 1) return false;
    const int first = kTriLeft ? m0 / BK : 0;
    kb0 = first + sc * sc_kb;
    kb1 = min(kb_total, kb0 + sc_kb);
    return kb0 < kb1;
  }
};

// Host-side description of one fp32 operand pair (hi, lo share the geometry).
struct Operand {
  const float* hi; const float* lo;
  int64_t rows, cols, ld;       // row-major [rows][cols], leading dimension ld (elements); cols = K
};

// acc = A * B^T over K = A.cols = B.cols; epi must accumulate (it is called once per super-chunk).
template <bool kTriLeft, bool kUpperOut, class EpiF>
gptq_status_t launch(const Operand& A, const Operand& B, int M, int N, EpiF epi, int* dev_info, cudaStream_t stream,
                     int reserve_sms = 0) {
  const int64_t K = A.cols;
  if (M <= 0 || N <= 0 || K <= 0) return GPTQ_OK;
  Traits::Maps maps;
  gptq_status_t st;
  auto mk = [&](CUtensorMap* m, const float* p, const Operand& o, uint32_t box_out) {
    return make_tmap_2d(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, p, (uint64_t)o.cols, (uint64_t)o.rows,
                        (uint64_t)o.ld * 4, BK, box_out);
  };
  if ((st = mk(&maps.a_hi, A.hi, A, BM)) != GPTQ_OK) return st;
  if ((st = mk(&maps.a_lo, A.lo, A, BM)) != GPTQ_OK) return st;
  if ((st = mk(&maps.b_hi, B.hi, B, BN)) != GPTQ_OK) return st;
  if ((st = mk(&maps.b_lo, B.lo, B, BN)) != GPTQ_OK) return st;
  TileItems<kTriLeft, kUpperOut> items{(M + BM - 1) / BM, (N + BN - 1) / BN, (int)((K + BK - 1) / BK), kSuperK / BK};
  const int n_sc = (items.kb_total + items.sc_kb - 1) / items.sc_kb;
  return pipe::launch_pipe<Traits>(maps, (int64_t)items.tiles_m * items.tiles_n * n_sc, items, epi, dev_info, stream,
                                   reserve_sms);
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
