// fp32-accurate tensor-core contraction from fp16 operand PAIRS ("3xFP16") on tcgen05 / TMEM / TMA,
// two-CTA form (umma_pipe2.cuh): a CTA pair owns a 256 x 256 output tile.
//
//   acc[m][n] = sum_k A[m][k] * B[n][k]  ~  Ahi*Bhi + Ahi*Blo + Alo*Bhi     (hi = fp16(x), lo = fp16(x - hi))
//
// An fp16 number carries 11 significant bits like a tf32 number, so hi + lo holds 22 bits and the
// dropped lo*lo term is of relative size 2^-22 -- the accuracy of three tf32 products of tf32 pairs
// -- while kind::f16 instructions run at twice the tf32 rate and the operands take half the bytes.
// Products of two fp16 values are exact in the fp32 accumulator.  The price is fp16's narrow exponent
// range: callers must scale their operands by powers of two (exact) so that the entries that matter
// sit well inside [2^-14, 2^15], and undo the scaling in the epilogue.  Entries far below a row's
// largest one lose relative precision gracefully (absolute error <= 2^-25 in scaled units); values
// beyond the range must be saturated by whoever writes the operands.
//
// Operand layouts: both row-major with K contiguous (A is [M][K], B is [N][K]).
// TMA boxes of 64 fp16 x 128 rows with 128-byte swizzle are the canonical K-major tiles.  Per CTA and
// 64-wide K block: its 128 rows of A (hi, lo) and its 128 of the tile's 256 rows of B (hi, lo) = 64 KB;
// twelve MMAs (four 16-wide K steps x three products) per K block go into one TMEM accumulator, which is
// drained into register running sums after every second K block, i.e. after 24 MMAs (see umma_pipe.cuh for
// why; draining after every block costs 7 % of a whole 175B-shaped step for an error that is already at the
// 1e-6 level of the factor either way: probe residual of U at 49152 columns 1.1e-6 against 1.8e-6).
#pragma once
#include <cstring>

#include "umma_pipe2.cuh"

namespace gptq {
namespace f16x3 {

constexpr int BM = 256, BN = 256, BK = 64;
constexpr int kSuperK = 4096;                 // K per work item: 32 register adds of 128-wide chunk sums

struct Traits {
  static constexpr int STAGES = 3;
  static constexpr int OP_BYTES = 128 * BK * 2;            // 16 KB: 128 rows x 64 fp16 (one of hi / lo, A or B half)
  static constexpr int STAGE_BYTES = 4 * OP_BYTES;         // 64 KB per CTA
  static constexpr int CHUNK_KB = 2;                       // 24 MMAs per TMEM accumulation
  static constexpr int EPI_SMEM = 8 * 4096;                // staging for epilogues that leave through TMA reductions
  struct Maps { CUtensorMap a_hi, a_lo, b_hi, b_lo, out; };  // out: the output, for those epilogues only

  static __device__ __forceinline__ void prefetch(const Maps& m) {
    umma::prefetch_tmap(&m.a_hi); umma::prefetch_tmap(&m.a_lo); umma::prefetch_tmap(&m.b_hi); umma::prefetch_tmap(&m.b_lo);
  }
  // m0: first row of this CTA's half of A; n0: first row (of B) of this CTA's half of the tile's columns
  static __device__ __forceinline__ void load(uint8_t* s, const Maps& m, int m0, int n0, int kb, uint64_t* bar) {
    const int k = kb * BK;
    umma::tma_load_2d_pair(s, &m.a_hi, k, m0, bar);
    umma::tma_load_2d_pair(s + OP_BYTES, &m.a_lo, k, m0, bar);
    umma::tma_load_2d_pair(s + 2 * OP_BYTES, &m.b_hi, k, n0, bar);
    umma::tma_load_2d_pair(s + 3 * OP_BYTES, &m.b_lo, k, n0, bar);
  }
  static __device__ __forceinline__ void mma(uint32_t d_tmem, uint32_t s, bool fresh) {
    using namespace umma;
    constexpr uint32_t idesc = make_idesc(kFmtF16, false, false, BM, BN);
    const uint32_t ahi = s, alo = s + OP_BYTES, bhi = s + 2 * OP_BYTES, blo = s + 3 * OP_BYTES;
#pragma unroll
    for (int ks = 0; ks < BK / 16; ++ks) {
      // K-major tiles: 16 fp16 = 32 bytes further along the swizzled row; 8-row groups 1024 B apart
      const uint64_t dah = make_desc_sw128(ahi + ks * 32, 0, 1024), dal = make_desc_sw128(alo + ks * 32, 0, 1024);
      const uint64_t dbh = make_desc_sw128(bhi + ks * 32, 0, 1024), dbl = make_desc_sw128(blo + ks * 32, 0, 1024);
      mma_f16_pair(d_tmem, dal, dbh, idesc, (fresh && ks == 0) ? 0u : 1u);   // small terms first
      mma_f16_pair(d_tmem, dah, dbl, idesc, 1u);
      mma_f16_pair(d_tmem, dah, dbh, idesc, 1u);
    }
  }
};

// Work items: 256 x 256 tiles x super-chunks of K, chunk-major; tiles column-major inside bands of 8 tile
// rows (operand reuse in L2).  kTriLeft: A is upper triangular (A[m][k] = 0 for k < m), so K starts at the
// tile's first row.  kUpperOut: only tiles that touch the upper triangle of the output are computed.
template <bool kTriLeft, bool kUpperOut>
struct TileItems {
  int tiles_m, tiles_n, kb_total, sc_kb;
  __device__ __forceinline__ bool operator()(int idx, int& m0, int& n0, int& kb0, int& kb1) const {
    const int n_tiles = tiles_m * tiles_n;
    const int sc = idx / n_tiles, t = idx % n_tiles;
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

// Host-side description of one operand pair (hi, lo share the geometry).
struct Operand {
  const __half* hi; const __half* lo;
  int64_t rows, cols, ld;       // row-major [rows][cols], leading dimension ld (elements, a multiple of 8); cols = K
};

// acc = A * B^T over K = A.cols = B.cols; epi must accumulate (it is called once per super-chunk).
template <bool kTriLeft, bool kUpperOut, class EpiF>
gptq_status_t launch(const Operand& A, const Operand& B, int M, int N, EpiF epi, int* dev_info, cudaStream_t stream,
                     int reserve_sms = 0, const CUtensorMap* out_map = nullptr) {
  const int64_t K = A.cols;
  if (M <= 0 || N <= 0 || K <= 0) return GPTQ_OK;
  static_assert(!pipe2::is_tile_epilogue<EpiF>::value || !kUpperOut, "tile epilogues write whole 32 x 32 blocks");
  if (pipe2::is_tile_epilogue<EpiF>::value != (out_map != nullptr)) return GPTQ_ERR_INVALID_ARG;
  Traits::Maps maps;
  if (out_map) maps.out = *out_map; else memset(&maps.out, 0, sizeof(maps.out));
  gptq_status_t st;
  auto mk = [&](CUtensorMap* m, const __half* p, const Operand& o) {
    return make_tmap_2d(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, p, (uint64_t)o.cols, (uint64_t)o.rows,
                        (uint64_t)o.ld * 2, BK, 128);
  };
  if ((st = mk(&maps.a_hi, A.hi, A)) != GPTQ_OK) return st;
  if ((st = mk(&maps.a_lo, A.lo, A)) != GPTQ_OK) return st;
  if ((st = mk(&maps.b_hi, B.hi, B)) != GPTQ_OK) return st;
  if ((st = mk(&maps.b_lo, B.lo, B)) != GPTQ_OK) return st;
  TileItems<kTriLeft, kUpperOut> items{(M + BM - 1) / BM, (N + BN - 1) / BN, (int)((K + BK - 1) / BK), kSuperK / BK};
  const int n_sc = (items.kb_total + items.sc_kb - 1) / items.sc_kb;
  return pipe2::launch_pipe2<Traits>(maps, (int64_t)items.tiles_m * items.tiles_n * n_sc, items, epi, dev_info, stream,
                                     reserve_sms);
}

// Epilogue that leaves through TMA reductions: out[row][col] += alpha * sa[row] * sb[col] * partial (sa, sb optional) for
// a row-major fp32 output described by Maps::out ({N, M}, 32 x 32 boxes, 128-byte swizzle).  The lanes write their rows
// into the warp's swizzled 4 KB staging tile and one lane sends it off; elements beyond M or N are dropped by the TMA
// unit.  L2 then adds whole 128-byte rows instead of 32 separate 16-byte pieces per instruction, which is what made
// per-lane reductions cost 13 us per 256 x 256 tile (this form: 5 us).
struct EpiTileAddF32 {
  static constexpr bool kTile = true;
  int M, N; float alpha;
  const float* sa; const float* sb;
  __device__ __forceinline__ void tile(const Traits::Maps& maps, uint8_t* buf, int row0, int col0, const float (&v)[32],
                                       int lane) const {
    if (row0 >= M || col0 >= N) return;          // (warp-uniform)
    const int row = row0 + lane;
    const float a = (sa != nullptr && row < M) ? alpha * sa[row] : alpha;
    if (lane == 0) umma::bulk_group_wait_read_all();     // the previous reduction has read the staging tile
    __syncwarp();
    const uint32_t base = umma::smem_u32(buf) + (uint32_t)lane * 128u;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      float4 b = make_float4(1.f, 1.f, 1.f, 1.f);
      if (sb != nullptr && col0 + 4 * g < N) b = *reinterpret_cast<const float4*>(sb + col0 + 4 * g);
      asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(base + (uint32_t)((g ^ (lane & 7)) << 4)),
                   "f"(v[4 * g] * a * b.x), "f"(v[4 * g + 1] * a * b.y), "f"(v[4 * g + 2] * a * b.z), "f"(v[4 * g + 3] * a * b.w)
                   : "memory");
    }
    umma::fence_proxy_async();
    __syncwarp();
    if (lane == 0) {
      umma::tma_reduce_add_2d(&maps.out, col0, row0, buf);
      umma::bulk_group_commit();
    }
  }
};
// The tensor map such an epilogue needs: `out` points at the output's first element, ld in elements (a multiple of 4).
inline gptq_status_t make_out_map_f32(CUtensorMap* m, float* out, int M, int N, int64_t ld) {
  return make_tmap_2d(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, out, (uint64_t)N, (uint64_t)M, (uint64_t)ld * 4, 32, 32);
}

// ---- splitting a (pre-scaled) fp32 value into an fp16 hi / lo pair --------------------------------
// Saturating conversions: a value beyond fp16's range becomes +-65504 instead of infinity; `sat` is set
// when that happened so the caller can report it.
__device__ __forceinline__ void split_f16(float x, __half& hi, __half& lo, bool& sat) {
  unsigned short h, l;
  asm("cvt.rn.satfinite.f16.f32 %0, %1;" : "=h"(h) : "f"(x));
  hi = __ushort_as_half(h);
  const float r = x - __half2float(hi);
  asm("cvt.rn.satfinite.f16.f32 %0, %1;" : "=h"(l) : "f"(r));
  lo = __ushort_as_half(l);
  sat |= !(fabsf(x) <= 65504.f);
}

}  // namespace f16x3
}  // namespace gptq
