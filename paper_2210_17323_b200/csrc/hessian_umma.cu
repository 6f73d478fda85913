// Stage 1 on the tensor pipe: H += 2 X X^T as a bf16 x bf16 -> fp32 contraction over tokens
// (Section 2: H = 2 X X^T).  tcgen05.mma with accumulators in tensor memory, operands staged by
// TMA into 128-byte-swizzled shared memory, one persistent CTA per SM (umma_pipe.cuh).
//
// Memory holds X token-major ([token][channel]), so for H = X X^T BOTH operands are contiguous
// along M/N (channels), not along K (tokens): both are fed as MN-major tiles and no transpose is
// ever materialised.  A TMA box of 64 channels x 64 tokens lands as 64 rows of 128 bytes, which
// is exactly the canonical MN-major 128B-swizzle layout (8-token groups 1024 B apart, 64-channel
// groups one box = 8192 B apart).
//
// Work decomposition: output tiles of 128 x 256 that touch the upper triangle, times super-chunks
// of up to 16384 tokens.  Accumulation is hierarchical: 512 tokens (32 MMAs) in a TMEM accumulator,
// chunk sums added round-to-nearest in registers over the super-chunk, super-chunk sums added to H
// with vector reductions (red.global.add.v4.f32).
#include "hessian_umma.cuh"
#include "umma_pipe.cuh"
#include "umma_pipe2.cuh"

namespace gptq {

namespace {

constexpr int BM = pipe::BM, BN = pipe::BN, BK = 64;
constexpr int BOX_BYTES = 64 * BK * 2;                    // one TMA box: 64 channels x 64 tokens bf16
constexpr int SUPER_ROWS = 16;                            // tile rows per rasterisation band

struct HessTraits {
  static constexpr int STAGES = 4;
  static constexpr int A_BYTES = (BM / 64) * BOX_BYTES;   // 16 KB
  static constexpr int B_BYTES = (BN / 64) * BOX_BYTES;   // 32 KB
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;   // 48 KB
  static constexpr int CHUNK_KB = 8;                      // 512 tokens = 32 MMAs per TMEM accumulation
  struct Maps { CUtensorMap x; };

  static __device__ __forceinline__ void prefetch(const Maps& m) { umma::prefetch_tmap(&m.x); }
  static __device__ __forceinline__ void load(uint8_t* s, const Maps& m, int m0, int n0, int kb, uint64_t* bar) {
    const int y = kb * BK;
#pragma unroll
    for (int j = 0; j < BM / 64; ++j) umma::tma_load_2d(s + j * BOX_BYTES, &m.x, m0 + 64 * j, y, bar);
#pragma unroll
    for (int j = 0; j < BN / 64; ++j) umma::tma_load_2d(s + A_BYTES + j * BOX_BYTES, &m.x, n0 + 64 * j, y, bar);
  }
  static __device__ __forceinline__ void mma(uint32_t d_tmem, uint32_t s, bool fresh) {
    using namespace umma;
    constexpr uint32_t idesc = make_idesc(kFmtBF16, true, true, BM, BN);
#pragma unroll
    for (int k = 0; k < BK / 16; ++k) {
      // 16 tokens per instruction = two 8-token groups (1024 B each)
      const uint64_t da = make_desc_sw128(s + k * 2048, BOX_BYTES, 1024);
      const uint64_t db = make_desc_sw128(s + A_BYTES + k * 2048, BOX_BYTES, 1024);
      mma_f16(d_tmem, da, db, idesc, (fresh && k == 0) ? 0u : 1u);
    }
  }
};

// Work item -> tile and token range.  Tiles are enumerated in bands of 16 tile rows, column by
// column inside a band, so CTAs that run at the same time share operand rows in L2; a few
// enumerated tiles lie wholly below the diagonal and are skipped.
struct HessItems {
  int tiles_m, tiles_n, n_enum, sc_kb, total_kb;
  __device__ __forceinline__ bool operator()(int idx, int& m0, int& n0, int& kb0, int& kb1) const {
    const int sc = idx / n_enum;
    int t = idx % n_enum, mi = 0, nj = 0;
    for (int s = 0; s * SUPER_ROWS < tiles_m; ++s) {
      const int rows = min(SUPER_ROWS, tiles_m - s * SUPER_ROWS);
      const int first = (s * SUPER_ROWS) >> 1;
      const int cnt = rows * (tiles_n - first);
      if (t < cnt) { nj = first + t / rows; mi = s * SUPER_ROWS + t % rows; break; }
      t -= cnt;
    }
    m0 = mi * BM; n0 = nj * BN;
    kb0 = sc * sc_kb;
    kb1 = min(total_kb, kb0 + sc_kb);
    return (mi >> 1) <= nj;          // tile touches the upper triangle: m0 <= n0 + BN - 1
  }
};

// ---- two-CTA variant: 256 x 256 tiles, each CTA stages 128 rows of A and 128 columns of B -------
struct HessPairTraits {
  static constexpr int STAGES = 6;
  static constexpr int A_BYTES = 2 * BOX_BYTES;           // 16 KB: this CTA's 128 rows
  static constexpr int B_BYTES = 2 * BOX_BYTES;           // 16 KB: this CTA's 128 of the 256 columns
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;   // 32 KB per CTA
  static constexpr int CHUNK_KB = 8;
  static constexpr int EPI_SMEM = 8 * 4096;               // one 32 x 32 fp32 staging tile per epilogue warp
  struct Maps { CUtensorMap x; CUtensorMap h; };          // X (bf16, 64 x 64 boxes), H (fp32, 32 x 32 boxes)

  static __device__ __forceinline__ void prefetch(const Maps& m) { umma::prefetch_tmap(&m.x); umma::prefetch_tmap(&m.h); }
  static __device__ __forceinline__ void load(uint8_t* s, const Maps& m, int m0, int n0, int kb, uint64_t* bar) {
    const int y = kb * BK;
#pragma unroll
    for (int j = 0; j < 2; ++j) umma::tma_load_2d_pair(s + j * BOX_BYTES, &m.x, m0 + 64 * j, y, bar);
#pragma unroll
    for (int j = 0; j < 2; ++j) umma::tma_load_2d_pair(s + A_BYTES + j * BOX_BYTES, &m.x, n0 + 64 * j, y, bar);
  }
  static __device__ __forceinline__ void mma(uint32_t d_tmem, uint32_t s, bool fresh) {
    using namespace umma;
    constexpr uint32_t idesc = make_idesc(kFmtBF16, true, true, 256, 256);
#pragma unroll
    for (int k = 0; k < BK / 16; ++k) {
      const uint64_t da = make_desc_sw128(s + k * 2048, BOX_BYTES, 1024);
      const uint64_t db = make_desc_sw128(s + A_BYTES + k * 2048, BOX_BYTES, 1024);
      mma_f16_pair(d_tmem, da, db, idesc, (fresh && k == 0) ? 0u : 1u);
    }
  }
};

// 256 x 256 tiles on or above the diagonal.  ONLY valid tiles are enumerated.  Order of the work items, which the
// dynamic item feed hands out in sequence so that the ~74 pairs always work on neighbouring items:
//   bands of `band` tile rows; inside a band the valid tiles column by column, cut into windows of `wt` tiles;
//   inside a window every token range (super-chunk) in turn; inside a token range the window's tiles.
// At any time the pairs therefore share the ~band + wt / band operand strips of one window over one or two token
// ranges (a few tens of MB, fetched from DRAM once and then read from L2), and the window's tiles of H stay in L2
// from one token range to the next, so that H goes to DRAM once per window and not once per token range.
struct HessPairItems {
  int tiles, n_enum, sc_kb, total_kb, band, wt, nsc;
  // valid tiles of band s: rows r0 .. r0+rows-1, columns r0 .. tiles-1, row <= column
  static __host__ __device__ __forceinline__ int band_count(int tiles, int band, int s) {
    const int r0 = s * band, rows = tiles - r0 < band ? tiles - r0 : band;
    return rows * (rows + 1) / 2 + rows * (tiles - r0 - rows);
  }
  __device__ __forceinline__ bool operator()(int idx, int& m0, int& n0, int& kb0, int& kb1) const {
    int mi = 0, nj = 0, sc = 0;
    for (int s = 0; s * band < tiles; ++s) {
      const int cnt = band_count(tiles, band, s);
      if (idx < cnt * nsc) {
        const int per_window = wt * nsc;
        const int j = idx / per_window, local = idx - j * per_window;
        const int n_w = cnt - j * wt < wt ? cnt - j * wt : wt;          // tiles in this window (the last one may be short)
        sc = local / n_w;
        const int t = j * wt + local - sc * n_w;
        const int r0 = s * band, rows = tiles - r0 < band ? tiles - r0 : band, tri = rows * (rows + 1) / 2;
        if (t < tri) {                     // diagonal part: column c (0-based inside the band) has c + 1 valid rows
          int c = 0;
          while ((c + 1) * (c + 2) / 2 <= t) ++c;
          nj = r0 + c; mi = r0 + t - c * (c + 1) / 2;
        } else {
          const int u = t - tri;
          nj = r0 + rows + u / rows; mi = r0 + u % rows;
        }
        break;
      }
      idx -= cnt * nsc;
    }
    m0 = mi * 256; n0 = nj * 256;
    kb0 = sc * sc_kb;
    kb1 = min(total_kb, kb0 + sc_kb);
    return true;
  }
};

// H[row][col..col+32) += 2 * partial, upper triangle only (4-wide groups that reach it).
struct EpiAddTwiceUpper {
  float* H; int C;
  __device__ __forceinline__ void operator()(int row, int col0, const float (&v)[32]) const {
    if (row >= C) return;
    float* hrow = H + (int64_t)row * C;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      const int col = col0 + 4 * g;
      if (col < C && col + 3 >= row)
        umma::red_add_v4(hrow + col, 2.f * v[4 * g], 2.f * v[4 * g + 1], 2.f * v[4 * g + 2], 2.f * v[4 * g + 3]);
    }
  }
};

// H[row0 .. +32)[col0 .. +32) += 2 * sums, one TMA reduction per warp and block: the lanes write their rows into a
// 128-byte-swizzled staging tile and one lane sends it off.  Blocks wholly below the diagonal are left out; the parts
// of diagonal blocks below it receive sums that the mirror pass overwrites.  The columns and rows beyond C are dropped
// by the TMA unit.
struct EpiAddTwiceTile {
  static constexpr bool kTile = true;
  int C;
  __device__ __forceinline__ void tile(const HessPairTraits::Maps& maps, uint8_t* buf, int row0, int col0,
                                       const float (&v)[32], int lane) const {
    if (row0 >= C || col0 >= C || col0 + 31 < row0) return;          // (warp-uniform)
    if (lane == 0) umma::bulk_group_wait_read_all();                  // the previous reduction has read the staging tile
    __syncwarp();
    const uint32_t base = umma::smem_u32(buf) + (uint32_t)lane * 128u;
#pragma unroll
    for (int g = 0; g < 8; ++g)
      asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(base + (uint32_t)((g ^ (lane & 7)) << 4)),
                   "f"(2.f * v[4 * g]), "f"(2.f * v[4 * g + 1]), "f"(2.f * v[4 * g + 2]), "f"(2.f * v[4 * g + 3]) : "memory");
    umma::fence_proxy_async();
    __syncwarp();
    if (lane == 0) {
      umma::tma_reduce_add_2d(&maps.h, col0, row0, buf);
      umma::bulk_group_commit();
    }
  }
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

}  // namespace

gptq_status_t make_tmap_2d(CUtensorMap* out, CUtensorMapDataType dtype, int elem_bytes, const void* base,
                           uint64_t inner, uint64_t outer, uint64_t row_stride_bytes,
                           uint32_t box_inner, uint32_t box_outer) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return GPTQ_ERR_CUDA;
  (void)elem_bytes;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {row_stride_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, dtype, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? GPTQ_OK : GPTQ_ERR_CUDA;
}

gptq_status_t make_tmap_3d_plain(CUtensorMap* out, CUtensorMapDataType dtype, const void* base, const uint64_t dims[3],
                                 const uint64_t strides_bytes[2], const uint32_t box[3]) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return GPTQ_ERR_CUDA;
  cuuint64_t d[3] = {dims[0], dims[1], dims[2]};
  cuuint64_t st[2] = {strides_bytes[0], strides_bytes[1]};
  cuuint32_t b[3] = {box[0], box[1], box[2]};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, dtype, 3, const_cast<void*>(base), d, st, b, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? GPTQ_OK : GPTQ_ERR_CUDA;
}

int device_sm_count() {
  // SM count of the CURRENT device, cached per device ordinal (a process may drive several GPUs).
  constexpr int kMaxDev = 64;
  static int sms_of[kMaxDev] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= kMaxDev) return 148;
  int sms = __atomic_load_n(&sms_of[dev], __ATOMIC_RELAXED);
  if (!sms) {
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) sms = 148;
    __atomic_store_n(&sms_of[dev], sms, __ATOMIC_RELAXED);
  }
  return sms;
}

bool hessian_umma_supported(int C, int64_t n_tokens) {
  return C % 32 == 0 && C >= 64 && n_tokens >= 1 && n_tokens < (int64_t)1 << 31;
}

gptq_status_t hessian_umma(float* H, const __nv_bfloat16* X, int64_t n_tokens, int C, int* dev_info,
                           cudaStream_t stream, bool mirror) {
  CUtensorMap tmap;
  gptq_status_t st = make_tmap_2d(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, (uint64_t)C, (uint64_t)n_tokens,
                                  (uint64_t)C * 2, 64, BK);
  if (st != GPTQ_OK) return st;
  const int sms = device_sm_count();
  const int total_kb = ceil_div(n_tokens, BK);
  int ck = C <= 8192 ? 256 : 128;       // one-CTA path: tokens per work item / 64
  if (C >= 512) {
    // two-CTA tiles of 256 x 256, dynamic item feed
    HessPairTraits::Maps maps;
    maps.x = tmap;
    st = make_tmap_2d(&maps.h, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, H, (uint64_t)C, (uint64_t)C, (uint64_t)C * 4, 32, 32);
    if (st != GPTQ_OK) return st;
    HessPairItems it;
    it.tiles = ceil_div(C, 256);
    it.band = 8;
    it.wt = 144;
    it.n_enum = it.tiles * (it.tiles + 1) / 2;
    ck = 128;                             // 8192 tokens per item
    while (ck > 8 && (int64_t)it.n_enum * ceil_div(total_kb, ck) < sms) ck >>= 1;
    while ((int64_t)it.n_enum * ceil_div(total_kb, ck) > 0x3FFFFFFF) ck <<= 1;     // (the grid has one cluster per item)
    it.total_kb = total_kb; it.sc_kb = ck; it.nsc = ceil_div(total_kb, ck);
    const int64_t n_items = (int64_t)it.n_enum * it.nsc;
    st = pipe2::launch_pipe2_dynamic<HessPairTraits>(maps, n_items, it, EpiAddTwiceTile{C}, dev_info, stream);
  } else {
    HessTraits::Maps maps{tmap};
    HessItems it;
    it.tiles_m = ceil_div(C, BM); it.tiles_n = ceil_div(C, BN);
    it.n_enum = 0;
    int n_valid = 0;
    for (int s = 0; s * SUPER_ROWS < it.tiles_m; ++s) {
      int rows = it.tiles_m - s * SUPER_ROWS < SUPER_ROWS ? it.tiles_m - s * SUPER_ROWS : SUPER_ROWS;
      it.n_enum += rows * (it.tiles_n - ((s * SUPER_ROWS) >> 1));
    }
    for (int mi = 0; mi < it.tiles_m; ++mi) n_valid += it.tiles_n - (mi >> 1);
    while (ck > 8 && (int64_t)n_valid * ceil_div(total_kb, ck) < 2 * sms) ck >>= 1;
    it.total_kb = total_kb; it.sc_kb = ck;
    st = pipe::launch_pipe<HessTraits>(maps, (int64_t)it.n_enum * ceil_div(total_kb, ck), it, EpiAddTwiceUpper{H, C},
                                       dev_info, stream);
  }
  if (st != GPTQ_OK) return st;
  if (mirror) GPTQ_CUDA_TRY(launch_mirror_upper_to_lower(H, C, stream));
  return GPTQ_OK;
}

cudaError_t hessian_set_wait_test_knobs(unsigned long long limit_ns, int skip_item) { return set_wait_test_knobs(limit_ns, skip_item); }

}  // namespace gptq

