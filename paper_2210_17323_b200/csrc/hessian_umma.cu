// Stage 1 on the tensor pipe: H += 2 X X^T as a bf16 x bf16 -> fp32 contraction over tokens
// (Section 2: H = 2 X X^T).  tcgen05.mma with accumulators in tensor memory, operands staged by
// TMA into 128-byte-swizzled shared memory, one persistent CTA per SM.
//
// Memory holds X token-major ([token][channel]), so for H = X X^T BOTH operands are contiguous
// along M/N (channels), not along K (tokens): both are fed as MN-major tiles and no transpose is
// ever materialised.  A TMA box of 64 channels x 64 tokens lands as 64 rows of 128 bytes, which
// is exactly the canonical MN-major 128B-swizzle layout (8-token groups 1024 B apart, 64-channel
// groups one box = 8192 B apart).
//
// Work decomposition: output tiles of 128 x 256 that touch the upper triangle, times chunks of
// tokens.  A chunk is accumulated in TMEM (fp32), then added to H with vector reductions
// (red.global.add.v4.f32), so accumulation is hierarchical: at most `chunk` tokens in one
// tensor-core accumulator, chunks summed in fp32 in memory.  Two TMEM accumulators (2 x 256
// columns) let the epilogue of one work item overlap the MMAs of the next.
#include "hessian_umma.cuh"
#include "umma.cuh"

namespace gptq {

namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int BOX_BYTES = 64 * BK * 2;                    // one TMA box: 64 channels x 64 tokens bf16
constexpr int A_BYTES = (BM / 64) * BOX_BYTES;            // 16 KB
constexpr int B_BYTES = (BN / 64) * BOX_BYTES;            // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;            // 48 KB
constexpr int SUPER_ROWS = 16;                            // tile rows per rasterisation band
constexpr int kThreads = 192;                             // warp 0: TMA, warp 1: MMA, warps 2-5: epilogue
constexpr size_t kSmemBytes = (size_t)STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;

struct Params {
  float* H;
  int C;
  int tiles_m, tiles_n;   // 128-row and 256-column tile counts
  int n_enum;             // enumerated tiles per chunk (includes a few below-diagonal ones that are skipped)
  int n_chunks;           // token chunks
  int chunk_kblocks;      // 64-token blocks per chunk
  int total_kblocks;
  int* dev_info;
};

struct Item { int m0, n0, kb0, kb1; bool valid; };

// Work item -> tile and token range.  Tiles are enumerated in bands of 16 tile rows, column by
// column inside a band, so CTAs that run at the same time share operand rows in L2.
__device__ __forceinline__ Item decode_item(const Params& p, int item) {
  Item it;
  int chunk = item / p.n_enum, t = item % p.n_enum;
  int mi = 0, nj = 0;
  for (int s = 0; s * SUPER_ROWS < p.tiles_m; ++s) {
    int rows = min(SUPER_ROWS, p.tiles_m - s * SUPER_ROWS);
    int first = (s * SUPER_ROWS) >> 1;
    int cnt = rows * (p.tiles_n - first);
    if (t < cnt) { nj = first + t / rows; mi = s * SUPER_ROWS + t % rows; break; }
    t -= cnt;
  }
  it.m0 = mi * BM; it.n0 = nj * BN;
  it.valid = (mi >> 1) <= nj;           // tile touches the upper triangle: m0 <= n0 + BN - 1
  it.kb0 = chunk * p.chunk_kblocks;
  it.kb1 = min(p.total_kblocks, it.kb0 + p.chunk_kblocks);
  return it;
}

__global__ void __launch_bounds__(kThreads, 1)
hessian_umma_kernel(const __grid_constant__ CUtensorMap tmap, const Params p) {
  using namespace umma;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + (size_t)STAGES * STAGE_BYTES);
  uint64_t* full = bars;                  // [STAGES] TMA -> MMA
  uint64_t* empty = bars + STAGES;        // [STAGES] MMA -> TMA
  uint64_t* acc_full = bars + 2 * STAGES; // [2] MMA -> epilogue
  uint64_t* acc_empty = acc_full + 2;     // [2] epilogue -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_items = p.n_enum * p.n_chunks;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 128); }
    fence_barrier_init();
    fence_proxy_async();
    prefetch_tmap(&tmap);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  fence_before_thread_sync();
  __syncthreads();
  fence_after_thread_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        Item it = decode_item(p, item);
        if (!it.valid) continue;
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait(&empty[stage], phase ^ 1)) { report_error(p.dev_info, GPTQ_ERR_TIMEOUT, 1); ok = false; break; }
          uint8_t* a = tiles + (size_t)stage * STAGE_BYTES;
          uint8_t* b = a + A_BYTES;
          mbar_arrive_expect_tx(&full[stage], STAGE_BYTES);
          const int y = kb * BK;
#pragma unroll
          for (int j = 0; j < BM / 64; ++j) tma_load_2d(a + j * BOX_BYTES, &tmap, it.m0 + 64 * j, y, &full[stage]);
#pragma unroll
          for (int j = 0; j < BN / 64; ++j) tma_load_2d(b + j * BOX_BYTES, &tmap, it.n0 + 64 * j, y, &full[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(kFmtBF16, true, true, BM, BN);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        Item it = decode_item(p, item);
        if (!it.valid) continue;
        if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1)) { report_error(p.dev_info, GPTQ_ERR_TIMEOUT, 2); break; }
        fence_after_thread_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!mbar_wait(&full[stage], phase)) { report_error(p.dev_info, GPTQ_ERR_TIMEOUT, 3); ok = false; break; }
          fence_after_thread_sync();
          const uint32_t a = smem_u32(tiles + (size_t)stage * STAGE_BYTES), b = a + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            // 16 tokens per instruction = two 8-token groups (1024 B each)
            uint64_t da = make_desc_sw128(a + k * 2048, BOX_BYTES, 1024);
            uint64_t db = make_desc_sw128(b + k * 2048, BOX_BYTES, 1024);
            mma_f16(d_tmem, da, db, idesc, (kb > it.kb0 || k > 0) ? 1u : 0u);
          }
          mma_commit(&empty[stage]);          // stage reusable once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        mma_commit(&acc_full[acc]);           // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue: TMEM -> H (+= 2 acc)
    const int q = warp & 3;                   // TMEM lane quarter this warp may read
    int acc = 0; uint32_t acc_phase = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
      Item it = decode_item(p, item);
      if (!it.valid) continue;
      if (!mbar_wait(&acc_full[acc], acc_phase)) { if (lane == 0) report_error(p.dev_info, GPTQ_ERR_TIMEOUT, 4); break; }
      fence_after_thread_sync();
      const int row = it.m0 + q * 32 + lane;
      float* hrow = p.H + (int64_t)row * p.C;
#pragma unroll 1
      for (int cc = 0; cc < BN; cc += 32) {
        float v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + cc), v);
        tmem_ld_wait();
        if (row < p.C) {
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const int col = it.n0 + cc + 4 * g;
            if (col < p.C && col + 3 >= row)
              red_add_v4(hrow + col, 2.f * v[4 * g], 2.f * v[4 * g + 1], 2.f * v[4 * g + 2], 2.f * v[4 * g + 3]);
          }
        }
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

int device_sm_count() {
  static int sms = 0;
  if (!sms) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) sms = 148;
  }
  return sms;
}

bool hessian_umma_supported(int C, int64_t n_tokens) {
  return C % 32 == 0 && C >= 64 && n_tokens >= 1 && n_tokens < (int64_t)1 << 31;
}

gptq_status_t hessian_umma(float* H, const __nv_bfloat16* X, int64_t n_tokens, int C, int* dev_info,
                           cudaStream_t stream) {
  CUtensorMap tmap;
  gptq_status_t st = make_tmap_2d(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, (uint64_t)C, (uint64_t)n_tokens,
                                  (uint64_t)C * 2, 64, BK);
  if (st != GPTQ_OK) return st;
  Params p;
  p.H = H; p.C = C; p.dev_info = dev_info;
  p.tiles_m = ceil_div(C, BM); p.tiles_n = ceil_div(C, BN);
  p.n_enum = 0;
  int n_valid = 0;
  for (int s = 0; s * SUPER_ROWS < p.tiles_m; ++s) {
    int rows = p.tiles_m - s * SUPER_ROWS < SUPER_ROWS ? p.tiles_m - s * SUPER_ROWS : SUPER_ROWS;
    p.n_enum += rows * (p.tiles_n - ((s * SUPER_ROWS) >> 1));
  }
  for (int mi = 0; mi < p.tiles_m; ++mi) n_valid += p.tiles_n - (mi >> 1);
  p.total_kblocks = ceil_div(n_tokens, BK);
  // tokens per chunk: at most 8192 (128 blocks); shorter when there are too few tiles to fill the GPU
  const int sms = device_sm_count();
  int ck = 128;
  while (ck > 8 && (int64_t)n_valid * ceil_div(p.total_kblocks, ck) < 2 * sms) ck >>= 1;
  p.chunk_kblocks = ck;
  p.n_chunks = ceil_div(p.total_kblocks, ck);
  const int64_t items = (int64_t)p.n_enum * p.n_chunks;
  const int grid = (int)(items < sms ? items : sms);
  GPTQ_CUDA_TRY(cudaFuncSetAttribute(hessian_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
  hessian_umma_kernel<<<grid, kThreads, kSmemBytes, stream>>>(tmap, p);
  GPTQ_LAUNCH_CHECK();
  GPTQ_CUDA_TRY(launch_mirror_upper_to_lower(H, C, stream));
  return GPTQ_OK;
}

}  // namespace gptq
