// Persistent, warp-specialised tensor-core pipeline, one-CTA form (128 x 256 tiles): the Hessian contraction
// (bf16) of layers with fewer than 512 channels.  umma_pipe2.cuh holds the two-CTA form that everything
// larger uses; the roles and the reasoning below are the same there.
//
//   warp 0      TMA producer: fills a ring of shared-memory stages with operand tiles
//   warp 1      MMA issuer: tcgen05.mma from shared memory into one of two TMEM accumulators
//   warps 2-9   epilogue: drain the TMEM accumulator into fp32 REGISTER running sums
//
// Why the register running sums: the tensor core adds each MMA's products into its fp32
// accumulator with truncation (measured: about half an ulp lost per instruction, always toward
// zero), so a long contraction kept in TMEM drifts by ~3e-8 x (number of MMAs).  Here TMEM only
// ever holds a short CHUNK of the contraction (<= 32 MMAs); the chunk sums are added with
// round-to-nearest in registers by the CUDA cores, and the running sum of one work item (a few
// thousand K) is handed to the epilogue functor, which folds it into memory (fp32 reduction or
// fp64 read-modify-write).  Two TMEM accumulators let the drain of one chunk overlap the MMAs of
// the next.
//
// A work item is an output tile (128 x 256) and a range of K blocks; ItemF maps a linear item
// index to it:   bool operator()(int idx, int& m0, int& n0, int& kb0, int& kb1) const
// (false = nothing to do).  EpiF receives, per thread, one row and 32 consecutive columns:
//   void operator()(int row, int col0, const float (&v)[32]) const   (does its own bounds checks)
//
// Traits supply the operand staging and the MMA sequence of one K block:
//   BK_STAGE_BYTES, STAGES, CHUNK_KB (K blocks accumulated in TMEM before a drain), Maps,
//   load(stage_ptr, maps, m0, n0, kb, bar), mma(d_tmem, stage_addr, fresh).
#pragma once
#include "umma.cuh"

namespace gptq {
namespace pipe {

constexpr int BM = 128, BN = 256;
constexpr int kThreads = 320;
constexpr int kEpiThreads = 256;

template <class Traits, class ItemF, class EpiF>
__global__ void __launch_bounds__(kThreads, 1)
umma_pipe_kernel(const __grid_constant__ typename Traits::Maps maps, const int n_items, const ItemF itemf,
                 const EpiF epi, int* dev_info) {
  using namespace umma;
  constexpr int STAGES = Traits::STAGES;
  constexpr int STAGE_BYTES = Traits::STAGE_BYTES;
  constexpr int CHUNK_KB = Traits::CHUNK_KB;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + (size_t)STAGES * STAGE_BYTES);
  uint64_t* full = bars;                   // [STAGES] TMA -> MMA
  uint64_t* empty = bars + STAGES;         // [STAGES] MMA -> TMA
  uint64_t* acc_full = bars + 2 * STAGES;  // [2] MMA -> epilogue (one chunk accumulated)
  uint64_t* acc_empty = acc_full + 2;      // [2] epilogue -> MMA (accumulator drained)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], kEpiThreads); }
    fence_barrier_init();
    fence_proxy_async();
    Traits::prefetch(maps);
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
      for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
        int m0, n0, kb0, kb1;
        if (!itemf(idx, m0, n0, kb0, kb1)) continue;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(&empty[stage], phase ^ 1)) { report_error(dev_info, GPTQ_ERR_TIMEOUT, 1); ok = false; break; }
          mbar_arrive_expect_tx(&full[stage], STAGE_BYTES);
          if (idx != g_skip_loads_of_item)      // (test knob: an item whose loads never come, see umma.cuh)
            Traits::load(tiles + (size_t)stage * STAGE_BYTES, maps, m0, n0, kb, &full[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
        int m0, n0, kb0, kb1;
        if (!itemf(idx, m0, n0, kb0, kb1)) continue;
        for (int cb = kb0; cb < kb1 && ok; cb += CHUNK_KB) {
          if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1)) { report_error(dev_info, GPTQ_ERR_TIMEOUT, 2); ok = false; break; }
          fence_after_thread_sync();
          const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
          const int ce = min(kb1, cb + CHUNK_KB);
          for (int kb = cb; kb < ce; ++kb) {
            if (!mbar_wait(&full[stage], phase)) { report_error(dev_info, GPTQ_ERR_TIMEOUT, 3); ok = false; break; }
            fence_after_thread_sync();
            Traits::mma(d_tmem, smem_u32(tiles + (size_t)stage * STAGE_BYTES), kb == cb);
            mma_commit(&empty[stage]);        // stage reusable once these MMAs have read it
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
          }
          if (!ok) break;
          mma_commit(&acc_full[acc]);         // chunk complete
          if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int q = warp & 3;                   // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;         // which 128 of the 256 accumulator columns
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
      int m0, n0, kb0, kb1;
      if (!itemf(idx, m0, n0, kb0, kb1)) continue;
      float sum[128];
#pragma unroll
      for (int i = 0; i < 128; ++i) sum[i] = 0.f;
      for (int cb = kb0; cb < kb1; cb += CHUNK_KB) {
        if (!mbar_wait(&acc_full[acc], acc_phase)) { if (lane == 0) report_error(dev_info, GPTQ_ERR_TIMEOUT, 4); ok = false; break; }
        fence_after_thread_sync();
        const uint32_t t0 = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN + half * 128);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float v[32];
          tmem_ld_32x32(t0 + 32 * c, v);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) sum[32 * c + j] += v[j];
        }
        fence_before_thread_sync();
        mbar_arrive(&acc_empty[acc]);
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
      if (!ok) break;
      const int row = m0 + q * 32 + lane;
#pragma unroll
      for (int c = 0; c < 4; ++c)
        epi(row, n0 + half * 128 + 32 * c, *reinterpret_cast<const float(*)[32]>(&sum[32 * c]));
    }
  }
  fence_before_thread_sync();
  __syncthreads();
  if (warp == 1) { fence_after_thread_sync(); tmem_dealloc(tmem_base, 512); }
}

template <class Traits, class ItemF, class EpiF>
gptq_status_t launch_pipe(const typename Traits::Maps& maps, int64_t n_items, ItemF itemf, EpiF epi, int* dev_info,
                          cudaStream_t stream, int reserve_sms = 0) {
  if (n_items <= 0) return GPTQ_OK;
  if (n_items > 0x7FFFFFFF) return GPTQ_ERR_UNSUPPORTED;
  constexpr size_t smem = (size_t)Traits::STAGES * Traits::STAGE_BYTES + 1024 + 256;
  int sms = device_sm_count() - reserve_sms;      // SMs left free for kernels running beside this one
  if (sms < 1) sms = 1;
  auto kern = umma_pipe_kernel<Traits, ItemF, EpiF>;
  GPTQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<(int)(n_items < sms ? n_items : sms), kThreads, smem, stream>>>(maps, (int)n_items, itemf, epi, dev_info);
  GPTQ_LAUNCH_CHECK();
  return GPTQ_OK;
}

}  // namespace pipe
}  // namespace gptq
