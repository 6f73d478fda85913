// Two-CTA variant of the persistent tensor-core pipeline (see umma_pipe.cuh for the roles and for
// why chunk sums are kept in registers).  A pair of CTAs in one cluster computes one 256 x 256
// output tile: CTA r of the pair owns rows [m0 + 128 r, +128) and stages its 128 rows of A and the
// columns [n0 + 128 r, +128) of B; tcgen05.mma.cta_group::2 (issued by the leader, rank 0) runs on
// both SMs' tensor cores, which exchange the B halves.  Per CTA and K block that is 32 KB of
// operands for the same 128 x 256 x 64 MACs that cost 48 KB in the one-CTA kernel -- the one-CTA
// kernel is bound by operand fill from L2, not by the tensor pipe -- and six stages fit.
//
// Synchronisation across the pair:
//   full[s]      lives in the leader; both CTAs' TMA loads credit their bytes to it
//   empty[s]     one per CTA; the leader's tcgen05.commit arrives on both (multicast commit)
//   acc_full[a]  one per CTA; multicast commit when a chunk is accumulated
//   acc_empty[a] lives in the leader; one arrival per epilogue warp of either CTA
// A cluster barrier brackets the kernel so neither CTA leaves (or frees TMEM / shared memory)
// while its peer can still touch it.  Every mbarrier wait is bounded.
#pragma once
#include "umma.cuh"

namespace gptq {
namespace pipe2 {

constexpr int BM_CTA = 128, BN = 256;      // per-CTA rows; tile is 256 x 256
constexpr int kThreads = 320;
constexpr int kEpiWarps = 8;

template <class Traits, class ItemF, class EpiF>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
umma_pipe2_kernel(const __grid_constant__ typename Traits::Maps maps, const int n_items, const ItemF itemf,
                  const EpiF epi, int* dev_info) {
  using namespace umma;
  constexpr int STAGES = Traits::STAGES;
  constexpr int STAGE_BYTES = Traits::STAGE_BYTES;     // per CTA
  constexpr int CHUNK_KB = Traits::CHUNK_KB;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + (size_t)STAGES * STAGE_BYTES);
  uint64_t* full = bars;
  uint64_t* empty = bars + STAGES;
  uint64_t* acc_full = bars + 2 * STAGES;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 2 * kEpiWarps); }
    fence_barrier_init();
    fence_proxy_async();
    Traits::prefetch(maps);
  }
  if (warp == 1) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
  fence_before_thread_sync();
  __syncthreads();
  cluster_sync();                       // peer's barriers are initialised before anything is sent to them
  fence_after_thread_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int idx = pair; idx < n_items && ok; idx += n_pairs) {
        int m0, n0, kb0, kb1;
        if (!itemf(idx, m0, n0, kb0, kb1)) continue;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(&empty[stage], phase ^ 1)) { report_error(dev_info, GPTQ_ERR_TIMEOUT, 21); ok = false; break; }
          if (rank == 0) mbar_arrive_expect_tx(&full[stage], 2 * STAGE_BYTES);   // bytes of both CTAs
          if (idx != g_skip_loads_of_item)      // (test knob: an item whose loads never come, see umma.cuh)
            Traits::load(tiles + (size_t)stage * STAGE_BYTES, maps, m0 + BM_CTA * (int)rank, n0 + (BN / 2) * (int)rank, kb,
                         &full[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      for (int idx = pair; idx < n_items && ok; idx += n_pairs) {
        int m0, n0, kb0, kb1;
        if (!itemf(idx, m0, n0, kb0, kb1)) continue;
        for (int cb = kb0; cb < kb1 && ok; cb += CHUNK_KB) {
          if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1)) { report_error(dev_info, GPTQ_ERR_TIMEOUT, 22); ok = false; break; }
          fence_after_thread_sync();
          const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
          const int ce = min(kb1, cb + CHUNK_KB);
          for (int kb = cb; kb < ce; ++kb) {
            if (!mbar_wait(&full[stage], phase)) { report_error(dev_info, GPTQ_ERR_TIMEOUT, 23); ok = false; break; }
            fence_after_thread_sync();
            Traits::mma(d_tmem, smem_u32(tiles + (size_t)stage * STAGE_BYTES), kb == cb);
            mma_commit_pair(&empty[stage]);
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
          }
          if (!ok) break;
          mma_commit_pair(&acc_full[acc]);
          if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (both CTAs, own rows)
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    for (int idx = pair; idx < n_items && ok; idx += n_pairs) {
      int m0, n0, kb0, kb1;
      if (!itemf(idx, m0, n0, kb0, kb1)) continue;
      float sum[128];
#pragma unroll
      for (int i = 0; i < 128; ++i) sum[i] = 0.f;
      for (int cb = kb0; cb < kb1; cb += CHUNK_KB) {
        if (!mbar_wait(&acc_full[acc], acc_phase)) { if (lane == 0) report_error(dev_info, GPTQ_ERR_TIMEOUT, 24); ok = false; break; }
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
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty[acc]), 0));
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
      if (!ok) break;
      const int row = m0 + BM_CTA * (int)rank + q * 32 + lane;
#pragma unroll
      for (int c = 0; c < 4; ++c)
        epi(row, n0 + half * 128 + 32 * c, *reinterpret_cast<const float(*)[32]>(&sum[32 * c]));
    }
  }
  fence_before_thread_sync();
  __syncthreads();
  cluster_sync();                       // the peer is done with this CTA's shared memory and barriers
  if (warp == 1) { fence_after_thread_sync(); tmem_dealloc_pair(tmem_base, 512); }
}

template <class Traits, class ItemF, class EpiF>
gptq_status_t launch_pipe2(const typename Traits::Maps& maps, int64_t n_items, ItemF itemf, EpiF epi, int* dev_info,
                           cudaStream_t stream, int reserve_sms = 0) {
  if (n_items <= 0) return GPTQ_OK;
  if (n_items > 0x7FFFFFFF) return GPTQ_ERR_UNSUPPORTED;
  constexpr size_t smem = (size_t)Traits::STAGES * Traits::STAGE_BYTES + 1024 + 256;
  int pairs_max = (device_sm_count() - reserve_sms) / 2;     // SMs left free for kernels running beside this one
  if (pairs_max < 1) pairs_max = 1;
  const int pairs = (int)(n_items < pairs_max ? n_items : pairs_max);
  auto kern = umma_pipe2_kernel<Traits, ItemF, EpiF>;
  GPTQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<2 * pairs, kThreads, smem, stream>>>(maps, (int)n_items, itemf, epi, dev_info);
  GPTQ_LAUNCH_CHECK();
  return GPTQ_OK;
}

}  // namespace pipe2
}  // namespace gptq
