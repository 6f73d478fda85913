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
//
// Work items reach the pairs in one of two ways (see "work-item feed" below): a persistent grid with a
// fixed round-robin assignment, or a grid of one cluster per item in which the running clusters take
// over the items of clusters that have not started (cluster launch control).
#pragma once
#include "umma.cuh"

namespace gptq {
namespace pipe2 {

constexpr int BM_CTA = 128, BN = 256;      // per-CTA rows; tile is 256 x 256
constexpr int kEpiWarps = 8;
// warps: 0 TMA producer, 1 MMA issuer, 2..9 epilogue, 10 work-item scheduler (dynamic form only)
constexpr int threads_of(bool dynamic) { return dynamic ? 352 : 320; }
constexpr int kThreads = threads_of(false);

// Optional members: Traits::EPI_SMEM (bytes of shared memory for the epilogue, 1024-byte aligned, behind the stages) and
// EpiF::kTile (the epilogue is called once per warp and 32 x 32 block of sums, with a 4 KB staging buffer of its own).
template <class T, class = void> struct epi_smem_of { static constexpr int value = 0; };
template <class T> struct epi_smem_of<T, decltype((void)T::EPI_SMEM)> { static constexpr int value = T::EPI_SMEM; };
template <class T, class = void> struct is_tile_epilogue { static constexpr bool value = false; };
template <class T> struct is_tile_epilogue<T, decltype((void)T::kTile)> { static constexpr bool value = T::kTile; };

// ---- work-item feed ------------------------------------------------------------------------------
// Static form: pair p takes items p, p + n_pairs, ... (a persistent grid of at most one pair per two SMs).
// Dynamic form: the grid has one cluster PER ITEM; a running cluster first takes the item of its own index
// and then keeps cancelling the launch of clusters that have not started yet (cluster launch control) and
// takes their items instead.  Items are therefore handed out in index order to whichever pair is free:
// the pairs in flight always work on a contiguous window of the item sequence however much their speeds
// differ, which is what lets the item order control what is shared through L2.  (With the static
// form the pairs of a 49152-channel Hessian launch drifted apart by up to 75 items, and two thirds of
// all operand loads went to DRAM.)  The scheduler thread of the leader CTA issues the cancel requests one
// item ahead of the producer, works out the item's tile and token range (so that no other role spends time on
// that at an item boundary) and hands both to the other roles of both CTAs through a two-slot ring:
//   sched_full[slot]   one per CTA; the scheduler arrives on both after writing idx[slot] and item[slot] in both CTAs
//   sched_empty[slot]  in the leader; one arrival per consumer (producer, MMA issuer, epilogue warps) of either CTA
struct SchedRing {
  uint64_t full[2];
  uint64_t empty[2];
  uint64_t clc_bar;
  uint64_t go;          // the leader's producer arrives when it starts an item: the request for the item after it may go out
  int idx[2];           // item index, -1: no more items
  int abort;            // leader's copy decides for the pair: a wait already ran out somewhere in this launch
  alignas(16) int4 item[2];           // the item's {m0, n0, kb0, kb1}, decoded once by the scheduler
  alignas(16) uint4 clc_response;
};
constexpr uint32_t kSchedConsumers = 2 * kEpiWarps + 3;   // both CTAs' epilogue warps and producers, the leader's MMA issuer

__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(umma::smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const uint64_t t0 = umma::global_timer_ns();
  const uint64_t limit = umma::g_wait_limit_ns;
  uint32_t spins = 0;
  while (!mbar_try_wait_cluster(bar, parity)) {
    if ((++spins & 0x3FF) == 0 && umma::global_timer_ns() - t0 > limit) return false;
  }
  return true;
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_v4(uint32_t cluster_addr, int4 v) {
  asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// Asks the hardware to cancel the launch of one not yet started cluster of this grid; the 16-byte answer
// lands in `response` (this CTA's shared memory) and completes 16 bytes on `bar`.
__device__ __forceinline__ void clc_try_cancel(uint4* response, uint64_t* bar) {
  asm volatile("clusterlaunchcontrol.try_cancel.async.shared::cta.mbarrier::complete_tx::bytes.b128 [%0], [%1];"
               ::"r"(umma::smem_u32(response)), "r"(umma::smem_u32(bar)) : "memory");
}
// Index (blockIdx.x of its first CTA) of the cancelled cluster, or -1 if nothing was left to cancel.
__device__ __forceinline__ int clc_decode(const uint4* response) {
  uint32_t x, valid;
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b128 r;\n\t"
      "ld.shared.b128 r, [%2];\n\t"
      "clusterlaunchcontrol.query_cancel.is_canceled.pred.b128 p, r;\n\t"
      "selp.u32 %1, 1, 0, p;\n\t"
      "mov.u32 %0, 0;\n\t"
      "@p clusterlaunchcontrol.query_cancel.get_first_ctaid::x.b32.b128 %0, r;\n\t}"
      : "=r"(x), "=r"(valid) : "r"(umma::smem_u32(response)) : "memory");
  return valid ? (int)x : -1;
}

// A role's position in the item sequence and the item it is working on.
struct Feed {
  int idx;       // index of the current item
  int fetch;     // items taken from the ring so far (dynamic form)
  int m0, n0, kb0, kb1;
};

// First item of a role: the pair's own index in both forms.
template <bool kDynamic, class ItemF>
__device__ __forceinline__ bool feed_first(Feed& f, int pair, int n_pairs, int n_items, const ItemF& itemf) {
  f.fetch = 0;
  for (f.idx = pair; f.idx < n_items; f.idx += n_pairs) {
    if (itemf(f.idx, f.m0, f.n0, f.kb0, f.kb1)) return true;
    if constexpr (kDynamic) break;
  }
  return false;
}
// The next item.  All lanes of a calling warp must call it together when `whole_warp`; lane 0 then signals the slot free.
template <bool kDynamic, class ItemF>
__device__ __forceinline__ bool feed_next(Feed& f, int n_pairs, int n_items, const ItemF& itemf, SchedRing* ring,
                                          bool whole_warp, bool& ok) {
  if constexpr (!kDynamic) {
    for (f.idx += n_pairs; f.idx < n_items; f.idx += n_pairs)
      if (itemf(f.idx, f.m0, f.n0, f.kb0, f.kb1)) return true;
    return false;
  } else {
    const int slot = f.fetch & 1;
    const uint32_t phase = (uint32_t)(f.fetch >> 1) & 1u;
    ++f.fetch;
    if (!mbar_wait_cluster(&ring->full[slot], phase)) { ok = false; return false; }
    int4 it;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(it.x), "=r"(it.y), "=r"(it.z), "=r"(it.w)
                 : "r"(umma::smem_u32(&ring->item[slot])) : "memory");
    f.idx = *reinterpret_cast<volatile int*>(&ring->idx[slot]);
    if (whole_warp) __syncwarp();
    if (!whole_warp || (threadIdx.x & 31) == 0)
      umma::mbar_arrive_cluster(umma::map_to_cta(umma::smem_u32(&ring->empty[slot]), 0));
    f.m0 = it.x; f.n0 = it.y; f.kb0 = it.z; f.kb1 = it.w;
    return f.idx >= 0;
  }
}

template <class Traits, class ItemF, class EpiF, bool kDynamic>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(threads_of(kDynamic), 1)
umma_pipe2_kernel(const __grid_constant__ typename Traits::Maps maps, const int n_items, const ItemF itemf,
                  const EpiF epi, int* dev_info) {
  using namespace umma;
  constexpr int STAGES = Traits::STAGES;
  constexpr int STAGE_BYTES = Traits::STAGE_BYTES;     // per CTA
  constexpr int CHUNK_KB = Traits::CHUNK_KB;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* epi_smem = tiles + (size_t)STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(epi_smem + epi_smem_of<Traits>::value);
  uint64_t* full = bars;
  uint64_t* empty = bars + STAGES;
  uint64_t* acc_full = bars + 2 * STAGES;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  SchedRing* ring = reinterpret_cast<SchedRing*>(reinterpret_cast<uint8_t*>(acc_empty + 2) + 16);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 2 * kEpiWarps); }
    if constexpr (kDynamic) {
      for (int a = 0; a < 2; ++a) { mbar_init(&ring->full[a], 1); mbar_init(&ring->empty[a], kSchedConsumers); }
      mbar_init(&ring->clc_bar, 1);
      mbar_init(&ring->go, 1);
      // Clusters that start after a wait has run out anywhere in this launch do nothing: otherwise every
      // remaining item of a broken launch would sit through its own time limit.
      ring->abort = (dev_info != nullptr && *reinterpret_cast<volatile int*>(dev_info) == GPTQ_ERR_TIMEOUT) ? 1 : 0;
    }
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
  bool abort = false;
  if constexpr (kDynamic) {
    uint32_t a;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(a) : "r"(map_to_cta(smem_u32(&ring->abort), 0)) : "memory");
    abort = a != 0;
  }

  if (abort) {
    // nothing: fall through to the closing barriers
  } else if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      Feed f;
      for (bool have = feed_first<kDynamic>(f, pair, n_pairs, n_items, itemf); have && ok;
           have = feed_next<kDynamic>(f, n_pairs, n_items, itemf, ring, false, ok)) {
        if constexpr (kDynamic) { if (rank == 0) mbar_arrive(&ring->go); }
        const int idx = f.idx, m0 = f.m0, n0 = f.n0, kb0 = f.kb0, kb1 = f.kb1;
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
      Feed f;
      for (bool have = feed_first<kDynamic>(f, pair, n_pairs, n_items, itemf); have && ok;
           have = feed_next<kDynamic>(f, n_pairs, n_items, itemf, ring, false, ok)) {
        const int kb0 = f.kb0, kb1 = f.kb1;
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
  } else if (warp < 2 + kEpiWarps) {
    // ------------------------------------------------------------------ epilogue (both CTAs, own rows)
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    Feed f;
    for (bool have = feed_first<kDynamic>(f, pair, n_pairs, n_items, itemf); have && ok;
         have = feed_next<kDynamic>(f, n_pairs, n_items, itemf, ring, true, ok)) {
      const int m0 = f.m0, n0 = f.n0, kb0 = f.kb0, kb1 = f.kb1;
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
      if constexpr (is_tile_epilogue<EpiF>::value) {
        static_assert(epi_smem_of<Traits>::value >= kEpiWarps * 4096, "tile epilogue: 4 KB of staging per epilogue warp");
#pragma unroll
        for (int c = 0; c < 4; ++c)
          epi.tile(maps, epi_smem + (warp - 2) * 4096, m0 + BM_CTA * (int)rank + q * 32, n0 + half * 128 + 32 * c,
                   *reinterpret_cast<const float(*)[32]>(&sum[32 * c]), lane);
      } else {
        const int row = m0 + BM_CTA * (int)rank + q * 32 + lane;
#pragma unroll
        for (int c = 0; c < 4; ++c)
          epi(row, n0 + half * 128 + 32 * c, *reinterpret_cast<const float(*)[32]>(&sum[32 * c]));
      }
    }
    if constexpr (is_tile_epilogue<EpiF>::value) { if (lane == 0) bulk_group_wait_all(); }
  } else if constexpr (kDynamic) {
    // ------------------------------------------------------------------ work-item scheduler (leader only)
    if (lane == 0 && rank == 0) {
      for (int k = 0;; ++k) {
        const int slot = k & 1;
        const uint32_t phase = (uint32_t)(k >> 1) & 1u;
        // every consumer of both CTAs has read what this slot held two items ago
        if (!mbar_wait_cluster(&ring->empty[slot], phase ^ 1)) { report_error(dev_info, GPTQ_ERR_TIMEOUT, 25); break; }
        if (!mbar_wait(&ring->go, (uint32_t)k & 1u)) { report_error(dev_info, GPTQ_ERR_TIMEOUT, 27); break; }
        mbar_arrive_expect_tx(&ring->clc_bar, 16);
        clc_try_cancel(&ring->clc_response, &ring->clc_bar);
        if (!mbar_wait(&ring->clc_bar, (uint32_t)k & 1u)) { report_error(dev_info, GPTQ_ERR_TIMEOUT, 26); break; }
        const int first_cta = clc_decode(&ring->clc_response);
        fence_proxy_async();              // the answer is read before the next request may overwrite it
        int next = first_cta < 0 ? -1 : (first_cta >> 1);
        int4 it = make_int4(0, 0, 0, 0);
        if (next >= n_items || (next >= 0 && !itemf(next, it.x, it.y, it.z, it.w))) it.w = it.z;   // (an empty item)
        ring->idx[slot] = next;
        ring->item[slot] = it;
        st_cluster_u32(map_to_cta(smem_u32(&ring->idx[slot]), 1), (uint32_t)next);
        st_cluster_v4(map_to_cta(smem_u32(&ring->item[slot]), 1), it);
        mbar_arrive_cluster(map_to_cta(smem_u32(&ring->full[slot]), 0));
        mbar_arrive_cluster(map_to_cta(smem_u32(&ring->full[slot]), 1));
        if (next < 0) break;              // after a failed request no further one may be issued
      }
    }
  }
  fence_before_thread_sync();
  __syncthreads();
  cluster_sync();                       // the peer is done with this CTA's shared memory and barriers
  if (warp == 1) { fence_after_thread_sync(); tmem_dealloc_pair(tmem_base, 512); }
}

constexpr size_t kBarrierBytes = 512;    // pipeline barriers, TMEM slot and the scheduler ring behind the stages

// Static form: a persistent grid of at most one CTA pair per two SMs (less `reserve_sms`, left free for kernels
// running beside this one); pair p takes items p, p + pairs, ...
template <class Traits, class ItemF, class EpiF>
gptq_status_t launch_pipe2(const typename Traits::Maps& maps, int64_t n_items, ItemF itemf, EpiF epi, int* dev_info,
                           cudaStream_t stream, int reserve_sms = 0) {
  if (n_items <= 0) return GPTQ_OK;
  if (n_items > 0x7FFFFFFF) return GPTQ_ERR_UNSUPPORTED;
  constexpr size_t smem = (size_t)Traits::STAGES * Traits::STAGE_BYTES + epi_smem_of<Traits>::value + 1024 + kBarrierBytes;
  int pairs_max = (device_sm_count() - reserve_sms) / 2;
  if (pairs_max < 1) pairs_max = 1;
  const int pairs = (int)(n_items < pairs_max ? n_items : pairs_max);
  auto kern = umma_pipe2_kernel<Traits, ItemF, EpiF, false>;
  GPTQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<2 * pairs, threads_of(false), smem, stream>>>(maps, (int)n_items, itemf, epi, dev_info);
  GPTQ_LAUNCH_CHECK();
  return GPTQ_OK;
}

// Dynamic form: one cluster per item; the running clusters take the items in index order (see above).
template <class Traits, class ItemF, class EpiF>
gptq_status_t launch_pipe2_dynamic(const typename Traits::Maps& maps, int64_t n_items, ItemF itemf, EpiF epi,
                                   int* dev_info, cudaStream_t stream) {
  if (n_items <= 0) return GPTQ_OK;
  if (n_items > 0x3FFFFFFF) return GPTQ_ERR_UNSUPPORTED;
  constexpr size_t smem = (size_t)Traits::STAGES * Traits::STAGE_BYTES + epi_smem_of<Traits>::value + 1024 + kBarrierBytes;
  auto kern = umma_pipe2_kernel<Traits, ItemF, EpiF, true>;
  GPTQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<(unsigned)(2 * n_items), threads_of(true), smem, stream>>>(maps, (int)n_items, itemf, epi, dev_info);
  GPTQ_LAUNCH_CHECK();
  return GPTQ_OK;
}

}  // namespace pipe2
}  // namespace gptq
