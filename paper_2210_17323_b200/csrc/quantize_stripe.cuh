// Row-stripe form of Algorithm 1's loops inside one outer block (included by quantize.cu, inside its
// namespace, after GridSpec / find_params).
//
// Rows of W are independent sub-problems (Section 2), so one CTA can own a stripe of 128 rows for a whole
// outer block of columns and run every inner block of it back to back with no other CTA involved:
//   for each inner block of B columns (the caller's block size, Section 3, Step 2):
//     (1) for each 16 columns of it: quantize them one after the other with immediate error feedback
//         (Algorithm 1's inner loop) -- ONE THREAD PER ROW, fp64, the 16 columns in registers -- then push
//         their 16 errors onto the rest of the block, which sits in shared memory;
//     (2) push the block's errors onto the remaining columns of the outer block for the stripe's rows
//         (Algorithm 1's lazy update, W[:, rest] -= E U[block, rest]).
// (The pushes of (1) accumulate in TMEM over the sub-blocks of a block; a thread subtracts the sum from its next 16
// columns when it reaches them, so the slab itself is never rewritten.)
// Both pushes are products of the stripe's errors with a panel of U and run on the tensor cores: the row
// threads write their scaled errors as an fp16 hi / lo pair into a 128-byte-swizzled K-major tile, which is
// the M = 128 left operand of tcgen05.mma (kind::f16, three products per term as in gemm_umma_f16.cuh);
// the scaled panel of U comes from the transposed fp16 pair quantize.cu prepares -- for (2) by TMA in
// 64-column tiles, for (1) as a small 16-deep slice copied with cp.async into the unswizzled core-matrix
// layout.  Sums form in TMEM (3 MMAs for (1), at most 24 for (2)), are read back with tcgen05.ld by the row
// threads, scaled, and subtracted: in (1) from the thread's own row of the shared-memory slab, in (2) from
// the fp64 working weights in global memory, through a shared-memory buffer and one bulk reduction
// (cp.reduce.async.bulk add.f64) per 32 columns, so that no thread waits for a memory round trip.
// The whole outer block is one launch instead of two per inner block, and nothing in it waits for another
// CTA.  Left-looking updates ACROSS outer blocks stay with the large two-CTA contraction.
//
// Threads: warps 0-3 own the rows (thread t <-> row t <-> TMEM lane t); warp 4 issues TMA and MMA.
#pragma once

constexpr int kStripeRows = 128;
constexpr int kStripeThreads = 160;
constexpr int kStripeSB = 16;                 // columns held in registers at a time
constexpr int kStripeMaxB = 128;              // widest inner block this form takes
constexpr int kStripeNT = 64;                 // columns of update (2) per TMEM accumulator / staged panel tile
constexpr int kStripeLD = kStripeRows;        // slab row stride (doubles): the slab is a verbatim copy of the stripe's columns
constexpr int kStripeMaxNb2 = 2048;           // widest outer block this form takes

struct StripeMaps { CUtensorMap p_hi, p_lo; };   // Pt[c - i2][k] of the outer block: boxes of 64 k x 64 columns

// Working weights of the outer block in STRIPE-MAJOR order: element (row, col) at ((row / 128) * ldw + col) * 128 + row % 128,
// so that the 128 row threads of a stripe read and write one column of it as 1 KB of consecutive doubles.
struct StripeArgs {
  double* Wblk; int64_t ldw; int nb2;         // working weights of the outer block (stripe-major, see above), its width
  const float* U; int C; int i2;              // first global column of the outer block
  int B;                                      // inner block width: multiple of 32, <= kStripeMaxB
  int R; GridSpec grid; int group;
  float* scales; float* zeros; int G;
  __half* Ehi; __half* Elo;                   // scaled errors E' (see quantize.cu), all columns
  const __half* Phi; const __half* Plo; int64_t ldp;   // scaled transposed panel of U: Pt[c - i2][k] (see quantize.cu)
  const float* sK; const float* sE; const float* sEinv; const float* sCinv;
  uint8_t* codes; double* loss; int* dev_info;
  int keep_errors;                            // 1: the scaled errors also go to Ehi / Elo in global memory (the left operand of
                                              // later outer blocks' contractions); 0: factor form, a separate kernel writes the
                                              // plain residuals there from the codes
};

// shared memory (from a 1024-byte aligned base):
//   [0, 64 KB)      E' tile: hi then lo, each two 64-wide K atoms of [128 rows][128 bytes], 128-byte swizzled
//   [64 KB, ...)    slab [B][kStripeLD] doubles; in phase (2) the same space holds two panel stages of 32 KB
//                   (hi and lo, each two K atoms of [64 columns][128 bytes]) and two 32 KB buffers of update values
//                   ([32 columns][128 rows] doubles) on their way to memory
//   then            Ud [B / 16][16][16] doubles (the 16 x 16 diagonal blocks of U), rdiag [B] doubles, sks [B] floats,
//                   two buffers for the 16-deep panel slices of (1) (hi and lo, [<= 112 columns][16 k] fp16 as 8 x 16-byte
//                   core matrices), barriers, TMEM slot
constexpr int kStripeETile = 65536;
constexpr int kStripeStage = 32768;
constexpr int kStripeDelta = 32768;
constexpr int kStripeSlice = (kStripeMaxB - kStripeSB) * kStripeSB * 2;   // 3584 bytes: one of hi / lo
__host__ __device__ constexpr size_t stripe_slab_bytes(int B) {
  return ((((size_t)B * kStripeLD * 8 > 2 * (size_t)(kStripeStage + kStripeDelta) ? (size_t)B * kStripeLD * 8
                                                                                  : 2 * (size_t)(kStripeStage + kStripeDelta)) + 1023) / 1024) * 1024;
}
__host__ __device__ constexpr size_t stripe_smem(int B) {
  return 1024 + kStripeETile + stripe_slab_bytes(B) + (size_t)B * kStripeSB * 8 + (size_t)B * 8 + (size_t)B * 4 +
         4 * (size_t)kStripeSlice + 256;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// Adds `bytes` of doubles in shared memory onto global memory (element-wise, performed by the memory system; no value comes
// back, so nothing waits for a round trip).  Both addresses 16-byte aligned, bytes a multiple of 16.  Issued by one thread.
__device__ __forceinline__ void bulk_reduce_add_f64(double* gdst, const void* ssrc, uint32_t bytes) {
  asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f64 [%0], [%1], %2;"
               ::"l"(gdst), "r"((uint32_t)__cvta_generic_to_shared(ssrc)), "r"(bytes) : "memory");
}
// Copies `bytes` (a multiple of 16, both addresses 16-byte aligned) from global to this CTA's shared memory; the bytes are
// credited to `bar`.  Issued by one thread.
__device__ __forceinline__ void bulk_copy_g2s(void* sdst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"((uint32_t)__cvta_generic_to_shared(sdst)), "l"(gsrc), "r"(bytes), "r"((uint32_t)__cvta_generic_to_shared(bar)) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void row_threads_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// 32 lanes x 16 consecutive fp32 columns of TMEM (warp w reads lanes 32 * (w % 4) ..)
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
// Shared-memory matrix descriptor of an UNSWIZZLED K-major operand: core matrices of 8 rows x 16 bytes, `k_step` bytes
// apart along K and `mn_step` bytes apart along M / N.
__device__ __forceinline__ uint64_t make_desc_plain(uint32_t saddr, uint32_t k_step, uint32_t mn_step) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((k_step >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((mn_step >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}

// Out-of-line pieces of the column loop (kept out of the unrolled body so that it stays small).
__device__ __noinline__ double exact_rne_quotient(double w, double scale) { return rint(w / scale); }
__device__ __noinline__ float2 find_params_outofline(double mn, double mx, GridSpec g) {
  float2 r;
  find_params(mn, mx, g, r.x, r.y);
  return r;
}

#ifdef GPTQ_EXP_TIMING
__device__ unsigned long long g_stripe_dbg[32];
#define TICK(var) const long long var = clock64()
#define TOCK(slot, var) do { if (blockIdx.x == 0 && (t == 0 || t == 128)) atomicAdd(&g_stripe_dbg[(slot) + (t == 128 ? 16 : 0)], (unsigned long long)(clock64() - (var))); } while (0)
#else
#define TICK(var)
#define TOCK(slot, var)
#endif

__global__ void __launch_bounds__(kStripeThreads, 1)
stripe_kernel(const __grid_constant__ StripeMaps maps, const StripeArgs a) {
  using namespace umma;
  constexpr int LD = kStripeLD;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int B = a.B;
  uint8_t* etile = base;                                                 // E' hi (32 KB) | E' lo (32 KB)
  uint8_t* stages = base + kStripeETile;                                 // phase (2): two panel stages
  double* delta = reinterpret_cast<double*>(stages + 2 * kStripeStage);  // phase (2): two buffers of update values [32][128]
  double* slab = reinterpret_cast<double*>(stages);                      // phase (1): [B][LD]
  double* Ud = reinterpret_cast<double*>(stages + stripe_slab_bytes(B)); // [B / 16][16][16]
  double* rdiag = Ud + (size_t)B * kStripeSB;                            // [B]
  float* sks = reinterpret_cast<float*>(rdiag + B);                      // [B]
  uint8_t* slices = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(sks + B) + 127) & ~(uintptr_t)127);   // [2][hi, lo][kStripeSlice]
  uint64_t* bars = reinterpret_cast<uint64_t*>(slices + 4 * kStripeSlice);
  uint64_t* full = bars;            // [2] TMA -> MMA
  uint64_t* empty = bars + 2;       // [2] MMA -> TMA
  uint64_t* acc_full = bars + 4;    // [2] MMA -> row threads
  uint64_t* acc_empty = bars + 6;   // [2] row threads -> MMA
  uint64_t* push_done = bars + 8;   // [1] MMA of a 16-column push -> row threads
  uint64_t* slab_full = bars + 9;   // [1] bulk copy of the slab -> row threads
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 10);

  const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
  const bool row_thread = warp < 4;
  const int r0 = blockIdx.x * kStripeRows, row = r0 + t;
  const bool live = row_thread && row < a.R;
  const int G = a.G, g = a.group;

  if (t == 0) {
    for (int s = 0; s < 2; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 4); }
    mbar_init(push_done, 1); mbar_init(slab_full, 1);
    fence_barrier_init();
    fence_proxy_async();
    prefetch_tmap(&maps.p_hi); prefetch_tmap(&maps.p_lo);
  }
  if (warp == 4) { tmem_alloc(tmem_slot, 256); tmem_relinquish(); }     // [0, 128) two accumulators of (2); [128, 256) the one of (1)
  fence_before_thread_sync();
  __syncthreads();
  fence_after_thread_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_lane = (uint32_t)((warp & 3) * 32) << 16;

  const float se_row = live ? a.sE[row] : 1.f;
  const double inv_se = live ? (double)a.sEinv[row] : 0.0;
  const double maxq = (double)a.grid.maxq;
  float scale_f = 1.f, zero_f = 0.f;
  if (live && g <= 0) { scale_f = a.scales[row]; zero_f = a.zeros[row]; }
  double scale = (double)scale_f, zero = (double)zero_f, rscale = 1.0 / scale;
  double loss = 0.0;
  bool bad = false;
  // columns of a 16-column sub-block at which a small group (4, 8 or 16 columns) starts
  const uint32_t small_group_starts = g == 4 ? 0x1111u : (g == 8 ? 0x0101u : (g == 16 ? 0x0001u : 0u));
  // pipeline state, carried across inner blocks
  int stage = 0; uint32_t stage_phase = 0;       // warp 4, lane 0: next stage to fill
  int acc = 0; uint32_t acc_phase = 0;           // everyone: next accumulator of (2)
  uint32_t push_phase = 0;                       // everyone: phase of push_done
  uint32_t slab_phase = 0;                       // everyone: phase of slab_full
  int dbuf = 0;                                  // row threads: next buffer of update values
  bool ok = true;

  for (int ib = 0; ib < a.nb2; ib += B) {                 // inner blocks of this outer block
    const int i = a.i2 + ib;                              // first global column of the inner block
    const int Bc = min(B, a.nb2 - ib);                    // its width (the last one of the matrix may be short)
    // ---------------------------------------------------------------- (1) the inner block, one thread per row
    if (t == 0) { bulk_wait<0>(); fence_proxy_async_all(); }   // the previous block's reductions into Wblk have been performed
    __syncthreads();                                      // phase (2) of the previous block is done with the shared buffers,
                                                          // and its updates to Wblk are visible to the whole CTA
    TICK(ts0);
    // 16-deep slice of the scaled panel for the push of sub-block s: Pt rows = the block's columns after the sub-block,
    // k = the sub-block's 16 columns; 16-byte pieces into 8 x 16-byte core matrices (K halves 128 B apart, 8-column groups
    // 256 B apart)
    auto stage_slice = [&](int s) {
      const int rem = Bc - 16 * (s + 1);
      uint8_t* dst = slices + (size_t)(s & 1) * 2 * kStripeSlice;
      for (int e = t; e < rem * 4; e += kStripeThreads) {
        const int c = e >> 2, kh = (e >> 1) & 1, hl = e & 1;
        const __half* src = (hl ? a.Plo : a.Phi) + (int64_t)(ib + 16 * (s + 1) + c) * a.ldp + i + 16 * s + 8 * kh;
        cp_async16(dst + hl * kStripeSlice + (c >> 3) * 256 + kh * 128 + (c & 7) * 16, src);
      }
    };
    stage_slice(0);
    if (t == 0) {
      // the block's columns of the stripe are Bc KB of consecutive doubles in memory and in the slab: bulk copies of 16 KB
      const double* src = a.Wblk + ((int64_t)blockIdx.x * a.ldw + ib) * kStripeRows;
      mbar_arrive_expect_tx(slab_full, (uint32_t)Bc * kStripeRows * 8);
      for (int c0 = 0; c0 < Bc; c0 += 16)
        bulk_copy_g2s(slab + (size_t)c0 * LD, src + (int64_t)c0 * kStripeRows, 16 * kStripeRows * 8, slab_full);
    }
    {
      // the 16 x 16 diagonal blocks of U of this inner block as doubles, 1 / U_jj and sK: loads first, then stores
      constexpr int PER = (kStripeMaxB * 4 + kStripeThreads - 1) / kStripeThreads;
      const int total = Bc * 4;                            // float4 pieces: (sub-block, row, quarter)
      float4 u4[PER];
#pragma unroll
      for (int it = 0; it < PER; ++it) {
        const int e = t + it * kStripeThreads, jr = e >> 2, q = e & 3;      // jr: row inside the block
        u4[it] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e < total) u4[it] = *reinterpret_cast<const float4*>(a.U + (int64_t)(i + jr) * a.C + i + (jr & ~15) + 4 * q);
      }
#pragma unroll
      for (int it = 0; it < PER; ++it) {
        const int e = t + it * kStripeThreads, jr = e >> 2, q = e & 3;
        if (e < total) {
          const float4 u = u4[it];
          double* d = Ud + jr * kStripeSB + 4 * q;
          d[0] = (double)u.x; d[1] = (double)u.y; d[2] = (double)u.z; d[3] = (double)u.w;
          const int dj = (jr & 15) - 4 * q;
          if (dj >= 0 && dj < 4) rdiag[jr] = 1.0 / (double)(dj == 0 ? u.x : (dj == 1 ? u.y : (dj == 2 ? u.z : u.w)));
        }
      }
      for (int c = t; c < Bc; c += kStripeThreads) sks[c] = a.sK[i + c];
    }
    // grid of a group wider than the block, starting here: min / max of the row's CURRENT weights (Section 5)
    if (g > B && (i % g) == 0 && row_thread) {
      double mn = INFINITY, mx = -INFINITY;
      if (live) {
        const double* p = a.Wblk + ((int64_t)blockIdx.x * a.ldw + ib) * kStripeRows + t;
        for (int c = 0; c < g; c += 4) {
          const double v0 = p[(int64_t)c * kStripeRows], v1 = p[(int64_t)(c + 1) * kStripeRows];
          const double v2 = p[(int64_t)(c + 2) * kStripeRows], v3 = p[(int64_t)(c + 3) * kStripeRows];
          mn = fmin(fmin(mn, fmin(v0, v1)), fmin(v2, v3)); mx = fmax(fmax(mx, fmax(v0, v1)), fmax(v2, v3));
        }
      }
      const float2 sz = find_params_outofline(mn, mx, a.grid);
      scale_f = sz.x; zero_f = sz.y;
      scale = (double)scale_f; zero = (double)zero_f; rscale = 1.0 / scale;
      if (live) { a.scales[(int64_t)row * G + i / g] = scale_f; a.zeros[(int64_t)row * G + i / g] = zero_f; }
    }   // (a wide group that started in an earlier inner block of this launch: its grid is still in registers)
    if (ok && !mbar_wait(slab_full, slab_phase)) { if (t == 0) report_error(a.dev_info, GPTQ_ERR_TIMEOUT, 37); ok = false; }
    slab_phase ^= 1;
    __syncthreads();                                      // slab, Ud, rdiag, sks staged
    TOCK(0, ts0);

    for (int j0 = 0; j0 < Bc; j0 += kStripeSB) {
      const int s = j0 >> 4, rem = Bc - j0 - kStripeSB;   // columns of the block after this sub-block
      if (row_thread) {
        TICK(ts2);
        // grid of a group that starts at this sub-block and lies inside the block (a multiple of 32 columns)
        if (g >= 32 && g <= B && ((i + j0) % g) == 0) {
          double mn = INFINITY, mx = -INFINITY;
          for (int c = j0; c < j0 + g; c += 16) {           // current weights = slab - accumulated pushes (none yet at j0 = 0)
            float v[16];
            if (j0 > 0) { tmem_ld_32x16(tmem_base + tmem_lane + 128 + c, v); tmem_ld_wait(); }
#pragma unroll
            for (int m = 0; m < 16; ++m) {
              double x = slab[(c + m) * LD + t];
              if (j0 > 0) x -= (double)(v[m] * __ldg(a.sCinv + i + c + m)) * inv_se;
              mn = fmin(mn, x); mx = fmax(mx, x);
            }
          }
          const float2 sz = find_params_outofline(mn, mx, a.grid);
          scale_f = sz.x; zero_f = sz.y;
          scale = (double)scale_f; zero = (double)zero_f; rscale = 1.0 / scale;
          if (live) { a.scales[(int64_t)row * G + (i + j0) / g] = scale_f; a.zeros[(int64_t)row * G + (i + j0) / g] = zero_f; }
        }
        double w[kStripeSB], err[kStripeSB];
#pragma unroll
        for (int m = 0; m < kStripeSB; ++m) w[m] = slab[(j0 + m) * LD + t];
        if (j0 > 0) {
          // minus the pushes of all earlier sub-blocks of this block, which accumulate in TMEM (column j of the block in
          // accumulator column j): sum / (sE[row] sC[column])
          float v[16];
          tmem_ld_32x16(tmem_base + tmem_lane + 128 + j0, v);
          tmem_ld_wait();
          const float* sci = a.sCinv + i + j0;
#pragma unroll
          for (int m = 0; m < kStripeSB; ++m) w[m] -= (double)(v[m] * __ldg(sci + m)) * inv_se;
        }
        uint32_t cw[kStripeSB / 4];
#pragma unroll
        for (int m = 0; m < kStripeSB / 4; ++m) cw[m] = 0;

        const double* ud = Ud + (size_t)j0 * kStripeSB;    // this sub-block's 16 x 16 block of U
#pragma unroll
        for (int jj = 0; jj < kStripeSB; ++jj) {
          if ((jj & 3) == 0 && ((small_group_starts >> jj) & 1u)) {   // small groups (4, 8, 16) live inside the registers
            double mn = INFINITY, mx = -INFINITY;
#pragma unroll
            for (int m = 0; m < kStripeSB; ++m)
              if (m >= jj && m < jj + g) { mn = fmin(mn, w[m]); mx = fmax(mx, w[m]); }
            const float2 sz = find_params_outofline(mn, mx, a.grid);
            scale_f = sz.x; zero_f = sz.y;
            scale = (double)scale_f; zero = (double)zero_f; rscale = 1.0 / scale;
            if (live) {
              const int gi = (i + j0 + jj) / g;
              a.scales[(int64_t)row * G + gi] = scale_f; a.zeros[(int64_t)row * G + gi] = zero_f;
            }
          }
          const double wj = w[jj];
          // code of this weight: rne(w / scale), the quotient formed with the reciprocal; only when it lands within
          // 1e-6 of a tie (where the reciprocal's last-bit error could change the rounding) is the division done
          const double tq = wj * rscale;
          double q = rint(tq);
          if (fabs(fabs(tq - q) - 0.5) < 1e-6) q = exact_rne_quotient(wj, scale);
          q += zero;
          q = fmin(fmax(q, 0.0), maxq);
          const double wq = scale * (q - zero);
          const double e = (wj - wq) * rdiag[j0 + jj];     // scaled error (w - q) / U_jj
          err[jj] = e;
          loss += e * e;
          bad |= !isfinite(e);
          cw[jj >> 2] |= (uint32_t)q << (8 * (jj & 3));
          const double* urow = ud + jj * kStripeSB;
#pragma unroll
          for (int m = 0; m < kStripeSB; ++m)             // immediate feedback onto the later columns in registers
            if (m > jj) w[m] -= e * urow[m];
        }
        if (!live) {
#pragma unroll
          for (int jj = 0; jj < kStripeSB; ++jj) err[jj] = 0.0;
          loss = 0.0; bad = false;
        }
        TOCK(2, ts2);
        TICK(ts4);
        // scaled errors as an fp16 hi / lo pair: into the swizzled K-major tile (row t, 16-byte chunk (k / 8) ^ (t & 7) of
        // the 128-byte row of K atom k / 64) and to global memory for the left-looking contractions of later outer blocks;
        // codes as bytes
        uint32_t hw[kStripeSB / 2], lw[kStripeSB / 2];
        bool sat = false;
#pragma unroll
        for (int u = 0; u < kStripeSB; u += 2) {
          __half h0, l0, h1, l1;
          f16x3::split_f16((float)err[u] * sks[j0 + u] * se_row, h0, l0, sat);
          f16x3::split_f16((float)err[u + 1] * sks[j0 + u + 1] * se_row, h1, l1, sat);
          hw[u >> 1] = (uint32_t)__half_as_ushort(h0) | ((uint32_t)__half_as_ushort(h1) << 16);
          lw[u >> 1] = (uint32_t)__half_as_ushort(l0) | ((uint32_t)__half_as_ushort(l1) << 16);
        }
        bad |= sat;
        const uint4 h_a = make_uint4(hw[0], hw[1], hw[2], hw[3]), h_b = make_uint4(hw[4], hw[5], hw[6], hw[7]);
        const uint4 l_a = make_uint4(lw[0], lw[1], lw[2], lw[3]), l_b = make_uint4(lw[4], lw[5], lw[6], lw[7]);
        const int atom = j0 >> 6, ch0 = (j0 & 63) >> 3;
        uint8_t* rowp = etile + atom * 16384 + t * 128;
        *reinterpret_cast<uint4*>(rowp + ((ch0 ^ (t & 7)) << 4)) = h_a;
        *reinterpret_cast<uint4*>(rowp + (((ch0 + 1) ^ (t & 7)) << 4)) = h_b;
        *reinterpret_cast<uint4*>(rowp + 32768 + ((ch0 ^ (t & 7)) << 4)) = l_a;
        *reinterpret_cast<uint4*>(rowp + 32768 + (((ch0 + 1) ^ (t & 7)) << 4)) = l_b;
        if (live) {
          const int64_t o = (int64_t)row * a.C + i + j0;
          uint4* gh = reinterpret_cast<uint4*>(a.Ehi + o);
          uint4* gl = reinterpret_cast<uint4*>(a.Elo + o);
          if (a.keep_errors) { gh[0] = h_a; gh[1] = h_b; gl[0] = l_a; gl[1] = l_b; }
          *reinterpret_cast<uint4*>(a.codes + o) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
        }
        TOCK(4, ts4);
      }
      if (rem <= 0) continue;                             // (uniform) last sub-block of the block: nothing left to push onto
      // ---- push the 16 errors onto the rest of the block: D = E'[:, sub-block] x (slice of the scaled panel)
      TICK(ts3);
      cp_async_wait_all();                                // this thread's pieces of the slice
      fence_proxy_async();                                // E' tile and slice were written through the generic proxy
      fence_before_thread_sync();                         // (the previous push's tcgen05.ld are done)
      __syncthreads();
      if (rem > kStripeSB) stage_slice(s + 1);            // next sub-block's slice, into the other buffer
      if (warp == 4 && lane == 0) {
        fence_after_thread_sync();
        const uint32_t idesc = make_idesc(kFmtF16, false, false, 128, rem);
        const uint32_t ea = smem_u32(etile) + (uint32_t)(s >> 2) * 16384 + (uint32_t)(s & 3) * 32;
        const uint32_t sl = smem_u32(slices + (size_t)(s & 1) * 2 * kStripeSlice);
        const uint64_t dah = make_desc_sw128(ea, 0, 1024), dal = make_desc_sw128(ea + 32768, 0, 1024);
        const uint64_t dbh = make_desc_plain(sl, 128, 256), dbl = make_desc_plain(sl + kStripeSlice, 128, 256);
        const uint32_t d_tmem = tmem_base + 128 + (uint32_t)(j0 + kStripeSB);   // accumulator column = column inside the block
        mma_f16(d_tmem, dal, dbh, idesc, s == 0 ? 0u : 1u);   // small terms first; the first sub-block's push initialises every column
        mma_f16(d_tmem, dah, dbl, idesc, 1u);
        mma_f16(d_tmem, dah, dbh, idesc, 1u);
        mma_commit(push_done);
      }
      if (row_thread) {
        if (ok && !mbar_wait(push_done, push_phase)) { if (lane == 0) report_error(a.dev_info, GPTQ_ERR_TIMEOUT, 36); ok = false; }
        fence_after_thread_sync();
      }
      push_phase ^= 1;
      TOCK(3, ts3);
    }

    // ---------------------------------------------------------------- (2) push the block's errors onto the rest of the outer block
    const int rest = a.nb2 - (ib + Bc);
    if (rest <= 0) continue;                              // (uniform across the CTA; otherwise Bc == B)
    TICK(ts5);
    fence_proxy_async();                                  // the E' tile (and the slab the stages overwrite) were written by plain stores
    fence_before_thread_sync();
    __syncthreads();
    TOCK(5, ts5);
    const int n_tiles = (rest + kStripeNT - 1) / kStripeNT;
    const int n_atoms = (B + 63) >> 6;                    // 64-wide K atoms in this block
    if (warp == 4) {
      if (lane == 0 && ok) {
        fence_after_thread_sync();
        constexpr uint32_t idesc = make_idesc(kFmtF16, false, false, 128, kStripeNT);
        auto load = [&](int tile, int st) {
          uint8_t* sp = stages + (size_t)st * kStripeStage;
          mbar_arrive_expect_tx(&full[st], (uint32_t)(n_atoms * 2 * 8192));
          for (int at = 0; at < n_atoms; ++at) {
            tma_load_2d(sp + at * 8192, &maps.p_hi, i + 64 * at, ib + B + tile * kStripeNT, &full[st]);
            tma_load_2d(sp + 16384 + at * 8192, &maps.p_lo, i + 64 * at, ib + B + tile * kStripeNT, &full[st]);
          }
        };
        int fill = stage; uint32_t fill_phase = stage_phase;
        // the stage ring is filled one tile ahead of the MMAs
        if (!mbar_wait(&empty[fill], fill_phase ^ 1)) { report_error(a.dev_info, GPTQ_ERR_TIMEOUT, 31); ok = false; }
        if (ok) load(0, fill);
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
          const int nf = fill ^ 1; const uint32_t nfp = fill_phase ^ (nf == 0 ? 1u : 0u);
          if (tl + 1 < n_tiles) {
            if (!mbar_wait(&empty[nf], nfp ^ 1)) { report_error(a.dev_info, GPTQ_ERR_TIMEOUT, 32); ok = false; break; }
            load(tl + 1, nf);
          }
          if (!mbar_wait(&full[fill], fill_phase)) { report_error(a.dev_info, GPTQ_ERR_TIMEOUT, 33); ok = false; break; }
          if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1)) { report_error(a.dev_info, GPTQ_ERR_TIMEOUT, 34); ok = false; break; }
          fence_after_thread_sync();
          TICK(tm3);
          const uint32_t d_tmem = tmem_base + (uint32_t)acc * kStripeNT;
          const uint32_t ea = smem_u32(etile), sb = smem_u32(stages + (size_t)fill * kStripeStage);
          for (int ks = 0; ks < B / 16; ++ks) {
            const uint32_t off = (uint32_t)(ks >> 2) * 16384 + (uint32_t)(ks & 3) * 32;
            const uint32_t offb = (uint32_t)(ks >> 2) * 8192 + (uint32_t)(ks & 3) * 32;
            const uint64_t dah = make_desc_sw128(ea + off, 0, 1024), dal = make_desc_sw128(ea + 32768 + off, 0, 1024);
            const uint64_t dbh = make_desc_sw128(sb + offb, 0, 1024), dbl = make_desc_sw128(sb + 16384 + offb, 0, 1024);
            mma_f16(d_tmem, dal, dbh, idesc, ks == 0 ? 0u : 1u);   // small terms first
            mma_f16(d_tmem, dah, dbl, idesc, 1u);
            mma_f16(d_tmem, dah, dbh, idesc, 1u);
          }
          mma_commit(&empty[fill]);
          mma_commit(&acc_full[acc]);
          TOCK(9, tm3);
          fill = nf; fill_phase = nfp;
          if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        stage = fill; stage_phase = fill_phase;
      } else {
        // the other lanes of warp 4 follow the accumulator sequence so that all threads agree on it
        for (int tl = 0; tl < n_tiles; ++tl) if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    } else {
      for (int tl = 0; tl < n_tiles && ok; ++tl) {
        TICK(te0);
        if (!mbar_wait(&acc_full[acc], acc_phase)) { if (lane == 0) report_error(a.dev_info, GPTQ_ERR_TIMEOUT, 35); ok = false; break; }
        fence_after_thread_sync();
        TOCK(6, te0);
        TICK(te1);
        const uint32_t t0 = tmem_base + tmem_lane + (uint32_t)(acc * kStripeNT);
        const int col_tile = ib + B + tl * kStripeNT;      // first column of this tile inside the outer block
#pragma unroll 1
        for (int c = 0; c < kStripeNT / 32; ++c) {
          if (col_tile + 32 * c >= a.nb2) break;           // (uniform across the row threads)
          float v[32];
          tmem_ld_32x32(t0 + 32 * c, v);
          tmem_ld_wait();
          // Wblk(row, columns) -= sum / (sE[row] sC[column]): the values go to a shared-memory buffer laid out like the
          // stripe in memory ([column][row], 32 KB) and are added to memory by one bulk reduction
          double* db = delta + (size_t)dbuf * (kStripeDelta / 8);
          if (t == 0) bulk_wait_read<1>();                 // the reduction issued from this buffer two rounds ago has read it
          row_threads_barrier();
          const float* sc = a.sCinv + a.i2 + col_tile + 32 * c;
#pragma unroll
          for (int u = 0; u < 32; ++u) db[u * kStripeRows + t] = -(double)(v[u] * __ldg(sc + u)) * inv_se;
          fence_proxy_async();
          row_threads_barrier();
          if (t == 0) {
            bulk_reduce_add_f64(a.Wblk + ((int64_t)blockIdx.x * a.ldw + col_tile + 32 * c) * kStripeRows, db, kStripeDelta);
            bulk_commit();
          }
          dbuf ^= 1;
        }
        TOCK(7, te1);
        fence_before_thread_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[acc]);
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
  }
  if (row_thread) {
    for (int o = 16; o > 0; o >>= 1) loss += __shfl_down_sync(0xffffffffu, loss, o);
    if (lane == 0 && loss != 0.0) atomicAdd(a.loss, loss);
    if (live && bad) report_error(a.dev_info, GPTQ_ERR_NONFINITE, row);
  }
  if (t == 0) bulk_wait<0>();                             // the last reductions have read their shared-memory buffers
  fence_before_thread_sync();
  __syncthreads();
  if (warp == 4) { fence_after_thread_sync(); tmem_dealloc(tmem_base, 256); }
}
