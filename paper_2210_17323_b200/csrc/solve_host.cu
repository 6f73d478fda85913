// Whole layer solve from HOST buffers: streams the calibration activations to the device in token
// chunks (double-buffered on a second stream so the copy of chunk k+1 overlaps the Hessian
// accumulation of chunk k), runs the three stages, and copies the results back.
// The stages themselves are the same entry points a device-side caller uses (Algorithm 1; Section 2).
#include "common.cuh"

namespace gptq {
namespace {

constexpr int64_t kChunkBytes = (int64_t)2048 << 20;  // per X staging buffer: every chunk costs one pass over H (read + write)

struct HostWs {
  float* H; float* U; __half* W; __nv_bfloat16* X[2];
  uint32_t* qweight; float* scales; float* zeros; double* loss; int* info;   // info: 3 x int[2]
  void* stage_ws; size_t stage_ws_bytes;
  int64_t chunk_tokens;
  size_t bytes;
};

inline int field_bits_h(int bits) { return bits == GPTQ_BITS_TERNARY ? 2 : bits; }

HostWs carve_host(void* ws, int R, int C, int64_t n_tokens, int n_grids, const int* bits_v, const int* group_v, int block) {
  WsCarver w(ws);
  HostWs o;
  int64_t ct = kChunkBytes / ((int64_t)C * 2);
  ct = ct / 64 * 64;
  if (ct < 64) ct = 64;
  if (ct > n_tokens) ct = n_tokens > 0 ? n_tokens : 1;
  o.chunk_tokens = ct;
  o.H = w.take<float>((size_t)C * C);
  o.U = w.take<float>((size_t)C * C);
  o.W = w.take<__half>((size_t)R * C);
  o.X[0] = w.take<__nv_bfloat16>((size_t)ct * C);
  o.X[1] = w.take<__nv_bfloat16>((size_t)ct * C);
  // one set of output buffers, sized for the widest grid, reused grid after grid
  int G = 1, f = 2;
  size_t s3 = 0;
  for (int i = 0; i < n_grids; ++i) {
    const int Gi = group_v[i] > 0 ? C / group_v[i] : 1;
    if (Gi > G) G = Gi;
    if (field_bits_h(bits_v[i]) > f) f = field_bits_h(bits_v[i]);
    const size_t q = gptq_quantize_workspace_bytes(R, C, bits_v[i], group_v[i], block);
    if (q > s3) s3 = q;
  }
  o.qweight = w.take<uint32_t>((size_t)R * (C * f / 32));
  o.scales = w.take<float>((size_t)R * G);
  o.zeros = w.take<float>((size_t)R * G);
  o.loss = w.take<double>(1);
  o.info = w.take<int>(8);
  size_t s1 = gptq_hessian_workspace_bytes(C, ct), s2 = gptq_prepare_hinv_workspace_bytes(C);
  o.stage_ws_bytes = s1 > s2 ? (s1 > s3 ? s1 : s3) : (s2 > s3 ? s2 : s3);
  if (o.stage_ws_bytes < kAlign) o.stage_ws_bytes = kAlign;
  o.stage_ws = w.take<unsigned char>(o.stage_ws_bytes);
  o.bytes = w.off;
  return o;
}

// First error wins across the Hessian calls of one solve: each call reports into `src` (which it clears
// first); a non-OK report is moved into `dst` unless `dst` already holds one.
__global__ void fold_info_kernel(int* __restrict__ dst, const int* __restrict__ src) {
  if (dst[0] == GPTQ_OK && src[0] != GPTQ_OK) { dst[1] = src[1]; dst[0] = src[0]; }
}

struct StreamGuard {
  cudaStream_t s = nullptr;
  cudaEvent_t loaded[2] = {nullptr, nullptr}, freed[2] = {nullptr, nullptr}, w_done = nullptr;
  ~StreamGuard() {
    for (int i = 0; i < 2; ++i) { if (loaded[i]) cudaEventDestroy(loaded[i]); if (freed[i]) cudaEventDestroy(freed[i]); }
    if (w_done) cudaEventDestroy(w_done);
    if (s) cudaStreamDestroy(s);
  }
};

}  // namespace
}  // namespace gptq

extern "C" size_t gptq_solve_layer_host_workspace_bytes(int R, int C, int64_t n_tokens, int bits, int group_size,
                                                        int block) {
  using namespace gptq;
  return gptq_solve_layer_host_grids_workspace_bytes(R, C, n_tokens, 1, &bits, &group_size, block);
}

extern "C" size_t gptq_solve_layer_host_grids_workspace_bytes(int R, int C, int64_t n_tokens, int n_grids, const int* bits,
                                                              const int* group_size, int block) {
  using namespace gptq;
  if (R <= 0 || C <= 0 || C % 32 != 0 || n_tokens < 0 || block <= 0 || n_grids <= 0 || !bits || !group_size) return 0;
  for (int i = 0; i < n_grids; ++i)
    if (gptq_quantize_workspace_bytes(R, C, bits[i], group_size[i], block) == 0) return 0;
  return carve_host(nullptr, R, C, n_tokens, n_grids, bits, group_size, block).bytes;
}

namespace gptq {
namespace {
gptq_status_t solve_layer_host_enqueue(const HostWs& w, StreamGuard& g, cudaStream_t s, const void* W_fp16_host,
                                       const void* X_bf16_host, int64_t n_tokens, int R, int C, float damp, int n_grids,
                                       const int* bits, const int* group_size, const int* sym, int block,
                                       uint32_t* const* qweight_host, float* const* scales_host, float* const* zeros_host,
                                       double* loss_host, int* info8_host);
}  // namespace
}  // namespace gptq

extern "C" gptq_status_t gptq_solve_layer_host(const void* W_fp16_host, const void* X_bf16_host, int64_t n_tokens,
                                               int R, int C, float damp, int bits, int group_size, int sym, int block,
                                               uint32_t* qweight_host, float* scales_host, float* zeros_host,
                                               double* loss_host, int* info_host, void* dev_ws, size_t dev_ws_bytes,
                                               void* stream) {
  return gptq_solve_layer_host_grids(W_fp16_host, X_bf16_host, n_tokens, R, C, damp, 1, &bits, &group_size, &sym, block,
                                     &qweight_host, &scales_host, &zeros_host, loss_host, info_host, dev_ws, dev_ws_bytes, stream);
}

extern "C" gptq_status_t gptq_solve_layer_host_grids(const void* W_fp16_host, const void* X_bf16_host, int64_t n_tokens,
                                                     int R, int C, float damp, int n_grids, const int* bits,
                                                     const int* group_size, const int* sym, int block,
                                                     uint32_t* const* qweight_host, float* const* scales_host,
                                                     float* const* zeros_host, double* loss_host, int* info_host,
                                                     void* dev_ws, size_t dev_ws_bytes, void* stream) {
  using namespace gptq;
  if (!W_fp16_host || !X_bf16_host || !qweight_host || !scales_host || !zeros_host || !loss_host || !info_host ||
      !bits || !group_size || !sym || n_grids <= 0 || R <= 0 || C <= 0 || C % 32 != 0 || n_tokens <= 0)
    return GPTQ_ERR_INVALID_ARG;
  for (int i = 0; i < n_grids; ++i)
    if (!qweight_host[i] || !scales_host[i] || !zeros_host[i]) return GPTQ_ERR_INVALID_ARG;
  const size_t need = gptq_solve_layer_host_grids_workspace_bytes(R, C, n_tokens, n_grids, bits, group_size, block);
  if (need == 0) return GPTQ_ERR_UNSUPPORTED;
  if (!dev_ws || !aligned_to(dev_ws, kAlign) || dev_ws_bytes < need) return GPTQ_ERR_WORKSPACE;
  HostWs w = carve_host(dev_ws, R, C, n_tokens, n_grids, bits, group_size, block);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  StreamGuard g;
  // the copy stream takes the caller's stream priority: of several calls in flight, the one on the higher-priority
  // stream gets its activations across first
  int prio = 0;
  GPTQ_CUDA_TRY(cudaStreamGetPriority(s, &prio));
  GPTQ_CUDA_TRY(cudaStreamCreateWithPriority(&g.s, cudaStreamNonBlocking, prio));
  for (int i = 0; i < 2; ++i) {
    GPTQ_CUDA_TRY(cudaEventCreateWithFlags(&g.loaded[i], cudaEventDisableTiming));
    GPTQ_CUDA_TRY(cudaEventCreateWithFlags(&g.freed[i], cudaEventDisableTiming));
  }
  GPTQ_CUDA_TRY(cudaEventCreateWithFlags(&g.w_done, cudaEventDisableTiming));

  int info[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  gptq_status_t st = solve_layer_host_enqueue(w, g, s, W_fp16_host, X_bf16_host, n_tokens, R, C, damp, n_grids, bits, group_size,
                                              sym, block, qweight_host, scales_host, zeros_host, loss_host, info);
  // Whatever happened, nothing of this call may still be in flight when it returns: the caller may free the host
  // buffers the copy stream reads, and the guard destroys that stream and its events.
  const cudaError_t e1 = cudaStreamSynchronize(s), e2 = cudaStreamSynchronize(g.s);
  if (st != GPTQ_OK) return st;
  if (e1 != cudaSuccess || e2 != cudaSuccess) return GPTQ_ERR_CUDA;
  info_host[0] = GPTQ_OK; info_host[1] = 0;
  for (int i = 0; i < 3; ++i)
    if (info[2 * i] != GPTQ_OK) { info_host[0] = info[2 * i]; info_host[1] = info[2 * i + 1]; break; }
  return GPTQ_OK;
}

namespace gptq {
namespace {
gptq_status_t solve_layer_host_enqueue(const HostWs& w, StreamGuard& g, cudaStream_t s, const void* W_fp16_host,
                                       const void* X_bf16_host, int64_t n_tokens, int R, int C, float damp, int n_grids,
                                       const int* bits, const int* group_size, const int* sym, int block,
                                       uint32_t* const* qweight_host, float* const* scales_host, float* const* zeros_host,
                                       double* loss_host, int* info8_host) {
  GPTQ_CUDA_TRY(cudaMemsetAsync(w.H, 0, (size_t)C * C * sizeof(float), s));
  GPTQ_CUDA_TRY(cudaMemsetAsync(w.info, 0, 8 * sizeof(int), s));
  const __nv_bfloat16* Xh = static_cast<const __nv_bfloat16*>(X_bf16_host);
  gptq_status_t st;
  // Chunks grow by a quarter each from 1/16 of the full chunk: the Hessian is under way after a few milliseconds, and a
  // chunk's copy does not outlast the accumulation of the chunk before it wherever accumulating is at least 1.25 x slower
  // than copying (wide layers); for narrow layers the copy is the bound either way.
  int k = 0;
  double grow = (double)w.chunk_tokens / 16.0;
  int64_t nt = 0;
  for (int64_t t0 = 0; t0 < n_tokens; t0 += nt, ++k) {
    const int b = k & 1;
    int64_t want = grow >= (double)w.chunk_tokens ? w.chunk_tokens : (int64_t)grow / 64 * 64;
    if (want < 64) want = 64;
    if (want > w.chunk_tokens) want = w.chunk_tokens;
    grow *= 1.25;
    nt = n_tokens - t0 < want ? n_tokens - t0 : want;
    if (k >= 2) GPTQ_CUDA_TRY(cudaStreamWaitEvent(g.s, g.freed[b], 0));       // buffer b consumed by chunk k-2
    GPTQ_CUDA_TRY(cudaMemcpyAsync(w.X[b], Xh + t0 * C, (size_t)nt * C * 2, cudaMemcpyHostToDevice, g.s));
    GPTQ_CUDA_TRY(cudaEventRecord(g.loaded[b], g.s));
    if (k == 0) {   // the weights ride behind the first chunk on the copy stream
      GPTQ_CUDA_TRY(cudaMemcpyAsync(w.W, W_fp16_host, (size_t)R * C * 2, cudaMemcpyHostToDevice, g.s));
      GPTQ_CUDA_TRY(cudaEventRecord(g.w_done, g.s));
    }
    GPTQ_CUDA_TRY(cudaStreamWaitEvent(s, g.loaded[b], 0));
    // every chunk reports into the spare slot info[6..7]; the first non-OK report is kept in info[0..1]
    // only the last chunk needs the pass that copies the upper triangle of H onto the lower one
    st = (t0 + nt < n_tokens ? gptq_hessian_accumulate_upper : gptq_hessian_accumulate)(w.H, w.X[b], nt, C, w.stage_ws, w.stage_ws_bytes,
                                                                                        w.info + 6, s);
    if (st != GPTQ_OK) return st;
    fold_info_kernel<<<1, 1, 0, s>>>(w.info, w.info + 6);
    GPTQ_LAUNCH_CHECK();
    GPTQ_CUDA_TRY(cudaEventRecord(g.freed[b], s));
  }
  GPTQ_CUDA_TRY(cudaStreamWaitEvent(s, g.w_done, 0));
  // Factor form (stage 2 without the rows of the inverse; same results, see gptq_prepare_factor) where stage 3 can run
  // it for every grid.
  bool factor = C > GPTQ_FACTOR_BLOCK && block > 0 && block <= 256 && GPTQ_FACTOR_BLOCK % block == 0;
  for (int gi = 0; gi < n_grids && factor; ++gi)
    if (group_size[gi] > block && GPTQ_FACTOR_BLOCK % group_size[gi] != 0) factor = false;
  st = factor ? gptq_prepare_factor(w.H, damp, C, w.U, w.stage_ws, w.stage_ws_bytes, w.info + 2, s)
              : gptq_prepare_hinv(w.H, damp, C, w.U, w.stage_ws, w.stage_ws_bytes, w.info + 2, s);
  if (st != GPTQ_OK) return st;
  // one Hessian and one factor serve every grid: quantize and copy back grid after grid (the device output buffers are
  // reused, the stream keeps a grid's copies ahead of the next grid's kernels)
  for (int gi = 0; gi < n_grids; ++gi) {
    st = (factor ? gptq_quantize_layer_factor : gptq_quantize_layer)(w.W, w.U, R, C, bits[gi], group_size[gi], sym[gi], block, w.qweight, w.scales, w.zeros, w.loss,
                             w.stage_ws, w.stage_ws_bytes, w.info + 6, s);
    if (st != GPTQ_OK) return st;
    fold_info_kernel<<<1, 1, 0, s>>>(w.info + 4, w.info + 6);
    GPTQ_LAUNCH_CHECK();
    const int G = group_size[gi] > 0 ? C / group_size[gi] : 1;
    GPTQ_CUDA_TRY(cudaMemcpyAsync(qweight_host[gi], w.qweight, (size_t)R * (C * field_bits_h(bits[gi]) / 32) * 4, cudaMemcpyDeviceToHost, s));
    GPTQ_CUDA_TRY(cudaMemcpyAsync(scales_host[gi], w.scales, (size_t)R * G * 4, cudaMemcpyDeviceToHost, s));
    GPTQ_CUDA_TRY(cudaMemcpyAsync(zeros_host[gi], w.zeros, (size_t)R * G * 4, cudaMemcpyDeviceToHost, s));
    GPTQ_CUDA_TRY(cudaMemcpyAsync(loss_host + gi, w.loss, sizeof(double), cudaMemcpyDeviceToHost, s));
  }
  GPTQ_CUDA_TRY(cudaMemcpyAsync(info8_host, w.info, 8 * sizeof(int), cudaMemcpyDeviceToHost, s));
  return GPTQ_OK;
}
}  // namespace
}  // namespace gptq
