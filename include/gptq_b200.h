/*
 * gptq_b200.h -- C ABI of the B200 (sm_100a) GPTQ layer solver.
 *
 * The library solves the layer-wise quantization problem of Section 2 (Eq. 1):
 * given a linear layer's weights W (d_row x d_col, here R x C) and calibration
 * inputs X, find grid-valued weights W^ minimising ||W X - W^ X||^2, with the
 * procedure of Algorithm 1 (Section 3).  Three calls, one per stage:
 *
 *   gptq_hessian_accumulate   H += 2 X X^T                 (Section 2; Alg. 1 caption)
 *   gptq_prepare_hinv         U = Cholesky((H + lambda I)^-1)^T   (Section 3 Step 3; Alg. 1)
 *   gptq_quantize_layer       Algorithm 1's two loops -> packed codes, scales,
 *                             zeros, loss
 *
 * Stages 2 and 3 also come as gptq_prepare_factor / gptq_quantize_layer_factor: the same results
 * without the factor's inverse (a reformulation of Algorithm 1's updates, described at gptq_prepare_factor).
 *
 * Conventions shared by every call
 *   - Every pointer except `stream` is DEVICE memory owned by the caller
 *     (unless a parameter says "host").  The library allocates no device
 *     memory: scratch comes from the caller's workspace `ws` (256-byte
 *     aligned, at least the size the matching *_workspace_bytes() reports).
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream) and the call returns without synchronising.
 *   - Argument errors are reported synchronously through the return value and
 *     nothing is enqueued.  Numerical / device-side conditions (a non-positive
 *     pivot, a bounded wait that ran out) are written to `dev_info` and are
 *     read by the caller after synchronising the stream; kernels never trap.
 *   - Matrices are dense row-major.  The paper's X is d_col x m; this API takes
 *     its transpose, token-major: X[t][c], t < n_tokens, c < C.
 *   - C must be a multiple of 32.
 *   - The device that owns the buffers and `stream` must be the CURRENT device of the calling
 *     thread (cudaSetDevice) for every call: per-device state inside the library (internal
 *     streams, SM count, the static scratch of gptq_prepare_hinv_static) is looked up by it.
 */
#ifndef GPTQ_B200_H_
#define GPTQ_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GPTQ_OK = 0,
  GPTQ_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, C % 32 != 0, misaligned pointer */
  GPTQ_ERR_UNSUPPORTED = 2, /* bits / group / block combination outside the supported set */
  GPTQ_ERR_NOT_PD = 3,      /* (dev_info only) H + lambda I is not positive definite */
  GPTQ_ERR_WORKSPACE = 4,   /* workspace missing, misaligned or too small */
  GPTQ_ERR_CUDA = 5,        /* a CUDA runtime / driver call failed */
  GPTQ_ERR_TIMEOUT = 6,     /* (dev_info only) a bounded device-side wait ran out */
  GPTQ_ERR_NONFINITE = 7    /* (dev_info only) a non-finite value was met */
} gptq_status_t;

/* bits value selecting the ternary grid {-1, 0, +1} x scale (Section 5, "Extreme
 * Quantization"); its codes 0, 1, 2 are stored in 2-bit fields. */
#define GPTQ_BITS_TERNARY (-1)

/* Bits of the `sym` argument of gptq_quantize_layer / gptq_rtn_layer / gptq_solve_layer_host (0 and 1 keep their
 * old meaning).  GPTQ_GRID_FP16_SCALES: every scale is rounded to the nearest fp16 value when the grid is
 * fixed -- before the zero-point is derived from it and before any weight is rounded on it -- so that a model stored
 * with one FP16 scale per group (the storage Section 5, "Extreme Quantization", counts) dequantizes to exactly the
 * values the solver compensated for.  The scale is still returned as fp32 (holding an fp16-representable value);
 * a scale that fp16 would flush to 0 or overflow stays fp32. */
#define GPTQ_GRID_SYMMETRIC 1
#define GPTQ_GRID_FP16_SCALES 2

/* Human-readable name of a status code (static storage, never NULL). */
const char* gptq_status_string(gptq_status_t status);

/* Diagnostic (no counterpart in the paper): number of CUDA kernels this library has
 * launched in the calling process so far.  Host-side counter; thread-safe. */
uint64_t gptq_launch_count(void);

/* Test hook (no counterpart in the paper).  Every wait inside the tensor-core kernels is bounded: when it runs out the
 * kernel records GPTQ_ERR_TIMEOUT in dev_info, every role leaves through its own bounded wait, tensor memory is freed and
 * the kernel returns -- it never hangs or traps.  This call lets a test see that path: it sets the limit of the waits
 * (nanoseconds; 0 restores the default of 4 s) and the index of one work item whose operand loads the producer leaves
 * out (-1: none), for kernels of the current device launched afterwards.  Synchronises the device.  Restore with (0, -1). */
gptq_status_t gptq_debug_wait_test(uint64_t wait_limit_ns, int skip_loads_of_item);

/* ------------------------------------------------------------------ stage 1
 * H += 2 * sum_t x_t x_t^T                     (Section 2: H_F = 2 X_F X_F^T;
 *                                               Algorithm 1 caption: 2 X X^T)
 *   H        [C x C] fp32, in/out.  The caller zeroes it before the first call;
 *            calls add, so calibration batches may arrive in any chunking
 *            (Section 5, Setup: Hessians are summed over calibration batches).  Both
 *            triangles are valid on return.  No 1/m normalisation.
 *   X_bf16   [n_tokens x C] bfloat16, row-major, 16-byte aligned.
 *   n_tokens >= 0 (0 is a no-op).
 *   dev_info int[2] or NULL: [0] = GPTQ_OK or GPTQ_ERR_TIMEOUT (a bounded wait inside the
 *            kernel ran out; H is then incomplete), [1] = which wait.
 * Products of bf16 values are exact in fp32; accumulation is fp32 and hierarchical: at most
 * 512 tokens in one tensor-core accumulator, those sums added round-to-nearest in registers
 * over at most 16384 tokens, and those added to H in memory. */
size_t gptq_hessian_workspace_bytes(int C, int64_t n_tokens);
gptq_status_t gptq_hessian_accumulate(float* H, const void* X_bf16, int64_t n_tokens, int C,
                                      void* ws, size_t ws_bytes, int* dev_info, void* stream);

/* The same sum for a caller that feeds one Hessian in several chunks (Section 5, Setup: Hessians are summed over
 * calibration batches).  Only tiles on or above the diagonal are computed; gptq_hessian_accumulate ends with a pass
 * that copies the upper triangle onto the lower one (2 C^2 floats of traffic), which only the last chunk needs.
 *   gptq_hessian_accumulate_upper  adds to the upper triangle (diagonal included) and leaves the strictly lower
 *                                  triangle as it is: it is stale until a later gptq_hessian_accumulate on the same H or
 *                                  gptq_hessian_symmetrize has run.  Arguments and errors as for gptq_hessian_accumulate.
 *   gptq_hessian_symmetrize        H[i][j] = H[j][i] for i > j (C % 32 == 0, H 16-byte aligned). */
gptq_status_t gptq_hessian_accumulate_upper(float* H, const void* X_bf16, int64_t n_tokens, int C,
                                            void* ws, size_t ws_bytes, int* dev_info, void* stream);
gptq_status_t gptq_hessian_symmetrize(float* H, int C, void* stream);

/* ------------------------------------------------------------------ stage 2
 * lambda = damp * mean(diag H);  H~ = H + lambda I          (Section 3, Step 3)
 * U = Cholesky(H~^-1)^T: upper triangular, positive diagonal, U^T U = H~^-1
 *                                                          (Algorithm 1, line 3)
 *   H        [C x C] fp32, symmetric (only its upper triangle is read); left intact unless U == H.
 *   U        [C x C] fp32, fully overwritten; the strict lower triangle is set to 0.
 *            U may be the same buffer as H (the factor then replaces the Hessian); partial overlap is not allowed.
 *   dev_info int[2]: [0] = GPTQ_OK or GPTQ_ERR_NOT_PD, [1] = index of the first
 *            non-positive pivot.  On NOT_PD the contents of U are unspecified
 *            but finite operations continue (no trap, no hang).  GPTQ_ERR_NONFINITE: an entry of
 *            the factor or of its inverse left the range of the scaled fp16 operand pairs the
 *            tensor-core contractions use for C > 1024 (a Hessian so ill-conditioned that entries of
 *            the inverse factor exceed ~100 times their row's diagonal entry); [1] = a row index.
 * Computed as the inverse of the upper factor of H~ = U~ U~^T, which equals
 * Cholesky(H~^-1)^T by uniqueness of the Cholesky factor.
 * Streams: for C > 1024 part of the work is enqueued on two internal streams (created once
 * per device on the first such call, never destroyed, they hold no device memory) that fork from
 * `stream` after the call's first kernels and join it again before the call returns, so the
 * caller sees ordinary single-stream ordering and the call can be captured into a CUDA graph
 * (make the first call for a device outside any capture).  The host-side enqueueing of
 * concurrent calls is serialised inside the library; calls on different streams still overlap on
 * the device as far as their workspaces are distinct. */
size_t gptq_prepare_hinv_workspace_bytes(int C);
gptq_status_t gptq_prepare_hinv(const float* H, float damp, int C, float* U,
                                void* ws, size_t ws_bytes, int* dev_info, void* stream);

/* Stage 2 without the inverse (a reformulation; Algorithm 1 itself asks for U).
 * Writing R = W - Q for the plain residuals (original weight minus quantized value) and E for Algorithm 1's scaled
 * errors, the update rule of Algorithm 1 gives Q + E U = W, i.e. E = R U~ with U~ = U^-1 the upper factor of
 * H~ = U~ U~^T.  For a block J of columns and the columns before it this reads
 *     (working weights of block J when the algorithm reaches it) = W_J + (R_before U~[before, J]) U_JJ,
 * where U_JJ = (U~_JJ)^-1 is the diagonal block of U.  So the solver needs U on the diagonal blocks and the products
 * U~[before, J] U_JJ above them -- what the backwards factorisation of H~ leaves when it stops before inverting, plus
 * one 1024-deep product per block column -- and the rows of the inverse (C^3 / 3 of stage 2's 2 C^3 / 3 flops) are
 * not needed.
 *   F   [C x C] fp32, fully overwritten: for diagonal blocks of GPTQ_FACTOR_BLOCK (1024) columns, block (J, J) holds
 *       U_JJ (upper triangular); the blocks above it hold U~[:, J] U_JJ; the strict lower triangle is 0.  For
 *       C <= 1024 F = U.
 *       F may be the same buffer as H.
 *   Everything else (H, damp, workspace, dev_info, streams, errors) as gptq_prepare_hinv; same workspace query.
 * Consumer: gptq_quantize_layer_factor. */
#define GPTQ_FACTOR_BLOCK 1024
gptq_status_t gptq_prepare_factor(const float* H, float damp, int C, float* F,
                                  void* ws, size_t ws_bytes, int* dev_info, void* stream);

/* gptq_prepare_hinv for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant, it computes exactly what gptq_prepare_hinv does.)
 *
 * Who needs it: code that may not call cudaMalloc -- a plug-in inside a framework whose
 * memory pool owns the whole device, a latency-critical loop where an allocation would
 * stall the GPU, a process with a fixed memory budget handed out at start-up.  Such a
 * caller has no workspace to pass, so the scratch lives inside the library, in one fixed
 * array in device global memory of 256 + 2 * 512 KiB = 1,048,832 bytes.
 *
 *   - Limit: C <= GPTQ_PREPARE_HINV_STATIC_MAX_C (1024); a larger C returns
 *     GPTQ_ERR_UNSUPPORTED and nothing is enqueued (use gptq_prepare_hinv with a workspace).
 *   - H, U, dev_info, stream, return value and dev_info contents: as gptq_prepare_hinv.
 *     The caller still owns and passes all inputs and outputs.
 *   - The call allocates nothing: no cudaMalloc / cudaFree and no allocating library routine.
 *   - Every GPU on which the library is loaded holds the array until the process exits.
 *   - The first call on each device resolves the array's device address (a one-time set-up,
 *     done with that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents.
 *     Nothing in it needs clearing (each call writes what it later reads), but two calls
 *     whose kernels overlap on the GPU -- different streams, or different host threads --
 *     race on it: serialise them on one stream. */
#define GPTQ_PREPARE_HINV_STATIC_MAX_C 1024
gptq_status_t gptq_prepare_hinv_static(const float* H, float damp, int C, float* U,
                                       int* dev_info, void* stream);

/* ------------------------------------------------------------------ stage 3
 * Algorithm 1: for each block of `block` columns, quantize column by column
 * (Q_j = quant(W_j); E_j = (W_j - Q_j) / U_jj; W[:, j:blockend] -= E_j U[j, j:blockend]),
 * then push the block's errors onto all later columns (W[:, blockend:] -= E U[block, blockend:]).
 *   W_fp16     [R x C] IEEE half, row-major, 16-byte aligned; not modified.
 *   U          [C x C] fp32 from gptq_prepare_hinv.
 *   bits       2, 3, 4, 8 or GPTQ_BITS_TERNARY.
 *   group_size <= 0: one grid per row, fixed from the original row before the
 *              process (Section 2; Section 5 Setup: per-row asymmetric min-max).
 *              > 0: g consecutive weights share a grid, taken at the group's first
 *              column from the weights as updated so far (Section 5, grouping).
 *              Must divide C, and nest with
 *              `block` (g % block == 0 or block % g == 0).  Supported sizes: 4, 8, 16
 *              or any multiple of 32 (the paper uses 8, 32, 64, 128, 1024); anything
 *              else returns GPTQ_ERR_UNSUPPORTED.
 *   sym        bit mask: 0: asymmetric min-max grid (range widened to contain 0, integer
 *              zero-point).  GPTQ_GRID_SYMMETRIC: symmetric grid, zero = (maxq+1)/2 (the ternary grid
 *              is always symmetric).  GPTQ_GRID_FP16_SCALES: see above.  Other bits: GPTQ_ERR_INVALID_ARG.
 *   block      B of Algorithm 1: a multiple of 32 in [32, 256].  The result does
 *              not depend on it (Section 3, Step 2) up to rounding.
 *   qweight    [R x C*f/32] uint32, f = field width (bits; 2 for ternary): per
 *              row a little-endian bit stream, code of column c in stream bits
 *              [c f, c f + f), word k = stream bits [32k, 32k+32).
 *   scales     [R x G] fp32, G = 1 (per row) or C / group_size.
 *   zeros      [R x G] fp32 holding integer zero-points in [0, maxq].
 *              The quantized weight is scales * (code - zeros).
 *   loss       double[1]: sum over all weights of E^2 = (w - q)^2 / U_jj^2 (Eq. 2 summed).
 *   dev_info   int[2], [0] = GPTQ_OK / GPTQ_ERR_NONFINITE / GPTQ_ERR_TIMEOUT.
 * All outputs are fully overwritten. */
size_t gptq_quantize_workspace_bytes(int R, int C, int bits, int group_size, int block);
gptq_status_t gptq_quantize_layer(const void* W_fp16, const float* U, int R, int C,
                                  int bits, int group_size, int sym, int block,
                                  uint32_t* qweight, float* scales, float* zeros, double* loss,
                                  void* ws, size_t ws_bytes, int* dev_info, void* stream);

/* gptq_quantize_layer on the output F of gptq_prepare_factor instead of U: same arguments, same outputs (codes, scales,
 * zero-points and loss agree with the U form up to fp32-level rounding of the update sums).  Across blocks of 1024
 * columns it feeds back the plain residuals w - q through the blocks of F above the diagonal (see gptq_prepare_factor);
 * inside a block it is Algorithm 1 as written.  Runs in the row-stripe form only: for C > 1024 the block size must divide 1024
 * (32, 64, 128, 256) and a group wider than the block must divide 1024 too, else GPTQ_ERR_UNSUPPORTED.
 * Workspace: gptq_quantize_workspace_bytes. */
gptq_status_t gptq_quantize_layer_factor(const void* W_fp16, const float* F, int R, int C,
                                         int bits, int group_size, int sym, int block,
                                         uint32_t* qweight, float* scales, float* zeros, double* loss,
                                         void* ws, size_t ws_bytes, int* dev_info, void* stream);

/* Which form of Algorithm 1's loops gptq_quantize_layer runs INSIDE an outer block of about 1024 columns (both are
 * exact regroupings of the same updates, Section 3 Step 2; updates ACROSS outer blocks are one large tensor-core
 * contraction per outer block either way):
 *   1 (default)  row-stripe form: rows are independent (Section 2), so one CTA owns a stripe of rows and runs all
 *                inner blocks of the outer block back to back in ONE launch -- the inner loop with one thread per
 *                row, the pushes of its errors with tcgen05 tensor-core instructions on the stripe's 128 rows.  A block
 *                of 256 columns runs there as two 128-column inner blocks (the same updates, regrouped).
 *   0            per inner block one in-block kernel and one small tcgen05 contraction (two launches per block).
 * Process-wide, takes effect for calls made afterwards; returns the previous value (any other argument only
 * queries).  Meant for side-by-side benchmarks; results of the two forms agree up to fp32-level rounding of the
 * update sums. */
int gptq_set_stage3_variant(int variant);

/* ------------------------------------------------------------------ round-to-nearest baseline
 * RTN (Section 5, Baselines): every weight rounded to the nearest value of the solver's own
 * grid -- per-row (group_size <= 0) or per-group min-max taken from the ORIGINAL weights -- with
 * no error feedback.  Equals gptq_quantize_layer for a diagonal Hessian.  Arguments and output
 * layout as in gptq_quantize_layer (any group size that divides C); no workspace, no dev_info. */
gptq_status_t gptq_rtn_layer(const void* W_fp16, int R, int C, int bits, int group_size, int sym,
                             uint32_t* qweight, float* scales, float* zeros, void* stream);

/* ------------------------------------------------------------------ using the packed weights
 * The two kernels the paper describes for running a quantized model (Section 5, "Practical
 * Speedups"; appendix on kernels), reading the packed layout gptq_quantize_layer writes.
 * Dequantized value: scales[r][gi] * (code - zeros[r][gi]), formed with one fp32 multiply.
 * group_size as in gptq_quantize_layer (<= 0: per row); 4, 8, 16 or a multiple of 32.
 *
 * gptq_dequantize: the whole matrix back to fp16 (round-to-nearest-even of the fp32 product).
 *   W_out_fp16 [R x C] half, starting on a 16-byte boundary (GPTQ_ERR_INVALID_ARG otherwise).
 * gptq_matvec: y = W^ x for ONE fp16 vector x (batch-1 generation: packed matrix times
 *   fp16 vector with dequantization on the fly, never materialising W^).
 *   x_fp16 [C] half, y [R] fp32; products exact, sums in fp32: per group the kernel forms
 *   sum q x and zero * sum x and combines them with the scale, so its rounding error is
 *   fp32-level relative to sum scale * (q + zero) * |x|.  Per-row grids and group sizes that
 *   are multiples of 128 run on the tensor cores (mma.sync f16), other group sizes on the
 *   CUDA cores.  C <= 51200 (x is staged in shared memory), else GPTQ_ERR_UNSUPPORTED; x and qweight
 *   must start on 16-byte boundaries (GPTQ_ERR_INVALID_ARG otherwise).  The tensor-core path moves
 *   the codes through shared-memory rings when a packed row is a whole number of 16-byte pieces,
 *   and through registers otherwise; the results are the same. */
gptq_status_t gptq_dequantize(const uint32_t* qweight, const float* scales, const float* zeros,
                              int R, int C, int bits, int group_size, void* W_out_fp16, void* stream);
gptq_status_t gptq_matvec(const uint32_t* qweight, const float* scales, const float* zeros,
                          const void* x_fp16, int R, int C, int bits, int group_size, float* y, void* stream);

/* ------------------------------------------------------------------ whole layer, host buffers
 * Stages 1-3 for one layer whose inputs and outputs live in HOST memory (Eq. 1's W and X in, the
 * packed W^ out): X is streamed to the device in token chunks of up to about 2 GiB (the first ones short,
 * growing by a quarter each, so that the accumulation starts after a few milliseconds), double-buffered on
 * an internal copy stream so that the transfer of a chunk overlaps the Hessian accumulation of the
 * previous one (Section 5, Setup: Hessians are accumulated over calibration batches); then
 * gptq_prepare_hinv and gptq_quantize_layer run and the results are copied back.
 *   W_fp16_host [R x C] half, X_bf16_host [n_tokens x C] bfloat16: host memory; page-locked memory
 *              is needed for the copies to overlap (pageable memory works, serialised).
 *   qweight_host, scales_host, zeros_host, loss_host: host outputs, shaped as in gptq_quantize_layer.
 *   info_host  int[2] (host): first non-OK device status of the three stages and its detail
 *              (for stage 1: of the first chunk that reported one).
 *   dev_ws     DEVICE workspace of gptq_solve_layer_host_workspace_bytes() bytes: holds H, U, W,
 *              two X staging buffers, the outputs and the stages' own workspaces.
 * Unlike the per-stage calls this one SYNCHRONISES `stream` before returning (the results are on
 * the host when it returns); it creates and destroys one internal stream and a few events per
 * call and allocates no device memory.  Calls from different host threads may be in flight at
 * the same time if each has its own `stream` and `dev_ws` (one layer's X then crosses PCIe while
 * another layer is factored and quantized). */
size_t gptq_solve_layer_host_workspace_bytes(int R, int C, int64_t n_tokens, int bits, int group_size, int block);
gptq_status_t gptq_solve_layer_host(const void* W_fp16_host, const void* X_bf16_host, int64_t n_tokens,
                                    int R, int C, float damp, int bits, int group_size, int sym, int block,
                                    uint32_t* qweight_host, float* scales_host, float* zeros_host,
                                    double* loss_host, int* info_host, void* dev_ws, size_t dev_ws_bytes,
                                    void* stream);

/* The same for SEVERAL grids of one layer (e.g. the 4-bit and the 3-bit model of the paper's tables from one calibration
 * pass): the activations cross to the device ONCE, one Hessian and one factor serve every grid (Algorithm 1's H^-1 does
 * not depend on the grid), and stage 3 runs and is copied back grid after grid.
 *   n_grids >= 1; bits / group_size / sym: host arrays of n_grids entries (as in gptq_quantize_layer);
 *   qweight_host / scales_host / zeros_host: host arrays of n_grids host pointers, each shaped for its grid;
 *   loss_host double[n_grids]; info_host int[2]: first non-OK device status of any stage or grid.
 * Everything else as gptq_solve_layer_host. */
size_t gptq_solve_layer_host_grids_workspace_bytes(int R, int C, int64_t n_tokens, int n_grids, const int* bits,
                                                   const int* group_size, int block);
gptq_status_t gptq_solve_layer_host_grids(const void* W_fp16_host, const void* X_bf16_host, int64_t n_tokens,
                                          int R, int C, float damp, int n_grids, const int* bits,
                                          const int* group_size, const int* sym, int block,
                                          uint32_t* const* qweight_host, float* const* scales_host,
                                          float* const* zeros_host, double* loss_host, int* info_host,
                                          void* dev_ws, size_t dev_ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GPTQ_B200_H_ */
