/*
 * ptq_linear.h -- C ABI of the B200 (sm_100a) PTS W8A8 linear layer.
 *
 * The operation is the quantized linear layer of PTQ4VM (arXiv 2412.20386),
 * Sec. 5.1 "Per-Token Static (PTS) Quantization":
 *
 *      Y  ~=  diag(Delta_W) . (W-bar . X-bar) . diag(Delta_X)
 *
 * with the SmoothQuant scale s of Sec. 2.4 (Eq. smooth_scale, Eq. smooth)
 * applied to the activations on the fly and assumed already folded into the
 * integer weight.  Written row-major, for token row m = b*T + t:
 *
 *   Q1  q[m,k]   = clamp( rne( (x[m,k] / s[k]) / dx[t] ), -128, 127 )      int8
 *   G1  acc[m,n] = sum_k q[m,k] * Wq[n,k]                                  int32
 *   E1  y[m,n]   = fp16( float(acc[m,n]) * dx[t] * dw[n] + bias[n] )       fp16
 *
 * Q1 uses two IEEE binary32 divisions in that order, round-to-nearest-even,
 * NaN -> 0, +-inf -> 127 / -128.  G1 is exact.  E1 is evaluated in binary32.
 * The four parts named in Appendix B.1 of the paper (activation smoothing,
 * quantization, integer GEMM, dequantization) map to Q1 (first two), G1, E1.
 *
 * Conventions
 *   - "host" / "device" in a parameter comment says where the pointer lives.
 *   - Every function returns a ptq_status_t; none throws, aborts or traps.
 *     ptq_last_error() gives a thread-local text for the last failure.
 *   - ptq_linear_create copies all parameters: the caller keeps its arrays.
 *   - The forward calls allocate nothing, enqueue work on the caller's stream
 *     and return without synchronising.  A handle is immutable after create,
 *     so concurrent forwards on different streams are allowed as long as they
 *     use different workspaces (each handle also carries one device status
 *     word that all its launches may set; see ptq_linear_device_status).
 *   - The quantize and GEMM kernels are launched with the programmatic-stream-serialization
 *     attribute: their set-up may run while the previous kernel on the stream drains, and each waits
 *     for that kernel's completion before it reads or writes any buffer.  Results and ordering are
 *     those of plain stream order.
 *   - Requires a device of compute capability 10.0 (sm_100a); create fails
 *     with PTQ_ERR_ARCH elsewhere.  There is no CPU or generic-GPU fallback.
 */
#ifndef PTQ_LINEAR_H_
#define PTQ_LINEAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ptq_linear ptq_linear_t;   /* opaque; owns device copies of all parameters */

typedef enum {
    PTQ_OK          = 0,
    PTQ_ERR_NULL    = 1,   /* a required pointer is NULL */
    PTQ_ERR_SHAPE   = 2,   /* a dimension is out of range, or the workspace is too small */
    PTQ_ERR_VALUE   = 3,   /* a parameter value is invalid (non-positive or non-finite step, weight code -128) */
    PTQ_ERR_ALIGN   = 4,   /* a device pointer is not aligned as required */
    PTQ_ERR_ARCH    = 5,   /* current device is not compute capability 10.0 */
    PTQ_ERR_CUDA    = 6,   /* a CUDA runtime / driver call failed; text in ptq_last_error() */
    PTQ_ERR_NOMEM   = 7,   /* device or host allocation failed (create / calibrate only) */
    PTQ_ERR_TIMEOUT = 8    /* a bounded device-side wait gave up (reported by ptq_linear_device_status) */
} ptq_status_t;

/* Flags for create / forward. */
#define PTQ_FLAG_NONE            0u
#define PTQ_FLAG_FUSED_PROLOGUE  1u   /* F1: quantize inside the GEMM kernel; no int8 round trip, no workspace
                                         (same bits; measured 2-3x slower than the two-kernel path) */
#define PTQ_FLAG_CTA_PAIR        2u   /* two-kernel path: run G1+E1 on CTA pairs (tcgen05 cta_group::2, 256-row tiles,
                                         half the weight bytes per CTA) when the batch has enough rows; same results */

/* Limits (create returns PTQ_ERR_SHAPE beyond them). */
#define PTQ_MAX_K   8192
#define PTQ_MAX_N   65536
#define PTQ_MAX_T   1048576

/*
 * Create a layer (Sec. 5.1; weight format of Sec. 2.3).
 *   K, N, T      input channels D_in, output channels D_out, token positions L per image
 *   w_q          host, [N,K] row-major int8, the folded integer weight W-bar = quant(W diag(s));
 *                values in [-127,127] (symmetric range of Sec. 2.3; -128 is rejected)
 *   w_step       host, [N] fp32, Delta_W per output channel, finite and > 0
 *   smooth       host, [K] fp32, smoothing scale s (Eq. smooth_scale), finite and > 0
 *   act_step     host, [T] fp32, Delta_X per token position, finite and > 0
 *   bias         host, [N] fp32 or NULL (added after the scaling, before the fp16 rounding)
 *   flags        reserved, pass PTQ_FLAG_NONE
 * The handle is bound to the device that is current at the time of the call.
 */
ptq_status_t ptq_linear_create(ptq_linear_t **out, int K, int N, int T,
                               const int8_t *w_q, const float *w_step,
                               const float *smooth, const float *act_step,
                               const float *bias, unsigned flags);

/*
 * Create a layer with ASYMMETRIC per-token-static activations: step and zero offset per token position,
 * which is what Sec. 5.1 allocates (both parameters for every token position; quantizer form of
 * Sec. 2.3 with the offset rounded to an integer):
 *   Q1  c[m,k]   = clip( rne( (x[m,k] / s[k]) / dx[t] ) + z[t], 0, 255 )           uint8
 *       (NaN -> z[t], +inf -> 255, -inf -> 0)
 *   G1  acc[m,n] = sum_k (c[m,k] - z[t]) * Wq[n,k]                                 int32
 *   E1  as for the symmetric layer
 *   act_zero   host, [T] int32, zero offsets z[t] in [0,255]
 * Everything else as ptq_linear_create.  The same forward / quantize / debug entry points serve the
 * handle; its codes are unsigned bytes.  PTQ_FLAG_FUSED_PROLOGUE and PTQ_FLAG_CTA_PAIR are accepted and
 * ignored for such a layer (it always runs the quantize kernel and the single-CTA GEMM kernel).
 */
ptq_status_t ptq_linear_create_asym(ptq_linear_t **out, int K, int N, int T,
                                    const int8_t *w_q, const float *w_step,
                                    const float *smooth, const float *act_step,
                                    const int32_t *act_zero, const float *bias, unsigned flags);

/* Release the handle and its device memory.  NULL is allowed. */
void ptq_linear_destroy(ptq_linear_t *h);

/*
 * Bytes of device workspace ptq_linear_forward needs for a batch of B images:
 * the int8 codes [B*T, Kpad] with Kpad = K rounded up to 16, or 0 with
 * PTQ_FLAG_FUSED_PROLOGUE on a layer the fused kernel covers.  The answer assumes a
 * 16-byte aligned x: an x that is only 2-byte aligned always takes the two-kernel path
 * and needs the size reported for PTQ_FLAG_NONE, whatever the flags.
 * Returns 0 for a NULL handle or B < 1.
 */
size_t ptq_linear_workspace_bytes(const ptq_linear_t *h, int B, unsigned flags);

/*
 * Forward pass Q1 -> G1 -> E1 (Sec. 5.1; Appendix B.1).
 *   x_fp16     device, [B,T,K] contiguous binary16, 2-byte aligned (16-byte alignment and K % 8 == 0
 *              enable the vectorised load path)
 *   y_fp16     device, [B,T,N] contiguous binary16; must not overlap x or the workspace
 *   workspace  device, at least ptq_linear_workspace_bytes(h,B,flags) bytes, 16-byte aligned;
 *              contents are scratch.  May be NULL with PTQ_FLAG_FUSED_PROLOGUE.
 *   flags      PTQ_FLAG_NONE: quantize kernel, then GEMM+dequant kernel (one of three variants chosen from
 *              the shape, all with the same bits: see ptq_linear_gemm_variant).
 *              PTQ_FLAG_FUSED_PROLOGUE: one kernel; same results bit for bit.  Layers whose shape the
 *              fused kernel does not cover fall back to the two-kernel path and then need the workspace
 *              (ptq_linear_fused_supported tells which).
 *   stream     cudaStream_t cast to void* (NULL = legacy default stream)
 */
ptq_status_t ptq_linear_forward(const ptq_linear_t *h, const void *x_fp16, int B,
                                void *y_fp16, void *workspace, size_t workspace_bytes,
                                unsigned flags, void *stream);

/*
 * Forward pass for callers that cannot allocate device memory.  (The paper has no counterpart of
 * this entry point; it computes exactly what ptq_linear_forward with PTQ_FLAG_NONE computes.)
 *
 * Some callers have no way to provide the workspace: code running where cudaMalloc is forbidden
 * (inside a latency-critical serving loop that must not touch the allocator, under a memory pool
 * that owns every byte of the device, or in a plugin that is handed only its input and output
 * buffers).  For them the int8 codes go to a scratch array that is part of the library image
 * itself: a file-scope __device__ array of PTQ_STATIC_SCRATCH_BYTES bytes, present on every GPU
 * that loads the library from load until process exit.
 *
 *   - B*T rows of ptq_linear_code_pitch(h) bytes must fit in PTQ_STATIC_SCRATCH_BYTES; larger
 *     batches are refused with PTQ_ERR_SHAPE (split the batch, or use ptq_linear_forward).
 *   - The call allocates nothing and frees nothing.  The first call on each device looks up the
 *     array's device address (a one-time, per-device set-up step done with that device current);
 *     make that first call before starting any stream capture.
 *   - All calls on one device, from every handle and every stream, share the same array, and it
 *     keeps whatever the previous call left in it.  Nothing in it needs to start at zero: each call
 *     writes every byte it later reads.  Two calls whose GPU work overlaps in time (different
 *     streams, no dependency between them) race on the array and corrupt each other's result; run
 *     them on one stream or order them with events.
 *   x_fp16, y_fp16, stream: as for ptq_linear_forward.
 */
#define PTQ_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
ptq_status_t ptq_linear_forward_static(const ptq_linear_t *h, const void *x_fp16, int B, void *y_fp16,
                                       void *stream);

/*
 * Comparator: per-token DYNAMIC quantization (the alternative that Sec. 4.1 and the latency table of
 * Sec. 6 set PTS against).  The layer's stored per-token-position steps are ignored; the step of every
 * token row is measured on that row at run time:
 *     u = x / s[k];   step[m] = max(max_k |u[m,k]|, 1e-5) / 127;   q = clamp(rne(u / step[m]), -128, 127)
 *     y[m,n] = fp16(float(sum_k q[m,k] Wq[n,k]) * step[m] * dw[n] + bias[n])
 * (binary32, same rounding and special-value rules as ptq_linear_forward).  The paper gives no
 * formula for its dynamic baseline; this is the usual symmetric min-max rule per token.
 *   h            a symmetric layer (ptq_linear_create); asymmetric layers give PTQ_ERR_VALUE
 *   x_fp16, B, y_fp16, stream   as for ptq_linear_forward
 *   workspace    device, 16-byte aligned, at least ptq_linear_workspace_bytes_dynamic(h, B) bytes
 *                (codes, then one float per row); caller-owned, contents undefined afterwards
 * The _debug form also copies out the codes (dense [B*T,K] int8), the int32 accumulators [B*T,N]
 * and the row steps ([B*T] float); each tap pointer may be NULL.
 */
size_t ptq_linear_workspace_bytes_dynamic(const ptq_linear_t *h, int B);
ptq_status_t ptq_linear_forward_dynamic(const ptq_linear_t *h, const void *x_fp16, int B, void *y_fp16,
                                        void *workspace, size_t workspace_bytes, void *stream);
ptq_status_t ptq_linear_forward_dynamic_debug(const ptq_linear_t *h, const void *x_fp16, int B, void *y_fp16,
                                              void *q_int8_out, void *acc_int32_out, void *step_fp32_out,
                                              void *workspace, size_t workspace_bytes, void *stream);

/* 1 if PTQ_FLAG_FUSED_PROLOGUE runs the single fused kernel for this layer (given a 16-byte aligned x;
 * any other x falls back to the two-kernel path and needs the workspace), 0 if the layer always falls back. */
int ptq_linear_fused_supported(const ptq_linear_t *h);

/*
 * Q1 alone (Appendix B.1, parts 1-2): q_int8 device [B,T,K] dense int8 codes.
 */
ptq_status_t ptq_quantize(const ptq_linear_t *h, const void *x_fp16, int B,
                          void *q_int8, void *stream);

/*
 * G1 + E1 alone (Sec. 5.1; Appendix B.1, parts 3-4): integer GEMM and dequantization on codes that
 * are already in device memory.
 *   q_int8     device, [B*T, pitch] int8 codes with pitch = ptq_linear_code_pitch(h) bytes per row
 *              (K rounded up to 16; bytes beyond K in a row are ignored), 16-byte aligned
 *   y_fp16     device, [B,T,N] binary16
 */
ptq_status_t ptq_linear_gemm_dequant(const ptq_linear_t *h, const void *q_int8, int B, void *y_fp16,
                                     void *stream);

/* Bytes per row of the code matrix that ptq_linear_gemm_dequant reads and the workspace holds. */
int ptq_linear_code_pitch(const ptq_linear_t *h);

/*
 * Which G1 + E1 kernel (Sec. 5.1; Appendix B.1, parts 3-4) a forward pass over B images takes on the
 * default path, assuming a 16-byte aligned y with N % 8 == 0 (otherwise always the first):
 *   0  ptq_gemm_dequant_kernel          operand stages streamed per tile, eight epilogue warps per tile
 *   1  ptq_gemm_dequant_kernel, teams   same, the epilogue warps in two teams, one per accumulator
 *                                       (K <= 384 and at least three tiles per SM)
 *   2  ptq_gemm_dequant_panel_kernel    the codes of a row panel resident in shared memory for a group
 *                                       of N tiles (512 <= K <= 768, several N tiles, many tiles per SM)
 * Returns -1 for a NULL handle or B < 1.  All variants produce the same bits.
 */
int ptq_linear_gemm_variant(const ptq_linear_t *h, int B);

/*
 * Measurement aid; the paper has no counterpart.  Times one of five stand-alone kernels that move bytes the way
 * the GEMM + dequantization kernel does (Sec. 5.1; Appendix B.1, parts 3-4) but compute nothing, so that a
 * roofline discussion can quote what THIS GPU does with nothing else running:
 *   kind 0  16-byte stores over buf                                      result: GB/s written
 *   kind 1  2-D TMA stores of 32 x 64 fp16 boxes over buf seen as y [M, 3072], in the epilogue's
 *           tile order, one CTA per SM, eight warps                      result: GB/s written
 *   kind 2  the operand stages of a [M, 768] x [3072, 768] problem (128 x 128 B + 256 x 128 B per k-block,
 *           four stages per CTA) pulled by 2-D tiled TMA loads           result: GB/s delivered to the SMs
 *   kind 3  an empty kernel, launches back to back                       result: microseconds per launch
 *   kind 4  the same with programmatic dependent launch                  result: microseconds per launch
 *   buf     device, 256-byte aligned scratch of `bytes` bytes (kinds 0-2; its contents are overwritten or
 *           ignored; the last 256 bytes hold a status word); kinds 1 and 2 use as many 128-row tiles as fit
 *   iters   timed launches (after three untimed ones), 1 .. 100000
 * Allocates no device memory.  Synchronises the stream.  PTQ_ERR_SHAPE if buf is too small.
 */
ptq_status_t ptq_probe(int kind, void *buf, size_t bytes, int iters, double *result, void *stream);

/*
 * Forward pass with parity taps.  Same as ptq_linear_forward, and additionally writes
 *   q_int8_out     device, [B,T,K] dense int8 codes of Q1, or NULL
 *                  (with PTQ_FLAG_FUSED_PROLOGUE the codes never exist in memory; they are then
 *                  produced by a separate run of the quantize kernel)
 *   acc_int32_out  device, [B,T,N] dense int32 accumulators of G1, or NULL
 * The workspace is required unless PTQ_FLAG_FUSED_PROLOGUE is set and q_int8_out is NULL.
 */
ptq_status_t ptq_linear_forward_debug(const ptq_linear_t *h, const void *x_fp16, int B,
                                      void *y_fp16, void *q_int8_out, void *acc_int32_out,
                                      void *workspace, size_t workspace_bytes,
                                      unsigned flags, void *stream);

/*
 * Q0: min-max calibration of the static parameters from a calibration batch
 * (Eq. smooth_scale with the given integer weights; PTS steps of Sec. 5.1 from
 * the min-max range of Sec. 2.3):
 *   maxX[k] = max |xcal[:,:,k]|,  maxW[k] = max_n |w_q[n,k]| * w_step[n]
 *   s[k]    = sqrt( max(maxX[k],1e-5) / max(maxW[k],1e-5) )
 *   dx[t]   = max( max_{b,k} |xcal[b,t,k] / s[k]|, 1e-5 ) / 127
 * all in binary32 with correctly rounded operations, so the result is unique.
 *   xcal_fp16     device, [Bc,T,K] contiguous binary16
 *   w_q, w_step   host
 *   smooth_out    host, [K];  act_step_out  host, [T]
 * Allocates temporary device memory and synchronises the stream before returning.
 */
ptq_status_t ptq_calibrate(int K, int N, int T, const void *xcal_fp16, int Bc,
                           const int8_t *w_q, const float *w_step,
                           float *smooth_out, float *act_step_out, void *stream);

/*
 * Comparator: per-TENSOR static quantization (the coarsest granularity of the latency table of Sec. 6
 * and of Fig. 5: one step for the whole activation tensor).  Same s[k] as ptq_calibrate, and
 *   step = max( max_{b,t,k} |xcal[b,t,k] / s[k]|, 1e-5 ) / 127
 * written to all T entries of act_step_out, so that the result feeds ptq_linear_create unchanged: a
 * per-tensor static layer is a PTS layer whose steps are all equal and runs the same kernels.
 * Arguments, ownership and errors as for ptq_calibrate.
 */
ptq_status_t ptq_calibrate_per_tensor(int K, int N, int T, const void *xcal_fp16, int Bc,
                                      const int8_t *w_q, const float *w_step,
                                      float *smooth_out, float *act_step_out, void *stream);

/*
 * W4A4 layers (the bit width of the paper's latency table; Appendix B.1, quantization part).  The
 * arithmetic is that of ptq_linear_create / ptq_linear_forward with the signed 4-bit range:
 *     q = clamp(rne((x / s[k]) / act_step[t]), -8, 7),   acc = sum_k q * w4,   y as before,
 * NaN -> 0, +inf -> 7, -inf -> -8.  Weights arrive packed two per byte as the paper states,
 *     byte = (w[n, 2i+1] << 4) | (w[n, 2i] & 15)      (low nibble = even column, two's complement),
 * rows of (K+1)/2 bytes, an odd K ending with an unused high nibble.  The integer tensor-core
 * instruction of sm_100 takes 8-bit operands, so the library unpacks the weights once at create and
 * keeps the activation codes one per byte in the workspace: 4-bit layers run at the speed of 8-bit
 * ones and save only the bytes of the stored weights.  All other entry points (workspace_bytes,
 * forward, forward_debug, quantize, gemm_dequant, forward_static) accept such a handle; the fused
 * prologue and CTA-pair flags are ignored, the dynamic comparator is refused.
 *   w_q_packed   host, [N, (K+1)/2] bytes
 *   act_step     host, [T]; ptq_calibrate_w4a4 returns the min-max steps max|x/s| / 7
 */
ptq_status_t ptq_linear_create_w4a4(ptq_linear_t **out, int K, int N, int T, const uint8_t *w_q_packed,
                                    const float *w_step, const float *smooth, const float *act_step,
                                    const float *bias, unsigned flags);
ptq_status_t ptq_calibrate_w4a4(int K, int N, int T, const void *xcal_fp16, int Bc, const uint8_t *w_q_packed,
                                const float *w_step, float *smooth_out, float *act_step_out, void *stream);
/*
 * Q1 of a W4A4 layer with the codes packed two per byte exactly as the paper's quantization step
 * writes them (byte = (q[m, 2i+1] << 4) | (q[m, 2i] & 15)), for storage or transport.
 *   q_packed    device, [B*T, (K+1)/2] bytes
 *   workspace   device, 16-byte aligned, at least ptq_linear_workspace_bytes(h, B, PTQ_FLAG_NONE) bytes
 */
ptq_status_t ptq_quantize_packed4(const ptq_linear_t *h, const void *x_fp16, int B, void *q_packed, void *workspace,
                                  size_t workspace_bytes, void *stream);

/*
 * Step-size search (Sec. 5.2, second stage; the "+Truncation" row of the ablation): for every token
 * position the candidate step
 *     Delta[t,j] = base_step[t] * (j / n_grid),   j = j_lo .. n_grid
 * that minimises the squared distance between the smoothed calibration activations u = x / s[k] and
 * their dequantized codes,
 *     loss[t,j] = sum_{b,k} (u - Delta[t,j] * clip(rne(u / Delta[t,j]), -128, 127))^2 ,
 * the largest j on equal losses.  Steps, quotients and the element error are binary32 (the error with
 * one rounding, as a fused multiply-add); the sum is binary64 and its order is fixed for a given
 * shape, but it is not the sequential order, so two candidates whose losses agree to about 1e-13
 * relative may be ranked either way.  Non-finite u do not enter the loss.  The paper states the
 * objective and that it is a grid search; the grid is this library's choice (a common one is
 * n_grid = 100, j_lo = 20 with base_step the min-max steps of ptq_calibrate: j = n_grid is "no
 * truncation").
 *   xcal_fp16     device, [Bc,T,K] contiguous binary16
 *   smooth        host, [K], positive finite;  base_step  host, [T], in [1e-30, inf)
 *   n_grid, j_lo  1 <= j_lo <= n_grid <= PTQ_MAX_SEARCH_GRID
 *   act_step_out  host, [T]: the chosen steps
 *   best_out      host, [T] int32: the chosen j, or NULL
 *   loss_out      host, [T, n_grid - j_lo + 1] binary64: every loss, or NULL
 * Allocates temporary device memory and synchronises the stream before returning.
 */
#define PTQ_MAX_SEARCH_GRID 4096
ptq_status_t ptq_search_act_step(int K, int T, const void *xcal_fp16, int Bc, const float *smooth,
                                 const float *base_step, int n_grid, int j_lo, float *act_step_out,
                                 int32_t *best_out, double *loss_out, void *stream);

/*
 * Q0 for asymmetric layers: s[k] as in ptq_calibrate; per token position the range [lo, hi] of x/s over
 * the calibration batch, widened to contain zero; dx[t] = max(hi - lo, 1e-5) / 255 and
 * z[t] = clip(rne(-lo / dx[t]), 0, 255)  (Delta_X and eps_X of Sec. 2.3 per token position, Sec. 5.1).
 *   act_zero_out  host, [T] int32
 */
ptq_status_t ptq_calibrate_asym(int K, int N, int T, const void *xcal_fp16, int Bc, const int8_t *w_q,
                                const float *w_step, float *smooth_out, float *act_step_out,
                                int32_t *act_zero_out, void *stream);

/*
 * Read and clear the handle's device status word.  Synchronises the device.  Returns PTQ_OK, or
 * PTQ_ERR_TIMEOUT if a kernel launched with this handle abandoned a bounded wait since the last
 * call (its output is then undefined), or PTQ_ERR_CUDA.
 */
ptq_status_t ptq_linear_device_status(const ptq_linear_t *h);

/*
 * Self-test of the failure path (no counterpart in the paper).  Every wait inside the kernels is
 * bounded: a wait that does not end sets the handle's status word and the CTA unwinds.  This call
 * makes that happen safely: it launches one tiny kernel that waits, for at most limit_us microseconds,
 * on a barrier that nothing ever signals and that no copy or tensor-core operation refers to, gives
 * up, and returns normally.  Afterwards ptq_linear_device_status(h) reports PTQ_ERR_TIMEOUT once and
 * PTQ_OK from then on, and the handle keeps working.
 *   limit_us   1 .. 100000
 *   result3    host, 3 words: what the short wait and a second, long wait on the same barrier
 *              returned (0 = gave up; the second leaves through the CTA-wide abort flag), and the
 *              nanoseconds the second one waited
 * Allocates 12 bytes of temporary device memory and synchronises the stream.
 */
ptq_status_t ptq_linear_selftest_wait_timeout(const ptq_linear_t *h, unsigned limit_us, unsigned *result3,
                                              void *stream);

/*
 * Write a one-line, human-readable description of the kernels and tilings chosen for this layer
 * (tile sizes, stage counts, whether PTQ_FLAG_FUSED_PROLOGUE has a kernel for it) into buf (at most
 * buf_bytes including the terminating NUL).  Returns the length the full text needs.
 */
int ptq_linear_describe(const ptq_linear_t *h, char *buf, int buf_bytes);

/* Number of kernels this library has launched in the calling process (all handles, all threads). */
unsigned long long ptq_kernel_launch_count(void);

const char *ptq_status_string(ptq_status_t st);
const char *ptq_last_error(void);   /* thread-local; valid until the next failing call on this thread */

#ifdef __cplusplus
}
#endif
#endif /* PTQ_LINEAR_H_ */
