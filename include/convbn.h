/*
 * convbn.h - C ABI of the B200 (sm_100a) Tune-mode Convolution-BatchNorm library.
 *
 * One ConvBN block (paper Sec. 3.1): a convolution with weight omega and optional bias b,
 * followed by a BatchNorm layer with FROZEN running statistics mu_hat / var_hat and affine
 * parameters gamma / beta.  Per output channel co:
 *
 *     r[co] = 1 / sqrt(var_hat[co] + eps)          s[co] = gamma[co] r[co]
 *     omega'[co,:] = s[co] omega[co,:]             b'[co] = (b[co] - mu_hat[co]) s[co] + beta[co]
 *
 * Conventions common to every entry point
 *   - The descriptor is read on the host.  EVERY OTHER POINTER IS A DEVICE POINTER (memory the
 *     current device can access) unless the argument is explicitly called "host".
 *   - The caller owns every buffer.  The library allocates no device memory, keeps no
 *     reference to a buffer after the call's kernels have run, and never writes the running
 *     statistics.  Work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = the
 *     default stream) and the call returns without synchronising.
 *   - Activations x / z / dz / dx / y have dtype `desc.dtype` and layout `desc.layout`:
 *         CONVBN_NCHW: [N][C][H][W]   weight: [C_out][C_in/G][kh][kw]
 *         CONVBN_NHWC: [N][H][W][C]   weight: [C_out][kh][kw][C_in/G]
 *     Weights passed in have the activation dtype.  b, gamma, beta, run_mean, run_var and
 *     every parameter gradient (dw in the weight's layout, db, dgamma, dbeta) are fp32.
 *     Supported pairs: (F32, NCHW) and (BF16, NHWC); others return CONVBN_EUNSUPPORTED.
 *   - Convolution hyper-parameters follow the usual deep-learning convention (the paper
 *     states only a kernel size): cross-correlation, zero padding, floor output size
 *     H_out = (H_in + 2 pad_h - dil_h (kh-1) - 1) / stride_h + 1, contiguous channel groups.
 *   - Activation and weight pointers must be 16-byte aligned, fp32 vectors 4-byte aligned.
 *   - `workspace` is scratch of at least convbn_workspace_bytes(desc, phase) bytes, 256-byte
 *     aligned; its contents are undefined after the call.  Calls that share a workspace must
 *     not overlap on the device.
 *   - Return value: a convbn_status.  Descriptor, pointer, alignment and workspace problems are
 *     found on the host before anything is launched.  A launch failure gives CONVBN_ECUDA.
 *     Device-side waits are bounded; one that expires sets a device error word which
 *     convbn_check() reports as CONVBN_ETIMEOUT.
 *   - Arithmetic: products of the storage type, fp32 accumulation, per-channel work in fp32,
 *     one rounding to the storage type when an activation is written.  Results are
 *     run-to-run deterministic (fixed reduction order, no floating-point atomics).
 */
#ifndef CONVBN_H_
#define CONVBN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CONVBN_OK = 0,
    CONVBN_EINVAL = 1,       /* bad descriptor or NULL pointer                      */
    CONVBN_EUNSUPPORTED = 2, /* dtype / layout pair not implemented                 */
    CONVBN_EWORKSPACE = 3,   /* workspace missing or too small                      */
    CONVBN_EALIGN = 4,       /* pointer not aligned as required                     */
    CONVBN_ECUDA = 5,        /* CUDA runtime / driver call failed                   */
    CONVBN_ETIMEOUT = 6,     /* a bounded device-side wait expired                  */
    CONVBN_ECAPACITY = 7     /* problem too large for the library's built-in scratch */
} convbn_status;

/* Storage type of x, w, z, dz, dx.  CONVBN_F16 (IEEE half; the paper's mixed-precision rows, Table 4: fp16 storage, fp32
 * accumulation, fp32 parameter gradients) is an NHWC storage type like CONVBN_BF16: every entry point that takes a
 * bf16 NHWC layer takes the same layer in half.  With CONVBN_NCHW it is refused: CONVBN_EUNSUPPORTED (the size
 * queries return 0). */
typedef enum { CONVBN_F32 = 0, CONVBN_BF16 = 1, CONVBN_F16 = 2 } convbn_dtype;
typedef enum { CONVBN_NCHW = 0, CONVBN_NHWC = 1 } convbn_layout;
typedef enum { CONVBN_MODE_TUNE = 0, CONVBN_MODE_EVAL = 1, CONVBN_MODE_DEPLOY = 2 } convbn_mode;

typedef enum {
    CONVBN_PHASE_TUNE_FWD = 0,
    CONVBN_PHASE_TUNE_BWD_DATA = 1,
    CONVBN_PHASE_TUNE_BWD_WEIGHT = 2,
    CONVBN_PHASE_EVAL_FWD = 3,
    CONVBN_PHASE_EVAL_BWD = 4,
    CONVBN_PHASE_DEPLOY_FWD = 5,
    CONVBN_PHASE_DEPLOY_BWD = 6,
    CONVBN_PHASE_TUNE_BWD = 7,
    CONVBN_PHASE_COUNT = 8
} convbn_phase;

/* Problem description (paper Sec. 3.1 and the shape annotations of Appendix C; stride, padding,
 * dilation and groups as in the convention above).  Plain data, read on the host.
 * Largest problems: X and Z at most 2^40 elements each, C_in / groups * kh * kw at most 2^30, padded input extents
 * (h_in + 2 pad_h, w_in + 2 pad_w) and filter spans (dil (k - 1)) at most 2^30; beyond that every entry point
 * returns CONVBN_EINVAL (the size queries 0). */
typedef struct convbn_desc {
    int n, c_in, h_in, w_in;   /* X is [N, C_in, H_in, W_in] logically                  */
    int c_out, kh, kw;         /* omega is [C_out, C_in/groups, kh, kw] logically        */
    int stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, groups;
    int dtype;                 /* convbn_dtype of activations and weights               */
    int layout;                /* convbn_layout                                         */
    double eps;                /* BatchNorm epsilon, added to the variance under the root */
} convbn_desc;

/* Output extent of the convolution (floor convention).  Host only.
 * CONVBN_EINVAL if the descriptor is inconsistent or the output would be empty. */
int convbn_out_shape(const convbn_desc *desc, int *h_out, int *w_out);

/* Linear-BN block (Sec. 3.2.2, last sentence: the associative law holds for a linear layer followed by
 * BatchNorm too): Y = X W^T + b on a [rows, in_features] matrix, W [out_features, in_features], BatchNorm over
 * the features.  That is the 1x1 block on `rows` images of one pixel, and in both supported layouts the
 * matrices already have the memory order the convolution entry points expect (X row-major [rows][in],
 * W row-major [out][in], Z [rows][out]).  Fills `desc` (host) so that every Tune / Eval / Deploy entry point
 * above serves the Linear-BN block; dtype CONVBN_BF16 selects the NHWC convention, CONVBN_F32 NCHW.
 * CONVBN_EINVAL for non-positive sizes or an unknown dtype. */
int convbn_linear_desc(int rows, int in_features, int out_features, int dtype, double eps, convbn_desc *desc);

/* Bytes of the opaque `saved` buffer that a forward call of `mode` (convbn_mode) writes for its
 * backward calls - the activation kept beside X (Sec. 3.3 / 3.4, Appendix M memory analysis):
 *   TUNE   : three fp32 vectors s, b', r (omega' is re-formed from omega in backward, it is
 *            never kept; no pre-normalisation tensor exists)
 *   EVAL   : the pre-normalisation output Y, N C_out H_out W_out elements of desc.dtype
 *   DEPLOY : 0
 * Returns 0 for an invalid descriptor. */
size_t convbn_saved_bytes(const convbn_desc *desc, int mode);

/* Scratch bytes a call of `phase` (convbn_phase) needs.  0 for an invalid descriptor/phase.
 * The split of the work over the SMs enters the size, so query it with the device that will run the
 * call current (with no device present the size for a 148-SM part is returned). */
size_t convbn_workspace_bytes(const convbn_desc *desc, int phase);

/* ---- Tune mode (Sec. 3.4; Table 2, Tune row) --------------------------------------------- */

/* Forward: forms s, b' and omega' from the CURRENT parameters at every call, then
 *     Z = omega' (*) X + b'.
 * in : x [activation], w [weight], b [C_out] or NULL (= no conv bias), gamma, beta, run_mean,
 *      run_var [C_out]
 * out: z [N, C_out, H_out, W_out]; saved (convbn_saved_bytes(desc, TUNE) bytes, 16-byte aligned) */
int convbn_tune_fwd(const convbn_desc *desc, const void *x, const void *w, const float *b,
                    const float *gamma, const float *beta, const float *run_mean,
                    const float *run_var, void *z, void *saved, void *workspace,
                    size_t workspace_bytes, void *stream);

/* Backward, data:  dX = omega'_rot (*) dZ  (the transposed convolution of dZ with omega').
 * in : dz, w (the same omega given to the forward), saved (from convbn_tune_fwd)
 * out: dx, same shape as x.  Every element of dx is written. */
int convbn_tune_bwd_data(const convbn_desc *desc, const void *dz, const void *w,
                         const void *saved, void *dx, void *workspace, size_t workspace_bytes,
                         void *stream);

/* Backward, parameters:
 *     domega' = dZ (.) X                      (cross-correlation over N, H_out, W_out)
 *     domega  = s domega'                     dbeta = sum dZ        db = s dbeta
 *     dgamma  = r ( sum_{ci,r,q} domega' omega + dbeta (b - mu_hat) )
 * in : dz, x, w, b (NULL iff the conv has no bias), run_mean, saved
 * out: dw [weight layout, fp32], db [C_out] (must be NULL iff b is NULL), dgamma, dbeta [C_out] */
int convbn_tune_bwd_weight(const convbn_desc *desc, const void *dz, const void *x,
                           const void *w, const float *b, const float *run_mean,
                           const void *saved, float *dw, float *db, float *dgamma,
                           float *dbeta, void *workspace, size_t workspace_bytes, void *stream);

/* Backward, both halves in one call (Table 2, Tune row; Sec. 3.2.1): dX and the parameter gradients exactly
 * as convbn_tune_bwd_data followed by convbn_tune_bwd_weight define them, same arguments, same outputs.
 * For the 1x1, stride-1 layers of a bottleneck (bf16 NHWC, one of C_in / C_out equal to 64 and the other
 * 128 or 256, at least 512 pixels) one kernel reads every dZ tile from memory ONCE and feeds both the
 * data-gradient and the weight-gradient GEMM from it (omega' = s omega is formed in shared memory and never
 * written); every other layer runs the two passes above SIDE BY SIDE: the parameter-gradient pass on a stream the library
 * owns (one per device and host thread, created on first use), forked from `stream` at the start of the call and joined
 * into it before the call returns, so the caller sees plain stream order (and a stream capture stays well-formed); each
 * pass has its own region of the workspace.  dx may not alias dz or x.
 * Workspace: convbn_workspace_bytes(desc, CONVBN_PHASE_TUNE_BWD). */
int convbn_tune_bwd(const convbn_desc *desc, const void *dz, const void *x, const void *w, const float *b,
                    const float *run_mean, const void *saved, void *dx, float *dw, float *db, float *dgamma,
                    float *dbeta, void *workspace, size_t workspace_bytes, void *stream);

/* Parameter gradients for callers that cannot allocate device memory (the paper has no counterpart
 * of this call; it exists for integration reasons only).
 *
 * convbn_tune_bwd_weight needs a scratch buffer for its partial sums, and somebody has to allocate
 * it.  Some users of this library cannot: code that runs where cudaMalloc is forbidden or would
 * stall the device (inside another framework's memory-pool callback, in a plug-in whose host owns
 * all device memory, in a real-time loop that must not touch the allocator).  For them this call
 * computes exactly what convbn_tune_bwd_weight computes, with the same kernels and the same
 * argument meaning, but takes no workspace: the scratch is a fixed 16 MiB array compiled into the
 * library (each GPU that loads the library holds those 16 MiB until the process ends).  The call
 * itself performs no cudaMalloc / cudaFree and calls no allocating routine.
 *
 *   - Limit: if convbn_workspace_bytes(desc, CONVBN_PHASE_TUNE_BWD_WEIGHT) exceeds 16 MiB
 *     (16 * 2^20 bytes) the call returns CONVBN_ECAPACITY and launches nothing.
 *   - The first call on each device looks up the array's device address (a runtime query, made with
 *     that device current).  Make that first call before starting any stream capture.
 *   - All calls share the one array.  It still holds the previous call's partial sums when a call
 *     starts; that is harmless, because every word the kernels read is first written by the same
 *     call, so nothing needs to be zeroed.  But two calls that overlap on the GPU (different
 *     streams, or different host threads without ordering) would overwrite each other's partial
 *     sums: callers must serialise them on the device. */
int convbn_tune_bwd_weight_noalloc(const convbn_desc *desc, const void *dz, const void *x,
                                   const void *w, const float *b, const float *run_mean,
                                   const void *saved, float *dw, float *db, float *dgamma,
                                   float *dbeta, void *stream);

/* ---- Eval mode comparator (Sec. 3.1; Table 2, Eval row) ---------------------------------- */

/* Y = omega (*) X + b is written to `y_saved` (the activation Eval mode keeps), then
 * Z = gamma (Y - mu_hat) r + beta.  y_saved: convbn_saved_bytes(desc, EVAL) bytes. */
int convbn_eval_fwd(const convbn_desc *desc, const void *x, const void *w, const float *b,
                    const float *gamma, const float *beta, const float *run_mean,
                    const float *run_var, void *z, void *y_saved, void *workspace,
                    size_t workspace_bytes, void *stream);

/* dY = s dZ; dX = omega_rot (*) dY; domega = dY (.) X; db = sum dY;
 * dgamma = sum dZ (Y - mu_hat) r; dbeta = sum dZ.   db may be NULL. */
int convbn_eval_bwd(const convbn_desc *desc, const void *dz, const void *x, const void *y_saved,
                    const void *w, const float *gamma, const float *run_mean,
                    const float *run_var, void *dx, float *dw, float *db, float *dgamma,
                    float *dbeta, void *workspace, size_t workspace_bytes, void *stream);

/* ---- Deploy mode comparator (Sec. 3.3; Table 2, Deploy row; Appendix C) -------------------- */

/* Once for all: w_fused = omega' (weight dtype and layout), b_fused = b' (fp32). */
int convbn_deploy_prepare(const convbn_desc *desc, const void *w, const float *b,
                          const float *gamma, const float *beta, const float *run_mean,
                          const float *run_var, void *w_fused, float *b_fused, void *stream);

/* Z = omega' (*) X + b' */
int convbn_deploy_fwd(const convbn_desc *desc, const void *x, const void *w_fused,
                      const float *b_fused, void *z, void *workspace, size_t workspace_bytes,
                      void *stream);

/* dX = omega'_rot (*) dZ; domega' = dZ (.) X; db' = sum dZ.  Gradients go to the FUSED
 * parameters only (which is what makes this mode unstable for training, Sec. 3.3). */
int convbn_deploy_bwd(const convbn_desc *desc, const void *dz, const void *x,
                      const void *w_fused, void *dx, float *dw_fused, float *db_fused,
                      void *workspace, size_t workspace_bytes, void *stream);

/* ---- one Tune-mode training step from HOST buffers ------------------------------------------- */

/* Device bytes convbn_tune_step_host needs in `device_arena`.  0 for an invalid descriptor. */
size_t convbn_host_step_arena_bytes(const convbn_desc *desc);

/* Forward, backward-data and backward-weight of one block (the three Tune-row calls above, Sec. 3.4
 * and Table 2) with every tensor in HOST memory: x, dz, w, b (NULL = no bias), gamma, beta,
 * run_mean, run_var are host inputs; z, dx, dw, db (NULL iff b is NULL), dgamma, dbeta are host
 * outputs, in the dtype / layout conventions above.  Copies are asynchronous (use page-locked host
 * memory for them to overlap).  The inputs go up on one library-owned stream, the results come down on another (one
 * pair per device and host thread, created on the first call there) and the kernels run on `stream` in between, each
 * step ordered behind what it needs: the uploads behind everything queued earlier on `stream`, the forward kernels
 * behind X and the parameters, the backward kernels behind dZ (which crosses the bus while Z comes back), the
 * downloads behind the kernels that produce them; finally `stream` waits for the last download.  Outputs are valid,
 * and the host inputs may be reused, once `stream` has been synchronised.  `device_arena` is caller-owned DEVICE
 * scratch of at least convbn_host_step_arena_bytes(desc) bytes, 256-byte aligned.
 *
 * convbn_tune_step_host_begin is the same call without that last wait: the next call's uploads (into ANOTHER arena)
 * then cross the bus while this call's results come down.  Host buffers, outputs and the arena belong to the library
 * until convbn_tune_step_host_join(stream) has made `stream` wait for every download begun by the calling host thread
 * on the current device; a later call that reuses an arena waits for the earlier call's downloads by itself. */
int convbn_tune_step_host(const convbn_desc *desc, const void *x, const void *dz, const void *w,
                          const float *b, const float *gamma, const float *beta,
                          const float *run_mean, const float *run_var, void *z, void *dx, float *dw,
                          float *db, float *dgamma, float *dbeta, void *device_arena,
                          size_t arena_bytes, void *stream);
int convbn_tune_step_host_begin(const convbn_desc *desc, const void *x, const void *dz, const void *w,
                                const float *b, const float *gamma, const float *beta,
                                const float *run_mean, const float *run_var, void *z, void *dx, float *dw,
                                float *db, float *dgamma, float *dbeta, void *device_arena,
                                size_t arena_bytes, void *stream);
int convbn_tune_step_host_join(void *stream);

/* Backward with the parameter gradients off the critical path (what a training step wants: dX feeds the layer below at
 * once, domega, db, dgamma, dbeta are needed by the optimiser only).  convbn_tune_bwd_begin takes the arguments of
 * convbn_tune_bwd and computes the same values, but returns with the parameter-gradient pass (the weight-gradient GEMM
 * and its epilogue, or for the single-kernel 1x1 path the epilogue alone) still running on the library's side stream:
 * when work queued on `stream` after the call runs, dx is complete, while dw, db, dgamma, dbeta and the workspace belong
 * to the library until convbn_tune_bwd_join(stream) has been called and the work it queues on `stream` has been reached.
 * convbn_tune_bwd_join makes `stream` wait for every pass begun by the calling host thread on the current device; it is
 * cheap, may be called with nothing pending, and must be called before a stream capture that contains begin calls ends.
 * Errors as for convbn_tune_bwd. */
int convbn_tune_bwd_begin(const convbn_desc *desc, const void *dz, const void *x, const void *w, const float *b,
                          const float *run_mean, const void *saved, void *dx, float *dw, float *db, float *dgamma,
                          float *dbeta, void *workspace, size_t workspace_bytes, void *stream);
int convbn_tune_bwd_join(void *stream);

/* ---- TransposedConv-BN in Tune mode (Sec. 3.2.2: the rewrite holds for any linear layer in front of a frozen BatchNorm;
 *      Sec. 3.3 definitions; Table 2, Tune row, with the transposed convolution in place of the convolution) ------------
 *
 * `desc` describes the TRANSPOSED convolution in its own terms: input [n][c_in][h_in][w_in] (logical), output
 * [n][c_out][h_out][w_out] with h_out = (h_in - 1) stride_h - 2 pad_h + dil_h (kh - 1) + 1 (no output padding), input pixel
 * (hi, wi) adding x[ci] w[ci][co][r][q] to output pixel (hi stride_h - pad_h + r dil_h, wi stride_w - pad_w + q dil_w).
 * Weights: NHWC descriptors [c_in][kh][kw][c_out/groups], NCHW descriptors [c_in][c_out/groups][kh][kw] (the layout of
 * the convolution this layer transposes, whose c_out is this c_in).  BatchNorm vectors, `saved` ([s | b' | r],
 * 3 c_out floats) and parameter gradients as in the convolution calls; dw has the layout of w, fp32.
 *   Z  = convT(X, s w) + b'                      convbn_tconv_tune_fwd  (writes z and saved)
 *   dX, dw = s dw', db = s dbeta, dgamma = r (sum dw' w + dbeta (b - mu_hat)), dbeta = sum dZ
 *                                                convbn_tconv_tune_bwd  (b and db both NULL or both non-NULL)
 * The transposed convolution runs on the kernels of the convolution it transposes (forward = that layer's backward data,
 * input gradient = its forward, weight gradient = its weight gradient with the two tensors exchanged); the scale, the bias
 * and the per-channel sums are separate small kernels.  One workspace size serves both calls.  Pointers: device, 16-byte
 * aligned (vectors 4), workspace 256.  Errors as for the convolution calls; nothing is launched after an error. */
int convbn_tconv_out_shape(const convbn_desc *desc, int *h_out, int *w_out);
size_t convbn_tconv_workspace_bytes(const convbn_desc *desc);
int convbn_tconv_tune_fwd(const convbn_desc *desc, const void *x, const void *w, const float *b, const float *gamma,
                          const float *beta, const float *run_mean, const float *run_var, void *z, void *saved,
                          void *workspace, size_t workspace_bytes, void *stream);
int convbn_tconv_tune_bwd(const convbn_desc *desc, const void *dz, const void *x, const void *w, const float *b,
                          const float *run_mean, const void *saved, void *dx, float *dw, float *db, float *dgamma,
                          float *dbeta, void *workspace, size_t workspace_bytes, void *stream);

/* ---- glue between blocks (Sec. 3.1: what surrounds a ConvBN block stays as it is) ------ */

/* Elementwise operations a residual network places between its ConvBN blocks, on `count` elements of `dtype`
 * (convbn_dtype), all pointers device, 16-byte aligned; `out` may alias `a` (in place) or `b`.
 *   convbn_relu          out = max(a, 0)
 *   convbn_add_relu      out = max(a + b, 0)                    (the end of a residual block)
 *   convbn_relu_bwd      out = a where y > 0, else 0            (a: gradient of the ReLU output y)
 *   convbn_add           out = a + b                            (gradients meeting at a fork)
 * A count of 0 is a no-op that looks at no pointer.  CONVBN_EINVAL for a negative count, an unknown dtype or (count > 0)
 * a NULL pointer; CONVBN_EALIGN; CONVBN_ECUDA. */
int convbn_relu(int dtype, const void *a, void *out, long long count, void *stream);
int convbn_add_relu(int dtype, const void *a, const void *b, void *out, long long count, void *stream);
int convbn_relu_bwd(int dtype, const void *a, const void *y, void *out, long long count, void *stream);
int convbn_add(int dtype, const void *a, const void *b, void *out, long long count, void *stream);

/* ---- measurement aid (the paper has no counterpart) ------------------------------------------ */

/* After convbn_profile_begin(), every kernel this library launches (from any thread) is bracketed
 * by a pair of CUDA events on its stream.  convbn_profile_end() stops that, synchronises the
 * device and writes one line per kernel family into `report` (host buffer, NUL-terminated,
 * truncated to report_bytes): "<name> <launches> <total milliseconds>\n", where <name> is
 * "<kernel family>@<shape key of the layer>#<phase of the call>".  At most 65536
 * launches are recorded between begin and end; later ones run unrecorded. */
int convbn_profile_begin(void);
int convbn_profile_end(char *report, size_t report_bytes);

/* ---- housekeeping -------------------------------------------------------------------------- */

/* Synchronises `stream`, then reads and clears the device error word of the current device.
 * CONVBN_OK, CONVBN_ETIMEOUT (a bounded wait in a kernel gave up; outputs of that call are
 * invalid) or CONVBN_ECUDA (the stream reported an error). */
int convbn_check(void *stream);

/* Self-test of the failure path (the paper has no counterpart): launches one block whose single bounded wait
 * - the same mbarrier wait the tensor-core kernels use, with a limit of about 100 microseconds - is on a
 * barrier that nobody arrives at.  The wait gives up, the kernel sets the device error word and returns
 * normally; nothing faults and the context stays usable.  The next convbn_check(stream) therefore reports
 * CONVBN_ETIMEOUT (and clears the word).  No copy or tensor-memory operation is in flight at any time. */
int convbn_selftest_wait_timeout(void *stream);

/* Static, NUL-terminated description of a status code. */
const char *convbn_status_string(int status);

/* Name of the kernel family the last call of `phase` selected on this thread, for logs and tests:
 * "direct", "umma", "umma-strip", "umma-strided", "umma-subpixel", "umma-stem", "stem-mma", "depthwise",
 * "grouped-mma", "grouped-umma", and for CONVBN_PHASE_TUNE_BWD "umma-fused-bwd" or "two-calls".
 * Static string, never NULL. */
const char *convbn_last_kernel(int phase);

#ifdef __cplusplus
}
#endif
#endif /* CONVBN_H_ */
