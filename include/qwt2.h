/*
 * qwt2.h -- C ABI of libqwt2: CWAC-fused quantized linear layer and CWAC calibration
 *           (QwT-v2, "channel-wise affine compensation") for NVIDIA B200 (sm_100a).
 *
 * General rules
 *   - Plain C.  No exceptions, no abort, nothing is printed.  Every call returns qwt_status.
 *   - Unless a parameter is marked HOST, every data pointer is a CUDA DEVICE pointer owned by the
 *     caller.  The library never frees caller memory and (except the *_host calls) never allocates
 *     device memory and never synchronises: work is enqueued on `stream` (a cudaStream_t passed as
 *     void*, NULL = the legacy default stream) and outputs are valid once that stream reaches the
 *     end of the call.
 *   - Matrices are row-major with the last index contiguous.
 *   - Argument errors are found on the host before anything is launched.
 *   - Inputs are assumed finite; NaN/Inf behaviour is unspecified.  Outputs must not alias inputs.
 *   - Calls may run concurrently on different streams if their workspaces are distinct.
 *   - Grids, workspace layouts and summation orders are functions of the problem shape only and are laid out for
 *     the 148 SMs of a B200; a call on a device with fewer SMs than its persistent grid returns QWT_ERR_ARCH.
 */
#ifndef QWT2_H_
#define QWT2_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t qwt_status;
enum {
  QWT_OK = 0,
  QWT_ERR_NULL = 1,        /* a required pointer is NULL */
  QWT_ERR_SHAPE = 2,       /* non-positive or overflowing dimension */
  QWT_ERR_ALIGN = 3,       /* base pointer or leading dimension not aligned as required */
  QWT_ERR_UNSUPPORTED = 4, /* dimension not a required multiple, unknown enum value */
  QWT_ERR_WORKSPACE = 5,   /* workspace too small */
  QWT_ERR_CUDA = 6,        /* a CUDA runtime/driver call failed; see qwt_last_cuda_error */
  QWT_ERR_TIMEOUT = 7,     /* a bounded device-side wait gave up (reported by qwt_qlinear_check_status) */
  QWT_ERR_ARCH = 8,        /* current device is not compute capability 10.x */
  QWT_ERR_TOO_LARGE = 9    /* problem exceeds the fixed scratch of qwt_cwac_calibrate_noalloc */
};

/* weight storage */
enum { QWT_W_INT8 = 0,         /* [N, K] int8 codes in [-127, 127] */
       QWT_W_INT4_PACKED = 1   /* [N, K/2] bytes, two's-complement nibbles, element 2j low, 2j+1 high */ };

/* output stage of the forward call */
enum { QWT_OUT_INT8_PER_TOKEN = 0, /* int8 codes [M, N] + float y_scale[M] (dynamic per-token absmax) */
       QWT_OUT_BF16 = 1,           /* bfloat16 [M, N], round to nearest even */
       QWT_OUT_FP32 = 2,           /* float [M, N]: the compensated real-valued output z */
       QWT_OUT_INT32_ACC = 3,      /* int32 [M, N]: raw integer accumulators (verification) */
       QWT_OUT_INT8_STATIC = 4     /* int8 codes [M, N] with STATIC scales: Eq. 10 as printed (see qwt_cwac_fold_static) */ };

const char* qwt_version(void);
const char* qwt_status_string(qwt_status s);
/* CUDA error code of the most recent QWT_ERR_CUDA on the calling thread (0 if none). */
qwt_status qwt_last_cuda_error(int* cuda_err /*HOST out*/);

/* ---------------------------------------------------------------------------------------------
 * CWAC calibration -- Section 3.3, Eq. 3-5.
 * For every output channel c the least-squares line through the calibration pairs
 *     (q_out[r, c], fp_out[r, c]),  r = 0..rows-1:
 *     a[c] = Cov(fp_out[:,c], q_out[:,c]) / Var(q_out[:,c]),   b[c] = E[fp_out[:,c]] - a[c] E[q_out[:,c]].
 * fp_out is the full-precision module output Y_full, q_out the quantized module's output Y_quant
 * on the same calibration tokens.
 *
 * The kernels make ONE pass over the two matrices and reduce them to five numbers per channel,
 * stats = double[5 * channels] laid out as [n | sum q | sum f | sum q*f | sum q*q] (each `channels`
 * long).  Eq. 4-5 are functions of exactly these, so calibration can be streamed batch by batch
 * (qwt_cwac_stats_accumulate per batch, qwt_cwac_solve at the end) or done in one call
 * (qwt_cwac_calibrate = zero stats in workspace + accumulate + solve).
 *
 * Degenerate channel (Var(q) <= 1e-12 * E[q^2], e.g. a constant column or rows == 1): every
 * (a, b = E[f] - a E[q]) minimises Eq. 3; a = 1 is returned.
 *
 *   fp_out, q_out : float [rows, ld], ld >= channels, ld % 4 == 0, base 16-byte aligned
 *   a, b          : float [channels] out
 *   n_degenerate  : int32 out (single value), may be NULL
 *   workspace     : >= qwt_cwac_workspace_bytes(rows, channels) bytes, 256-byte aligned
 * Errors: NULL, SHAPE (rows < 1, channels < 1, ld < channels), ALIGN, WORKSPACE, ARCH, CUDA.
 * Results are bitwise reproducible for fixed (rows, channels, ld).
 */
size_t qwt_cwac_workspace_bytes(int64_t rows, int32_t channels);
qwt_status qwt_cwac_calibrate(const float* fp_out, const float* q_out, int64_t rows, int32_t channels,
                              int64_t ld, float* a, float* b, int32_t* n_degenerate,
                              void* workspace, size_t workspace_bytes, void* stream);
/* stats += statistics of this batch.  The caller zeroes stats (5*channels doubles) before the first batch. */
qwt_status qwt_cwac_stats_accumulate(const float* fp_out, const float* q_out, int64_t rows, int32_t channels,
                                     int64_t ld, double* stats, void* workspace, size_t workspace_bytes,
                                     void* stream);
/* Closed form of Eq. 4-5 from the statistics (float64 arithmetic, float32 results). */
qwt_status qwt_cwac_solve(const double* stats, int32_t channels, float* a, float* b, int32_t* n_degenerate,
                          void* stream);
/* Calibration with HOST matrices: fp_out/q_out are host pointers (pinned memory recommended); they are
 * streamed to the device in row chunks through `staging` (device, >= qwt_cwac_host_staging_bytes) while
 * earlier chunks are reduced.  a, b, n_degenerate are HOST outputs, valid on return (the call waits). */
size_t qwt_cwac_host_staging_bytes(int64_t rows, int32_t channels);
qwt_status qwt_cwac_calibrate_host(const float* fp_out /*HOST*/, const float* q_out /*HOST*/, int64_t rows,
                                   int32_t channels, int64_t ld, float* a /*HOST*/, float* b /*HOST*/,
                                   int32_t* n_degenerate /*HOST, may be NULL*/,
                                   void* staging, size_t staging_bytes, void* stream);

/* Calibration of several layers in one call (the layers of a model on one calibration set): one statistics launch
 * and one reduce / solve launch for all of them, instead of two (three with the fold) per layer.  Every problem is
 * cut and summed exactly as its own qwt_cwac_calibrate call would cut and sum it, so the results are bit for bit
 * the same; what goes away is a launch, a ramp and a tail per layer.
 *   problems : HOST array of `count` descriptors (read during the call only); the pointers inside are DEVICE
 *              pointers with the meaning and alignment of qwt_cwac_calibrate / qwt_cwac_fold.  w_scale != NULL
 *              asks for the fold of that layer as well: fscale = a * w_scale, fbias = a * bias + b (bias may be NULL).
 *   n_degenerate : DEVICE int32, total over all problems, may be NULL
 *   workspace    : device, 256-byte aligned, >= qwt_cwac_calibrate_batch_workspace_bytes(problems, count) */
typedef struct qwt_calib_problem {
  const float* fp_out;
  const float* q_out;
  int64_t rows;
  int64_t ld;
  int32_t channels;
  float* a;
  float* b;
  const float* w_scale;
  const float* bias;
  float* fscale;
  float* fbias;
} qwt_calib_problem;
size_t qwt_cwac_calibrate_batch_workspace_bytes(const qwt_calib_problem* problems /*HOST*/, int32_t count);
qwt_status qwt_cwac_calibrate_batch(const qwt_calib_problem* problems /*HOST*/, int32_t count,
                                    int32_t* n_degenerate, void* workspace, size_t workspace_bytes, void* stream);

/* Calibration without any workspace argument (the paper has no counterpart: this is a packaging variant of
 * qwt_cwac_calibrate, same kernels, same results within the library's calibration tolerance).
 * For callers that cannot allocate device memory -- e.g. a plug-in confined to a host program's fixed
 * memory arena, or a service that must not call cudaMalloc while it is serving.  The per-chunk partial sums
 * live in a fixed array of QWT_NOALLOC_SCRATCH_BYTES inside the library image; every GPU that loads the
 * library holds that array until the process exits.  The call itself allocates nothing.
 *   - Limit: channels (rounded up to 128) * 48 bytes must fit the array, i.e. at most 131072 channels;
 *     otherwise QWT_ERR_TOO_LARGE.  Long inputs are cut into fewer, longer row chunks so that they fit.
 *   - The first call on each device looks up the array's device address (with that device current); make
 *     that first call before any stream capture is started.
 *   - The address is kept per device ordinal for the life of the process.  It belongs to the device's primary
 *     context as it was at that first call: after cudaDeviceReset, or under another (non-primary) context on the same
 *     device, it is stale and the entry point must not be used in that process any more.
 *   - All calls share the one array.  Nothing in it has to be cleared between calls (each call overwrites
 *     what it reads), but two calls that overlap on the GPU -- different streams, or different host threads
 *     -- race on it: serialise them, or use qwt_cwac_calibrate with separate workspaces.
 * Arguments and other errors as for qwt_cwac_calibrate. */
#define QWT_NOALLOC_SCRATCH_BYTES (6u << 20)
qwt_status qwt_cwac_calibrate_noalloc(const float* fp_out, const float* q_out, int64_t rows, int32_t channels,
                                      int64_t ld, float* a, float* b, int32_t* n_degenerate, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Fold -- Section 3.4, Eq. 9-11.  CWAC is absorbed into the layer's requantization parameters:
 * alpha joins the multiplier (Eq. 11, M' = alpha S_x S_W / S_r), beta joins the additive term.
 * With per-token S_x and S_r that are only known at run time the static parts are
 *     fscale[n] = a[n] * w_scale[n],     fbias[n] = a[n] * bias[n] + b[n]
 * (CWAC acts on the module output, which includes the layer bias).
 *   w_scale [n] float (S_W); bias [n] float or NULL (= 0); a, b [n] float or both NULL (= 1, 0)
 *   fscale, fbias [n] float out.
 * Errors: NULL (w_scale, fscale, fbias; or exactly one of a, b), SHAPE (n < 1), ARCH, CUDA.
 */
qwt_status qwt_cwac_fold(const float* w_scale, const float* bias, const float* a, const float* b, int32_t n,
                         float* fscale, float* fbias, void* stream);

/* Fold for an engine with STATIC per-tensor scales -- Section 3.4, Eq. 10-11 exactly as printed (zero-points 0):
 *     mult[n]   = a[n] * S_x * w_scale[n] / S_r                               (the multiplier M' of Eq. 11)
 *     offset[n] = rne((a[n] * bias[n] + b[n]) / (a[n] * S_x * w_scale[n]))    (the rounded term of Eq. 10, INT32;
 *                 the layer bias rides with beta because CWAC acts on the module output)
 * computed in float64 on the device.  A channel whose a * S_x * w_scale is 0 gets offset 0.
 * The forward call with QWT_OUT_INT8_STATIC then produces
 *     Y[m, n] = clip(rne(mult[n] * (acc[m, n] + offset[n])), -127, 127)
 * (the sum in exact integer arithmetic, the product in FP32), i.e. S_r * Y approximates the compensated output
 * with beta off by at most half an accumulator step, |a S_x w_scale| / 2 (Section 3.4).
 *   S_x, S_r > 0: static activation / output scales; bias [n] or NULL; a, b [n] or both NULL (= 1, 0)
 *   mult float [n] out, offset int32 [n] out.
 * Errors: NULL, SHAPE (n < 1, S_x <= 0, S_r <= 0), ARCH, CUDA. */
qwt_status qwt_cwac_fold_static(const float* w_scale, const float* bias, const float* a, const float* b, int32_t n,
                                float S_x, float S_r, float* mult, int32_t* offset, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Forward -- Section 3.4, Eq. 6-11 with all zero-points 0 (symmetric codes).
 *     acc[m, n] = sum_k X[m, k] * W[n, k]                       (int8 x int8 -> int32, exact; the W_q x_q of Eq. 7)
 *     z[m, n]   = fma((float)acc[m, n] * x_scale[m], fscale[n], fbias[n])      (Eq. 9 after the fold)
 *   QWT_OUT_INT8_PER_TOKEN: y_scale[m] = max_n |z[m, n]| / 127;  Y[m, n] = clip(rne(z / y_scale[m]), -127, 127)
 *                           (Eq. 1-2 applied to the output with zero-point 0: the 1/S_r of Eq. 10-11, per token);
 *                           a row of zeros gives y_scale 0 and codes 0.  The kernel rounds z * (1 / y_scale[m])
 *                           (FP32 reciprocal, one fused multiply-add), which differs from the FP32 quotient by
 *                           one step in about one code per million.
 *   QWT_OUT_BF16 / FP32   : Y = z rounded to bfloat16 / as is.       QWT_OUT_INT32_ACC: Y = acc.
 *   QWT_OUT_INT8_STATIC   : Y[m, n] = clip(rne(fscale[n] * (acc[m, n] + offset[n])), -127, 127) with fscale = mult and
 *                           fbias = the INT32 offset array of qwt_cwac_fold_static passed through the same pointer
 *                           (reinterpreted); x_scale and y_scale are not used (NULL).  No workspace traffic.
 *
 *   X [M, K] int8; x_scale [M] float (may be NULL for INT32_ACC)
 *   W [N, K] int8, or [N, K/2] packed int4 (expanded to int8 on chip: tile by tile, or once per CTA where the layer
 *     runs on CTA pairs that keep their W halves in shared memory; otherwise, with 1024 rows or more, once per call
 *     into the workspace, which qwt_qlinear_workspace_bytes sizes for it)
 *   fscale, fbias [N] float (may be NULL for INT32_ACC)
 *   Y [M, N] of the output type; y_scale [M] float out, INT8 mode only (else NULL)
 *   K % 16 == 0 (int8) or K % 32 == 0 (packed int4); X, W, Y bases 16-byte aligned;
 *   N % 16 == 0 (int8 out), N % 8 == 0 (bf16), N % 4 == 0 (fp32 / int32).
 *   workspace >= qwt_qlinear_workspace_bytes(...), 256-byte aligned; its content is scratch
 *   (a status word, per-row maxima, per-strip counters) that the call re-initialises itself.
 * Errors: NULL, SHAPE, ALIGN, UNSUPPORTED, WORKSPACE, ARCH, CUDA.  Device-side waits are bounded; if one
 * gives up the kernel records it in the workspace status word and exits; qwt_qlinear_check_status
 * reports that as QWT_ERR_TIMEOUT.
 */
size_t qwt_qlinear_workspace_bytes(int32_t M, int32_t N, int32_t K, int32_t wfmt, int32_t out_mode);
qwt_status qwt_qlinear_cwac_forward(const int8_t* X, const float* x_scale, const void* W, int32_t wfmt,
                                    const float* fscale, const float* fbias, int32_t M, int32_t N, int32_t K,
                                    int32_t out_mode, void* Y, float* y_scale,
                                    void* workspace, size_t workspace_bytes, void* stream);
/* Waits for `stream`, then reads the status word of a forward workspace.  QWT_OK or QWT_ERR_TIMEOUT.
 * device_status (HOST out, may be NULL) receives the raw word (0 = clean). */
qwt_status qwt_qlinear_check_status(const void* workspace, void* stream, int32_t* device_status);
/* Forward with HOST activations: X, x_scale are host inputs, Y, y_scale host outputs (pinned memory
 * recommended); W, fscale, fbias stay DEVICE resident (they are model parameters).  `staging` is device
 * scratch >= qwt_qlinear_host_staging_bytes(...).  The call copies in, runs the same kernel, copies out
 * and waits for the stream, so the outputs are valid on return.  More than 4096 rows are cut into row chunks
 * (exact: a row's scale needs that row only) that alternate over two helper streams of the library, ordered after
 * the work already queued on `stream`, so that the copy-in of a chunk, the kernel of the one before and the
 * copy-out of the one before that overlap; the streams and events are created on the thread's first such call
 * on a device and kept. */
size_t qwt_qlinear_host_staging_bytes(int32_t M, int32_t N, int32_t K, int32_t wfmt, int32_t out_mode);
qwt_status qwt_qlinear_cwac_forward_host(const int8_t* X /*HOST*/, const float* x_scale /*HOST*/, const void* W,
                                         int32_t wfmt, const float* fscale, const float* fbias, int32_t M,
                                         int32_t N, int32_t K, int32_t out_mode, void* Y /*HOST*/,
                                         float* y_scale /*HOST*/, void* staging, size_t staging_bytes,
                                         void* stream);

/* ---------------------------------------------------------------------------------------------
 * Calibration fused into the layer (Section 3.3 applied to the layer of Eq. 6-8, in one pass):
 * the quantized layer runs on the calibration rows and, instead of writing its output
 *     q[m, n] = S_x[m] S_W[n] acc[m, n] + bias[n]              (the layer before compensation, FP32)
 * the kernel reads the stored full-precision output fp_out[m, n] of the same rows and accumulates the
 * per-channel sums of Eq. 4-5 in its epilogue; q never exists in memory.  Results equal
 * qwt_qlinear_cwac_forward(QWT_OUT_FP32, fscale = w_scale, fbias = bias) followed by qwt_cwac_calibrate
 * within the calibration tolerance (same q values, different but fixed summation order: strips of 128 rows,
 * then the strips in order; results are bitwise reproducible).
 *   X, x_scale, W, w_format : as for qwt_qlinear_cwac_forward (x_scale required)
 *   w_scale  float [N]      : S_W;   bias float [N] or NULL (= 0)
 *   fp_out   float [M, ld]  : 16-byte aligned, ld >= N, ld % 4 == 0;   N % 4 == 0
 *   stats    float64 [5 * N] or NULL: running statistics, updated in place (layout of qwt_cwac_stats_accumulate)
 *   a, b     float [N] or both NULL : solved from (stats + this call) when given; one of stats / (a, b) is required
 *   n_degenerate            : as for qwt_cwac_calibrate, may be NULL
 *   workspace               : device, 256-byte aligned, >= qwt_qlinear_cwac_calibrate_workspace_bytes; its first
 *                             word is the status word of qwt_qlinear_check_status
 */
size_t qwt_qlinear_cwac_calibrate_workspace_bytes(int32_t M, int32_t N, int32_t K, int32_t w_format);
qwt_status qwt_qlinear_cwac_calibrate(const int8_t* X, const float* x_scale, const void* W, int32_t w_format,
                                      const float* w_scale, const float* bias, const float* fp_out, int64_t ld,
                                      int32_t M, int32_t N, int32_t K, double* stats, float* a, float* b,
                                      int32_t* n_degenerate, void* workspace, size_t workspace_bytes,
                                      void* stream);

/* ---------------------------------------------------------------------------------------------
 * Support: symmetric row-wise quantizer -- Eq. 1-2 with zero-point 0 and signed codes.
 *     scale[r] = max_c |X[r, c]| / qmax;   Xq[r, c] = clip(rne(X[r, c] / scale[r]), -qmax, qmax)
 * Per-token activations: X = activations, qmax = 127.  Per-channel weights: X = W [N, K], qmax = 127 or 7.
 *   X float [rows, ld] (ld >= cols); Xq int8 [rows, cols]; scale float [rows].  A zero row gives scale 0, codes 0.
 * qwt_pack_int4: codes int8 [rows, cols] in [-8, 7], cols even -> packed [rows, cols/2].
 */
qwt_status qwt_quantize_rows_i8(const float* X, int64_t rows, int32_t cols, int64_t ld, int32_t qmax,
                                int8_t* Xq, float* scale, void* stream);
qwt_status qwt_pack_int4(const int8_t* codes, int64_t rows, int32_t cols, uint8_t* packed, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Asymmetric (unsigned) codes -- Eq. 1-2 and Eq. 6-7 as printed, with non-zero zero-points:
 *     acc[m, n] = sum_k (W_q[n, k] - Z_W[n]) (x_q[m, k] - Z_x[m])
 *               = sum_k W_q x_q  -  Z_W[n] sum_k x_q[m, k]  -  Z_x[m] sum_k W_q[n, k]  +  K Z_x[m] Z_W[n]      (Eq. 7)
 * (codes in [0, 255]; Z_x per token -- pass the same value for every token for the paper's per-tensor activation
 * zero-point -- and Z_W per output channel).  The unsigned product runs on the tensor cores, the three zero-point
 * terms are added in the epilogue in exact integer arithmetic; everything after that (x_scale, fscale, fbias, the
 * output stages) is as in qwt_qlinear_cwac_forward.
 *
 * qwt_quantize_rows_u8   Eq. 1-2 per row: scale[r] = (max - min) / 255 (1 for a constant row),
 *                        zero[r] = clip(rne(-min / scale), 0, 255), Xq = clip(rne(x / scale) + zero, 0, 255);
 *                        rowsum[r] = sum_c Xq[r, c] (may be NULL).  Rows = tokens for activations, output
 *                        channels for weights.
 * qwt_asym_weight_terms  w_terms int32 [2 N]: w_terms[n] = -Z_W[n], w_terms[N + n] = K Z_W[n] - sum_k W_q[n, k];
 *                        computed once per layer.
 * qwt_qlinear_cwac_forward_asym   X uint8 [M, K], x_zero / x_rowsum int32 [M], W uint8 [N, K] (no packed int4),
 *                        out_mode any but QWT_OUT_INT8_STATIC; K <= 33000; other arguments, workspace and errors as
 *                        for qwt_qlinear_cwac_forward.
 */
qwt_status qwt_quantize_rows_u8(const float* X, int64_t rows, int32_t cols, int64_t ld, uint8_t* Xq, float* scale,
                                int32_t* zero, int32_t* rowsum, void* stream);
qwt_status qwt_asym_weight_terms(const uint8_t* W, const int32_t* w_zero, int32_t N, int32_t K, int32_t* w_terms,
                                 void* stream);
qwt_status qwt_qlinear_cwac_forward_asym(const uint8_t* X, const float* x_scale, const int32_t* x_zero,
                                         const int32_t* x_rowsum, const uint8_t* W, const int32_t* w_terms,
                                         const float* fscale, const float* fbias, int32_t M, int32_t N, int32_t K,
                                         int32_t out_mode, void* Y, float* y_scale, void* workspace,
                                         size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Convolutions (the paper places CWAC after every quantized convolution too, Section 3.3).  In NHWC layout a 1x1
 * convolution is qwt_qlinear_cwac_forward itself with M = batch*H*W, K = C_in, N = C_out.  For a kh x kw
 * convolution qwt_im2col_i8 writes the patch matrix
 *     patches[(b, ho, wo), (i, j, c)] = X[b, ho*stride + i - pad, wo*stride + j - pad, c]   (0 outside the image)
 * of shape [batch*Ho*Wo, kh*kw*C] (Ho = (H + 2 pad - kh) / stride + 1, likewise Wo), after which the convolution is
 * the same forward call with K = kh*kw*C and the weights laid out [C_out, kh, kw, C_in].  The per-token scale of
 * the layer's input belongs to the pixel the patch is centred on only if the scale is per tensor: use one
 * x_scale value for all rows (the paper's per-tensor activation scale).  Symmetric codes (zero-point 0).
 *   X int8 [batch, H, W, C], C % 16 == 0, 16-byte aligned; patches int8, 16-byte aligned.
 * Errors: NULL, SHAPE, UNSUPPORTED (C % 16), ALIGN, ARCH, CUDA. */
qwt_status qwt_im2col_i8(const int8_t* X, int32_t batch, int32_t H, int32_t W, int32_t C, int32_t kh, int32_t kw,
                         int32_t stride, int32_t pad, int8_t* patches, void* stream);

/* Convolution without the patch matrix (the same layer as an implicit GEMM): the kernel of qwt_qlinear_cwac_forward
 * reads the activations straight from the NHWC tensor -- a tile's A operand is, per filter tap and block of 128 input
 * channels, a block of input pixels fetched by one rank-4 tensor-map copy (every `stride`-th position; positions outside
 * the image read 0, the zero-point of the symmetric codes) -- and writes the output tensor through a rank-4 map as well.
 *     acc[b, ho, wo, n] = sum_{i, j, c} X[b, ho*stride + i - pad, wo*stride + j - pad, c] * Wt[n, i, j, c]
 *     z = fma((float)acc * x_scale, fscale[n], fbias[n]),  then the output stage as in qwt_qlinear_cwac_forward
 * with ONE activation scale x_scale for the whole tensor (the paper's per-tensor S_x; a per-pixel scale would not
 * factor out of the sum over taps) and, for QWT_OUT_INT8_PER_TOKEN, one output scale per output pixel.
 *   X  int8 [batch, H, W, C], C % 128 == 0;   Wt int8 [Cout, kh, kw, C];   fscale, fbias float [Cout]
 *   Y  [batch, Ho, Wo, Cout] of the output type (Ho = (H + 2 pad - kh) / stride + 1, likewise Wo)
 *   y_scale float [batch * Ho * Wo], QWT_OUT_INT8_PER_TOKEN only
 *   out_mode: INT8_PER_TOKEN, BF16, FP32 or INT32_ACC;   stride <= 8;   kh * kw * C <= 131072
 *   workspace >= qwt_qconv2d_workspace_bytes(...), 256-byte aligned; status word as for the forward call.
 * Other channel counts (C % 16 == 0) go through qwt_im2col_i8.
 * Errors: NULL, SHAPE, UNSUPPORTED (C % 128, Cout multiple, stride, out_mode), ALIGN, WORKSPACE, ARCH, CUDA. */
size_t qwt_qconv2d_workspace_bytes(int32_t batch, int32_t H, int32_t W, int32_t C, int32_t Cout, int32_t kh, int32_t kw,
                                   int32_t stride, int32_t pad, int32_t out_mode);
qwt_status qwt_qconv2d_cwac_forward(const int8_t* X, float x_scale, const int8_t* Wt, const float* fscale,
                                    const float* fbias, int32_t batch, int32_t H, int32_t W, int32_t C, int32_t Cout,
                                    int32_t kh, int32_t kw, int32_t stride, int32_t pad, int32_t out_mode, void* Y,
                                    float* y_scale, void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Test hooks (the paper has no counterpart).  Host-side, process-wide switches that exist so that the give-up path of
 * the bounded device-side waits can be exercised without faulting or hanging a GPU; both are 0 in normal operation.
 *   qwt_test_set_wait_limit_ns  bound of every device-side wait of the forward calls issued afterwards, in
 *                               nanoseconds; 0 restores the default (QWT_TIMEOUT_MS from the environment, else 2 s).
 *   qwt_test_set_phantom_units  per-token INT8 forward calls planned afterwards expect n (0..4) more 128-column units
 *                               per row strip than the layer has.  Nothing ever publishes a row maximum for them, so
 *                               the exchange of a layer wider than 128 columns cannot complete: every CTA's wait runs
 *                               out after the limit, the kernel records a code in the workspace status word, tears
 *                               down and returns, and qwt_qlinear_check_status reports QWT_ERR_TIMEOUT; Y and y_scale
 *                               are then undefined.  Workspace sizes are planned with the same n. */
void qwt_test_set_wait_limit_ns(uint64_t ns);
void qwt_test_set_phantom_units(int32_t n);

/* Kernels launched by this library on the calling thread since the last reset (for launch accounting). */
int64_t qwt_launch_count(void);
void qwt_launch_count_reset(void);

#ifdef __cplusplus
}
#endif
#endif /* QWT2_H_ */
