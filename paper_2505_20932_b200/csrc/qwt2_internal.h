// Internal declarations shared by the translation units of libqwt2 (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "qwt2.h"

namespace qwt {

// Plans (tile walk, grids, workspace layouts, summation order) are functions of the problem shape only, laid out for
// this many SMs, so that workspace sizes and the bits of the results do not depend on the device that happens to be
// current; a call checks that the device has at least as many SMs as its plan's persistent grid.
constexpr int kPlanSMs = 148;

// Process-wide test hooks (qwt_test_* in the C ABI); both zero in normal operation.
struct TestHooks {
  std::atomic<unsigned long long> wait_limit_ns;   // != 0: bound of every device-side wait of later forward calls
  std::atomic<int> phantom_units;                  // per-token INT8: units a row strip expects beyond those that exist
};
TestHooks& test_hooks();

// thread-local record of the last CUDA failure and of the number of kernels launched
void set_cuda_error(int err);
void count_launch(int n = 1);

#define QWT_CUDA_TRY(expr)                                   \
  do {                                                       \
    cudaError_t _e = (expr);                                 \
    if (_e != cudaSuccess) {                                 \
      ::qwt::set_cuda_error((int)_e);                        \
      return QWT_ERR_CUDA;                                   \
    }                                                        \
  } while (0)

// after a kernel launch
#define QWT_LAUNCH_CHECK()                                   \
  do {                                                       \
    cudaError_t _e = cudaGetLastError();                     \
    if (_e != cudaSuccess) {                                 \
      ::qwt::set_cuda_error((int)_e);                        \
      return QWT_ERR_CUDA;                                   \
    }                                                        \
    ::qwt::count_launch();                                   \
  } while (0)

struct DeviceInfo {
  int device;
  int sm_count;
  int cc_major;
  int cc_minor;
  int max_smem_optin;
};
// Properties of the current device (cached per device). Returns QWT_ERR_ARCH when it is not CC 10.x.
qwt_status current_device(DeviceInfo* out);

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// ---- calibration (cwac_kernels.cu)
// Values per (row chunk, channel) in the partial sums of the statistics pass: four sums of shifted values
// (dq, df, dq df, dq dq) and the two shifts.
constexpr int kPartialValues = 6;
struct CwacPlan {
  int slabs;        // column slabs of 128 channels
  int chunks;       // row chunks
  int64_t chunk_rows;
  size_t partial_bytes;  // double[chunks][kPartialValues][channels_padded]
  int cpad;         // channels rounded up to 128
};
CwacPlan cwac_plan(int64_t rows, int32_t channels, int sm_count);
qwt_status launch_cwac_stats(const float* fp_out, const float* q_out, int64_t rows, int32_t channels, int64_t ld,
                             double* stats, void* workspace, const CwacPlan& plan, cudaStream_t st);
struct CalibBatchItem {
  const float* fp_out;
  const float* q_out;
  int64_t rows, ld;
  int32_t channels;
  float* a;
  float* b;
  const float* w_scale;   // non-NULL: fold as well (Eq. 11) into fscale / fbias
  const float* bias;
  float* fscale;
  float* fbias;
};
size_t cwac_batch_workspace_bytes(const CalibBatchItem* items, int32_t count);
qwt_status launch_cwac_calibrate_batch(const CalibBatchItem* items, int32_t count, int32_t* n_degenerate,
                                       void* workspace, cudaStream_t st);
qwt_status launch_cwac_solve(const double* stats, int32_t channels, float* a, float* b, int32_t* n_degenerate,
                             cudaStream_t st);
qwt_status launch_cwac_fold(const float* w_scale, const float* bias, const float* a, const float* b, int32_t n,
                            float* fscale, float* fbias, cudaStream_t st);
qwt_status launch_cwac_fold_static(const float* w_scale, const float* bias, const float* a, const float* b, int32_t n,
                                   float S_x, float S_r, float* mult, int32_t* offset, cudaStream_t st);
qwt_status launch_quantize_rows(const float* X, int64_t rows, int32_t cols, int64_t ld, int32_t qmax, int8_t* Xq,
                                float* scale, cudaStream_t st);
qwt_status launch_im2col_i8(const int8_t* X, int32_t Bn, int32_t H, int32_t W, int32_t C, int32_t kh, int32_t kw,
                            int32_t stride, int32_t pad, int8_t* P, cudaStream_t st);
qwt_status launch_unpack_int4(const void* packed, int64_t rows, int32_t cols, int8_t* codes, cudaStream_t st);
qwt_status launch_pack_int4(const int8_t* codes, int64_t rows, int32_t cols, uint8_t* packed, cudaStream_t st);

// ---- forward (qlinear_tcgen05.cu)
struct QlinearPlan {
  int bn;            // CTA tile width (128 or 256)
  int tiles_m, tiles_n;
  int grid;
  bool fused_requant;    // cross-CTA row-max protocol inside the GEMM kernel
  int gather_words;      // INT8 output: exchange words per row (one per 128-column unit; 0 = counter protocol)
  int strip_units;       // 128-column units of a row strip (whose row maxima the per-token INT8 exchange waits for)
  bool w_resident;       // grid is a multiple of tiles_n: a CTA's W tile can stay in shared memory
  bool own_strips;       // per-token INT8 with two column tiles per strip: a CTA takes whole strips
  bool pair;             // CTA pairs (clusters of two, MMAs of M = 256 issued by the even CTA); the grid is even
  bool w4_expand;        // packed int4 weights are expanded to int8 in the workspace first (many rows: the GEMM is
                         // compute-bound and the int8 mainloop is twice as fast as the one that converts on chip)
  bool w4_res;           // packed int4 weights, CTA pairs with resident W halves: every CTA expands its half once, on
                         // chip, and the int8 pair kernel runs on the resident operand (no workspace copy of W)
  size_t ws_status_off, ws_partial_off, ws_z_off, ws_w_off, ws_total;
};
// plain: every CTA streams both operands for single tiles b, b + G, ... (no resident W tile, own strips or CTA pairs)
qwt_status qlinear_plan(int32_t M, int32_t N, int32_t K, int32_t wfmt, int32_t out_mode, const DeviceInfo& dev,
                        QlinearPlan* plan, bool plain = false);
// Convolution as an implicit GEMM: geometry of the tiles (blocks of 2^bw_log x 2^bh_log output positions of
// 128 >> (bw_log + bh_log) images) over an NHWC tensor.
struct QconvArgs {
  int B, H, W, C, Ho, Wo;
  int kh, kw, stride, pad;
  int bw_log, bh_log, tiles_w, tiles_h, tiles_b;
  float x_scale;
};
// The block shape that wastes the fewest tile rows for this output size (ties: the widest block).
void qconv_tiling(int B, int Ho, int Wo, int stride, QconvArgs* out);
// Internal output mode of the forward kernel: no output matrix, the per-channel sums of Eq. 4-5 instead.
constexpr int kOutCalibStats = 5;
struct QlinearStatsArgs {
  const float* F;      // [M, ldf] full-precision output
  int64_t ldf;
  double* sums;        // [tiles_m][kPartialValues][cpad] partials, one per strip of 128 rows
  int cpad;
};
qwt_status launch_qlinear(const int8_t* X, const float* x_scale, const void* W, int32_t wfmt, const float* fscale,
                          const float* fbias, int32_t M, int32_t N, int32_t K, int32_t out_mode, void* Y,
                          float* y_scale, void* workspace, const QlinearPlan& plan, cudaStream_t st,
                          const int32_t* x_zero = nullptr, const int32_t* x_rowsum = nullptr,
                          const int32_t* w_terms = nullptr, const QlinearStatsArgs* stats = nullptr,
                          const QconvArgs* conv = nullptr);
qwt_status launch_quantize_rows_u8(const float* X, int64_t rows, int32_t cols, int64_t ld, uint8_t* Xq, float* scale,
                                   int32_t* zero, int32_t* rowsum, cudaStream_t st);
qwt_status launch_asym_weight_terms(const uint8_t* W, const int32_t* w_zero, int32_t N, int32_t K, int32_t* w_terms,
                                    cudaStream_t st);

}  // namespace qwt
