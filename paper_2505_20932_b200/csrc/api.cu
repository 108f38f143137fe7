// extern "C" entry points of libqwt2: argument validation on the host, then kernel launches.
#include <cuda_runtime.h>
#include <stdlib.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "qwt2_internal.h"

namespace qwt {

static thread_local int tl_cuda_error = 0;
static thread_local int64_t tl_launches = 0;

TestHooks& test_hooks() {
  static TestHooks hooks;     // zero-initialised
  return hooks;
}

void set_cuda_error(int err) { tl_cuda_error = err; }
void count_launch(int n) { tl_launches += n; }

qwt_status current_device(DeviceInfo* out) {
  static std::mutex mu;
  static DeviceInfo cache[64];
  static bool have[64] = {false};
  int dev = 0;
  QWT_CUDA_TRY(cudaGetDevice(&dev));
  std::lock_guard<std::mutex> lock(mu);
  if (dev < 0 || dev >= 64) return QWT_ERR_ARCH;
  if (!have[dev]) {
    DeviceInfo d{};
    d.device = dev;
    QWT_CUDA_TRY(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
    QWT_CUDA_TRY(cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev));
    QWT_CUDA_TRY(cudaDeviceGetAttribute(&d.cc_minor, cudaDevAttrComputeCapabilityMinor, dev));
    QWT_CUDA_TRY(cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    cache[dev] = d;
    have[dev] = true;
  }
  *out = cache[dev];
  if (out->cc_major != 10) return QWT_ERR_ARCH;
  return QWT_OK;
}

static inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }

static qwt_status check_calib_args(const float* fp_out, const float* q_out, int64_t rows, int32_t channels,
                                   int64_t ld) {
  if (fp_out == nullptr || q_out == nullptr) return QWT_ERR_NULL;
  if (rows < 1 || channels < 1 || ld < channels) return QWT_ERR_SHAPE;
  if (!aligned(fp_out, 16) || !aligned(q_out, 16) || (ld % 4) != 0) return QWT_ERR_ALIGN;
  return QWT_OK;
}

qwt_status launch_cwac_reduce(const void* workspace, const CwacPlan& plan, int32_t channels, int64_t rows,
                              double* stats_io, float* a, float* b, int32_t* n_degenerate, cudaStream_t st);

}  // namespace qwt

using namespace qwt;

extern "C" {

const char* qwt_version(void) { return "qwt2-b200 0.1 (sm_100a)"; }

const char* qwt_status_string(qwt_status s) {
  switch (s) {
    case QWT_OK: return "ok";
    case QWT_ERR_NULL: return "required pointer is NULL";
    case QWT_ERR_SHAPE: return "invalid dimension";
    case QWT_ERR_ALIGN: return "pointer or leading dimension not aligned";
    case QWT_ERR_UNSUPPORTED: return "unsupported size multiple or enum value";
    case QWT_ERR_WORKSPACE: return "workspace too small or misaligned";
    case QWT_ERR_CUDA: return "CUDA call failed";
    case QWT_ERR_TIMEOUT: return "device-side wait timed out";
    case QWT_ERR_ARCH: return "device is not compute capability 10.x";
    case QWT_ERR_TOO_LARGE: return "problem exceeds the fixed scratch array of the no-allocation entry point";
    default: return "unknown status";
  }
}

qwt_status qwt_last_cuda_error(int* cuda_err) {
  if (cuda_err == nullptr) return QWT_ERR_NULL;
  *cuda_err = tl_cuda_error;
  return QWT_OK;
}

void qwt_test_set_wait_limit_ns(uint64_t ns) { test_hooks().wait_limit_ns.store(ns, std::memory_order_relaxed); }
void qwt_test_set_phantom_units(int32_t n) {
  test_hooks().phantom_units.store(n < 0 ? 0 : (n > 4 ? 4 : n), std::memory_order_relaxed);
}

int64_t qwt_launch_count(void) { return tl_launches; }
void qwt_launch_count_reset(void) { tl_launches = 0; }

// ------------------------------------------------------------------------------------------------ calibration

size_t qwt_cwac_workspace_bytes(int64_t rows, int32_t channels) {
  if (rows < 1 || channels < 1) return 0;
  return cwac_plan(rows, channels, kPlanSMs).partial_bytes;
}

qwt_status qwt_cwac_calibrate(const float* fp_out, const float* q_out, int64_t rows, int32_t channels, int64_t ld,
                              float* a, float* b, int32_t* n_degenerate, void* workspace, size_t workspace_bytes,
                              void* stream) {
  qwt_status s = check_calib_args(fp_out, q_out, rows, channels, ld);
  if (s != QWT_OK) return s;
  if (a == nullptr || b == nullptr || workspace == nullptr) return QWT_ERR_NULL;
  const CwacPlan plan = cwac_plan(rows, channels, kPlanSMs);
  if (workspace_bytes < plan.partial_bytes || !aligned(workspace, 256)) return QWT_ERR_WORKSPACE;
  DeviceInfo dev;
  if ((s = current_device(&dev)) != QWT_OK) return s;
  if ((s = launch_cwac_stats(fp_out, q_out, rows, channels, ld, nullptr, workspace, plan, as_stream(stream))) != QWT_OK)
    return s;
  return launch_cwac_reduce(workspace, plan, channels, rows, nullptr, a, b, n_degenerate, as_stream(stream));
}

static_assert(sizeof(qwt_calib_problem) == sizeof(CalibBatchItem), "the ABI struct and the internal one are the same");

static qwt_status check_batch(const qwt_calib_problem* p, int32_t count) {
  if (p == nullptr) return QWT_ERR_NULL;
  if (count < 1 || count > 4096) return QWT_ERR_SHAPE;
  for (int32_t i = 0; i < count; ++i) {
    qwt_status s = check_calib_args(p[i].fp_out, p[i].q_out, p[i].rows, p[i].channels, p[i].ld);
    if (s != QWT_OK) return s;
    if (p[i].a == nullptr || p[i].b == nullptr) return QWT_ERR_NULL;
    if (p[i].w_scale != nullptr && (p[i].fscale == nullptr || p[i].fbias == nullptr)) return QWT_ERR_NULL;
  }
  return QWT_OK;
}

size_t qwt_cwac_calibrate_batch_workspace_bytes(const qwt_calib_problem* problems, int32_t count) {
  if (check_batch(problems, count) != QWT_OK) return 0;
  return cwac_batch_workspace_bytes(reinterpret_cast<const CalibBatchItem*>(problems), count);
}

qwt_status qwt_cwac_calibrate_batch(const qwt_calib_problem* problems, int32_t count, int32_t* n_degenerate,
                                    void* workspace, size_t workspace_bytes, void* stream) {
  qwt_status s = check_batch(problems, count);
  if (s != QWT_OK) return s;
  if (workspace == nullptr) return QWT_ERR_NULL;
  const CalibBatchItem* items = reinterpret_cast<const CalibBatchItem*>(problems);
  if (workspace_bytes < cwac_batch_workspace_bytes(items, count) || !aligned(workspace, 256)) return QWT_ERR_WORKSPACE;
  DeviceInfo dev;
  if ((s = current_device(&dev)) != QWT_OK) return s;
  return launch_cwac_calibrate_batch(items, count, n_degenerate, workspace, as_stream(stream));
}

qwt_status qwt_cwac_stats_accumulate(const float* fp_out, const float* q_out, int64_t rows, int32_t channels,
                                     int64_t ld, double* stats, void* workspace, size_t workspace_bytes,
                                     void* stream) {
  qwt_status s = check_calib_args(fp_out, q_out, rows, channels, ld);
  if (s != QWT_OK) return s;
  if (stats == nullptr || workspace == nullptr) return QWT_ERR_NULL;
  const CwacPlan plan = cwac_plan(rows, channels, kPlanSMs);
  if (workspace_bytes < plan.partial_bytes || !aligned(workspace, 256)) return QWT_ERR_WORKSPACE;
  DeviceInfo dev;
  if ((s = current_device(&dev)) != QWT_OK) return s;
  if ((s = launch_cwac_stats(fp_out, q_out, rows, channels, ld, nullptr, workspace, plan, as_stream(stream))) != QWT_OK)
    return s;
  return launch_cwac_reduce(workspace, plan, channels, rows, stats, nullptr, nullptr, nullptr, as_stream(stream));
}

qwt_status qwt_cwac_solve(const double* stats, int32_t channels, float* a, float* b, int32_t* n_degenerate,
                          void* stream) {
  if (stats == nullptr || a == nullptr || b == nullptr) return QWT_ERR_NULL;
  if (channels < 1) return QWT_ERR_SHAPE;
  DeviceInfo dev;
  qwt_status s = current_device(&dev);
  if (s != QWT_OK) return s;
  return launch_cwac_solve(stats, channels, a, b, n_degenerate, as_stream(stream));
}

// Host-matrix calibration: rows are cut into chunks; chunk i is copied into one of two staging slots while
// chunk i-1 is reduced.  Staging layout: [stats 5*C doubles][out a,b,n_deg][2 slots x (fp, q) chunk][partials].
namespace {
struct HostCalibLayout {
  int64_t chunk_rows;
  size_t off_stats, off_out, off_slot[2], slot_bytes, off_ws, ws_bytes, total;
};
HostCalibLayout host_calib_layout(int64_t rows, int32_t channels) {
  HostCalibLayout L{};
  const int64_t target_bytes = 64ll << 20;   // per matrix per slot
  int64_t cr = target_bytes / ((int64_t)channels * 4);
  if (cr < 128) cr = 128;
  if (cr > rows) cr = rows;
  L.chunk_rows = cr;
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  size_t off = 0;
  L.off_stats = off; off += up((size_t)5 * channels * 8);
  L.off_out = off; off += up((size_t)2 * channels * 4 + 16);
  L.slot_bytes = up((size_t)cr * channels * 4);
  for (int i = 0; i < 2; ++i) { L.off_slot[i] = off; off += 2 * L.slot_bytes; }
  L.ws_bytes = cwac_plan(cr, channels, kPlanSMs).partial_bytes;
  L.off_ws = off; off += up(L.ws_bytes);
  L.total = off;
  return L;
}
}  // namespace

size_t qwt_cwac_host_staging_bytes(int64_t rows, int32_t channels) {
  if (rows < 1 || channels < 1) return 0;
  return host_calib_layout(rows, channels).total;
}

qwt_status qwt_cwac_calibrate_host(const float* fp_out, const float* q_out, int64_t rows, int32_t channels,
                                   int64_t ld, float* a, float* b, int32_t* n_degenerate, void* staging,
                                   size_t staging_bytes, void* stream) {
  if (fp_out == nullptr || q_out == nullptr || a == nullptr || b == nullptr || staging == nullptr) return QWT_ERR_NULL;
  if (rows < 1 || channels < 1 || ld < channels) return QWT_ERR_SHAPE;
  if ((channels % 4) != 0) return QWT_ERR_ALIGN;   // staged rows are packed with ld = channels
  const HostCalibLayout L = host_calib_layout(rows, channels);
  if (staging_bytes < L.total || !aligned(staging, 256)) return QWT_ERR_WORKSPACE;
  DeviceInfo dev;
  qwt_status s = current_device(&dev);
  if (s != QWT_OK) return s;
  cudaStream_t st = as_stream(stream);
  uint8_t* base = static_cast<uint8_t*>(staging);
  double* stats = reinterpret_cast<double*>(base + L.off_stats);
  float* d_a = reinterpret_cast<float*>(base + L.off_out);
  float* d_b = d_a + channels;
  int32_t* d_nd = reinterpret_cast<int32_t*>(d_b + channels);

  // a second stream carries the copies so that they overlap the reduction of the previous chunk
  cudaStream_t copy_st;
  cudaEvent_t copied[2], reduced[2];
  QWT_CUDA_TRY(cudaStreamCreateWithFlags(&copy_st, cudaStreamNonBlocking));
  for (int i = 0; i < 2; ++i) {
    cudaEventCreateWithFlags(&copied[i], cudaEventDisableTiming);
    cudaEventCreateWithFlags(&reduced[i], cudaEventDisableTiming);
  }
  qwt_status rc = QWT_OK;
  cudaEvent_t start;
  cudaEventCreateWithFlags(&start, cudaEventDisableTiming);
  auto cleanup = [&]() {
    cudaStreamSynchronize(copy_st);
    cudaStreamDestroy(copy_st);
    for (int i = 0; i < 2; ++i) { cudaEventDestroy(copied[i]); cudaEventDestroy(reduced[i]); }
    cudaEventDestroy(start);
  };
#define QWT_HC_TRY(expr) do { cudaError_t _e = (expr); if (_e != cudaSuccess) { set_cuda_error((int)_e); rc = QWT_ERR_CUDA; goto done; } } while (0)
  {
    QWT_HC_TRY(cudaMemsetAsync(stats, 0, (size_t)5 * channels * 8, st));
    QWT_HC_TRY(cudaEventRecord(start, st));
    QWT_HC_TRY(cudaStreamWaitEvent(copy_st, start, 0));
    int64_t r0 = 0;
    for (int i = 0; r0 < rows; ++i, r0 += L.chunk_rows) {
      const int slot = i & 1;
      const int64_t nr = (rows - r0 < L.chunk_rows) ? rows - r0 : L.chunk_rows;
      float* d_fp = reinterpret_cast<float*>(base + L.off_slot[slot]);
      float* d_q = reinterpret_cast<float*>(base + L.off_slot[slot] + L.slot_bytes);
      if (i >= 2) QWT_HC_TRY(cudaStreamWaitEvent(copy_st, reduced[slot], 0));
      QWT_HC_TRY(cudaMemcpy2DAsync(d_fp, (size_t)channels * 4, fp_out + r0 * ld, (size_t)ld * 4, (size_t)channels * 4,
                                   (size_t)nr, cudaMemcpyHostToDevice, copy_st));
      QWT_HC_TRY(cudaMemcpy2DAsync(d_q, (size_t)channels * 4, q_out + r0 * ld, (size_t)ld * 4, (size_t)channels * 4,
                                   (size_t)nr, cudaMemcpyHostToDevice, copy_st));
      QWT_HC_TRY(cudaEventRecord(copied[slot], copy_st));
      QWT_HC_TRY(cudaStreamWaitEvent(st, copied[slot], 0));
      const CwacPlan plan = cwac_plan(nr, channels, kPlanSMs);
      if ((rc = launch_cwac_stats(d_fp, d_q, nr, channels, channels, nullptr, base + L.off_ws, plan, st)) != QWT_OK) goto done;
      if ((rc = launch_cwac_reduce(base + L.off_ws, plan, channels, nr, stats, nullptr, nullptr, nullptr, st)) != QWT_OK) goto done;
      QWT_HC_TRY(cudaEventRecord(reduced[slot], st));
    }
    if ((rc = launch_cwac_solve(stats, channels, d_a, d_b, d_nd, st)) != QWT_OK) goto done;
    QWT_HC_TRY(cudaMemcpyAsync(a, d_a, (size_t)channels * 4, cudaMemcpyDeviceToHost, st));
    QWT_HC_TRY(cudaMemcpyAsync(b, d_b, (size_t)channels * 4, cudaMemcpyDeviceToHost, st));
    if (n_degenerate != nullptr) QWT_HC_TRY(cudaMemcpyAsync(n_degenerate, d_nd, 4, cudaMemcpyDeviceToHost, st));
    QWT_HC_TRY(cudaStreamSynchronize(st));
  }
done:
#undef QWT_HC_TRY
  cleanup();
  return rc;
}

// ------------------------------------------------------------------------------------------------ fold

qwt_status qwt_cwac_fold(const float* w_scale, const float* bias, const float* a, const float* b, int32_t n,
                         float* fscale, float* fbias, void* stream) {
  if (w_scale == nullptr || fscale == nullptr || fbias == nullptr) return QWT_ERR_NULL;
  if ((a == nullptr) != (b == nullptr)) return QWT_ERR_NULL;
  if (n < 1) return QWT_ERR_SHAPE;
  DeviceInfo dev;
  qwt_status s = current_device(&dev);
  if (s != QWT_OK) return s;
  return launch_cwac_fold(w_scale, bias, a, b, n, fscale, fbias, as_stream(stream));
}

qwt_status qwt_cwac_fold_static(const float* w_scale, const float* bias, const float* a, const float* b, int32_t n,
                                float S_x, float S_r, float* mult, int32_t* offset, void* stream) {
  if (w_scale == nullptr || mult == nullptr || offset == nullptr) return QWT_ERR_NULL;
  if ((a == nullptr) != (b == nullptr)) return QWT_ERR_NULL;
  if (n < 1 || !(S_x > 0.f) || !(S_r > 0.f)) return QWT_ERR_SHAPE;
  DeviceInfo dev;
  qwt_status s = current_device(&dev);
  if (s != QWT_OK) return s;
  return launch_cwac_fold_static(w_scale, bias, a, b, n, S_x, S_r, mult, offset, as_stream(stream));
}

// ------------------------------------------------------------------------------------------------ forward

static qwt_status check_forward_args(const void* X, const float* x_scale, const void* W, int32_t wfmt,
                                     const float* fscale, const float* fbias, int32_t M, int32_t N, int32_t K,
                                     int32_t out_mode, const void* Y, const float* y_scale, bool host_io) {
  if (X == nullptr || W == nullptr || Y == nullptr) return QWT_ERR_NULL;
  if (wfmt != QWT_W_INT8 && wfmt != QWT_W_INT4_PACKED) return QWT_ERR_UNSUPPORTED;
  if (out_mode < QWT_OUT_INT8_PER_TOKEN || out_mode > QWT_OUT_INT8_STATIC) return QWT_ERR_UNSUPPORTED;
  if (out_mode != QWT_OUT_INT32_ACC && (fscale == nullptr || fbias == nullptr)) return QWT_ERR_NULL;
  if (out_mode != QWT_OUT_INT32_ACC && out_mode != QWT_OUT_INT8_STATIC && x_scale == nullptr) return QWT_ERR_NULL;
  if (out_mode == QWT_OUT_INT8_PER_TOKEN && y_scale == nullptr) return QWT_ERR_NULL;
  if (M < 1 || N < 1 || K < 1) return QWT_ERR_SHAPE;
  if ((int64_t)M * (int64_t)N >= (int64_t)1 << 40) return QWT_ERR_SHAPE;
  if (K > 131072) return QWT_ERR_SHAPE;   // 127^2 * K must stay below 2^31
  const int kmul = wfmt == QWT_W_INT8 ? 16 : 32;
  if (K % kmul != 0) return QWT_ERR_UNSUPPORTED;
  const bool codes = out_mode == QWT_OUT_INT8_PER_TOKEN || out_mode == QWT_OUT_INT8_STATIC;
  const int nmul = codes ? 16 : (out_mode == QWT_OUT_BF16 ? 8 : 4);
  if (N % nmul != 0) return QWT_ERR_UNSUPPORTED;
  if (!aligned(W, 16)) return QWT_ERR_ALIGN;
  if (!host_io && (!aligned(X, 16) || !aligned(Y, 16))) return QWT_ERR_ALIGN;
  return QWT_OK;
}

size_t qwt_qlinear_workspace_bytes(int32_t M, int32_t N, int32_t K, int32_t wfmt, int32_t out_mode) {
  if (M < 1 || N < 1 || K < 1) return 0;
  DeviceInfo dev{};
  dev.sm_count = kPlanSMs;
  QlinearPlan plan;
  if (qlinear_plan(M, N, K, wfmt, out_mode, dev, &plan) != QWT_OK) return 0;
  return plan.ws_total;
}

qwt_status qwt_qlinear_cwac_forward(const int8_t* X, const float* x_scale, const void* W, int32_t wfmt,
                                    const float* fscale, const float* fbias, int32_t M, int32_t N, int32_t K,
                                    int32_t out_mode, void* Y, float* y_scale, void* workspace,
                                    size_t workspace_bytes, void* stream) {
  qwt_status s = check_forward_args(X, x_scale, W, wfmt, fscale, fbias, M, N, K, out_mode, Y, y_scale, false);
  if (s != QWT_OK) return s;
  if (workspace == nullptr) return QWT_ERR_NULL;
  DeviceInfo dev{};
  dev.sm_count = kPlanSMs;
  QlinearPlan plan;
  if ((s = qlinear_plan(M, N, K, wfmt, out_mode, dev, &plan)) != QWT_OK) return s;
  if (workspace_bytes < plan.ws_total || !aligned(workspace, 256)) return QWT_ERR_WORKSPACE;
  DeviceInfo real;
  if ((s = current_device(&real)) != QWT_OK) return s;
  if (real.sm_count < plan.grid) return QWT_ERR_ARCH;   // the persistent grid must be co-resident
  return launch_qlinear(X, x_scale, W, wfmt, fscale, fbias, M, N, K, out_mode, Y, y_scale, workspace, plan,
                        as_stream(stream));
}

qwt_status qwt_qlinear_cwac_forward_asym(const uint8_t* X, const float* x_scale, const int32_t* x_zero,
                                         const int32_t* x_rowsum, const uint8_t* W, const int32_t* w_terms,
                                         const float* fscale, const float* fbias, int32_t M, int32_t N, int32_t K,
                                         int32_t out_mode, void* Y, float* y_scale, void* workspace,
                                         size_t workspace_bytes, void* stream) {
  if (out_mode == QWT_OUT_INT8_STATIC) return QWT_ERR_UNSUPPORTED;
  qwt_status s = check_forward_args(X, x_scale, W, QWT_W_INT8, fscale, fbias, M, N, K, out_mode, Y, y_scale, false);
  if (s != QWT_OK) return s;
  if (x_zero == nullptr || x_rowsum == nullptr || w_terms == nullptr || workspace == nullptr) return QWT_ERR_NULL;
  if (K > 33000) return QWT_ERR_SHAPE;   // 255^2 * K must stay below 2^31
  DeviceInfo dev{};
  dev.sm_count = kPlanSMs;
  QlinearPlan plan;
  if ((s = qlinear_plan(M, N, K, QWT_W_INT8, out_mode, dev, &plan)) != QWT_OK) return s;
  if (workspace_bytes < plan.ws_total || !aligned(workspace, 256)) return QWT_ERR_WORKSPACE;
  DeviceInfo real;
  if ((s = current_device(&real)) != QWT_OK) return s;
  if (real.sm_count < plan.grid) return QWT_ERR_ARCH;
  return launch_qlinear(reinterpret_cast<const int8_t*>(X), x_scale, W, QWT_W_INT8, fscale, fbias, M, N, K, out_mode,
                        Y, y_scale, workspace, plan, as_stream(stream), x_zero, x_rowsum, w_terms);
}

// Calibration fused into the layer (Section 3.3 on top of Eq. 6-8): workspace = [status 256 B][partials].
namespace {
struct FusedCalibLayout {
  QlinearPlan plan;
  CwacPlan red;          // the strips of 128 rows play the part of the row chunks
  size_t off_partial, total;
};
qwt_status fused_calib_layout(int32_t M, int32_t N, int32_t K, int32_t wfmt, FusedCalibLayout* L) {
  DeviceInfo dev{};
  dev.sm_count = kPlanSMs;
  qwt_status s = qlinear_plan(M, N, K, wfmt, kOutCalibStats, dev, &L->plan);
  if (s != QWT_OK) return s;
  L->red = CwacPlan{};
  L->red.slabs = (N + 127) / 128;
  L->red.cpad = L->red.slabs * 128;
  L->red.chunks = L->plan.tiles_m;
  L->red.chunk_rows = 128;
  L->red.partial_bytes = (size_t)L->red.chunks * kPartialValues * L->red.cpad * sizeof(double);
  L->off_partial = 256;
  // the expanded int8 copy of packed weights (if the plan asks for one) goes behind the partials
  L->plan.ws_w_off = (L->off_partial + L->red.partial_bytes + 255) / 256 * 256;
  L->total = L->plan.ws_w_off + (L->plan.w4_expand ? (size_t)N * (size_t)K : 0);
  return QWT_OK;
}
}  // namespace

size_t qwt_qlinear_cwac_calibrate_workspace_bytes(int32_t M, int32_t N, int32_t K, int32_t wfmt) {
  if (M < 1 || N < 1 || K < 1) return 0;
  FusedCalibLayout L;
  if (fused_calib_layout(M, N, K, wfmt, &L) != QWT_OK) return 0;
  return L.total;
}

qwt_status qwt_qlinear_cwac_calibrate(const int8_t* X, const float* x_scale, const void* W, int32_t wfmt,
                                      const float* w_scale, const float* bias, const float* fp_out, int64_t ld,
                                      int32_t M, int32_t N, int32_t K, double* stats, float* a, float* b,
                                      int32_t* n_degenerate, void* workspace, size_t workspace_bytes, void* stream) {
  if (X == nullptr || x_scale == nullptr || W == nullptr || w_scale == nullptr || fp_out == nullptr ||
      workspace == nullptr)
    return QWT_ERR_NULL;
  if (stats == nullptr && (a == nullptr || b == nullptr)) return QWT_ERR_NULL;
  if ((a == nullptr) != (b == nullptr)) return QWT_ERR_NULL;
  if (wfmt != QWT_W_INT8 && wfmt != QWT_W_INT4_PACKED) return QWT_ERR_UNSUPPORTED;
  if (M < 1 || N < 1 || K < 1 || ld < N || K > 131072) return QWT_ERR_SHAPE;
  if (K % (wfmt == QWT_W_INT8 ? 16 : 32) != 0 || N % 4 != 0 || ld % 4 != 0) return QWT_ERR_UNSUPPORTED;
  if (!aligned(X, 16) || !aligned(W, 16) || !aligned(fp_out, 16)) return QWT_ERR_ALIGN;
  FusedCalibLayout L;
  qwt_status s = fused_calib_layout(M, N, K, wfmt, &L);
  if (s != QWT_OK) return s;
  if (workspace_bytes < L.total || !aligned(workspace, 256)) return QWT_ERR_WORKSPACE;
  DeviceInfo real;
  if ((s = current_device(&real)) != QWT_OK) return s;
  if (real.sm_count < L.plan.grid) return QWT_ERR_ARCH;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  QlinearStatsArgs sa{fp_out, ld, reinterpret_cast<double*>(ws + L.off_partial), L.red.cpad};
  cudaStream_t st = as_stream(stream);
  if ((s = launch_qlinear(X, x_scale, W, wfmt, w_scale, bias, M, N, K, kOutCalibStats, nullptr, nullptr, workspace,
                          L.plan, st, nullptr, nullptr, nullptr, &sa)) != QWT_OK)
    return s;
  return launch_cwac_reduce(ws + L.off_partial, L.red, N, M, stats, a, b, n_degenerate, st);
}

qwt_status qwt_asym_weight_terms(const uint8_t* W, const int32_t* w_zero, int32_t N, int32_t K, int32_t* w_terms,
                                 void* stream) {
  if (W == nullptr || w_zero == nullptr || w_terms == nullptr) return QWT_ERR_NULL;
  if (N < 1 || K < 1 || K > 33000) return QWT_ERR_SHAPE;
  DeviceInfo dev;
  qwt_status s = current_device(&dev);
  if (s != QWT_OK) return s;
  return launch_asym_weight_terms(W, w_zero, N, K, w_terms, as_stream(stream));
}

qwt_status qwt_quantize_rows_u8(const float* X, int64_t rows, int32_t cols, int64_t ld, uint8_t* Xq, float* scale,
                                int32_t* zero, int32_t* rowsum, void* stream) {
  if (X == nullptr || Xq == nullptr || scale == nullptr || zero == nullptr) return QWT_ERR_NULL;
  if (rows < 1 || cols < 1 || ld < cols || rows > (int64_t)8 * 2147483647) return QWT_ERR_SHAPE;
  DeviceInfo dev;
  qwt_status s = current_device(&dev);
  if (s != QWT_OK) return s;
  return launch_quantize_rows_u8(X, rows, cols, ld, Xq, scale, zero, rowsum, as_stream(stream));
}

qwt_status qwt_qlinear_check_status(const void* workspace, void* stream, int32_t* device_status) {
  if (workspace == nullptr) return QWT_ERR_NULL;
  QWT_CUDA_TRY(cudaStreamSynchronize(as_stream(stream)));
  uint32_t word = 0;
  QWT_CUDA_TRY(cudaMemcpy(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost));
  if (device_status != nullptr) *device_status = (int32_t)word;
  return word == 0 ? QWT_OK : QWT_ERR_TIMEOUT;
}

namespace {
// Rows of a chunk of the host-buffer forward: inputs of chunk c + 1 travel to the device while chunk c is computed
// and the outputs of chunk c - 1 travel back (a row's per-token scale needs that row only, so row chunks are exact).
constexpr int32_t kHostChunkRows = 4096;

struct HostFwdLayout {
  size_t off_x, off_xs, off_y, off_ys, off_ws[2], ws_bytes, total;
  size_t esz;
  int32_t chunk_rows, chunks;
};
HostFwdLayout host_fwd_layout(int32_t M, int32_t N, int32_t K, int32_t wfmt, int32_t out_mode) {
  HostFwdLayout L{};
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  L.esz = (out_mode == QWT_OUT_INT8_PER_TOKEN || out_mode == QWT_OUT_INT8_STATIC)
              ? 1 : (out_mode == QWT_OUT_BF16 ? 2 : 4);
  L.chunk_rows = M > kHostChunkRows ? kHostChunkRows : M;
  L.chunks = (M + L.chunk_rows - 1) / L.chunk_rows;
  size_t off = 0;
  L.off_x = off; off += up((size_t)M * K);
  L.off_xs = off; off += up((size_t)M * 4);
  L.off_y = off; off += up((size_t)M * N * L.esz);
  L.off_ys = off; off += up((size_t)M * 4);
  L.ws_bytes = up(qwt_qlinear_workspace_bytes(L.chunk_rows, N, K, wfmt, out_mode));
  L.off_ws[0] = off; off += L.ws_bytes;
  L.off_ws[1] = off; off += L.chunks > 1 ? L.ws_bytes : 0;
  L.total = off;
  return L;
}

// Two helper streams and three events per host thread and device, created on first use and kept.
struct HostPipe {
  cudaStream_t s[2];
  cudaEvent_t start, done[2];
  bool ready;
};
qwt_status host_pipe(HostPipe** out) {
  static thread_local HostPipe pipes[64] = {};
  int dev = 0;
  QWT_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return QWT_ERR_ARCH;
  HostPipe& hp = pipes[dev];
  if (!hp.ready) {
    for (int i = 0; i < 2; ++i) {
      QWT_CUDA_TRY(cudaStreamCreateWithFlags(&hp.s[i], cudaStreamNonBlocking));
      QWT_CUDA_TRY(cudaEventCreateWithFlags(&hp.done[i], cudaEventDisableTiming));
    }
    QWT_CUDA_TRY(cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming));
    hp.ready = true;
  }
  *out = &hp;
  return QWT_OK;
}
}  // namespace

size_t qwt_qlinear_host_staging_bytes(int32_t M, int32_t N, int32_t K, int32_t wfmt, int32_t out_mode) {
  if (M < 1 || N < 1 || K < 1) return 0;
  return host_fwd_layout(M, N, K, wfmt, out_mode).total;
}

qwt_status qwt_qlinear_cwac_forward_host(const int8_t* X, const float* x_scale, const void* W, int32_t wfmt,
                                         const float* fscale, const float* fbias, int32_t M, int32_t N, int32_t K,
                                         int32_t out_mode, void* Y, float* y_scale, void* staging,
                                         size_t staging_bytes, void* stream) {
  qwt_status s = check_forward_args(X, x_scale, W, wfmt, fscale, fbias, M, N, K, out_mode, Y, y_scale, true);
  if (s != QWT_OK) return s;
  if (staging == nullptr) return QWT_ERR_NULL;
  const HostFwdLayout L = host_fwd_layout(M, N, K, wfmt, out_mode);
  if (staging_bytes < L.total || !aligned(staging, 256)) return QWT_ERR_WORKSPACE;
  cudaStream_t st = as_stream(stream);
  uint8_t* base = static_cast<uint8_t*>(staging);
  int8_t* d_x = reinterpret_cast<int8_t*>(base + L.off_x);
  float* d_xs = reinterpret_cast<float*>(base + L.off_xs);
  uint8_t* d_y = base + L.off_y;
  float* d_ys = reinterpret_cast<float*>(base + L.off_ys);
  const bool per_token = out_mode == QWT_OUT_INT8_PER_TOKEN;
  // one chunk of rows [r0, r0 + rows): copy in, compute, copy out, all on stream cs
  auto chunk = [&](int32_t r0, int32_t rows, void* ws, cudaStream_t cs) -> qwt_status {
    QWT_CUDA_TRY(cudaMemcpyAsync(d_x + (size_t)r0 * K, X + (size_t)r0 * K, (size_t)rows * K, cudaMemcpyHostToDevice, cs));
    const size_t y_off = (size_t)r0 * N * L.esz;
    qwt_status r = qwt_qlinear_cwac_forward(d_x + (size_t)r0 * K, x_scale ? d_xs + r0 : nullptr, W, wfmt, fscale, fbias,
                                            rows, N, K, out_mode, d_y + y_off, per_token ? d_ys + r0 : nullptr, ws,
                                            L.ws_bytes, cs);
    if (r != QWT_OK) return r;
    QWT_CUDA_TRY(cudaMemcpyAsync(static_cast<uint8_t*>(Y) + y_off, d_y + y_off, (size_t)rows * N * L.esz,
                                 cudaMemcpyDeviceToHost, cs));
    return QWT_OK;
  };
  // the per-row scales travel once, whole: in before the first chunk, out after the last
  if (x_scale != nullptr) QWT_CUDA_TRY(cudaMemcpyAsync(d_xs, x_scale, (size_t)M * 4, cudaMemcpyHostToDevice, st));
  if (L.chunks == 1) {
    if ((s = chunk(0, M, base + L.off_ws[0], st)) != QWT_OK) return s;
    if (per_token) QWT_CUDA_TRY(cudaMemcpyAsync(y_scale, d_ys, (size_t)M * 4, cudaMemcpyDeviceToHost, st));
    QWT_CUDA_TRY(cudaStreamSynchronize(st));
    return QWT_OK;
  }
  // several chunks: they alternate over two helper streams that start after the work already queued on `stream`
  HostPipe* hp = nullptr;
  if ((s = host_pipe(&hp)) != QWT_OK) return s;
  QWT_CUDA_TRY(cudaEventRecord(hp->start, st));
  for (int i = 0; i < 2; ++i) QWT_CUDA_TRY(cudaStreamWaitEvent(hp->s[i], hp->start, 0));
  qwt_status rc = QWT_OK;
  for (int32_t c = 0; c < L.chunks && rc == QWT_OK; ++c) {
    const int32_t r0 = c * L.chunk_rows;
    const int32_t rows = M - r0 < L.chunk_rows ? M - r0 : L.chunk_rows;
    rc = chunk(r0, rows, base + L.off_ws[c & 1], hp->s[c & 1]);
  }
  for (int i = 0; i < 2; ++i) {
    QWT_CUDA_TRY(cudaEventRecord(hp->done[i], hp->s[i]));
    QWT_CUDA_TRY(cudaStreamWaitEvent(st, hp->done[i], 0));
  }
  if (per_token && rc == QWT_OK)
    QWT_CUDA_TRY(cudaMemcpyAsync(y_scale, d_ys, (size_t)M * 4, cudaMemcpyDeviceToHost, st));
  QWT_CUDA_TRY(cudaStreamSynchronize(st));
  return rc;
}

// ------------------------------------------------------------------------------------------------ support

qwt_status qwt_quantize_rows_i8(const float* X, int64_t rows, int32_t cols, int64_t ld, int32_t qmax, int8_t* Xq,
                                float* scale, void* stream) {
  if (X == nullptr || Xq == nullptr || scale == nullptr) return QWT_ERR_NULL;
  if (rows < 1 || cols < 1 || ld < cols || rows > (int64_t)8 * 2147483647) return QWT_ERR_SHAPE;
  if (qmax < 1 || qmax > 127) return QWT_ERR_UNSUPPORTED;
  DeviceInfo dev;
  qwt_status s = current_device(&dev);
  if (s != QWT_OK) return s;
  return launch_quantize_rows(X, rows, cols, ld, qmax, Xq, scale, as_stream(stream));
}

qwt_status qwt_im2col_i8(const int8_t* X, int32_t batch, int32_t H, int32_t W, int32_t C, int32_t kh, int32_t kw,
                         int32_t stride, int32_t pad, int8_t* patches, void* stream) {
  if (X == nullptr || patches == nullptr) return QWT_ERR_NULL;
  if (batch < 1 || H < 1 || W < 1 || C < 1 || kh < 1 || kw < 1 || stride < 1 || pad < 0) return QWT_ERR_SHAPE;
  if (H + 2 * pad < kh || W + 2 * pad < kw) return QWT_ERR_SHAPE;
  if ((C % 16) != 0) return QWT_ERR_UNSUPPORTED;
  if (!aligned(X, 16) || !aligned(patches, 16)) return QWT_ERR_ALIGN;
  DeviceInfo dev;
  qwt_status s = current_device(&dev);
  if (s != QWT_OK) return s;
  return launch_im2col_i8(X, batch, H, W, C, kh, kw, stride, pad, patches, as_stream(stream));
}

namespace {
// Geometry, plan and argument checks shared by the size query and the call.
qwt_status qconv_setup(int32_t batch, int32_t H, int32_t W, int32_t C, int32_t Cout, int32_t kh, int32_t kw,
                       int32_t stride, int32_t pad, int32_t out_mode, QconvArgs* cv, QlinearPlan* plan, int32_t* m_eff,
                       int32_t* K) {
  if (batch < 1 || H < 1 || W < 1 || C < 1 || Cout < 1 || kh < 1 || kw < 1 || stride < 1 || pad < 0) return QWT_ERR_SHAPE;
  if (H + 2 * pad < kh || W + 2 * pad < kw) return QWT_ERR_SHAPE;
  if (out_mode != QWT_OUT_INT8_PER_TOKEN && out_mode != QWT_OUT_BF16 && out_mode != QWT_OUT_FP32 &&
      out_mode != QWT_OUT_INT32_ACC)
    return QWT_ERR_UNSUPPORTED;
  if ((C % 128) != 0 || stride > 8) return QWT_ERR_UNSUPPORTED;
  const int nmul = out_mode == QWT_OUT_INT8_PER_TOKEN ? 16 : (out_mode == QWT_OUT_BF16 ? 8 : 4);
  if (Cout % nmul != 0) return QWT_ERR_UNSUPPORTED;
  const int64_t k = (int64_t)kh * kw * C;
  if (k > 131072) return QWT_ERR_SHAPE;
  *cv = QconvArgs{};
  cv->B = batch; cv->H = H; cv->W = W; cv->C = C;
  cv->Ho = (H + 2 * pad - kh) / stride + 1;
  cv->Wo = (W + 2 * pad - kw) / stride + 1;
  cv->kh = kh; cv->kw = kw; cv->stride = stride; cv->pad = pad;
  qconv_tiling(batch, cv->Ho, cv->Wo, stride, cv);
  const int64_t tiles = (int64_t)cv->tiles_w * cv->tiles_h * cv->tiles_b;
  if (tiles * 128 >= ((int64_t)1 << 31) || tiles * 128 * (int64_t)Cout >= ((int64_t)1 << 40)) return QWT_ERR_SHAPE;
  *m_eff = (int32_t)(tiles * 128);
  *K = (int32_t)k;
  DeviceInfo dev{};
  dev.sm_count = kPlanSMs;
  qwt_status s = qlinear_plan(*m_eff, Cout, *K, QWT_W_INT8, out_mode, dev, plan, /*plain=*/true);
  if (s != QWT_OK) return s;
  if (out_mode == QWT_OUT_INT8_PER_TOKEN && !plan->fused_requant) return QWT_ERR_UNSUPPORTED;   // more column tiles than CTAs
  return QWT_OK;
}
}  // namespace

size_t qwt_qconv2d_workspace_bytes(int32_t batch, int32_t H, int32_t W, int32_t C, int32_t Cout, int32_t kh, int32_t kw,
                                   int32_t stride, int32_t pad, int32_t out_mode) {
  QconvArgs cv;
  QlinearPlan plan;
  int32_t m_eff = 0, K = 0;
  if (qconv_setup(batch, H, W, C, Cout, kh, kw, stride, pad, out_mode, &cv, &plan, &m_eff, &K) != QWT_OK) return 0;
  return plan.ws_total;
}

qwt_status qwt_qconv2d_cwac_forward(const int8_t* X, float x_scale, const int8_t* Wt, const float* fscale,
                                    const float* fbias, int32_t batch, int32_t H, int32_t W, int32_t C, int32_t Cout,
                                    int32_t kh, int32_t kw, int32_t stride, int32_t pad, int32_t out_mode, void* Y,
                                    float* y_scale, void* workspace, size_t workspace_bytes, void* stream) {
  if (X == nullptr || Wt == nullptr || Y == nullptr || workspace == nullptr) return QWT_ERR_NULL;
  if (out_mode != QWT_OUT_INT32_ACC && (fscale == nullptr || fbias == nullptr)) return QWT_ERR_NULL;
  if (out_mode == QWT_OUT_INT8_PER_TOKEN && y_scale == nullptr) return QWT_ERR_NULL;
  QconvArgs cv;
  QlinearPlan plan;
  int32_t m_eff = 0, K = 0;
  qwt_status s = qconv_setup(batch, H, W, C, Cout, kh, kw, stride, pad, out_mode, &cv, &plan, &m_eff, &K);
  if (s != QWT_OK) return s;
  if (!aligned(X, 16) || !aligned(Wt, 16) || !aligned(Y, 16)) return QWT_ERR_ALIGN;
  if (workspace_bytes < plan.ws_total || !aligned(workspace, 256)) return QWT_ERR_WORKSPACE;
  DeviceInfo real;
  if ((s = current_device(&real)) != QWT_OK) return s;
  if (real.sm_count < plan.grid) return QWT_ERR_ARCH;
  cv.x_scale = x_scale;
  return launch_qlinear(X, nullptr, Wt, QWT_W_INT8, fscale, fbias, m_eff, Cout, K, out_mode, Y, y_scale, workspace, plan,
                        as_stream(stream), nullptr, nullptr, nullptr, nullptr, &cv);
}

qwt_status qwt_pack_int4(const int8_t* codes, int64_t rows, int32_t cols, uint8_t* packed, void* stream) {
  if (codes == nullptr || packed == nullptr) return QWT_ERR_NULL;
  if (rows < 1 || cols < 2) return QWT_ERR_SHAPE;
  if ((cols % 2) != 0) return QWT_ERR_UNSUPPORTED;
  DeviceInfo dev;
  qwt_status s = current_device(&dev);
  if (s != QWT_OK) return s;
  return launch_pack_int4(codes, rows, cols, packed, as_stream(stream));
}

}  // extern "C"
