// qwt_cwac_calibrate_noalloc: one-shot CWAC calibration for callers that cannot hand the library a
// workspace because they are not allowed to allocate device memory themselves -- for instance a plug-in
// that lives inside another program's pre-partitioned memory arena, or a service that must not call
// cudaMalloc (an implicitly synchronising call) once it is serving.  The scratch that qwt_cwac_calibrate
// takes from the caller lives here in a fixed array inside the library image instead.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "qwt2_internal.h"

namespace qwt {
qwt_status launch_cwac_reduce(const void* workspace, const CwacPlan& plan, int32_t channels, int64_t rows,
                              double* stats_io, float* a, float* b, int32_t* n_degenerate, cudaStream_t st);
}

namespace {

// 6 MiB of per-chunk partial sums (double[chunks][6][channels padded to 128]).  Every GPU that loads the
// library carries this array until the process exits.
constexpr size_t kScratchBytes = QWT_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_calib_scratch[kScratchBytes];

// Device address of g_calib_scratch per device.  In host code the array's name is only a handle for the
// runtime, not an address a kernel could use, so the address is asked for once per device.
qwt_status scratch_address(void** out) {
  static std::mutex mu;
  static void* addr[64] = {nullptr};
  int dev = 0;
  QWT_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return QWT_ERR_ARCH;
  std::lock_guard<std::mutex> lock(mu);
  if (addr[dev] == nullptr) {
    void* p = nullptr;
    QWT_CUDA_TRY(cudaGetSymbolAddress(&p, g_calib_scratch));
    addr[dev] = p;
  }
  *out = addr[dev];
  return QWT_OK;
}

}  // namespace

extern "C" qwt_status qwt_cwac_calibrate_noalloc(const float* fp_out, const float* q_out, int64_t rows,
                                                 int32_t channels, int64_t ld, float* a, float* b,
                                                 int32_t* n_degenerate, void* stream) {
  using namespace qwt;
  if (fp_out == nullptr || q_out == nullptr || a == nullptr || b == nullptr) return QWT_ERR_NULL;
  if (rows < 1 || channels < 1 || ld < channels) return QWT_ERR_SHAPE;
  if (!aligned(fp_out, 16) || !aligned(q_out, 16) || (ld % 4) != 0) return QWT_ERR_ALIGN;

  // Same plan as qwt_cwac_calibrate, with fewer (longer) row chunks when its partial sums would not fit.
  CwacPlan plan = cwac_plan(rows, channels, kPlanSMs);
  const size_t per_chunk = (size_t)kPartialValues * plan.cpad * sizeof(double);
  if (per_chunk > kScratchBytes) return QWT_ERR_TOO_LARGE;       // more than 131072 channels
  if (plan.partial_bytes > kScratchBytes) {
    const int64_t max_chunks = (int64_t)(kScratchBytes / per_chunk);
    int64_t chunk_rows = (rows + max_chunks - 1) / max_chunks;
    chunk_rows = (chunk_rows + 7) / 8 * 8;
    plan.chunk_rows = chunk_rows;
    plan.chunks = (int)((rows + chunk_rows - 1) / chunk_rows);
    plan.partial_bytes = (size_t)plan.chunks * per_chunk;
  }

  DeviceInfo dev;
  qwt_status s = current_device(&dev);
  if (s != QWT_OK) return s;
  void* scratch = nullptr;
  if ((s = scratch_address(&scratch)) != QWT_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The statistics kernel writes every partial that the reduction reads, so nothing left in the array by
  // an earlier call can leak into this one and nothing has to be cleared first.
  if ((s = launch_cwac_stats(fp_out, q_out, rows, channels, ld, nullptr, scratch, plan, st)) != QWT_OK) return s;
  return launch_cwac_reduce(scratch, plan, channels, rows, nullptr, a, b, n_degenerate, st);
}
