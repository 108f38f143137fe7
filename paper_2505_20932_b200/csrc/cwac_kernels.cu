// CWAC calibration (Section 3.3, Eq. 3-5), fold (Section 3.4, Eq. 9-11) and the symmetric
// row quantizer (Eq. 1-2 with zero-point 0).  All kernels here are bandwidth bound.
#include <cuda_runtime.h>
#include <stdint.h>

#include "qwt2_internal.h"

namespace qwt {

// ------------------------------------------------------------------------------------------------
// Statistics pass.
//
// Grid = (column slabs of 128 channels) x (row chunks).  A block is 32 x 8 threads: a warp reads one
// row's 128 channels of q and of f as two coalesced 512-byte requests (16 bytes per lane); the eight
// warps of the block walk eight rows at a time.  Every thread owns 4 channels and keeps, for each of
// them, four running sums of the values *shifted by the chunk's first row* (dq = q - q0, df = f - f0):
//     sum dq, sum df, sum dq*df, sum dq*dq.
// The sums run in FP32 for FLUSH rows and are then added to FP64 accumulators, so FP32 only ever adds
// a handful of terms of the size of the channel's spread (the shift removes the mean), which keeps the
// variance and covariance accurate for channels whose mean is far from zero.  At the end of the chunk
// the four shifted sums and the two shifts are written as one partial per (chunk, value, channel), still in
// shifted form: a second kernel re-references every chunk to the shift of chunk 0 (a change of the size of the
// channel's spread, not of its mean), adds the chunks in a fixed order and solves Eq. 4-5 from sums that
// never held the square of the mean -- var(q) = E[q^2] - E[q]^2 on raw FP64 sums loses log10((mean/std)^2)
// digits.  No atomics, so results are reproducible.
// ------------------------------------------------------------------------------------------------
// Descriptors of a batched launch (passed by value as kernel parameters).
constexpr int kMaxBatch = 48;        // 48 descriptors of 80 bytes + the block offsets stay below the 4 KB of kernel parameters
struct StatsProblem {
  const float* fp_out;
  const float* q_out;
  double* partial;
  int64_t rows, ld, chunk_rows;
  int channels, cpad, slabs, pad_;
};
struct StatsBatch {
  int count;
  int block0[kMaxBatch + 1];
  StatsProblem prob[kMaxBatch];
};
struct ReduceProblem {
  const double* partial;
  float* a;
  float* b;
  const float* w_scale;
  const float* bias;
  float* fscale;
  float* fbias;
  double n_rows;
  int chunks, cpad, channels, chunk_rows;
};
struct ReduceBatch {
  int count;
  int block0[kMaxBatch + 1];
  ReduceProblem prob[kMaxBatch];
};
static_assert(sizeof(ReduceBatch) + sizeof(int*) <= 4096 && sizeof(StatsBatch) <= 4096, "kernel parameter space");

constexpr int kStatsTX = 32;
constexpr int kStatsTY = 8;
constexpr int kStatsThreads = kStatsTX * kStatsTY;
constexpr int kSlabChannels = kStatsTX * 4;
constexpr int kFlushRows = 16;   // rows per thread between FP32 -> FP64 flushes
constexpr int kBatchRows = 4;    // rows per thread whose loads are issued together

__device__ __forceinline__ float4 ld_stream(const float* p) {
  return __ldcs(reinterpret_cast<const float4*>(p));
}

// One block's work: column slab `slab`, row chunk `chunk` of one (fp_out, q_out) pair.
__device__ __forceinline__ void cwac_stats_block(const float* __restrict__ fp_out, const float* __restrict__ q_out,
                                                 int64_t rows, int channels, int64_t ld, int64_t chunk_rows,
                                                 double* __restrict__ partial, int cpad, int slab, int chunk) {
  const int tx = threadIdx.x & (kStatsTX - 1);
  const int ty = threadIdx.x / kStatsTX;
  const int c0 = slab * kSlabChannels + tx * 4;
  const int64_t r0 = (int64_t)chunk * chunk_rows;
  const int64_t r1 = (r0 + chunk_rows < rows) ? r0 + chunk_rows : rows;
  // c0 + 3 may pass `channels`, but ld % 4 == 0 and ld >= channels keep the 16-byte load inside the row
  const bool active = c0 < channels;

  float kq[4] = {0.f, 0.f, 0.f, 0.f}, kf[4] = {0.f, 0.f, 0.f, 0.f};
  if (active) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(q_out + r0 * ld + c0));
    const float4 b = __ldg(reinterpret_cast<const float4*>(fp_out + r0 * ld + c0));
    kq[0] = a.x; kq[1] = a.y; kq[2] = a.z; kq[3] = a.w;
    kf[0] = b.x; kf[1] = b.y; kf[2] = b.z; kf[3] = b.w;
  }

  // FP64 accumulators: one private slot per thread and sum in shared memory (the same array the block reduction
  // reads at the end), touched once per kFlushRows rows; in registers they would cost 32 of the thread's 128
  __shared__ double red[kStatsTY][16][kStatsTX];
#pragma unroll
  for (int i = 0; i < 16; ++i) red[ty][i][tx] = 0.0;

  if (active) {
    const float* qp = q_out + c0;
    const float* fp = fp_out + c0;
    for (int64_t rb = r0 + ty; rb < r1; rb += (int64_t)kStatsTY * kFlushRows) {
      float s[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) s[i] = 0.f;
#pragma unroll
      for (int g = 0; g < kFlushRows / kBatchRows; ++g) {
        float4 qv[kBatchRows], fv[kBatchRows];
#pragma unroll
        for (int i = 0; i < kBatchRows; ++i) {
          const int64_t r = rb + (int64_t)(g * kBatchRows + i) * kStatsTY;
          if (r < r1) {
            qv[i] = ld_stream(qp + r * ld);
            fv[i] = ld_stream(fp + r * ld);
          } else {  // shifted value 0: contributes nothing
            qv[i] = make_float4(kq[0], kq[1], kq[2], kq[3]);
            fv[i] = make_float4(kf[0], kf[1], kf[2], kf[3]);
          }
        }
#pragma unroll
        for (int i = 0; i < kBatchRows; ++i) {
          const float qa[4] = {qv[i].x, qv[i].y, qv[i].z, qv[i].w};
          const float fa[4] = {fv[i].x, fv[i].y, fv[i].z, fv[i].w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float dq = qa[j] - kq[j];
            const float df = fa[j] - kf[j];
            s[0 + j] += dq;
            s[4 + j] += df;
            s[8 + j] = fmaf(dq, df, s[8 + j]);
            s[12 + j] = fmaf(dq, dq, s[12 + j]);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < 16; ++i) red[ty][i][tx] += (double)s[i];
    }
  }

  // block reduction over the 8 row lanes, in a fixed order
  __shared__ float shift_q[kSlabChannels], shift_f[kSlabChannels];
  if (ty == 0) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      shift_q[tx * 4 + j] = kq[j];
      shift_f[tx * 4 + j] = kf[j];
    }
  }
  __syncthreads();
  if (threadIdx.x < kSlabChannels) {
    const int ch = threadIdx.x;           // channel inside the slab
    const int ltx = ch >> 2, j = ch & 3;
    const int c = slab * kSlabChannels + ch;
    double sd[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      double t = 0.0;
#pragma unroll
      for (int y = 0; y < kStatsTY; ++y) t += red[y][s * 4 + j][ltx];
      sd[s] = t;
    }
    // shifted sums and the shifts themselves (kPartialValues per chunk and channel)
    double* out = partial + (size_t)chunk * kPartialValues * cpad + c;
    out[0 * (size_t)cpad] = sd[0];
    out[1 * (size_t)cpad] = sd[1];
    out[2 * (size_t)cpad] = sd[2];
    out[3 * (size_t)cpad] = sd[3];
    out[4 * (size_t)cpad] = (double)shift_q[ch];
    out[5 * (size_t)cpad] = (double)shift_f[ch];
  }
}

// (two blocks per SM: 256 threads x 128 registers each is the whole register file)
__global__ void __launch_bounds__(kStatsThreads, 2)
cwac_stats_kernel(const float* __restrict__ fp_out, const float* __restrict__ q_out, int64_t rows, int channels,
                  int64_t ld, int64_t chunk_rows, double* __restrict__ partial, int cpad) {
  cwac_stats_block(fp_out, q_out, rows, channels, ld, chunk_rows, partial, cpad, (int)blockIdx.x, (int)blockIdx.y);
}

// Several pairs in one launch (the layers of a model): block b belongs to the problem p with
// block0[p] <= b < block0[p + 1] and does exactly what block (slab, chunk) of that problem's own launch would do,
// so the results are bit for bit those of the single calls; what goes away is one launch, ramp and tail per layer.
__global__ void __launch_bounds__(kStatsThreads, 2)
cwac_stats_batch_kernel(const __grid_constant__ StatsBatch sb) {
  int p = 0;
  while (p + 1 < sb.count && (int)blockIdx.x >= sb.block0[p + 1]) ++p;
  const StatsProblem pr = sb.prob[p];
  const int local = (int)blockIdx.x - sb.block0[p];
  cwac_stats_block(pr.fp_out, pr.q_out, pr.rows, pr.channels, pr.ld, pr.chunk_rows, pr.partial, pr.cpad,
                   local % pr.slabs, local / pr.slabs);
}

// Closed form of Eq. 4-5 from the five sums of one channel.
__device__ __forceinline__ void cwac_solve_channel(double n, double Sq, double Sf, double Sqf, double Sqq,
                                                   float* a, float* b, int* degenerate) {
  const double mq = Sq / n, mf = Sf / n;
  const double msq = Sqq / n;
  const double var = msq - mq * mq;
  const double cov = Sqf / n - mq * mf;
  double alpha;
  if (var <= 1e-12 * msq) {   // constant column / single row: every alpha minimises Eq. 3, take 1
    alpha = 1.0;
    *degenerate = 1;
  } else {
    alpha = cov / var;
    *degenerate = 0;
  }
  *a = (float)alpha;
  *b = (float)(mf - alpha * mq);
}

// The same from sums of values shifted by (Kq, Kf): variance and covariance do not see the shift, the means do.
__device__ __forceinline__ void cwac_solve_channel_shifted(double n, double s0, double s1, double s2, double s3,
                                                           double Kq, double Kf, float* a, float* b, int* degenerate) {
  const double dq = s0 / n, df = s1 / n;            // means of the shifted values
  const double var = s3 / n - dq * dq;
  const double cov = s2 / n - dq * df;
  const double mq = Kq + dq, mf = Kf + df;
  const double msq = var + mq * mq;                  // E[q^2]
  double alpha;
  if (var <= 1e-12 * msq) {
    alpha = 1.0;
    *degenerate = 1;
  } else {
    alpha = cov / var;
    *degenerate = 0;
  }
  *a = (float)alpha;
  *b = (float)(mf - alpha * mq);
}

// Adds the partials of all row chunks.  A block owns 32 channels; its 32 row lanes each add every 32nd
// chunk, then the lanes are combined in a fixed order, so the result does not depend on scheduling.
// stats_io (may be NULL): running statistics to update.  a, b (may be NULL): solve after the reduction.
constexpr int kRedTX = 32;
constexpr int kRedTY = 32;
__device__ __forceinline__ void cwac_reduce_block(const double* __restrict__ partial, int chunks, int cpad,
                                                  int channels, double n_rows, int chunk_rows,
                                                  double* __restrict__ stats_io,
                                                  float* __restrict__ a, float* __restrict__ b,
                                                  int* __restrict__ n_degenerate, int block,
                                                  const float* __restrict__ w_scale, const float* __restrict__ bias,
                                                  float* __restrict__ fscale, float* __restrict__ fbias) {
  const int tx = threadIdx.x & (kRedTX - 1);
  const int ty = threadIdx.x / kRedTX;
  const int c = block * kRedTX + tx;            // < cpad by construction of the grid
  double s[4] = {0.0, 0.0, 0.0, 0.0};
  double K0q = 0.0, K0f = 0.0;                  // reference shift: that of chunk 0
  if (c < channels) {
    K0q = partial[(size_t)4 * cpad + c];
    K0f = partial[(size_t)5 * cpad + c];
    for (int k = ty; k < chunks; k += kRedTY) {
      const double* p = partial + (size_t)k * kPartialValues * cpad + c;
      const double left = n_rows - (double)k * (double)chunk_rows;
      const double nb = left < (double)chunk_rows ? left : (double)chunk_rows;      // rows of this chunk
      const double d0 = p[0], d1 = p[(size_t)cpad], d2 = p[2 * (size_t)cpad], d3 = p[3 * (size_t)cpad];
      const double dq = p[4 * (size_t)cpad] - K0q, df = p[5 * (size_t)cpad] - K0f;
      s[0] += d0 + nb * dq;
      s[1] += d1 + nb * df;
      s[2] += d2 + df * d0 + dq * d1 + nb * dq * df;
      s[3] += d3 + 2.0 * dq * d0 + nb * dq * dq;
    }
  }
  __shared__ double red[kRedTY][4][kRedTX];
#pragma unroll
  for (int i = 0; i < 4; ++i) red[ty][i][tx] = s[i];
  __syncthreads();
  if (ty != 0 || c >= channels) return;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    double t = 0.0;
#pragma unroll 4      // (fully unrolled, the 128 loads of the four sums are hoisted and spill)
    for (int y = 0; y < kRedTY; ++y) t += red[y][i][tx];
    s[i] = t;
  }
  double n = n_rows;
  if (stats_io == nullptr && a != nullptr) {     // one-shot fit: solve from the shifted sums
    int deg;
    cwac_solve_channel_shifted(n, s[0], s[1], s[2], s[3], K0q, K0f, &a[c], &b[c], &deg);
    if (deg && n_degenerate != nullptr) atomicAdd(n_degenerate, 1);
    if (w_scale != nullptr) {     // Eq. 11 at once, the arithmetic of cwac_fold_kernel
      const float ai = a[c], bi = b[c];
      const float bs = bias ? bias[c] : 0.0f;
      fscale[c] = ai * w_scale[c];
      fbias[c] = fmaf(ai, bs, bi);
    }
    return;
  }
  {   // running statistics are raw sums (the interface of the streaming calls): undo the reference shift
    const double r0 = s[0], r1 = s[1];
    s[0] = r0 + n * K0q;
    s[1] = r1 + n * K0f;
    s[2] = s[2] + K0f * r0 + K0q * r1 + n * K0q * K0f;
    s[3] = s[3] + 2.0 * K0q * r0 + n * K0q * K0q;
  }
  if (stats_io != nullptr) {
    n += stats_io[c];
#pragma unroll
    for (int i = 0; i < 4; ++i) s[i] += stats_io[(size_t)(i + 1) * channels + c];
    stats_io[c] = n;
#pragma unroll
    for (int i = 0; i < 4; ++i) stats_io[(size_t)(i + 1) * channels + c] = s[i];
  }
  if (a != nullptr) {
    int deg;
    cwac_solve_channel(n, s[0], s[1], s[2], s[3], &a[c], &b[c], &deg);
    if (deg && n_degenerate != nullptr) atomicAdd(n_degenerate, 1);
    if (w_scale != nullptr) {     // Eq. 11 at once, the arithmetic of cwac_fold_kernel
      const float ai = a[c], bi = b[c];
      const float bs = bias ? bias[c] : 0.0f;
      fscale[c] = ai * w_scale[c];
      fbias[c] = fmaf(ai, bs, bi);
    }
  }
}

__global__ void __launch_bounds__(kRedTX * kRedTY)
cwac_reduce_kernel(const double* __restrict__ partial, int chunks, int cpad, int channels, double n_rows,
                   int chunk_rows, double* __restrict__ stats_io, float* __restrict__ a, float* __restrict__ b,
                   int* __restrict__ n_degenerate) {
  cwac_reduce_block(partial, chunks, cpad, channels, n_rows, chunk_rows, stats_io, a, b, n_degenerate, (int)blockIdx.x,
                    nullptr, nullptr, nullptr, nullptr);
}

__global__ void __launch_bounds__(kRedTX * kRedTY)
cwac_reduce_batch_kernel(const __grid_constant__ ReduceBatch rb, int* __restrict__ n_degenerate) {
  int p = 0;
#pragma unroll 1
  while (p + 1 < rb.count && (int)blockIdx.x >= rb.block0[p + 1]) ++p;
  const ReduceProblem* pr = rb.prob + p;
  cwac_reduce_block(pr->partial, pr->chunks, pr->cpad, pr->channels, pr->n_rows, pr->chunk_rows, nullptr, pr->a, pr->b,
                    n_degenerate,
                    (int)blockIdx.x - rb.block0[p], pr->w_scale, pr->bias, pr->fscale, pr->fbias);
}

__global__ void __launch_bounds__(128)
cwac_solve_kernel(const double* __restrict__ stats, int channels, float* __restrict__ a, float* __restrict__ b,
                  int* __restrict__ n_degenerate) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= channels) return;
  int deg;
  cwac_solve_channel(stats[c], stats[(size_t)channels + c], stats[2 * (size_t)channels + c],
                     stats[3 * (size_t)channels + c], stats[4 * (size_t)channels + c], &a[c], &b[c], &deg);
  if (deg && n_degenerate != nullptr) atomicAdd(n_degenerate, 1);
}

// Eq. 11: the static part of the multiplier and the additive term.
__global__ void __launch_bounds__(256)
cwac_fold_kernel(const float* __restrict__ w_scale, const float* __restrict__ bias, const float* __restrict__ a,
                 const float* __restrict__ b, int n, float* __restrict__ fscale, float* __restrict__ fbias) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float ai = a ? a[i] : 1.0f;
  const float bi = b ? b[i] : 0.0f;
  const float bs = bias ? bias[i] : 0.0f;
  fscale[i] = ai * w_scale[i];
  fbias[i] = fmaf(ai, bs, bi);
}

// Eq. 10-11 as printed, static scales: multiplier M' and the rounded accumulator offset, in float64.
__global__ void __launch_bounds__(256)
cwac_fold_static_kernel(const float* __restrict__ w_scale, const float* __restrict__ bias, const float* __restrict__ a,
                        const float* __restrict__ b, int n, double S_x, double S_r, float* __restrict__ mult,
                        int32_t* __restrict__ offset) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const double ai = a ? (double)a[i] : 1.0;
  const double bi = b ? (double)b[i] : 0.0;
  const double bs = bias ? (double)bias[i] : 0.0;
  const double step = ai * S_x * (double)w_scale[i];      // real value of one accumulator step after compensation
  mult[i] = (float)(step / S_r);
  const double off = step != 0.0 ? rint((ai * bs + bi) / step) : 0.0;
  offset[i] = (int32_t)fmin(fmax(off, -2147483647.0), 2147483647.0);
}

// Eq. 1-2 with zero-point 0: one warp per row, two passes over the row (the second hits cache).  VEC: 16-byte
// loads and 4-byte stores (cols and ld multiples of 4, 16-byte aligned X, 4-byte aligned Xq); same arithmetic
// per element either way.
template <bool VEC>
__global__ void __launch_bounds__(256)
quantize_rows_kernel(const float* __restrict__ X, int64_t rows, int cols, int64_t ld, float qmax,
                     int8_t* __restrict__ Xq, float* __restrict__ scale) {
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= rows) return;
  const float* x = X + r * ld;
  float m = 0.f;
  if (VEC) {
    const float4* x4 = reinterpret_cast<const float4*>(x);
    for (int c = lane; c < cols / 4; c += 32) {
      const float4 v = x4[c];
      m = fmaxf(fmaxf(m, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
    }
  } else {
    for (int c = lane; c < cols; c += 32) m = fmaxf(m, fabsf(x[c]));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  const float s = __fdiv_rn(m, qmax);
  if (lane == 0) scale[r] = s;
  int8_t* q = Xq + r * (int64_t)cols;
  auto code = [&](float xv) -> int {
    float v = rintf(__fdiv_rn(xv, s));
    v = fminf(fmaxf(v, -qmax), qmax);
    return (int)v;
  };
  if (VEC) {
    const float4* x4 = reinterpret_cast<const float4*>(x);
    uint32_t* q4 = reinterpret_cast<uint32_t*>(q);
    for (int c = lane; c < cols / 4; c += 32) {
      uint32_t w = 0u;
      if (s > 0.f) {
        const float4 v = x4[c];
        w = (uint32_t)(code(v.x) & 0xff) | ((uint32_t)(code(v.y) & 0xff) << 8) | ((uint32_t)(code(v.z) & 0xff) << 16) |
            ((uint32_t)(code(v.w) & 0xff) << 24);
      }
      q4[c] = w;
    }
  } else if (s > 0.f) {
    for (int c = lane; c < cols; c += 32) q[c] = (int8_t)code(x[c]);
  } else {
    for (int c = lane; c < cols; c += 32) q[c] = 0;
  }
}

// Eq. 1-2 as printed, one row at a time (one warp per row): s = (max - min) / 255, z = clip(rne(-min / s), 0, 255),
// code = clip(rne(x / s) + z, 0, 255); a constant row gets s = 1.  Also leaves the row's code sum, one of the
// terms of Eq. 7.
__global__ void __launch_bounds__(256)
quantize_rows_u8_kernel(const float* __restrict__ X, int64_t rows, int cols, int64_t ld, uint8_t* __restrict__ Xq,
                        float* __restrict__ scale, int32_t* __restrict__ zero, int32_t* __restrict__ rowsum) {
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= rows) return;
  const float* x = X + r * ld;
  float lo = x[0], hi = x[0];
  for (int c = lane; c < cols; c += 32) {
    lo = fminf(lo, x[c]);
    hi = fmaxf(hi, x[c]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
  }
  float s = __fdiv_rn(__fsub_rn(hi, lo), 255.f);
  if (!(s > 0.f)) s = 1.f;
  const float zf = fminf(fmaxf(rintf(__fdiv_rn(-lo, s)), 0.f), 255.f);
  uint8_t* q = Xq + r * (int64_t)cols;
  int sum = 0;
  for (int c = lane; c < cols; c += 32) {
    const float v = fminf(fmaxf(__fadd_rn(rintf(__fdiv_rn(x[c], s)), zf), 0.f), 255.f);
    q[c] = (uint8_t)(int)v;
    sum += (int)v;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) {
    scale[r] = s;
    zero[r] = (int)zf;
    if (rowsum != nullptr) rowsum[r] = sum;
  }
}

// Weight-side terms of Eq. 7, one warp per output channel: terms[n] = -Z_W[n], terms[N + n] = K Z_W[n] - sum_k W_q[n, k].
__global__ void __launch_bounds__(256)
asym_weight_terms_kernel(const uint8_t* __restrict__ W, const int32_t* __restrict__ w_zero, int N, int K,
                         int32_t* __restrict__ terms) {
  const int lane = threadIdx.x & 31;
  const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (n >= N) return;
  const uint8_t* w = W + (size_t)n * K;
  int sum = 0;
  for (int k = lane; k < K; k += 32) sum += w[k];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) {
    const int z = w_zero[n];
    terms[n] = -z;
    terms[N + n] = K * z - sum;
  }
}

// Patch matrix of a convolution (NHWC codes, zero-point 0): row (b, ho, wo), column (i, j, c) holds
// X[b, ho*stride + i - pad, wo*stride + j - pad, c], 0 outside the image.  16 bytes per thread (C % 16 == 0).
__global__ void __launch_bounds__(256)
im2col_i8_kernel(const int8_t* __restrict__ X, int Bn, int H, int W, int C, int kh, int kw, int stride, int pad, int Ho,
                 int Wo, int8_t* __restrict__ P) {
  const int chunks = C >> 4;                                   // 16-byte chunks per pixel
  const int64_t per_row = (int64_t)kh * kw * chunks;
  const int64_t total = (int64_t)Bn * Ho * Wo * per_row;
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= total) return;
  const int64_t rowi = t / per_row;
  const int rem = (int)(t - rowi * per_row);
  const int tap = rem / chunks, ch = rem - tap * chunks;
  const int i = tap / kw, j = tap - i * kw;
  const int wo = (int)(rowi % Wo);
  const int64_t bh = rowi / Wo;
  const int ho = (int)(bh % Ho), b = (int)(bh / Ho);
  const int y = ho * stride + i - pad, x = wo * stride + j - pad;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (y >= 0 && y < H && x >= 0 && x < W)
    v = *reinterpret_cast<const uint4*>(X + (((int64_t)b * H + y) * W + x) * C + ch * 16);
  *reinterpret_cast<uint4*>(P + rowi * ((int64_t)kh * kw * C) + (int64_t)tap * C + ch * 16) = v;
}

__global__ void __launch_bounds__(256)
pack_int4_kernel(const int8_t* __restrict__ codes, int64_t n_bytes, uint8_t* __restrict__ packed) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_bytes) return;
  const int lo = codes[2 * i], hi = codes[2 * i + 1];
  packed[i] = (uint8_t)((lo & 0xF) | ((hi & 0xF) << 4));
}

// Packed int4 -> int8 codes (two's-complement nibbles, even element in the low half): 16 packed bytes per thread.
__global__ void __launch_bounds__(256)
unpack_int4_kernel(const uint4* __restrict__ packed, int64_t n_vec, uint4* __restrict__ codes) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_vec) return;
  const uint4 w = __ldg(packed + i);
  const uint32_t in[4] = {w.x, w.y, w.z, w.w};
  uint32_t out[8];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    // sign extension of a nibble n: (n ^ 8) - 8, on four bytes at a time
    const uint32_t lo = __vsub4((in[k] & 0x0F0F0F0Fu) ^ 0x08080808u, 0x08080808u);         // even elements
    const uint32_t hi = __vsub4(((in[k] >> 4) & 0x0F0F0F0Fu) ^ 0x08080808u, 0x08080808u);  // odd elements
    out[2 * k] = __byte_perm(lo, hi, 0x5140);
    out[2 * k + 1] = __byte_perm(lo, hi, 0x7362);
  }
  codes[2 * i] = make_uint4(out[0], out[1], out[2], out[3]);
  codes[2 * i + 1] = make_uint4(out[4], out[5], out[6], out[7]);
}

// ------------------------------------------------------------------------------------------------ host side

CwacPlan cwac_plan(int64_t rows, int32_t channels, int /*sm_count*/) {
  // The plan is a function of the shape only, so that the workspace size and the summation order
  // (hence the bits of the result) do not depend on the device.  The statistics kernel keeps two
  // blocks resident per SM (148 x 2 = 296); the number of row chunks is chosen so that the grid fills
  // whole waves of 296 blocks as well as possible with as few chunks as possible.
  CwacPlan p;
  p.slabs = (channels + kSlabChannels - 1) / kSlabChannels;
  p.cpad = p.slabs * kSlabChannels;
  const int64_t resident = 296;
  const int64_t min_chunk = (int64_t)kStatsTY * kFlushRows;     // at least one full flush per thread
  const int64_t max_chunks = (rows + min_chunk - 1) / min_chunk;
  int64_t best_chunks = 1;
  double best_eff = -1.0;
  for (int waves = 1; waves <= 8; ++waves) {
    int64_t chunks = waves * resident / p.slabs;
    if (chunks < 1) chunks = 1;
    if (chunks > max_chunks) chunks = max_chunks;
    const int64_t blocks = chunks * p.slabs;
    const double eff = (double)blocks / (double)(((blocks + resident - 1) / resident) * resident);
    if (eff > best_eff + 0.02) {
      best_eff = eff;
      best_chunks = chunks;
    }
  }
  int64_t chunk_rows = (rows + best_chunks - 1) / best_chunks;
  chunk_rows = (chunk_rows + kStatsTY - 1) / kStatsTY * kStatsTY;
  p.chunk_rows = chunk_rows;
  p.chunks = (int)((rows + chunk_rows - 1) / chunk_rows);
  p.partial_bytes = (size_t)p.chunks * kPartialValues * p.cpad * sizeof(double);
  return p;
}

qwt_status launch_cwac_stats(const float* fp_out, const float* q_out, int64_t rows, int32_t channels, int64_t ld,
                             double* /*unused*/, void* workspace, const CwacPlan& plan, cudaStream_t st) {
  dim3 grid(plan.slabs, plan.chunks);
  cwac_stats_kernel<<<grid, kStatsThreads, 0, st>>>(fp_out, q_out, rows, channels, ld, plan.chunk_rows,
                                                    static_cast<double*>(workspace), plan.cpad);
  QWT_LAUNCH_CHECK();
  return QWT_OK;
}

qwt_status launch_cwac_reduce(const void* workspace, const CwacPlan& plan, int32_t channels, int64_t rows,
                              double* stats_io, float* a, float* b, int32_t* n_degenerate, cudaStream_t st) {
  if (a != nullptr && n_degenerate != nullptr) QWT_CUDA_TRY(cudaMemsetAsync(n_degenerate, 0, sizeof(int32_t), st));
  if (plan.chunk_rows > 0x7fffffffll) return QWT_ERR_SHAPE;
  cwac_reduce_kernel<<<(channels + kRedTX - 1) / kRedTX, kRedTX * kRedTY, 0, st>>>(
      static_cast<const double*>(workspace), plan.chunks, plan.cpad, channels, (double)rows, (int)plan.chunk_rows, stats_io,
      a, b, n_degenerate);
  QWT_LAUNCH_CHECK();
  return QWT_OK;
}

size_t cwac_batch_workspace_bytes(const CalibBatchItem* items, int32_t count) {
  size_t total = 0;
  for (int32_t i = 0; i < count; ++i)
    total += (cwac_plan(items[i].rows, items[i].channels, kPlanSMs).partial_bytes + 255) / 256 * 256;
  return total;
}

// Statistics of all problems in one launch, reduction + solve (+ fold) of all problems in a second one; more than
// kMaxBatch problems go in groups.
qwt_status launch_cwac_calibrate_batch(const CalibBatchItem* items, int32_t count, int32_t* n_degenerate,
                                       void* workspace, cudaStream_t st) {
  if (n_degenerate != nullptr) QWT_CUDA_TRY(cudaMemsetAsync(n_degenerate, 0, sizeof(int32_t), st));
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  size_t off = 0;
  for (int32_t g0 = 0; g0 < count; g0 += kMaxBatch) {
    const int n = count - g0 < kMaxBatch ? count - g0 : kMaxBatch;
    StatsBatch sb{};
    ReduceBatch rb{};
    sb.count = rb.count = n;
    int sblocks = 0, rblocks = 0;
    for (int i = 0; i < n; ++i) {
      const CalibBatchItem& it = items[g0 + i];
      const CwacPlan plan = cwac_plan(it.rows, it.channels, kPlanSMs);
      double* partial = reinterpret_cast<double*>(ws + off);
      off += (plan.partial_bytes + 255) / 256 * 256;
      sb.block0[i] = sblocks;
      sb.prob[i] = StatsProblem{it.fp_out, it.q_out, partial, it.rows, it.ld, plan.chunk_rows, it.channels, plan.cpad,
                                plan.slabs, 0};
      sblocks += plan.slabs * plan.chunks;
      rb.block0[i] = rblocks;
      if (plan.chunk_rows > 0x7fffffffll) return QWT_ERR_SHAPE;
      rb.prob[i] = ReduceProblem{partial, it.a, it.b, it.w_scale, it.bias, it.fscale, it.fbias, (double)it.rows,
                                 plan.chunks, plan.cpad, it.channels, (int)plan.chunk_rows};
      rblocks += (it.channels + kRedTX - 1) / kRedTX;
    }
    sb.block0[n] = sblocks;
    rb.block0[n] = rblocks;
    cwac_stats_batch_kernel<<<sblocks, kStatsThreads, 0, st>>>(sb);
    QWT_LAUNCH_CHECK();
    cwac_reduce_batch_kernel<<<rblocks, kRedTX * kRedTY, 0, st>>>(rb, n_degenerate);
    QWT_LAUNCH_CHECK();
  }
  return QWT_OK;
}

qwt_status launch_cwac_solve(const double* stats, int32_t channels, float* a, float* b, int32_t* n_degenerate,
                             cudaStream_t st) {
  if (n_degenerate != nullptr) QWT_CUDA_TRY(cudaMemsetAsync(n_degenerate, 0, sizeof(int32_t), st));
  cwac_solve_kernel<<<(channels + 127) / 128, 128, 0, st>>>(stats, channels, a, b, n_degenerate);
  QWT_LAUNCH_CHECK();
  return QWT_OK;
}

qwt_status launch_cwac_fold(const float* w_scale, const float* bias, const float* a, const float* b, int32_t n,
                            float* fscale, float* fbias, cudaStream_t st) {
  cwac_fold_kernel<<<(n + 255) / 256, 256, 0, st>>>(w_scale, bias, a, b, n, fscale, fbias);
  QWT_LAUNCH_CHECK();
  return QWT_OK;
}

qwt_status launch_cwac_fold_static(const float* w_scale, const float* bias, const float* a, const float* b, int32_t n,
                                   float S_x, float S_r, float* mult, int32_t* offset, cudaStream_t st) {
  cwac_fold_static_kernel<<<(n + 255) / 256, 256, 0, st>>>(w_scale, bias, a, b, n, (double)S_x, (double)S_r, mult,
                                                          offset);
  QWT_LAUNCH_CHECK();
  return QWT_OK;
}

qwt_status launch_quantize_rows(const float* X, int64_t rows, int32_t cols, int64_t ld, int32_t qmax, int8_t* Xq,
                                float* scale, cudaStream_t st) {
  const int rows_per_block = 8;
  const int64_t blocks = (rows + rows_per_block - 1) / rows_per_block;
  const bool vec = (cols % 4) == 0 && (ld % 4) == 0 && aligned(X, 16) && aligned(Xq, 4);
  if (vec) quantize_rows_kernel<true><<<(unsigned)blocks, rows_per_block * 32, 0, st>>>(X, rows, cols, ld, (float)qmax, Xq, scale);
  else quantize_rows_kernel<false><<<(unsigned)blocks, rows_per_block * 32, 0, st>>>(X, rows, cols, ld, (float)qmax, Xq, scale);
  QWT_LAUNCH_CHECK();
  return QWT_OK;
}

qwt_status launch_quantize_rows_u8(const float* X, int64_t rows, int32_t cols, int64_t ld, uint8_t* Xq, float* scale,
                                   int32_t* zero, int32_t* rowsum, cudaStream_t st) {
  const int rows_per_block = 8;
  const int64_t blocks = (rows + rows_per_block - 1) / rows_per_block;
  quantize_rows_u8_kernel<<<(unsigned)blocks, rows_per_block * 32, 0, st>>>(X, rows, cols, ld, Xq, scale, zero, rowsum);
  QWT_LAUNCH_CHECK();
  return QWT_OK;
}

qwt_status launch_asym_weight_terms(const uint8_t* W, const int32_t* w_zero, int32_t N, int32_t K, int32_t* w_terms,
                                    cudaStream_t st) {
  asym_weight_terms_kernel<<<(N + 7) / 8, 256, 0, st>>>(W, w_zero, N, K, w_terms);
  QWT_LAUNCH_CHECK();
  return QWT_OK;
}

qwt_status launch_im2col_i8(const int8_t* X, int32_t Bn, int32_t H, int32_t W, int32_t C, int32_t kh, int32_t kw,
                            int32_t stride, int32_t pad, int8_t* P, cudaStream_t st) {
  const int Ho = (H + 2 * pad - kh) / stride + 1, Wo = (W + 2 * pad - kw) / stride + 1;
  const int64_t total = (int64_t)Bn * Ho * Wo * kh * kw * (C / 16);
  im2col_i8_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(X, Bn, H, W, C, kh, kw, stride, pad, Ho, Wo, P);
  QWT_LAUNCH_CHECK();
  return QWT_OK;
}

qwt_status launch_pack_int4(const int8_t* codes, int64_t rows, int32_t cols, uint8_t* packed, cudaStream_t st) {
  const int64_t n_bytes = rows * (int64_t)(cols / 2);
  pack_int4_kernel<<<(unsigned)((n_bytes + 255) / 256), 256, 0, st>>>(codes, n_bytes, packed);
  QWT_LAUNCH_CHECK();
  return QWT_OK;
}

// packed: [rows, cols / 2] with cols % 32 == 0, 16-byte aligned; codes: int8 [rows, cols], 16-byte aligned
qwt_status launch_unpack_int4(const void* packed, int64_t rows, int32_t cols, int8_t* codes, cudaStream_t st) {
  const int64_t n_vec = rows * (int64_t)(cols / 32);
  unpack_int4_kernel<<<(unsigned)((n_vec + 255) / 256), 256, 0, st>>>(static_cast<const uint4*>(packed), n_vec,
                                                                     reinterpret_cast<uint4*>(codes));
  QWT_LAUNCH_CHECK();
  return QWT_OK;
}

}  // namespace qwt
