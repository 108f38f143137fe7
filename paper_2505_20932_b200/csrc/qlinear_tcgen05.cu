// CWAC-fused quantized linear layer (Section 3.4, Eq. 6-11 with zero-points 0) for sm_100a.
//
// One persistent, warp-specialised kernel:
//   warp 0      TMA producer: per-CTA cp.async.bulk.tensor loads of the X tile [128 x 128 B] and the
//               W tile [BN x 128 B] into a ring of 128-byte-swizzled shared-memory stages
//   warp 1      MMA issuer: one thread issues tcgen05.mma kind::i8 (128 x BN x 32 per instruction) into a
//               TMEM accumulator; tcgen05.commit releases the stage / publishes the accumulator
//   warp 18     strip coordinator (per-token INT8 output only), see below
//   warps 19-22 (packed int4 weights only) expand the W tile to int8 in shared memory before the MMA
//   warps 2-17  epilogue: tcgen05.ld of the INT32 accumulators, z = fma(float(acc) * x_scale[m], fscale[n],
//               fbias[n]) (the folded M' and offset of Eq. 10-11), then the output stage.  TMEM holds
//               512 / BN accumulator buffers so the next tile's mainloop overlaps this epilogue.
//
// Per-token INT8 output needs max_n |z[m, n]| over the whole row, but a CTA owns only BN columns of it.
// Tiles are numbered strip-major (all column tiles of rows 0-127, then of rows 128-255, ...) and CTA c
// takes tiles c, c + G, c + 2G, ...  An epilogue warp computes z for its 32 x (BN/4) slice, keeps it in
// registers, releases the TMEM buffer, publishes its per-row maxima with atomicMax on the float bit
// pattern (non-negative floats order like unsigned integers) and increments its strip's arrival counter;
// it then waits until the counter shows every slice of the strip and emits the codes with the final row
// scale.  Progress: take the lowest-numbered tile t that has not published.  Its CTA's epilogue can only
// be waiting on an earlier tile t - kG, whose strip ends before t whenever tiles_n <= G, so every tile of
// that strip has published and the wait ends; the mainloop of t needs nothing but TMEM buffers that
// lower-numbered tiles free without waiting.  The grid is launched cooperatively so all G CTAs are
// resident.  Every wait is bounded; a wait that gives up records a code in the workspace status word and
// the CTA tears down normally.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include <mutex>

#include "ptx_sm100.cuh"
#include "qwt2_internal.h"

namespace qwt {

namespace {

constexpr int kBM = 128;           // rows of a CTA tile (= TMEM lanes)
constexpr int kBK = 128;           // bytes of K per stage: one 128-byte swizzle row
constexpr int kUmmaK = 32;         // K of one kind::i8 instruction
constexpr int kTmemCols = 512;
constexpr int kNumEpilogueWarps = 16;
constexpr int kCoordWarp = 2 + kNumEpilogueWarps;      // warp that talks to the other CTAs of a row strip
constexpr int kConvWarp0 = kCoordWarp + 1;              // first of 4 W4 -> INT8 converter warps (packed weights only)
constexpr int kNumConvWarps = 4;
constexpr int kThreadsW8 = 32 * (3 + kNumEpilogueWarps);
constexpr int kThreadsW4 = kThreadsW8 + 32 * kNumConvWarps;
constexpr int kABytes = kBM * kBK;

// status word codes (0 = clean)
enum : uint32_t {
  kStWaitEmpty = 1, kStWaitFull = 2, kStWaitTmemEmpty = 3, kStWaitTmemFull = 4, kStWaitStrip = 5,
};

struct QlParams {
  const float* x_scale;
  const float* fscale;
  const float* fbias;
  void* Y;
  float* y_scale;
  int M, N, K;
  int tiles_n, num_tiles, num_kb;
  uint32_t* status;
  uint32_t* rowmax;     // [M] bit patterns of non-negative floats
  uint32_t* counters;   // [tiles_m] tiles of the strip that have published their row maxima
  uint32_t* flags;      // [tiles_m] set by the last tile of the strip
  uint32_t counter_target;
  unsigned long long timeout_ns;
};

template <int BN, bool W4>
struct SmemLayout {
  static constexpr int kBBytes = BN * kBK;                 // expanded (int8) W tile of one stage
  static constexpr int kPBytes = W4 ? BN * (kBK / 2) : 0;  // packed (int4) W tile of one stage
  static constexpr int kStages = W4 ? ((BN == 256) ? 3 : 5) : ((BN == 256) ? 4 : 6);
  static constexpr int kAcc = kTmemCols / BN;
  static constexpr int kOffA = 0;
  static constexpr int kOffB = kOffA + kStages * kABytes;
  static constexpr int kOffP = kOffB + kStages * kBBytes;
  static constexpr int kOffFS = kOffP + kStages * kPBytes;         // float [epilogue warp][BN / 4], private per warp
  static constexpr int kOffFB = kOffFS + kNumEpilogueWarps * (BN / 4) * 4;
  static constexpr int kOffBars = kOffFB + kNumEpilogueWarps * (BN / 4) * 4;
  // full[S], empty[S], conv[S], tfull[A], tempty[A], drain, published, strip ready
  static constexpr int kNumBars = 3 * kStages + 2 * kAcc + 3;
  static constexpr int kOffMisc = kOffBars + kNumBars * 8;         // tmem base, abort word
  static constexpr int kTotal = kOffMisc + 16;
  static constexpr int kDynamic = kTotal + 1024;                   // slack to align the base to 1024
  static_assert(kDynamic <= 232448, "shared memory budget of one CTA");
};

__device__ __forceinline__ float epilogue_z(uint32_t acc_bits, float xs, float fs, float fb) {
  // Eq. 9 after the fold: (S_x acc) * (alpha S_W) + (alpha bias + beta)
  return fmaf(__fmul_rn(__int2float_rn((int)acc_bits), xs), fs, fb);
}

__device__ __forceinline__ void st_v4(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  *reinterpret_cast<uint4*>(p) = make_uint4(a, b, c, d);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int BN, int OUT, bool RCP, bool W4>
__global__ void __launch_bounds__(W4 ? kThreadsW4 : kThreadsW8, 1)
qlinear_cwac_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const QlParams p) {
  using L = SmemLayout<BN, W4>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem + L::kOffA;
  uint8_t* sB = smem + L::kOffB;
  uint8_t* sP = smem + L::kOffP;     // packed int4 tiles (W4 only)
  float* sFS = reinterpret_cast<float*>(smem + L::kOffFS);
  float* sFB = reinterpret_cast<float*>(smem + L::kOffFB);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::kOffBars);
  uint64_t* empty = full + L::kStages;
  uint64_t* conv = empty + L::kStages;     // W4 only: the stage's W tile has been expanded to int8
  uint64_t* tfull = conv + L::kStages;
  uint64_t* tempty = tfull + L::kAcc;
  uint64_t* drain = tempty + L::kAcc;
  uint64_t* pub_bar = drain + 1;     // 16 arrivals: every epilogue warp has issued its atomicMax
  uint64_t* ready_bar = drain + 2;   // 1 arrival: the strip's row maxima are final
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kOffMisc);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(smem + L::kOffMisc + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint64_t tmo = p.timeout_ns;

  if (threadIdx.x == 0) {
    for (int i = 0; i < L::kStages; ++i) {
      ptx::mbar_init(&full[i], 1);
      ptx::mbar_init(&empty[i], 1);
      ptx::mbar_init(&conv[i], kNumConvWarps);
    }
    for (int i = 0; i < L::kAcc; ++i) {
      ptx::mbar_init(&tfull[i], 1);
      ptx::mbar_init(&tempty[i], kNumEpilogueWarps);
    }
    ptx::mbar_init(drain, 1);
    ptx::mbar_init(pub_bar, kNumEpilogueWarps);
    ptx::mbar_init(ready_bar, 1);
    *cta_abort = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  auto give_up = [&](uint32_t code) {
    *cta_abort = 1;
    atomicCAS(p.status, 0u, code);
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t kbi = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x) {
        const int m0 = (tile / p.tiles_n) * kBM;
        const int n0 = (tile % p.tiles_n) * BN;
        for (int kb = 0; kb < p.num_kb; ++kb, ++kbi) {
          const uint32_t s = kbi % L::kStages;
          if (!ptx::mbar_wait_bounded(&empty[s], ((kbi / L::kStages) & 1u) ^ 1u, cta_abort, tmo)) {
            give_up(kStWaitEmpty);
            ok = false;
            break;
          }
          ptx::mbar_arrive_expect_tx(&full[s], kABytes + (W4 ? L::kPBytes : L::kBBytes));
          ptx::tma_load_2d(sA + s * kABytes, &tmA, kb * kBK, m0, &full[s]);
          if (W4) ptx::tma_load_2d(sP + s * L::kPBytes, &tmB, kb * (kBK / 2), n0, &full[s]);
          else ptx::tma_load_2d(sB + s * L::kBBytes, &tmB, kb * kBK, n0, &full[s]);
        }
      }
      if (*cta_abort != 0) {
        // let copies still in flight land before the CTA's shared memory is released
        const uint32_t first = kbi > (uint32_t)L::kStages ? kbi - L::kStages : 0u;
        for (uint32_t j = first; j < kbi; ++j) {
          uint32_t polls = 0;
          while (!ptx::mbar_try_wait(&full[j % L::kStages], (j / L::kStages) & 1u) && ++polls < (1u << 16)) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_i8(kBM, BN);
      const uint32_t a_base = ptx::smem_u32(sA), b_base = ptx::smem_u32(sB);
      uint32_t kbi = 0, it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x, ++it) {
        const uint32_t buf = it % L::kAcc;
        if (!ptx::mbar_wait_bounded(&tempty[buf], ((it / L::kAcc) & 1u) ^ 1u, cta_abort, tmo)) {
          give_up(kStWaitTmemEmpty);
          break;
        }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = 0; kb < p.num_kb; ++kb, ++kbi) {
          const uint32_t s = kbi % L::kStages;
          if (!ptx::mbar_wait_bounded(W4 ? &conv[s] : &full[s], (kbi / L::kStages) & 1u, cta_abort, tmo)) {
            give_up(kStWaitFull);
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint64_t a_desc = ptx::make_kmajor_sw128_desc(a_base + s * kABytes);
          const uint64_t b_desc = ptx::make_kmajor_sw128_desc(b_base + s * L::kBBytes);
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            // next 32 bytes of K inside the swizzled 128-byte row: start address + 32 B (>> 4 = 2)
            ptx::mma_i8_ss(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          ptx::tc_commit(&empty[s]);
        }
        if (ok) ptx::tc_commit(&tfull[buf]);
      }
      if (*cta_abort != 0) {
        // make sure no MMA is still running when TMEM is released
        ptx::tc_commit(drain);
        uint32_t polls = 0;
        while (!ptx::mbar_try_wait(drain, 0) && ++polls < (1u << 16)) {
        }
      }
    }
  } else if (W4 && warp >= kConvWarp0) {
    // ------------------------------------------------------------------ W4 -> INT8 converter warps
    // The packed tile (64 bytes per row, two's-complement nibbles, even element low) is expanded into the
    // 128-byte-swizzled operand tile the MMA descriptor expects.  Each nibble is moved to the HIGH half of
    // its byte, i.e. the operand holds 16 x code (|16 code| <= 112 fits int8); the factor 1/16 is exact in
    // the epilogue (fscale / 16, or an arithmetic shift of the raw accumulators).
    const int ct = threadIdx.x - kConvWarp0 * 32;          // 0..127
    uint32_t kbi = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x) {
      for (int kb = 0; kb < p.num_kb; ++kb, ++kbi) {
        const uint32_t s = kbi % L::kStages;
        if (!ptx::mbar_wait_bounded(&full[s], (kbi / L::kStages) & 1u, cta_abort, tmo)) {
          give_up(kStWaitFull);
          ok = false;
          break;
        }
        const uint8_t* src = sP + s * L::kPBytes;
        uint8_t* dst = sB + s * L::kBBytes;
#pragma unroll 2
        for (int q = ct; q < BN * 4; q += 32 * kNumConvWarps) {
          const int n = q >> 2, c = q & 3;                 // row of the tile, 16-byte chunk of the packed row
          const uint4 w = *reinterpret_cast<const uint4*>(src + n * 64 + c * 16);
          const uint32_t in[4] = {w.x, w.y, w.z, w.w};
          uint32_t out[8];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t lo = (in[i] << 4) & 0xF0F0F0F0u;   // even elements, nibble in the high half
            const uint32_t hi = in[i] & 0xF0F0F0F0u;          // odd elements
            out[2 * i] = __byte_perm(lo, hi, 0x5140);         // e0 e1 e2 e3
            out[2 * i + 1] = __byte_perm(lo, hi, 0x7362);     // e4 e5 e6 e7
          }
          uint8_t* row = dst + n * 128;
          const int sw = n & 7;                              // 128-byte swizzle: chunk ^= row % 8
          *reinterpret_cast<uint4*>(row + (((2 * c) ^ sw) << 4)) = make_uint4(out[0], out[1], out[2], out[3]);
          *reinterpret_cast<uint4*>(row + (((2 * c + 1) ^ sw) << 4)) = make_uint4(out[4], out[5], out[6], out[7]);
        }
        ptx::fence_proxy_async_smem();     // generic-proxy writes -> visible to the tensor core's async proxy
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&conv[s]);
      }
    }
  } else if (warp == kCoordWarp) {
    // ------------------------------------------------------------------ strip coordinator (INT8 output only)
    // One thread per CTA speaks for the tile: once the 16 epilogue warps have issued their row maxima it
    // counts the tile as published; the last tile of a strip raises the strip's flag, the others poll the
    // flag (a different word than the counter, with a back-off, so that arrivals are not queued behind
    // polls) and then release the epilogue warps.
    if (OUT == QWT_OUT_INT8_PER_TOKEN && lane == 0) {
      uint32_t it = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x, ++it) {
        const int tm = tile / p.tiles_n;
        if (!ptx::mbar_wait_bounded(pub_bar, it & 1u, cta_abort, tmo)) {
          give_up(kStWaitStrip);
          break;
        }
        __threadfence();     // the warps' atomicMax (seen through the barrier) before the count
        const uint32_t old = atomicAdd(p.counters + tm, 1u);
        if (old + 1u == p.counter_target) {
          __threadfence();
          ptx::st_release_gpu(p.flags + tm, 1u);
        } else {
          uint32_t polls = 0;
          uint64_t t0 = 0;
          bool failed = false;
          while (ptx::ld_acquire_gpu(p.flags + tm) == 0u) {
            __nanosleep(64);
            if ((++polls & 63u) == 0u) {
              const uint64_t now = ptx::globaltimer_ns();
              if (t0 == 0) t0 = now;
              if (*cta_abort != 0 || now - t0 > tmo || ptx::ld_acquire_gpu(p.status) != 0u) {
                failed = true;
                break;
              }
            }
          }
          if (failed) {
            give_up(kStWaitStrip);
            break;
          }
        }
        __threadfence();
        ptx::mbar_arrive(ready_bar);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    // 16 warps: TMEM lane quadrant = warp % 4 (hardware rule), column group = (warp - 2) / 4.
    // A warp owns 32 rows x CW columns of the tile; a thread owns one row of that.
    constexpr int CW = BN / (kNumEpilogueWarps / 4);
    const int qd = warp & 3;
    const int cg = (warp - 2) >> 2;
    // each warp stages its slice of fscale / fbias privately (no cross-warp barrier to get stuck on)
    float* fs = sFS + (warp - 2) * CW;
    float* fb = sFB + (warp - 2) * CW;
    uint32_t it = 0;
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x, ++it) {
      const uint32_t buf = it % L::kAcc;
      const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
      const int m0 = tm * kBM;
      const int n0 = tn * BN + cg * CW;          // first column of this warp's slice
      __syncwarp();   // every lane is done with the previous tile's slice
      if (OUT != QWT_OUT_INT32_ACC) {
        for (int i = lane; i < CW; i += 32) {
          const int c = n0 + i;
          fs[i] = c < p.N ? __ldg(p.fscale + c) * (W4 ? 0.0625f : 1.0f) : 0.f;   // W4 operands hold 16 x code
          fb[i] = c < p.N ? __ldg(p.fbias + c) : 0.f;
        }
      }
      __syncwarp();
      const int row = m0 + qd * 32 + lane;
      const bool row_ok = row < p.M;
      float xs = 0.f;
      if (OUT != QWT_OUT_INT32_ACC && row_ok) xs = __ldg(p.x_scale + row);

      if (!ptx::mbar_wait_bounded(&tfull[buf], (it / L::kAcc) & 1u, cta_abort, tmo)) {
        give_up(kStWaitTmemFull);
        break;
      }
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(qd * 32) << 16) + buf * BN + cg * CW;

      if (OUT == QWT_OUT_INT8_PER_TOKEN) {
        // z of the whole slice stays in registers; the accumulator buffer is released before the wait
        float z[CW];
        float amax = 0.f;
#pragma unroll
        for (int h = 0; h < CW / 32; ++h) {
          uint32_t r[32];
          ptx::tmem_ld_32x32b_x32(taddr + h * 32, r);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float4 f4 = *reinterpret_cast<const float4*>(fs + h * 32 + j);
            const float4 b4 = *reinterpret_cast<const float4*>(fb + h * 32 + j);
            z[h * 32 + j + 0] = epilogue_z(r[j + 0], xs, f4.x, b4.x);   // columns >= N give 0 * 0 + 0
            z[h * 32 + j + 1] = epilogue_z(r[j + 1], xs, f4.y, b4.y);
            z[h * 32 + j + 2] = epilogue_z(r[j + 2], xs, f4.z, b4.z);
            z[h * 32 + j + 3] = epilogue_z(r[j + 3], xs, f4.w, b4.w);
            amax = fmaxf(fmaxf(amax, fmaxf(fabsf(z[h * 32 + j]), fabsf(z[h * 32 + j + 1]))),
                         fmaxf(fabsf(z[h * 32 + j + 2]), fabsf(z[h * 32 + j + 3])));
          }
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&tempty[buf]);

        if (row_ok) atomicMax(p.rowmax + row, __float_as_uint(amax));
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(pub_bar);
        // the coordinator warp publishes the tile and waits for the rest of the strip
        if (!ptx::mbar_wait_bounded(ready_bar, it & 1u, cta_abort, tmo)) {
          give_up(kStWaitStrip);
          break;
        }
        float ys = 0.f;
        if (row_ok) {
          ys = __fdiv_rn(__uint_as_float(__ldcg(p.rowmax + row)), 127.f);
          if (tn == 0 && cg == 0) p.y_scale[row] = ys;
        }
        const float den = ys > 0.f ? ys : 1.f;       // a zero row has z == 0 everywhere: codes 0
        const float inv = __fdiv_rn(1.f, den);
        int8_t* yrow = static_cast<int8_t*>(p.Y) + (size_t)row * p.N + n0;
#pragma unroll
        for (int g = 0; g < CW / 16; ++g) {
          uint32_t w[4];
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            int q[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float zz = z[g * 16 + t * 4 + j];
              q[j] = __float2int_rn(RCP ? __fmul_rn(zz, inv) : __fdiv_rn(zz, den));   // |q| <= 127 by construction
            }
            const uint32_t lo = __byte_perm((uint32_t)q[0], (uint32_t)q[1], 0x0040);
            const uint32_t hi = __byte_perm((uint32_t)q[2], (uint32_t)q[3], 0x0040);
            w[t] = __byte_perm(lo, hi, 0x5410);
          }
          if (row_ok && n0 + g * 16 + 16 <= p.N) st_v4(yrow + g * 16, w[0], w[1], w[2], w[3]);
        }
      } else {
#pragma unroll
        for (int h = 0; h < CW / 32; ++h) {
          uint32_t r[32];
          ptx::tmem_ld_32x32b_x32(taddr + h * 32, r);
          ptx::tmem_ld_wait();
          const int c0 = n0 + h * 32;
          if (OUT == QWT_OUT_INT32_ACC) {
            if (W4) {
#pragma unroll
              for (int j = 0; j < 32; ++j) r[j] = (uint32_t)((int)r[j] >> 4);   // exact: every term is a multiple of 16
            }
            if (row_ok) {
              int32_t* yrow = static_cast<int32_t*>(p.Y) + (size_t)row * p.N + c0;
#pragma unroll
              for (int g = 0; g < 8; ++g)
                if (c0 + g * 4 + 4 <= p.N) st_v4(yrow + g * 4, r[g * 4], r[g * 4 + 1], r[g * 4 + 2], r[g * 4 + 3]);
            }
          } else {
            float z[32];
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const float4 f4 = *reinterpret_cast<const float4*>(fs + h * 32 + j);
              const float4 b4 = *reinterpret_cast<const float4*>(fb + h * 32 + j);
              z[j + 0] = epilogue_z(r[j + 0], xs, f4.x, b4.x);
              z[j + 1] = epilogue_z(r[j + 1], xs, f4.y, b4.y);
              z[j + 2] = epilogue_z(r[j + 2], xs, f4.z, b4.z);
              z[j + 3] = epilogue_z(r[j + 3], xs, f4.w, b4.w);
            }
            if (OUT == QWT_OUT_FP32) {
              if (row_ok) {
                float* yrow = static_cast<float*>(p.Y) + (size_t)row * p.N + c0;
#pragma unroll
                for (int g = 0; g < 8; ++g)
                  if (c0 + g * 4 + 4 <= p.N)
                    st_v4(yrow + g * 4, __float_as_uint(z[g * 4]), __float_as_uint(z[g * 4 + 1]),
                          __float_as_uint(z[g * 4 + 2]), __float_as_uint(z[g * 4 + 3]));
              }
            } else {  // BF16
              if (row_ok) {
                __nv_bfloat16* yrow = static_cast<__nv_bfloat16*>(p.Y) + (size_t)row * p.N + c0;
#pragma unroll
                for (int g = 0; g < 4; ++g)
                  if (c0 + g * 8 + 8 <= p.N)
                    st_v4(yrow + g * 8, pack_bf16x2(z[g * 8], z[g * 8 + 1]), pack_bf16x2(z[g * 8 + 2], z[g * 8 + 3]),
                          pack_bf16x2(z[g * 8 + 4], z[g * 8 + 5]), pack_bf16x2(z[g * 8 + 6], z[g * 8 + 7]));
              }
            }
          }
        }
        // accumulator buffer is free again
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&tempty[buf]);
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  });
  return fn;
}

// Row-major byte matrix [rows, row_bytes] -> map with a box of {box_bytes, box_rows}.
bool make_byte_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t row_bytes, uint32_t box_bytes,
                   uint32_t box_rows, CUtensorMapSwizzle swz) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {row_bytes, rows};
  cuuint64_t strides[1] = {row_bytes};
  cuuint32_t box[2] = {box_bytes, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

unsigned long long timeout_ns_from_env() {
  static unsigned long long v = [] {
    const char* e = getenv("QWT_TIMEOUT_MS");
    unsigned long long ms = 2000;
    if (e != nullptr) {
      const long long x = atoll(e);
      if (x > 0) ms = (unsigned long long)x;
    }
    return ms * 1000000ull;
  }();
  return v;
}

// QWT_REQUANT_RECIPROCAL=1 replaces the division z / y_scale by a multiplication with 1 / y_scale
// (codes may then differ from the division by one step on a few elements per million).
bool requant_by_reciprocal() {
  static const bool v = [] {
    const char* e = getenv("QWT_REQUANT_RECIPROCAL");
    return e != nullptr && e[0] == '1';
  }();
  return v;
}

template <int BN, int OUT, bool RCP, bool W4>
qwt_status launch_inst(const CUtensorMap& tmA, const CUtensorMap& tmB, const QlParams& prm, int grid,
                       bool cooperative, cudaStream_t st) {
  using L = SmemLayout<BN, W4>;
  constexpr int kThreads = W4 ? kThreadsW4 : kThreadsW8;
  auto kern = qlinear_cwac_kernel<BN, OUT, RCP, W4>;
  // per device and cheap, so it is simply set on every launch
  QWT_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamic));
  if (cooperative) {
    void* args[] = {(void*)&tmA, (void*)&tmB, (void*)&prm};
    QWT_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)kern, dim3(grid), dim3(kThreads), args, L::kDynamic, st));
    count_launch();
  } else {
    kern<<<grid, kThreads, L::kDynamic, st>>>(tmA, tmB, prm);
    QWT_LAUNCH_CHECK();
  }
  return QWT_OK;
}

template <int BN, bool W4>
qwt_status launch_bn(int out_mode, const CUtensorMap& tmA, const CUtensorMap& tmB, const QlParams& prm, int grid,
                     cudaStream_t st) {
  switch (out_mode) {
    case QWT_OUT_INT8_PER_TOKEN:
      if (requant_by_reciprocal())
        return launch_inst<BN, QWT_OUT_INT8_PER_TOKEN, true, W4>(tmA, tmB, prm, grid, true, st);
      return launch_inst<BN, QWT_OUT_INT8_PER_TOKEN, false, W4>(tmA, tmB, prm, grid, true, st);
    case QWT_OUT_BF16:
      return launch_inst<BN, QWT_OUT_BF16, false, W4>(tmA, tmB, prm, grid, false, st);
    case QWT_OUT_FP32:
      return launch_inst<BN, QWT_OUT_FP32, false, W4>(tmA, tmB, prm, grid, false, st);
    case QWT_OUT_INT32_ACC:
      return launch_inst<BN, QWT_OUT_INT32_ACC, false, W4>(tmA, tmB, prm, grid, false, st);
  }
  return QWT_ERR_UNSUPPORTED;
}

}  // namespace

qwt_status qlinear_plan(int32_t M, int32_t N, int32_t K, int32_t wfmt, int32_t out_mode, const DeviceInfo& dev,
                        QlinearPlan* plan) {
  (void)K;
  QlinearPlan pl{};
  pl.tiles_m = (M + kBM - 1) / kBM;
  // 256-wide tiles keep the tensor pipe ahead of shared-memory bandwidth; 128-wide ones are used when
  // the wider tile would leave many SMs without work.
  const int sms = dev.sm_count > 0 ? dev.sm_count : 148;
  auto score = [&](int bn) {
    const long tn = (N + bn - 1) / bn;
    const long tiles = (long)pl.tiles_m * tn;
    const long waves = (tiles + sms - 1) / sms;
    const double wave_eff = (double)tiles / (double)(waves * sms);   // SMs busy in the last round
    const double pad_eff = (double)N / (double)(tn * bn);            // useful columns of the tiles
    return wave_eff * pad_eff;
  };
  pl.bn = (N > 128 && score(256) + 0.05 >= score(128)) ? 256 : 128;
  const char* force = getenv("QWT_FORCE_BN");
  if (force != nullptr) {
    const int f = atoi(force);
    if (f == 128 || f == 256) pl.bn = f;
  }
  pl.tiles_n = (N + pl.bn - 1) / pl.bn;
  const long tiles = (long)pl.tiles_m * pl.tiles_n;
  pl.grid = (int)(tiles < sms ? tiles : sms);
  const bool w4 = wfmt == QWT_W_INT4_PACKED;
  pl.smem_bytes = pl.bn == 256 ? (w4 ? SmemLayout<256, true>::kDynamic : SmemLayout<256, false>::kDynamic)
                               : (w4 ? SmemLayout<128, true>::kDynamic : SmemLayout<128, false>::kDynamic);
  pl.fused_requant = (out_mode == QWT_OUT_INT8_PER_TOKEN) && (pl.tiles_n <= pl.grid);
  size_t off = 0;
  pl.ws_status_off = off;
  off += 256;
  pl.ws_rowmax_off = off;
  off += ((size_t)M * 4 + 255) / 256 * 256;
  pl.ws_counter_off = off;
  off += ((size_t)pl.tiles_m * 4 + 255) / 256 * 256;
  pl.ws_flag_off = off;
  off += ((size_t)pl.tiles_m * 4 + 255) / 256 * 256;
  pl.ws_z_off = off;
  if (out_mode == QWT_OUT_INT8_PER_TOKEN && !pl.fused_requant) off += (size_t)M * N * 4;
  pl.ws_total = off;
  *plan = pl;
  return QWT_OK;
}

qwt_status launch_qlinear(const int8_t* X, const float* x_scale, const void* W, int32_t wfmt, const float* fscale,
                          const float* fbias, int32_t M, int32_t N, int32_t K, int32_t out_mode, void* Y,
                          float* y_scale, void* workspace, const QlinearPlan& plan, cudaStream_t st) {
  const bool w4 = wfmt == QWT_W_INT4_PACKED;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  CUtensorMap tmA, tmB;
  const bool okA = make_byte_map(&tmA, X, (uint64_t)M, (uint64_t)K, kBK, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
  const bool okB = w4 ? make_byte_map(&tmB, W, (uint64_t)N, (uint64_t)K / 2, kBK / 2, (uint32_t)plan.bn,
                                      CU_TENSOR_MAP_SWIZZLE_NONE)
                      : make_byte_map(&tmB, W, (uint64_t)N, (uint64_t)K, kBK, (uint32_t)plan.bn,
                                      CU_TENSOR_MAP_SWIZZLE_128B);
  if (!okA || !okB) {
    set_cuda_error((int)cudaErrorInvalidValue);
    return QWT_ERR_CUDA;
  }
  // status word, row maxima and strip counters start at zero
  QWT_CUDA_TRY(cudaMemsetAsync(ws, 0, plan.ws_z_off, st));

  QlParams prm{};
  prm.x_scale = x_scale;
  prm.fscale = fscale;
  prm.fbias = fbias;
  prm.Y = Y;
  prm.y_scale = y_scale;
  prm.M = M;
  prm.N = N;
  prm.K = K;
  prm.tiles_n = plan.tiles_n;
  prm.num_tiles = plan.tiles_m * plan.tiles_n;
  prm.num_kb = (K + kBK - 1) / kBK;
  prm.status = reinterpret_cast<uint32_t*>(ws + plan.ws_status_off);
  prm.rowmax = reinterpret_cast<uint32_t*>(ws + plan.ws_rowmax_off);
  prm.counters = reinterpret_cast<uint32_t*>(ws + plan.ws_counter_off);
  prm.flags = reinterpret_cast<uint32_t*>(ws + plan.ws_flag_off);
  prm.counter_target = (uint32_t)plan.tiles_n;
  prm.timeout_ns = timeout_ns_from_env();

  int mode = out_mode;
  if (out_mode == QWT_OUT_INT8_PER_TOKEN && !plan.fused_requant) {
    // very wide layers (more column tiles than CTAs): z goes through FP32 scratch and a row quantizer
    mode = QWT_OUT_FP32;
    prm.Y = ws + plan.ws_z_off;
  }
  qwt_status s;
  if (w4) s = plan.bn == 256 ? launch_bn<256, true>(mode, tmA, tmB, prm, plan.grid, st)
                             : launch_bn<128, true>(mode, tmA, tmB, prm, plan.grid, st);
  else s = plan.bn == 256 ? launch_bn<256, false>(mode, tmA, tmB, prm, plan.grid, st)
                          : launch_bn<128, false>(mode, tmA, tmB, prm, plan.grid, st);
  if (s != QWT_OK) return s;
  if (mode != out_mode)
    return launch_quantize_rows(reinterpret_cast<const float*>(ws + plan.ws_z_off), M, N, N, 127,
                                static_cast<int8_t*>(Y), y_scale, st);
  return QWT_OK;
}

}  // namespace qwt
