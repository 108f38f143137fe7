// CWAC-fused quantized linear layer (Section 3.4, Eq. 6-11 with zero-points 0) for sm_100a.
//
// One persistent, warp-specialised kernel; CTA c takes the 128 x BN output tiles c, c + G, c + 2G, ...
// (tiles are numbered strip-major: all column tiles of rows 0-127, then of rows 128-255, ...):
//   warp 0      TMA producer: per-CTA cp.async.bulk.tensor loads of the X tile [128 x 128 B] and the
//               W tile [BN x 128 B] into a ring of 128-byte-swizzled shared-memory stages.  For short K
//               the CTA's W tile is loaded once and stays resident; the ring then carries X only.
//   warp 1      MMA issuer: one thread issues tcgen05.mma kind::i8 (128 x BN x 32 per instruction) into one of
//               kAcc = 512 / BN TMEM accumulator buffers; tcgen05.commit releases the stage / publishes the buffer
//   warps 2-17  epilogue: 4 groups of 4 warps.  The work item of a group is a unit = 128 columns of a tile;
//               the CTA's units are dealt to the groups round-robin (the 512 TMEM columns hold 4 units).
//               Inside a group the warp's TMEM lane quadrant is warp % 4.  The accumulators are read with
//               tcgen05.ld.16x256b (the m16n8 fragment layout): a thread sees four rows and a quarter of the
//               columns, so a per-column parameter is loaded once and used four times -- with one row per
//               thread every lane needs every column's fscale/fbias and the shared-memory pipe bounds the
//               epilogue.  It forms z = fma(float(acc) * x_scale[m], fscale[n], fbias[n])
//               (the folded M' and offset of Eq. 10-11, two elements per packed-FP32 instruction), converts,
//               writes its words into a swizzled 32-row box in shared memory; the warp then re-deals its
//               lanes so that each global store instruction covers whole box rows (row-contiguous writes; rows
//               >= M and chunks >= N are predicated off).  The groups run out of phase, so the fixed
//               latencies of one group (waits, exchange) are covered by the arithmetic of the others.
//   warps 18-21 (packed int4 weights only) expand the W tile to int8 in shared memory before the MMA
//
// Per-token INT8 output needs max_n |z[m, n]| over the whole row, but a CTA owns only BN columns of it.
// The epilogue of a tile therefore has two phases and the accumulators stay in TMEM between them:
//   phase 1  z from the accumulators (written back to TMEM in their place) -> row maxima of the unit (combined
//            over the four lanes that share a row) -> published to the other CTAs of the strip:
//            as a tagged 8-byte word per row and unit (strips of at most 32 units), or by atomicMax on
//            rowmax[m] plus a strip counter and flag (wider layers); a row that lies inside one tile is settled
//            inside the CTA (one unit: nothing to do; two units: through shared memory), and so is a row of
//            exactly two tiles when the CTA takes whole strips (own strips);
//   phase 2  once the maxima of every unit of the strip are there, the rows' scales follow (the unit at column
//            0 writes y_scale); z is read back from TMEM, divided, rounded and stored as codes; only then is
//            the TMEM buffer released.
// While a group waits for its strip the other groups work on the following tiles.  Progress: phase 1 of
// tile t needs (a) its group, i.e. phase 2 of tile t - kAcc*G finished, and (b) its accumulator, whose
// buffer is released by that same phase 2; phase 2 of a tile u needs phase 1 of the tiles of u's strip, all
// numbered below u + tiles_n <= u + G.  Every dependency of phase 1 of t is thus a phase 1 of a lower-numbered
// tile, so by induction every phase 1 and then every phase 2 completes, provided all G CTAs are resident:
// the grid is launched cooperatively with G <= number of SMs and one CTA per SM.  Every wait is bounded; a
// wait that gives up records a code in the workspace status word and the CTA tears down normally.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include <atomic>
#include <mutex>
#include <type_traits>

#include "ptx_sm100.cuh"
#include "qwt2_internal.h"

namespace qwt {

namespace {

constexpr int kBM = 128;           // rows of a CTA tile (= TMEM lanes)
constexpr int kBK = 128;           // bytes of K per stage: one 128-byte swizzle row
constexpr int kUmmaK = 32;         // K of one kind::i8 instruction
constexpr int kTmemCols = 512;
constexpr int kMaxGatherWords = 32;   // per-token INT8: strips of up to this many units exchange tagged words
constexpr int kGroupWarps = 4;        // warps of an epilogue group (one per TMEM lane quadrant)
constexpr int kGroups = 4;            // epilogue groups; a group works on one 128-column unit of a tile at a time
// Columns of an epilogue unit: 128 in every mode (512 TMEM columns = 4 units in flight, one per group).  64-column
// units, which let the four groups share one tile, were measured slower on short-K layers and are left selectable here.
__host__ __device__ constexpr int unit_cols(int /*out_mode*/) { return 128; }
constexpr int kEpiWarps = kGroupWarps * kGroups;
constexpr int kNumConvWarps = 4;      // W4 -> INT8 converter warps (packed weights only)
constexpr int kABytes = kBM * kBK;
constexpr int kSmemBudget = 232448 - 1024;            // opt-in maximum of one CTA minus the slack to align the base

// status word codes (0 = clean)
enum : uint32_t {
  kStWaitEmpty = 1, kStWaitFull = 2, kStWaitTmemEmpty = 3, kStWaitTmemFull = 4, kStWaitStrip = 5, kStWaitParam = 6,
};

struct QlParams {
  const float* x_scale;
  const float* fscale;
  const float* fbias;
  void* Y;
  float* y_scale;
  int M, N, K;
  int tiles_n, num_tiles, num_kb;
  // the CTA's tile walk without divisions: CTA b has nl_mul * (nl_base + (b < nl_rem)) tiles; from one tile to the next
  // the (row strip, column tile) pair moves by (step_q, step_r) with carry (default walk: b, b + G, ...)
  int nl_base, nl_rem, nl_mul, step_q, step_r;
  int stages;           // depth of the operand ring in shared memory
  int res_kb;           // > 0: the CTA's W tile (all res_kb k-blocks) stays resident, the ring holds X only
  // Packed int4 weights with a resident W tile (CTA pairs): the tile arrives packed, once, and the epilogue warps expand
  // it into the resident buffer before their first unit; the operands then hold 16 x code and the epilogue divides
  // by 16 (w4_mul = 1/16 on fscale, offsets x 16, raw accumulators >> 4), exactly as with the converter warps.
  int w4_res;
  float w4_mul;
  uint32_t* status;
  unsigned long long* partial;   // [tiles_m][units per strip][128]: (tag, row maximum of the unit), zero = not yet there
  uint32_t counter_target;       // units of a row strip that lie inside the matrix
  int gather_words;              // exchange words per row: one per unit, or 0 = counter protocol for wide layers
  uint32_t* rowmax;              // counter protocol: [M] bit patterns of non-negative floats
  uint32_t* counters;            // [tiles_m] units of the strip that have published their row maxima
  uint32_t* flags;               // [tiles_m] raised by the unit that completes the strip
  unsigned long long timeout_ns;
  // asymmetric (unsigned) codes, Eq. 7 in full: acc = sum W_q x_q - Z_W[n] rsx[m] + Z_x[m] (K Z_W[n] - csw[n])
  const int* x_zero;             // [M] Z_x per token
  const int* x_rowsum;           // [M] rsx[m] = sum_k x_q[m, k]
  const int* w_terms;            // [2 N]: -Z_W[n], then K Z_W[n] - sum_k W_q[n, k]
  int local_pair;                // per-token INT8: a strip is one 256-wide tile of two units, exchanged inside the CTA
  int own_strips;                // per-token INT8: a strip is two 256-wide tiles, both taken by the same CTA
  // Convolution as an implicit GEMM (NHWC activations, rank-4 tensor maps): a tile's 128 rows are the output pixels of
  // a block of cv_bw x cv_bh positions of cv_bn images (powers of two, product 128; row r of the tile is pixel
  // (r % bw, (r / bw) % bh, r / (bw * bh)) of the block); a k-block is 128 input channels of one filter tap.
  struct Conv {
    int on;
    int bw_log, bh_log;            // log2 of the block's width and height (the rest of the 128 rows: images)
    int tiles_w, tiles_h;          // blocks per image row / column (row-strip index = (image block, block row, block column))
    int Wo, Ho, B;                 // output width, height, images
    int stride, pad, kw, cpb;      // cpb: 128-channel blocks per pixel
    int sub_w, sub_h;              // the 32 rows of an epilogue warp as (sub_w, sub_h, 32 / (sub_w * sub_h)) positions
    float x_scale;                 // per-tensor activation scale S_x
  } cv;
  // calibration statistics instead of an output matrix (Section 3.3, Eq. 4-5)
  const float* F;                // [M, ldf] full-precision output of the same layer on the same rows
  long long ldf;
  double* sums;                  // [tiles_m][6][cpad]: shifted sums of q, f, q f, q q over the rows of a strip, and the two shifts
  int cpad;
};

// Compile-time geometry of one instantiation.
template <int BN, int OUT, bool W4, int WIDE, bool ASYM = false, bool PAIR = false>
struct Cfg {
  // PAIR: two CTAs of a cluster work on two row strips of the same column tile; the even CTA issues MMAs of
  // M = 256 (tcgen05 cta_group::2) that take the A tile and half of the W tile from each CTA's shared memory
  static_assert(!PAIR || (!ASYM && OUT != kOutCalibStats && BN == 256), "CTA pairs: symmetric codes, 256-wide tiles");
  static constexpr bool kInt8Out = OUT == QWT_OUT_INT8_PER_TOKEN;     // dynamic per-token scale: two-phase epilogue
  static constexpr bool kStatic8 = OUT == QWT_OUT_INT8_STATIC;       // Eq. 10 as printed: static multiplier + offset
  static constexpr bool kCodes = kInt8Out || kStatic8;               // one byte per output element
  static constexpr bool kStats = OUT == kOutCalibStats;              // no output matrix: per-channel sums of Eq. 4-5
  static constexpr bool kTmaStore = !kStatic8 && !kStats;            // staging boxes leave by cp.async.bulk.tensor
  static constexpr bool kHasParams = OUT != QWT_OUT_INT32_ACC;       // x_scale / fscale / fbias are used
  static constexpr bool kNeedSlice = kHasParams || ASYM;             // per-column values staged in shared memory
  static constexpr int kEsz = kCodes ? 1 : (OUT == QWT_OUT_BF16 ? 2 : 4);
  static constexpr int kAcc = kTmemCols / BN;                        // accumulator buffers (tiles) in TMEM
  static constexpr int kUnitN = unit_cols(OUT);                      // columns of an epilogue unit
  static constexpr int kUPT = BN / kUnitN;                           // epilogue units per tile
  // Warps in groups of four (the unit of register reallocation): warps 0-3 = TMA producer, MMA issuer and two idle
  // warps; warps 4-19 = the four epilogue groups; warps 20-23 = the converter warps (packed weights only).
  static constexpr int kEpiWarp0 = 4;
  static constexpr int kConvWarp0 = kEpiWarp0 + kEpiWarps;           // first converter warp (W4 only)
  static constexpr int kThreads = 32 * (kEpiWarp0 + kEpiWarps + (W4 ? kNumConvWarps : 0));
  // Registers: the CTA starts with kLaunchRegs per thread (what the launch bounds allow); once the roles are known
  // the warps that need few give theirs back to the CTA's pool (setmaxnreg.dec) and the epilogue warps take them
  // (setmaxnreg.inc waits until the pool holds enough -- the pool is the CTA's own allocation and nothing else, so
  // the budgets below must add up to no more than the CTA started with):
  //   int8 weights   640 threads x 96 = 61440;  4 x 32 x 56 + 16 x 32 x 104 = 60416
  //   packed weights 768 threads x 80: left as launched (the converter warps want their 80, measured)
  static constexpr int kLaunchRegs = (65536 / kThreads) / 8 * 8;
  static constexpr int kRegsService = W4 ? kLaunchRegs : 56;
  static constexpr int kRegsConv = kLaunchRegs;
  static constexpr int kRegsEpi = W4 ? kLaunchRegs : 104;
  static_assert(kRegsService <= kLaunchRegs && kRegsConv <= kLaunchRegs && kRegsEpi >= kLaunchRegs, "dec / inc directions");
  static_assert(32 * (kEpiWarp0 * kRegsService + kEpiWarps * kRegsEpi + (W4 ? kNumConvWarps * kRegsConv : 0)) <=
                    kThreads * kLaunchRegs,
                "register budgets exceed what the CTA was launched with: setmaxnreg.inc would wait for ever");
  // output staging: one box of 32 rows per epilogue warp, through which a warp turns "thread = row" into
  // row-contiguous global stores.  128-byte rows for 128-wide tiles; 256-wide tiles use 32-byte rows when the
  // operand ring needs the room (long K: the epilogue hides behind the mainloop) and 64-byte rows otherwise
  // (statistics: the slot holds the warp's four sums and two shifts of the unit's 128 columns, 3 KB)
  static constexpr int kBoxBytes = kStats ? 96 : (BN == 128 ? (kStatic8 && kUnitN < 128 ? 64 : 128) : (WIDE == 1 ? 64 : 32));
  static constexpr int kBC = kBoxBytes / kEsz;                       // columns per box
  static constexpr int kSlotBytes = 32 * kBoxBytes;
  static constexpr int kStagingBytes = kEpiWarps * kSlotBytes;
  static constexpr int kBRows = PAIR ? BN / 2 : BN;                   // rows of the W tile this CTA loads
  static constexpr int kBBytes = kBRows * kBK;                       // expanded (int8) W tile of one stage
  static constexpr int kPBytes = W4 ? kBRows * (kBK / 2) : 0;        // packed (int4) W tile of one stage
  static constexpr int kStageBytes = kABytes + kBBytes + kPBytes;
  // per group and unit: fscale | fbias, and with asymmetric codes also the two integer column terms of Eq. 7
  static constexpr int kParamArrays = ASYM ? 4 : 2;
  static constexpr int kParamBytes = kGroups * kParamArrays * kUnitN * 4;
  // per-token INT8 with the whole row inside one tile: the tile's two units exchange their row maxima here
  // ([2 pairs of groups][2 buffers][2 units][128 rows] floats)
  static constexpr int kPairBytes = kInt8Out ? 2 * 2 * 2 * kBM * 4 : 0;
  static constexpr int kBarBytes = 512;
  static constexpr int kFixedBytes = kStagingBytes + kParamBytes + kPairBytes + kBarBytes;
  static constexpr int kMaxStages = 12;
  // full[S], empty[S], conv[S], tfull[A], tempty[A], pfull[4], pub[4], ready[4], gdone[4], drain, wfull
  static constexpr int kNumBars = 3 * kMaxStages + 2 * kAcc + 4 * kGroups + 2;
  static_assert(kNumBars * 8 + 16 <= kBarBytes, "barrier block");
  // Shared memory, in this order (every block a multiple of 1024 bytes):
  //   [resident W: res_kb x kBBytes] [X ring: stages x kABytes] [W ring: stages x kBBytes, streaming only]
  //   [packed W ring, int4 only] [output staging] [fscale|fbias] [barriers]
  // Streaming: every stage carries an X and a W k-block.  Resident: the CTA's W tile is loaded once.
  __host__ __device__ static constexpr int stage_bytes(bool resident) { return resident ? kABytes : kStageBytes; }
  __host__ __device__ static constexpr int stages_for(int res_kb) {
    const int avail = kSmemBudget - kFixedBytes - res_kb * kBBytes;
    if (avail <= 0) return 0;
    const int n = avail / stage_bytes(res_kb > 0);
    return n > kMaxStages ? kMaxStages : n;
  }
  __host__ __device__ static constexpr int ring_bytes(int stages, int res_kb) {
    return res_kb * kBBytes + stages * stage_bytes(res_kb > 0);
  }
  __host__ __device__ static constexpr int dynamic_bytes(int stages, int res_kb) {
    return ring_bytes(stages, res_kb) + kFixedBytes + 1024;         // slack to align the base to 1024
  }
  static_assert(stages_for(0) >= 3, "shared memory budget of one CTA");
};

// 16-byte chunk index XOR of the TMA shared-memory swizzle for a dense box whose rows are BOXB bytes long.
template <int BOXB>
__device__ __forceinline__ uint32_t swizzle_xor(int row) {
  return BOXB == 32 ? ((row >> 2) & 1) : (BOXB == 64 ? ((row >> 1) & 3) : (row & 7));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Eq. 9 after the fold for two neighbouring columns: (S_x acc) * (alpha S_W) + (alpha bias + beta)
__device__ __forceinline__ float2 z_pair(uint32_t a0, uint32_t a1, float2 xs2, float f0, float f1, float b0,
                                         float b1) {
  const float2 a = make_float2(__int2float_rn((int)a0), __int2float_rn((int)a1));
  return __ffma2_rn(__fmul2_rn(a, xs2), make_float2(f0, f1), make_float2(b0, b1));
}

// The tiles of one CTA in the order it takes them, as (row strip, column tile), advanced without divisions.
// Default: tiles b, b + G, b + 2G, ... of the strip-major numbering.  Own strips: the strips b, b + G, ... and every
// column tile of each in turn.
struct TileWalk {
  int tm, tn;        // current tile
  int ord;           // own strips: ordinal of the current strip among this CTA's strips
  int tiles_n, step_q, step_r, G;
  bool own;
  __device__ __forceinline__ void init(const QlParams& p, int b, int G_) {
    tiles_n = p.tiles_n;
    step_q = p.step_q;
    step_r = p.step_r;
    G = G_;
    own = p.own_strips != 0;
    ord = 0;
    if (own) {
      tm = b;
      tn = 0;
    } else {
      tm = b / tiles_n;            // the only division of the walk
      tn = b - tm * tiles_n;
    }
  }
  __device__ __forceinline__ void advance() {
    if (own) {
      if (++tn == tiles_n) {
        tn = 0;
        tm += G;
        ++ord;
      }
    } else {
      tn += step_r;
      tm += step_q;
      if (tn >= tiles_n) {
        tn -= tiles_n;
        ++tm;
      }
    }
  }
  __device__ __forceinline__ void advance(int n) {
    for (int i = 0; i < n; ++i) advance();
  }
};

template <int BN, int OUT, bool W4, int WIDE, bool ASYM, bool PAIR>
__global__ void __launch_bounds__((Cfg<BN, OUT, W4, WIDE, ASYM, PAIR>::kThreads), 1)
qlinear_cwac_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmY, const QlParams p) {
  using C = Cfg<BN, OUT, W4, WIDE, ASYM, PAIR>;
  constexpr int kAcc = C::kAcc;
  constexpr int kMaxStages = C::kMaxStages;
  const int stages = p.stages;
  const bool resident = p.res_kb > 0;      // the CTA's W tile is loaded once; the ring carries X only
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sWres = smem;                                               // [res_kb][BN x 128 B]
  uint8_t* sA = sWres + p.res_kb * C::kBBytes;                         // [stages][128 x 128 B]
  uint8_t* sB = sA + stages * kABytes;                                 // [stages][BN x 128 B] (streaming)
  uint8_t* sP = sB + (resident ? 0 : stages * C::kBBytes);             // [stages][BN x 64 B] packed int4 (W4 only)
  uint8_t* sStage = smem + C::ring_bytes(stages, p.res_kb);
  float* sParam = reinterpret_cast<float*>(sStage + C::kStagingBytes);      // [group][fscale 128 | fbias 128]
  float* sPair = reinterpret_cast<float*>(sStage + C::kStagingBytes + C::kParamBytes);
  uint8_t* sBars = sStage + C::kStagingBytes + C::kParamBytes + C::kPairBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(sBars);
  uint64_t* empty = full + kMaxStages;
  uint64_t* conv = empty + kMaxStages;   // W4 only: the stage's W tile has been expanded to int8
  uint64_t* tfull = conv + kMaxStages;   // accumulator buffer complete (MMA -> epilogue)
  uint64_t* tempty = tfull + kAcc;       // accumulator buffer free (every warp that read it -> MMA)
  uint64_t* pfull = tempty + kAcc;       // per group: fscale / fbias slice of its unit is in shared memory (lead warp)
  uint64_t* pub = pfull + kGroups;       // per group: its 4 warps have issued the unit's row maxima
  uint64_t* ready = pub + kGroups;       // per group: the strip's row maxima are final
  uint64_t* gdone = ready + kGroups;     // per group: its 4 warps have finished the unit (parameter slice reusable)
  uint64_t* drain = gdone + kGroups;
  uint64_t* wfull = drain + 1;           // resident W tile has landed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sBars + C::kBarBytes - 16);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(sBars + C::kBarBytes - 12);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint64_t tmo = p.timeout_ns;
  // CTA pairs: the pair is the unit of the tile walk; this CTA's row strip is 2 * (the walk's strip) + its rank
  const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;
  const int G = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int walker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;      // index of this CTA (pair) in the walk
  auto strip_of = [&](int walk_tm) { return PAIR ? 2 * walk_tm + (int)rank : walk_tm; };
  // Tiles of this CTA, in the order it takes them.  Default: b, b + G, b + 2G, ...  With own strips (per-token INT8
  // whose rows span exactly two column tiles): the strips b, b + G, ... and both column tiles of each in turn, so
  // that a row's maxima never leave the CTA.
  const int n_local = p.nl_mul * (p.nl_base + (walker < p.nl_rem ? 1 : 0));

  if (warp == 0) {
    // the barriers lie one after the other in shared memory; the lanes of warp 0 initialise them side by side
    // (one thread doing all of them costs the CTA most of a microsecond before its first load)
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmA);
      ptx::prefetch_tensormap(&tmB);
      if (C::kTmaStore) ptx::prefetch_tensormap(&tmY);
      *cta_abort = 0;
    }
    for (int i = lane; i < C::kNumBars; i += 32) {
      uint32_t count = 1;                                            // full, empty, tfull, pfull, ready, drain, wfull
      if (i >= 2 * kMaxStages && i < 3 * kMaxStages) count = (kNumConvWarps / 2) * (PAIR ? 2 : 1);   // conv: a team
      // packed resident tile: conv[0] counts the packed tile's bytes, conv[1] this CTA's expanding warps (the ring is
      // free for X), conv[2] (even CTA) the expanding warps of both CTAs (the MMAs may start)
      if (!W4 && p.w4_res && i >= 2 * kMaxStages && i < 2 * kMaxStages + 3)
        count = i == 2 * kMaxStages ? 1 : (i == 2 * kMaxStages + 1 ? kEpiWarps : 2 * kEpiWarps);
      else if (i >= 3 * kMaxStages + kAcc && i < 3 * kMaxStages + 2 * kAcc)
        count = kGroupWarps * C::kUPT * (PAIR ? 2 : 1);              // tempty (pairs: the warps of both CTAs)
      else if (i >= 3 * kMaxStages + 2 * kAcc + kGroups && i < 3 * kMaxStages + 2 * kAcc + 2 * kGroups)
        // pub (in-CTA exchange of a tile's two units: pub[g & ~1] counts the warps of both groups; own strips:
        // pub[0] counts the warps of all the strip's units)
        count = p.own_strips ? kGroupWarps * p.counter_target : (p.local_pair ? 2 * kGroupWarps : kGroupWarps);
      else if (i >= 3 * kMaxStages + 2 * kAcc + 3 * kGroups && i < 3 * kMaxStages + 2 * kAcc + 4 * kGroups)
        count = kGroupWarps;                                                                       // gdone
      ptx::mbar_init(&full[i], count);
    }
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    if (PAIR) {
      ptx::tmem_alloc_pair(tmem_slot, kTmemCols);
      ptx::tmem_relinquish_pair();
    } else {
      ptx::tmem_alloc(tmem_slot, kTmemCols);
      ptx::tmem_relinquish();
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (PAIR) {       // the peer's barriers must exist before anything of this CTA signals them
    ptx::cluster_arrive();
    ptx::cluster_wait();
  }
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Everything above touched only this CTA's shared and tensor memory.  From here on global memory is read and written:
  // with a programmatic launch (the kernel may have started under the tail of the one before it in the stream) wait for
  // that kernel to finish first.
  ptx::grid_dependency_wait();

  // Without the INT8 exchange nothing else in the workspace is used: the first CTA clears the status word
  // (a wait can only give up seconds later).
  if ((!C::kInt8Out || p.counter_target <= 1u || p.local_pair || p.own_strips) && blockIdx.x == 0 && threadIdx.x == 0)
    *p.status = 0u;

  auto give_up = [&](uint32_t code) {
    *cta_abort = 1;
    if (PAIR) ptx::st_shared_cluster_u32(ptx::mapa_shared(ptx::smem_u32(const_cast<int*>(cta_abort)), rank ^ 1u), 1u);
    atomicCAS(p.status, 0u, code);
  };

  // Registers move from the service (and converter) warps to the epilogue warps; each group of four warps does so at
  // the top of its own branch, so that the compiler budgets the code below it accordingly.
  if (warp < C::kEpiWarp0) {
  if (C::kRegsService < C::kLaunchRegs) ptx::setmaxnreg_dec<C::kRegsService>();
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      if (resident) {
        // With a grid that is a multiple of tiles_n every tile of this CTA has the same column tile: its W
        // tile is loaded once and the ring below streams X only (half the bytes per tile through the SM's
        // load port, which is what bounds short-K layers).
        const int n0 = (walker % p.tiles_n) * BN + (int)rank * C::kBRows;      // (one modulo per call)
        if (PAIR && !W4 && p.w4_res) {
          // the packed half tile (64 bytes per row and k-block) lands in the top end of the still unused X ring; the
          // stages it covers are filled with X only when the epilogue warps have expanded it into the resident buffer
          // (the first X loads, into the stages below it, are under way meanwhile)
          constexpr int kPackedKb = C::kBRows * (kBK / 2);
          uint8_t* const packed = sA + stages * kABytes - p.res_kb * kPackedKb;
          ptx::mbar_arrive_expect_tx(&conv[0], (uint32_t)(p.res_kb * kPackedKb));
          for (int kb = 0; kb < p.res_kb; ++kb) ptx::tma_load_2d(packed + kb * kPackedKb, &tmB, kb * (kBK / 2), n0, &conv[0]);
        } else if (PAIR) {
          // each CTA keeps its half of the pair's W tile; both halves are counted on the even CTA's barrier
          const uint32_t lead_wfull = ptx::mapa_shared(ptx::smem_u32(wfull), 0u);
          if (rank == 0u) ptx::mbar_arrive_expect_tx(wfull, 2u * (uint32_t)(p.res_kb * C::kBBytes));
          for (int kb = 0; kb < p.res_kb; ++kb)
            ptx::tma_load_2d_pair(sWres + kb * C::kBBytes, &tmB, kb * kBK, n0, lead_wfull);
        } else {
          ptx::mbar_arrive_expect_tx(wfull, (uint32_t)(p.res_kb * C::kBBytes));
          for (int kb = 0; kb < p.res_kb; ++kb) ptx::tma_load_2d(sWres + kb * C::kBBytes, &tmB, kb * kBK, n0, wfull);
        }
      }
      uint32_t issued = 0, s = 0, ph = 0;
      bool ok = true;
      // packed resident tile: first ring stage that overlaps the packed tile's landing area
      const uint32_t held_from = (PAIR && !W4 && p.w4_res)
                                     ? (uint32_t)((stages * kABytes - p.res_kb * C::kBRows * (kBK / 2)) / kABytes)
                                     : 0xffffffffu;
      TileWalk walk;
      walk.init(p, walker, G);
      for (int jt = 0; ok && jt < n_local; ++jt, walk.advance()) {
        // With its last tile under way this CTA lets the kernel behind this one in the stream begin: that kernel's CTAs
        // take the SMs as they fall free, do their set-up and wait for this kernel's end before they touch global
        // memory.  (Earlier would be no use, a waiting CTA only holds an SM that another stream's kernel could work on.)
        if (jt + 1 >= n_local) ptx::grid_launch_dependents();
        const int m0 = strip_of(walk.tm) * kBM;
        const int n0 = walk.tn * BN;
        for (int kb = 0; kb < p.num_kb; ++kb, ++issued) {
          if (!ptx::mbar_wait_bounded(&empty[s], ph ^ 1u, cta_abort, tmo)) {
            give_up(kStWaitEmpty);
            ok = false;
            break;
          }
          if (issued == held_from && !ptx::mbar_wait_bounded(&conv[1], 0, cta_abort, tmo)) {
            give_up(kStWaitFull);
            ok = false;
            break;
          }
          if (!PAIR && !W4 && p.cv.on) {
            // implicit GEMM: the activations of one filter tap, 128 channels, for the tile's block of output pixels
            // (zero outside the image: the zero-point of the symmetric codes)
            const int tap = kb / p.cv.cpb, cb = kb - tap * p.cv.cpb;
            const int fi = tap / p.cv.kw, fj = tap - fi * p.cv.kw;
            const int tw = walk.tm % p.cv.tiles_w, t2 = walk.tm / p.cv.tiles_w;
            const int th = t2 % p.cv.tiles_h, tb = t2 / p.cv.tiles_h;
            ptx::mbar_arrive_expect_tx(&full[s], kABytes + C::kBBytes);
            ptx::tma_load_4d(sA + s * kABytes, &tmA, cb * kBK, ((tw << p.cv.bw_log) * p.cv.stride) + fj - p.cv.pad,
                             ((th << p.cv.bh_log) * p.cv.stride) + fi - p.cv.pad,
                             tb << (7 - p.cv.bw_log - p.cv.bh_log), &full[s]);
            ptx::tma_load_2d(sB + s * C::kBBytes, &tmB, kb * kBK, n0, &full[s]);
          } else if (PAIR && W4) {
            // packed weights: a CTA's loads are counted on its own barrier, for its own converter warps, which then
            // report to the even CTA
            ptx::mbar_arrive_expect_tx(&full[s], kABytes + C::kPBytes);
            ptx::tma_load_2d(sA + s * kABytes, &tmA, kb * kBK, m0, &full[s]);
            ptx::tma_load_2d(sP + s * C::kPBytes, &tmB, kb * (kBK / 2), n0 + (int)rank * C::kBRows, &full[s]);
          } else if (PAIR) {
            // both CTAs' loads of the stage are counted on the even CTA's barrier, where the MMAs are issued
            const uint32_t lead_full = ptx::mapa_shared(ptx::smem_u32(&full[s]), 0u);
            if (rank == 0u) ptx::mbar_arrive_expect_tx(&full[s], 2u * (kABytes + (resident ? 0 : C::kBBytes)));
            ptx::tma_load_2d_pair(sA + s * kABytes, &tmA, kb * kBK, m0, lead_full);
            if (!resident)
              ptx::tma_load_2d_pair(sB + s * C::kBBytes, &tmB, kb * kBK, n0 + (int)rank * C::kBRows, lead_full);
          } else if (resident) {
            ptx::mbar_arrive_expect_tx(&full[s], kABytes);
            ptx::tma_load_2d(sA + s * kABytes, &tmA, kb * kBK, m0, &full[s]);
          } else {
            ptx::mbar_arrive_expect_tx(&full[s], kABytes + (W4 ? C::kPBytes : C::kBBytes));
            ptx::tma_load_2d(sA + s * kABytes, &tmA, kb * kBK, m0, &full[s]);
            if (W4) ptx::tma_load_2d(sP + s * C::kPBytes, &tmB, kb * (kBK / 2), n0, &full[s]);
            else ptx::tma_load_2d(sB + s * C::kBBytes, &tmB, kb * kBK, n0, &full[s]);
          }
          if (++s == (uint32_t)stages) {
            s = 0;
            ph ^= 1u;
          }
        }
      }
      if (*cta_abort != 0 && !W4 && p.w4_res) {      // the packed tile's copies (counted in this CTA)
        uint32_t polls = 0;
        while (!ptx::mbar_try_wait(&conv[0], 0) && ++polls < (1u << 16)) {
        }
      }
      if (*cta_abort != 0 && (rank == 0u || W4)) {
        // let copies still in flight land before the CTA's shared memory is released (pairs: the even CTA's
        // barriers count the loads of both, and the odd CTA stays until the pair's final synchronisation)
        const uint32_t back = issued < (uint32_t)stages ? issued : (uint32_t)stages;
        for (uint32_t j = 0; j < back; ++j) {
          // walk back over the last `back` issues: stage and phase of issue number issued - 1 - j
          const uint32_t n = issued - 1 - j;
          uint32_t polls = 0;
          while (!ptx::mbar_try_wait(&full[n % stages], (n / stages) & 1u) && ++polls < (1u << 16)) {
          }
        }
        if (resident && !(!W4 && p.w4_res)) {
          uint32_t polls = 0;
          while (!ptx::mbar_try_wait(wfull, 0) && ++polls < (1u << 16)) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0u) {
      constexpr uint32_t idesc = ASYM ? ptx::make_idesc_u8(kBM, BN) : ptx::make_idesc_i8(PAIR ? 2 * kBM : kBM, BN);
      const uint32_t a_base = ptx::smem_u32(sA), b_base = ptx::smem_u32(sB), w_base = ptx::smem_u32(sWres);
      uint32_t s = 0, ph = 0, it = 0;
      bool ok = true;
      if (resident && !ptx::mbar_wait_bounded((!W4 && p.w4_res) ? &conv[2] : wfull, 0, cta_abort, tmo)) {
        give_up(kStWaitFull);
        ok = false;
      }
      for (int jt = 0; ok && jt < n_local; ++jt, ++it) {
        const uint32_t buf = it % kAcc;
        if (!ptx::mbar_wait_bounded(&tempty[buf], ((it / kAcc) & 1u) ^ 1u, cta_abort, tmo)) {
          give_up(kStWaitTmemEmpty);
          break;
        }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = 0; kb < p.num_kb; ++kb) {
          if (!ptx::mbar_wait_bounded(W4 ? &conv[s] : &full[s], ph, cta_abort, tmo)) {
            give_up(kStWaitFull);
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint64_t a_desc = ptx::make_kmajor_sw128_desc(a_base + s * kABytes);
          const uint64_t b_desc = ptx::make_kmajor_sw128_desc(resident ? w_base + kb * C::kBBytes : b_base + s * C::kBBytes);
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            // next 32 bytes of K inside the swizzled 128-byte row: start address + 32 B (>> 4 = 2)
            if (PAIR) ptx::mma_i8_ss_pair(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
            else ptx::mma_i8_ss(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          if (PAIR) ptx::tc_commit_pair_mc(&empty[s], 3);     // the stage is free in both CTAs
          else ptx::tc_commit(&empty[s]);
          if (++s == (uint32_t)stages) {
            s = 0;
            ph ^= 1u;
          }
        }
        if (ok) {
          if (PAIR) ptx::tc_commit_pair_mc(&tfull[buf], 3);   // the accumulator is complete in both CTAs
          else ptx::tc_commit(&tfull[buf]);
        }
      }
      if (*cta_abort != 0) {
        // make sure no MMA is still running when TMEM is released
        if (PAIR) ptx::tc_commit_pair(drain);
        else ptx::tc_commit(drain);
        uint32_t polls = 0;
        while (!ptx::mbar_try_wait(drain, 0) && ++polls < (1u << 16)) {
        }
      }
    }
  }   // (warps 2 and 3 are idle: they fill the first group of four and wait at the end)
  } else if (W4 && warp >= C::kConvWarp0) {
    if (C::kRegsConv < C::kLaunchRegs) ptx::setmaxnreg_dec<C::kRegsConv>();
    // ------------------------------------------------------------------ W4 -> INT8 converter warps
    // The packed tile (64 bytes per row, two's-complement nibbles, even element low) is expanded into the
    // 128-byte-swizzled operand tile the MMA descriptor expects.  Each nibble is moved to the HIGH half of
    // its byte, i.e. the operand holds 16 x code (|16 code| <= 112 fits int8); the factor 1/16 is exact in
    // the epilogue (fscale / 16, or an arithmetic shift of the raw accumulators).
    // Two teams of two warps take the k-blocks alternately, so that two stages are being expanded at any time: a
    // team's pass over a stage is mostly latency (the wait for the load, the shared-memory round trip, the proxy
    // fence), which the other team's pass covers.
    constexpr int kTeams = 2, kTeamThreads = 32 * kNumConvWarps / kTeams;
    const int cw = warp - C::kConvWarp0;
    const int team = cw / (kNumConvWarps / kTeams);
    const int lt = threadIdx.x - (C::kConvWarp0 + team * (kNumConvWarps / kTeams)) * 32;       // 0..63 inside the team
    uint32_t s = (uint32_t)team, ph = 0;                   // (the ring has at least three stages)
    const int total_kb = n_local * p.num_kb;
    for (int n = team; n < total_kb; n += kTeams) {
      if (!ptx::mbar_wait_bounded(&full[s], ph, cta_abort, tmo)) {
        give_up(kStWaitFull);
        break;
      }
      const uint8_t* src = sP + s * C::kPBytes;
      uint8_t* dst = sB + s * C::kBBytes;
#pragma unroll 4
      for (int q = lt; q < C::kBRows * 4; q += kTeamThreads) {
        const int n_row = q >> 2, c = q & 3;               // row of the tile, 16-byte chunk of the packed row
        const uint4 w = *reinterpret_cast<const uint4*>(src + n_row * 64 + c * 16);
        const uint32_t in[4] = {w.x, w.y, w.z, w.w};
        uint32_t out[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t lo = (in[i] << 4) & 0xF0F0F0F0u;   // even elements, nibble in the high half
          const uint32_t hi = in[i] & 0xF0F0F0F0u;          // odd elements
          out[2 * i] = __byte_perm(lo, hi, 0x5140);         // e0 e1 e2 e3
          out[2 * i + 1] = __byte_perm(lo, hi, 0x7362);     // e4 e5 e6 e7
        }
        uint8_t* row = dst + n_row * 128;
        const int sw = n_row & 7;                            // 128-byte swizzle: chunk ^= row % 8
        *reinterpret_cast<uint4*>(row + (((2 * c) ^ sw) << 4)) = make_uint4(out[0], out[1], out[2], out[3]);
        *reinterpret_cast<uint4*>(row + (((2 * c + 1) ^ sw) << 4)) = make_uint4(out[4], out[5], out[6], out[7]);
      }
      ptx::fence_proxy_async_smem();     // generic-proxy writes -> visible to the tensor core's async proxy
      __syncwarp();
      if (lane == 0) {
        // (pairs: the MMAs are issued by the even CTA, which reads this CTA's tiles as well)
        if (PAIR) ptx::mbar_arrive_cluster(ptx::mapa_shared(ptx::smem_u32(&conv[s]), 0u));
        else ptx::mbar_arrive(&conv[s]);
      }
      s += kTeams;
      if (s >= (uint32_t)stages) {
        s -= (uint32_t)stages;
        ph ^= 1u;
      }
    }
  } else {
    if (C::kRegsEpi > C::kLaunchRegs) ptx::setmaxnreg_inc<C::kRegsEpi>();
    // ------------------------------------------------------------------ epilogue warps
    // Work item = one unit: kUnitN columns of a tile.  The CTA's units are numbered u = j * kUPT + part
    // (j = local tile); group g takes u = g, g + 4, ...  Unit u lives in its tile's accumulator buffer, part by part.
    constexpr int UPT = C::kUPT;
    constexpr int kUnitN = C::kUnitN;
    constexpr int BOXB = C::kBoxBytes;
    constexpr int BC = C::kBC;              // columns per staging box
    constexpr int ESZ = C::kEsz;
    const int ew = warp - C::kEpiWarp0;
    const int g = ew / kGroupWarps;
    const int qd = warp & 3;                // TMEM lane quadrant (hardware rule: warp % 4)
    const bool lead = qd == 0;              // stages fscale / fbias and speaks for the group to the other CTAs
    uint8_t* stg = sStage + ew * C::kSlotBytes;
    const uint32_t swz = swizzle_xor<BOXB>(lane);
    float* const ps_fs = sParam + g * C::kParamArrays * kUnitN;   // this group's fscale slice, then its fbias slice
    float* const ps_fb = ps_fs + kUnitN;
    int* const ps_c1 = reinterpret_cast<int*>(ps_fs + 2 * kUnitN);   // ASYM: -Z_W, then K Z_W - column sum of W_q
    int* const ps_cd = ps_c1 + kUnitN;
    int pre_c1[kUnitN / 32], pre_cd[kUnitN / 32];
    const uint32_t taddr_q = tmem_base + ((uint32_t)(qd * 32) << 16);   // this warp's lane quadrant, column 0
    const int n_units = n_local * UPT;
    float pre_fs[kUnitN / 32], pre_fb[kUnitN / 32];

    // the group's walk over its units g, g + 4, ...: `walk` stands on the tile of the current unit, `next` on the
    // tile of the group's next unit (for the parameter prefetch)
    constexpr int kTileStep = kGroups / UPT;                 // tiles between two units of a group
    TileWalk walk, next;
    walk.init(p, walker, G);
    walk.advance(g / UPT);
    next = walk;
    next.advance(kTileStep);
    auto col0_at = [&](const TileWalk& w, int u) {           // first column of unit u (whose tile w stands on)
      return w.tn * BN + (u % UPT) * kUnitN;
    };
    auto prefetch_params = [&](int n0) {
#pragma unroll
      for (int i = 0; i < kUnitN / 32; ++i) {
        const int c = n0 + i * 32 + lane;
        if (ASYM) {
          pre_c1[i] = c < p.N ? __ldg(p.w_terms + c) : 0;
          pre_cd[i] = c < p.N ? __ldg(p.w_terms + p.N + c) : 0;
        }
        if (!C::kHasParams) continue;
        pre_fs[i] = c < p.N ? __ldg(p.fscale + c) * (W4 ? 0.0625f : p.w4_mul) : 0.f;   // W4 operands hold 16 x code
        if (C::kStatic8) {   // integer accumulator offsets travel as bit patterns (x16 with the x16 W4 operands)
          const int o = c < p.N ? __ldg(reinterpret_cast<const int*>(p.fbias) + c) : 0;
          pre_fb[i] = __int_as_float((W4 || p.w4_res) ? o * 16 : o);
        } else {
          pre_fb[i] = (c < p.N && p.fbias != nullptr) ? __ldg(p.fbias + c) : 0.f;   // statistics: no bias = 0
        }
      }
    };
    int pre_n0 = -1;                        // lead warp: first column of the unit the prefetch registers hold
    if (C::kNeedSlice && lead && g < n_units) {
      pre_n0 = col0_at(walk, g);
      prefetch_params(pre_n0);
    }

    // Writes the warp's box (32 rows x BOXB bytes, swizzled in its staging slot) to global memory: lanes are
    // re-dealt so that one store instruction covers whole box rows (BOXB contiguous bytes each).
    // x_bytes / y = position of the box in the output matrix, in bytes / rows.
    auto store_box = [&](int x_bytes, int y) {
      constexpr int CPR = BOXB / 16;                 // 16-byte chunks per box row
      constexpr int RPI = 32 / CPR;                  // rows per store instruction
      __syncwarp();
      const int chunk = lane % CPR;
      const int xb = x_bytes + chunk * 16;
      const bool col_ok = xb < p.N * ESZ;            // N * ESZ is a multiple of 16: a chunk is all in or all out
      uint8_t* out = static_cast<uint8_t*>(p.Y) + xb;
#pragma unroll
      for (int i = 0; i < CPR; ++i) {
        const int r = i * RPI + lane / CPR;
        uint4 v = *reinterpret_cast<const uint4*>(stg + r * BOXB + ((chunk ^ swizzle_xor<BOXB>(r)) << 4));
        // static-scale INT8 boxes: rows 8-15 and 24-31 were written with the 8-byte halves of every chunk exchanged
        if (C::kStatic8 && (r & 8) != 0) v = make_uint4(v.z, v.w, v.x, v.y);
        if (col_ok && y + r < p.M) *reinterpret_cast<uint4*>(out + (size_t)(y + r) * p.N * ESZ) = v;
      }
      __syncwarp();                                  // the slot may be rewritten
    };

    // The same box by a bulk tensor store issued by one lane: the LSU sees nothing of it and the warp goes on
    // at once.  The staging slot may be rewritten when the copy has read it: slot_free() before the next box's
    // first write (by then the copy has usually had the next box's TMEM load and arithmetic to finish reading).
    int box_w = 0, box_h = 0, box_b = 0;             // convolution: output position of the warp's 32 rows
    auto tma_box = [&](int x_bytes, int y) {
      ptx::fence_proxy_async_smem();                 // this lane's writes to the slot, for the async proxy
      __syncwarp();
      if (lane == 0) {
        if (p.cv.on) {
          if (box_w < p.cv.Wo && box_h < p.cv.Ho && box_b < p.cv.B)
            ptx::tma_store_4d(&tmY, stg, x_bytes, box_w, box_h, box_b);
        } else if (y < p.M) {
          ptx::tma_store_2d(&tmY, stg, x_bytes, y);
        }
        ptx::bulk_commit_group();
      }
    };
    auto slot_free = [&]() {
      if (lane == 0) ptx::bulk_wait_read_all();
      __syncwarp();
    };

    if (PAIR && !W4 && p.w4_res) {
      // Packed resident tile: all sixteen epilogue warps expand this CTA's half (two's-complement nibbles, even element
      // low, each moved to the HIGH half of its byte: the operand holds 16 x code) from the X ring, where it landed,
      // into the resident buffer in the 128-byte-swizzled layout of the MMA descriptor; then the ring is free for X
      // and, once both CTAs are through, the even CTA's MMAs may start.
      bool fine = ptx::mbar_wait_bounded(&conv[0], 0, cta_abort, tmo);
      if (fine) {
        constexpr int kPackedKb = C::kBRows * (kBK / 2);
        const uint8_t* const packed = sA + stages * kABytes - p.res_kb * kPackedKb;    // top end of the X ring
        const int t = (int)threadIdx.x - C::kEpiWarp0 * 32;
        const int items = p.res_kb * C::kBRows * 4;          // 16-byte chunks of the packed tile
        for (int it = t; it < items; it += kEpiWarps * 32) {
          const int kb = it / (C::kBRows * 4), rem = it - kb * (C::kBRows * 4);
          const int n_row = rem >> 2, ch = rem & 3;
          const uint4 w = *reinterpret_cast<const uint4*>(packed + kb * kPackedKb + n_row * 64 + ch * 16);
          const uint32_t in[4] = {w.x, w.y, w.z, w.w};
          uint32_t out[8];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t lo = (in[i] << 4) & 0xF0F0F0F0u;   // even elements, nibble in the high half
            const uint32_t hi = in[i] & 0xF0F0F0F0u;          // odd elements
            out[2 * i] = __byte_perm(lo, hi, 0x5140);
            out[2 * i + 1] = __byte_perm(lo, hi, 0x7362);
          }
          uint8_t* row = sWres + kb * C::kBBytes + n_row * 128;
          const int sw = n_row & 7;
          *reinterpret_cast<uint4*>(row + (((2 * ch) ^ sw) << 4)) = make_uint4(out[0], out[1], out[2], out[3]);
          *reinterpret_cast<uint4*>(row + (((2 * ch + 1) ^ sw) << 4)) = make_uint4(out[4], out[5], out[6], out[7]);
        }
        ptx::fence_proxy_async_smem();     // generic-proxy writes -> visible to the tensor core's async proxy
      }
      __syncwarp();
      if (lane == 0) {
        if (fine) {
          ptx::mbar_arrive(&conv[1]);
          ptx::mbar_arrive_cluster(ptx::mapa_shared(ptx::smem_u32(&conv[2]), 0u));
        } else {
          give_up(kStWaitFull);
        }
      }
    }

    int use = 0;                            // units this group has handled
    int xuse = 0;                           // ... of which through the counter exchange (phases of pub / ready there:
                                            // a unit right of the matrix handles nothing and arrives on neither)
    int slice_n0 = -1;                      // first column of the unit whose parameters are in the group's slice
    int reloads = 0;                        // times the slice has been (re)loaded
    for (int u = g; u < n_units; u += kGroups, ++use, walk = next, next.advance(kTileStep)) {
      const int j = u / UPT;
      const int tm = strip_of(walk.tm);
      const int n0 = col0_at(walk, u);
      const uint32_t buf = j % kAcc, tpar = (j / kAcc) & 1u, upar = use & 1u;
      const int y0 = tm * kBM + qd * 32;
      const uint32_t taddr = taddr_q + buf * BN + (uint32_t)(u % UPT) * kUnitN;   // the unit's columns in TMEM
      float xs4[4] = {0.f, 0.f, 0.f, 0.f};    // x_scale of the thread's four rows, requested before the waits below
      if (C::kHasParams && !C::kStatic8) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int r = y0 + (lane >> 2) + 8 * k;
          if (p.cv.on) xs4[k] = p.cv.x_scale;
          else if (r < p.M) xs4[k] = __ldg(p.x_scale + r);
        }
      }
      // convolution: the tile's block of output pixels, and where row r of the tile lies in the output
      int cv_w0 = 0, cv_h0 = 0, cv_b0 = 0;
      if (p.cv.on) {
        const int tw = tm % p.cv.tiles_w, t2 = tm / p.cv.tiles_w;
        cv_w0 = tw << p.cv.bw_log;
        cv_h0 = (t2 % p.cv.tiles_h) << p.cv.bh_log;
        cv_b0 = (t2 / p.cv.tiles_h) << (7 - p.cv.bw_log - p.cv.bh_log);
      }
      auto cv_pixel = [&](int r, int& w, int& h, int& b) {        // r = row inside the tile
        w = cv_w0 + (r & ((1 << p.cv.bw_log) - 1));
        h = cv_h0 + ((r >> p.cv.bw_log) & ((1 << p.cv.bh_log) - 1));
        b = cv_b0 + (r >> (p.cv.bw_log + p.cv.bh_log));
      };
      if (p.cv.on) cv_pixel(qd * 32, box_w, box_h, box_b);
      // statistics: the thread's rows inside the matrix, and the first step's values of f (requested before the
      // waits below; every later step is requested one step ahead)
      constexpr int NB = 2;                   // statistics: 8-column blocks per step
      bool rv[4] = {true, true, true, true};
      const bool rows_full = y0 + 32 <= p.M;
      float2 fnext[NB][4];
      auto load_f = [&](int col0, float2 (&dst)[NB][4]) {
#pragma unroll
        for (int i = 0; i < NB; ++i) {
          const int col = col0 + 8 * i + 2 * (lane & 3);    // N is even: a column pair is all in or all out
#pragma unroll
          for (int k = 0; k < 4; ++k)
            dst[i][k] = (col < p.N && rv[k]) ? __ldcs(reinterpret_cast<const float2*>(
                                                   p.F + (size_t)(y0 + (lane >> 2) + 8 * k) * (size_t)p.ldf + col))
                                             : make_float2(0.f, 0.f);
        }
      };
      if constexpr (C::kStats) {
#pragma unroll
        for (int k = 0; k < 4; ++k) rv[k] = y0 + (lane >> 2) + 8 * k < p.M;
        load_f(n0, fnext);
      }
      int zx4[4] = {0, 0, 0, 0}, rs4[4] = {0, 0, 0, 0};   // ASYM: zero-point and code sum of the four rows
      if (ASYM) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int r = y0 + (lane >> 2) + 8 * k;
          if (r < p.M) {
            zx4[k] = __ldg(p.x_zero + r);
            rs4[k] = __ldg(p.x_rowsum + r);
          }
        }
      }
      // The slice is reloaded only when the unit's columns differ from those of the group's previous unit: with a
      // resident W tile every tile of the CTA has the same columns, and the group's slice is loaded once per call.
      const bool reload = C::kNeedSlice && n0 != slice_n0;
      if (reload) {
        slice_n0 = n0;
        const uint32_t ppar = (uint32_t)(reloads++) & 1u;
        if (lead) {
          if (pre_n0 != n0) prefetch_params(n0);     // not fetched ahead (never the case with a regular tile walk)
          // the slice is free once the group's 4 warps have finished the unit that used it before
          if (!ptx::mbar_wait_bounded(&gdone[g], upar ^ 1u, cta_abort, tmo)) {
            give_up(kStWaitParam);
            break;
          }
#pragma unroll
          for (int i = 0; i < kUnitN / 32; ++i) {
            if (C::kHasParams) {
              ps_fs[i * 32 + lane] = pre_fs[i];
              ps_fb[i * 32 + lane] = pre_fb[i];
            }
            if (ASYM) {
              ps_c1[i * 32 + lane] = pre_c1[i];
              ps_cd[i * 32 + lane] = pre_cd[i];
            }
          }
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&pfull[g]);
          if (u + kGroups < n_units && col0_at(next, u + kGroups) != n0) {
            pre_n0 = col0_at(next, u + kGroups);
            prefetch_params(pre_n0);
          }
        }
        if (!ptx::mbar_wait_bounded(&pfull[g], ppar, cta_abort, tmo)) {
          give_up(kStWaitParam);
          break;
        }
      }
      if (!ptx::mbar_wait_bounded(&tfull[buf], tpar, cta_abort, tmo)) {
        give_up(kStWaitTmemFull);
        break;
      }
      ptx::tc_fence_after();
      // Fragment geometry of this thread (see tmem_ld_frag): it sees the unit's columns 8i + 2c, 8i + 2c + 1 and
      // the four rows q + 8k (k = 0..3) of the warp's 32.  Per-column parameters are then loaded once per column
      // pair and used for four rows, which is what keeps the shared-memory pipe from bounding the epilogue.
      const int q = lane >> 2, c = lane & 3;
      const float2 xs2[4] = {make_float2(xs4[0], xs4[0]), make_float2(xs4[1], xs4[1]), make_float2(xs4[2], xs4[2]),
                             make_float2(xs4[3], xs4[3])};
      // a unit entirely right of the matrix (or, for the odd CTA of a pair, below it) has nothing to compute or store
      const bool in_range = n0 < p.N && (!PAIR || tm * kBM < p.M);
      // z of one 8-column block for the thread's four rows; a = registers of lanes q, q + 8 (half 0) and of
      // lanes q + 16, q + 24 (half 1); col = first column of the block inside the unit
      // Eq. 7: the unsigned product plus the three zero-point terms, for the block's two columns and four rows
      // (in place, exact integer arithmetic): acc += -Z_W[n] rsx[m] + Z_x[m] (K Z_W[n] - csw[n])
      auto asym_fix = [&](uint32_t* a0, uint32_t* a1, int col) {
        const int2 c1 = *reinterpret_cast<const int2*>(ps_c1 + col + 2 * c);
        const int2 cd = *reinterpret_cast<const int2*>(ps_cd + col + 2 * c);
        auto fix = [&](uint32_t& v0, uint32_t& v1, int k) {
          v0 = (uint32_t)((int)v0 + c1.x * rs4[k] + zx4[k] * cd.x);
          v1 = (uint32_t)((int)v1 + c1.y * rs4[k] + zx4[k] * cd.y);
        };
        fix(a0[0], a0[1], 0);
        fix(a0[2], a0[3], 1);
        fix(a1[0], a1[1], 2);
        fix(a1[2], a1[3], 3);
      };
      auto z_block = [&](const uint32_t* a0, const uint32_t* a1, int col, float2 (&z)[4]) {
        const float2 f2 = *reinterpret_cast<const float2*>(ps_fs + col + 2 * c);
        const float2 b2 = *reinterpret_cast<const float2*>(ps_fb + col + 2 * c);
        if (C::kStatic8) {
          // Eq. 10: M' (acc + offset); the sum is exact integer arithmetic, the product one FP32 rounding
          const int o0 = __float_as_int(b2.x), o1 = __float_as_int(b2.y);
          auto mo = [&](uint32_t x0, uint32_t x1) {
            return __fmul2_rn(make_float2(__int2float_rn((int)x0 + o0), __int2float_rn((int)x1 + o1)), f2);
          };
          z[0] = mo(a0[0], a0[1]);
          z[1] = mo(a0[2], a0[3]);
          z[2] = mo(a1[0], a1[1]);
          z[3] = mo(a1[2], a1[3]);
          return;
        }
        z[0] = z_pair(a0[0], a0[1], xs2[0], f2.x, f2.y, b2.x, b2.y);     // columns >= N give 0 * 0 + 0
        z[1] = z_pair(a0[2], a0[3], xs2[1], f2.x, f2.y, b2.x, b2.y);
        z[2] = z_pair(a1[0], a1[1], xs2[2], f2.x, f2.y, b2.x, b2.y);
        z[3] = z_pair(a1[2], a1[3], xs2[3], f2.x, f2.y, b2.x, b2.y);
      };

      // The accumulator buffer is handed back to the tensor pipe as soon as this warp has read the last of it
      // (the arithmetic and the stores of the last box then overlap the next tile's MMAs).
      bool released = false;
      auto release_acc = [&]() {
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (PAIR) ptx::mbar_arrive_cluster(ptx::mapa_shared(ptx::smem_u32(&tempty[buf]), 0u));   // the even CTA issues the MMAs
          else ptx::mbar_arrive(&tempty[buf]);
        }
        released = true;
      };
      const int boxes_in = in_range ? ((p.N - n0 + BC - 1) / BC < kUnitN / BC ? (p.N - n0 + BC - 1) / BC : kUnitN / BC) : 0;
      float den_row = 1.f, inv_row = 1.f;
      bool slow = false;
      if (C::kInt8Out && in_range) {
        // ---------------------------------------------------------------- phase 1: row maxima of the unit
        float amax[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
        for (int h = 0; h < kUnitN / 32; ++h) {
          uint32_t a0[16], a1[16];
          ptx::tmem_ld_16x256b_x4(taddr + h * 32, a0);
          ptx::tmem_ld_16x256b_x4(taddr + (16u << 16) + h * 32, a1);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float2 z[4];
            if (ASYM) asym_fix(a0 + 4 * i, a1 + 4 * i, h * 32 + 8 * i);
            z_block(a0 + 4 * i, a1 + 4 * i, h * 32 + 8 * i, z);
#pragma unroll
            for (int k = 0; k < 4; ++k) amax[k] = ptx::max3_abs(amax[k], z[k].x, z[k].y);
            // z replaces the accumulators in TMEM: phase 2 reads it back instead of recomputing it
            a0[4 * i] = __float_as_uint(z[0].x);
            a0[4 * i + 1] = __float_as_uint(z[0].y);
            a0[4 * i + 2] = __float_as_uint(z[1].x);
            a0[4 * i + 3] = __float_as_uint(z[1].y);
            a1[4 * i] = __float_as_uint(z[2].x);
            a1[4 * i + 1] = __float_as_uint(z[2].y);
            a1[4 * i + 2] = __float_as_uint(z[3].x);
            a1[4 * i + 3] = __float_as_uint(z[3].y);
          }
          ptx::tmem_st_16x256b_x4(taddr + h * 32, a0);
          ptx::tmem_st_16x256b_x4(taddr + (16u << 16) + h * 32, a1);
        }
        ptx::tmem_st_wait();
        // the four lanes that share a row (same q) combine; lane (q, c) then speaks for row q + 8c
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          amax[k] = fmaxf(amax[k], __shfl_xor_sync(0xffffffffu, amax[k], 1));
          amax[k] = fmaxf(amax[k], __shfl_xor_sync(0xffffffffu, amax[k], 2));
        }
        const float amax_mine = c == 0 ? amax[0] : (c == 1 ? amax[1] : (c == 2 ? amax[2] : amax[3]));
        const int my = q + 8 * c;             // row (inside the warp's 32) this lane publishes and fetches
        const int row = y0 + my;
        // Exchange of the row maxima between the CTAs of a row strip (all words start at zero):
        //  - up to 32 units per strip: every unit stores (tag 1, its maximum) in an 8-byte word of its own per
        //    row -- a single aligned 8-byte access is indivisible, so no fence is needed -- and a thread polls
        //    the words of its row until all are tagged (one store, then loads that hit L2);
        //  - wider layers (their long mainloop hides the extra round trips): atomicMax into rowmax[m] (a
        //    non-negative float orders like its bit pattern), then the group's lead warp counts the unit on
        //    the strip's counter; the unit that completes the strip raises the strip's flag, the others poll it.
        const int strip_units = (int)p.counter_target;            // units of a row strip inside the matrix
        const int words = p.gather_words;                         // words per row: strip_units, or 0
        unsigned long long* slot = p.partial + ((size_t)tm * words) * kBM + qd * 32 + my;
        float amax_row = 0.f;
        int good = 1;
        if (strip_units == 1) {
          amax_row = amax_mine;      // the unit is the whole row: nothing to exchange (and nothing was cleared)
        } else if (p.own_strips) {
          // the row is this CTA's two tiles of the strip: all its units (up to 4, one per group) meet in shared
          // memory (two buffers by the strip's ordinal: a group can be one strip ahead of the readers of the last)
          const uint32_t xp = (uint32_t)walk.ord & 1u;
          float* const sbuf = sPair + xp * 4 * kBM;                                   // [unit of the strip][row]
          sbuf[(uint32_t)(walk.tn * UPT + u % UPT) * kBM + qd * 32 + my] = amax_mine;
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&pub[0]);
          if (!ptx::mbar_wait_bounded(&pub[0], xp, cta_abort, tmo)) {
            good = 0;
          } else {
            amax_row = amax_mine;
            for (int v = 0; v < strip_units; ++v) amax_row = fmaxf(amax_row, sbuf[v * kBM + qd * 32 + my]);
          }
        } else if (p.local_pair) {
          // the row is this tile's two units, handled by the groups g and g ^ 1: through shared memory (two
          // buffers: the pair's next tile comes two tiles later, when everybody has long read this one)
          const uint32_t xp = (uint32_t)(j >> 1) & 1u;
          float* const pbuf = sPair + ((uint32_t)(g >> 1) * 2 + xp) * 2 * kBM;      // [unit of the tile][row]
          float* mine = pbuf + (uint32_t)(u % UPT) * kBM + qd * 32 + my;
          *mine = amax_mine;
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&pub[g & ~1]);
          if (!ptx::mbar_wait_bounded(&pub[g & ~1], xp, cta_abort, tmo)) good = 0;
          else amax_row = fmaxf(amax_mine, pbuf[(uint32_t)((u % UPT) ^ 1) * kBM + qd * 32 + my]);
        } else if (words > 0) {
          ptx::st_relaxed_gpu_u64(slot + (size_t)(n0 / kUnitN) * kBM,
                                  (1ull << 32) | (unsigned long long)__float_as_uint(amax_mine));
          // all words of the row are requested together (one L2 round trip when they are all there)
          uint32_t polls = 0;
          uint64_t t0 = 0;
          while (true) {
            bool all = true;
            float m = 0.f;
            // 16 words at a time, every batch in flight at once; narrow strips (the common case) take one batch
            auto batch = [&](int v0) {
              unsigned long long w[16];
#pragma unroll
              for (int v = 0; v < 16; ++v)
                w[v] = v0 + v < strip_units ? ptx::ld_relaxed_gpu_u64(slot + (size_t)(v0 + v) * kBM) : (1ull << 32);
#pragma unroll
              for (int v = 0; v < 16; ++v) {
                all = all && (w[v] >> 32) != 0ull;
                m = fmaxf(m, __uint_as_float((uint32_t)w[v]));
              }
            };
            batch(0);
            if (strip_units > 16) batch(16);
            if (all) {
              amax_row = m;
              break;
            }
            __nanosleep(20);
            if ((++polls & 127u) == 0u) {
              const uint64_t now = ptx::globaltimer_ns();
              if (t0 == 0) t0 = now;
              if (*cta_abort != 0 || now - t0 > tmo) {
                good = 0;
                break;
              }
            }
          }
        } else {
          if (row < p.M) atomicMax(p.rowmax + row, __float_as_uint(amax_mine));
          __syncwarp();
          if (lane == 0) {
            __threadfence();                  // this warp's maxima before the arrival below
            ptx::mbar_arrive(&pub[g]);
          }
          if (lead) {
            // the lead warp counts the unit once the whole group has published, then waits for the strip
            if (lane == 0) {
              int fine = ptx::mbar_wait_bounded(&pub[g], (uint32_t)xuse & 1u, cta_abort, tmo) ? 1 : 0;
              if (fine) {
                __threadfence();
                const uint32_t old = atomicAdd(p.counters + tm, 1u);
                if (old + 1u == p.counter_target) {
                  __threadfence();
                  ptx::st_release_gpu(p.flags + tm, 1u);
                } else {
                  uint32_t polls = 0;
                  uint64_t t0 = 0;
                  while (ptx::ld_acquire_gpu(p.flags + tm) == 0u) {
                    __nanosleep(32);
                    if ((++polls & 63u) == 0u) {
                      const uint64_t now = ptx::globaltimer_ns();
                      if (t0 == 0) t0 = now;
                      if (*cta_abort != 0 || now - t0 > tmo || ptx::ld_acquire_gpu(p.status) != 0u) {
                        fine = 0;
                        break;
                      }
                    }
                  }
                }
                __threadfence();
              }
              if (fine) ptx::mbar_arrive(&ready[g]);
              else give_up(kStWaitStrip);
            }
            __syncwarp();     // the other lanes wait here, not in a spin loop beside lane 0
          }
          if (!ptx::mbar_wait_bounded(&ready[g], (uint32_t)xuse & 1u, cta_abort, tmo)) good = 0;
          else amax_row = row < p.M ? __uint_as_float(__ldcg(p.rowmax + row)) : 0.f;
          ++xuse;
        }
        if (!__all_sync(0xffffffffu, good)) {
          if (lane == 0) give_up(kStWaitStrip);
          break;
        }
        // ---------------------------------------------------------------- phase 2: scale, codes
        const float ys = __fdiv_rn(amax_row, 127.f);
        if (p.cv.on) {
          int pw, ph_, pb;
          cv_pixel(qd * 32 + my, pw, ph_, pb);
          if (n0 == 0 && pw < p.cv.Wo && ph_ < p.cv.Ho && pb < p.cv.B)
            p.y_scale[((size_t)pb * p.cv.Ho + ph_) * p.cv.Wo + pw] = ys;
        } else if (n0 == 0 && row < p.M) {
          p.y_scale[row] = ys;
        }
        const float den_mine = ys > 0.f ? ys : 1.f;          // a zero row has z == 0 everywhere: codes 0
        const float inv_mine = __frcp_rn(den_mine);
        // a scale so small that its reciprocal overflows (never on real data): divide directly
        slow = __any_sync(0xffffffffu, !(inv_mine <= 3.0e38f));
        // phase 2 works on row `lane` of the warp's 32; that row's maximum sits in lane (q, c) = (lane % 8, lane / 8)
        den_row = __shfl_sync(0xffffffffu, den_mine, 4 * (lane & 7) + (lane >> 3));
        inv_row = __shfl_sync(0xffffffffu, inv_mine, 4 * (lane & 7) + (lane >> 3));
      }

      if constexpr (C::kStats) {
        // -------------------------------------------------------------- calibration statistics of the unit
        // q = the layer's quantized output before compensation (fscale = S_W, fbias = bias), f = the stored
        // full-precision output of the same rows.  Eq. 4-5 need, per channel, the sums of q, f, q f and q q.
        // A warp shifts q and f by their values in its own first row (a constant column then sums to exactly
        // zero, as Eq. 4's degenerate case needs), adds the shifted terms in FP32 over its 32 rows (4 in the
        // thread, then a halving butterfly over the 8 lanes that share a column pair: pairwise order, at most
        // 5 roundings deep) and leaves sums and shifts in shared memory; the group's 128 threads then take one
        // column each, undo the shifts in FP64, add the four warps in order and write the strip's partial.  A
        // second kernel adds the strips in a fixed order.  Rows >= M and columns >= N contribute nothing.
        float* const wsum = reinterpret_cast<float*>(stg);      // [4 sums | shift of q | shift of f][128 columns]
        // The slots of the group's four warps are read by all four after pub[g]: a warp may rewrite its own slot only
        // when every warp of the group has finished the previous unit (the lead warp's wait above covers only the
        // units whose columns change).
        if (!ptx::mbar_wait_bounded(&gdone[g], upar ^ 1u, cta_abort, tmo)) {
          give_up(kStWaitParam);
          break;
        }
        if (in_range) {
#pragma unroll 2
          for (int h = 0; h < kUnitN / (8 * NB); ++h) {
            const int c0 = h * 8 * NB;                          // first column of the step inside the unit
            float2 fv[NB][4];
#pragma unroll
            for (int i = 0; i < NB; ++i)
#pragma unroll
              for (int k = 0; k < 4; ++k) fv[i][k] = fnext[i][k];
            if (h + 1 < kUnitN / (8 * NB)) load_f(n0 + c0 + 8 * NB, fnext);   // in flight during this step
            uint32_t a0[4 * NB], a1[4 * NB];
            ptx::tmem_ld_frag<NB>(taddr + c0, a0);
            ptx::tmem_ld_frag<NB>(taddr + (16u << 16) + c0, a1);
            ptx::tmem_ld_wait();
            if (h + 1 == kUnitN / (8 * NB)) release_acc();
            float v[8 * NB];                                    // [(block, column of the pair)][sum]
#pragma unroll
            for (int i = 0; i < NB; ++i) {
              float2 z[4];
              z_block(a0 + 4 * i, a1 + 4 * i, c0 + 8 * i, z);
              // the warp's first row sits in lanes 0-3 (q = 0), row slot k = 0
              const float2 kq = make_float2(__shfl_sync(0xffffffffu, z[0].x, c), __shfl_sync(0xffffffffu, z[0].y, c));
              const float2 kf = make_float2(__shfl_sync(0xffffffffu, fv[i][0].x, c),
                                            __shfl_sync(0xffffffffu, fv[i][0].y, c));
              if (q == 0) {
                *reinterpret_cast<float2*>(wsum + 4 * kUnitN + c0 + 8 * i + 2 * c) = kq;
                *reinterpret_cast<float2*>(wsum + 5 * kUnitN + c0 + 8 * i + 2 * c) = kf;
              }
              if (!rows_full) {                                 // last strip only: rows >= M get shifted value 0
#pragma unroll
                for (int k = 0; k < 4; ++k)
                  if (!rv[k]) {
                    z[k] = kq;
                    fv[i][k] = kf;
                  }
              }
              const float2 nkq = make_float2(-kq.x, -kq.y), nkf = make_float2(-kf.x, -kf.y);
              float2 s0 = make_float2(0.f, 0.f), s1 = s0, s2 = s0, s3 = s0;     // .x / .y = the pair's two columns
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const float2 dq = __fadd2_rn(z[k], nkq);
                const float2 df = __fadd2_rn(fv[i][k], nkf);
                s0 = __fadd2_rn(s0, dq);
                s1 = __fadd2_rn(s1, df);
                s2 = __ffma2_rn(dq, df, s2);
                s3 = __ffma2_rn(dq, dq, s3);
              }
              float* o = v + (2 * i) * 4;
              o[0] = s0.x; o[1] = s1.x; o[2] = s2.x; o[3] = s3.x;
              o[4] = s0.y; o[5] = s1.y; o[6] = s2.y; o[7] = s3.y;
            }
            // halving butterfly over lane bits 4, 3, 2 (the row index q): at every level a lane hands one half
            // of its values to its partner and adds the partner's other half to the half it keeps
#pragma unroll
            for (int lvl = 0; lvl < 3; ++lvl) {
              const int mask = 16 >> lvl;
              const int half = (8 * NB) >> (lvl + 1);
              const bool up = (lane & mask) != 0;
#pragma unroll
              for (int j = 0; j < half; ++j) {
                const float lo = v[j], hi = v[j + half];
                const float got = __shfl_xor_sync(0xffffffffu, up ? lo : hi, mask);
                v[j] = (up ? hi : lo) + got;
              }
            }
            // the lane is left with values j + NB q of the original numbering
#pragma unroll
            for (int j = 0; j < NB; ++j) {
              const int idx = j + NB * q;
              const int ie = idx >> 2;
              wsum[(idx & 3) * kUnitN + c0 + 8 * (ie >> 1) + 2 * c + (ie & 1)] = v[j];
            }
          }
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&pub[g]);
        if (!ptx::mbar_wait_bounded(&pub[g], upar, cta_abort, tmo)) {
          give_up(kStWaitStrip);
          break;
        }
        const int t = qd * 32 + lane;                           // the group's 128 threads take one column each
        if (in_range && n0 + t < p.N) {
          // The four warps in the order of their rows (TMEM quadrant 0 first: its first row is the strip's first
          // row, which always lies inside the matrix), every warp re-referenced to the shifts of quadrant 0 -- a
          // change of the size of the channel's spread -- so that the strip's partial stays in shifted form.
          double S0 = 0.0, S1 = 0.0, S2 = 0.0, S3 = 0.0, K0q = 0.0, K0f = 0.0;
#pragma unroll
          for (int qi = 0; qi < kGroupWarps; ++qi) {
            // the slot of epilogue warp g * 4 + w holds the rows of TMEM quadrant w
            const int w = qi;
            const int left = p.M - (tm * kBM + qi * 32);
            if (left <= 0) continue;                            // nothing of this warp is inside the matrix
            const double nw = (double)(left < 32 ? left : 32);
            const float* ws4 = reinterpret_cast<const float*>(sStage + (g * kGroupWarps + w) * C::kSlotBytes) + t;
            const double d0 = ws4[0], d1 = ws4[kUnitN], d2 = ws4[2 * kUnitN], d3 = ws4[3 * kUnitN];
            if (qi == 0) {
              K0q = ws4[4 * kUnitN];
              K0f = ws4[5 * kUnitN];
            }
            const double dq = (double)ws4[4 * kUnitN] - K0q, df = (double)ws4[5 * kUnitN] - K0f;
            S0 += d0 + nw * dq;
            S1 += d1 + nw * df;
            S2 += d2 + df * d0 + dq * d1 + nw * dq * df;
            S3 += d3 + 2.0 * dq * d0 + nw * dq * dq;
          }
          double* out = p.sums + (size_t)tm * kPartialValues * (size_t)p.cpad + n0 + t;
          out[0] = S0;
          out[(size_t)p.cpad] = S1;
          out[2 * (size_t)p.cpad] = S2;
          out[3 * (size_t)p.cpad] = S3;
          out[4 * (size_t)p.cpad] = K0q;
          out[5 * (size_t)p.cpad] = K0f;
        }
      } else if (C::kInt8Out && in_range) {
        // ---------------------------------------------------------------- phase 2: codes, box by box
        // z is read back in the 32x32b layout: thread = row, 32 consecutive columns in registers, so a row has
        // one scale and its codes leave the thread as whole 16-byte pieces (no per-column value is needed any
        // more).  code = rne(z * (1 / y_scale)) in one fused multiply-add: adding 1.5 * 2^23 leaves the integer
        // in the low mantissa bits (|z / y_scale| <= 127 by construction).
        auto codes_and_store = [&](auto slow_tag) {
          constexpr bool SLOW = decltype(slow_tag)::value;
          const float2 magic2 = make_float2(12582912.f, 12582912.f);
          const float2 inv2 = make_float2(inv_row, inv_row);
          auto two = [&](uint32_t x, uint32_t y) -> uint32_t {        // two codes in the low 16 bits
            const float2 z2 = make_float2(__uint_as_float(x), __uint_as_float(y));
            const float2 m = SLOW ? __fadd2_rn(make_float2(__fdiv_rn(z2.x, den_row), __fdiv_rn(z2.y, den_row)), magic2)
                                  : __ffma2_rn(z2, inv2, magic2);
            return __byte_perm(__float_as_uint(m.x), __float_as_uint(m.y), 0x0040);
          };
          uint8_t* const row_base = stg + lane * BOXB;
#pragma unroll 1
          for (int bx = 0; bx < kUnitN / BC; ++bx) {
            if (n0 + bx * BC >= p.N) break;
#pragma unroll 1
            for (int h = 0; h < BC / 32; ++h) {
              uint32_t zr[32];
              ptx::tmem_ld_32x32b_x32(taddr + bx * BC + h * 32, zr);
              ptx::tmem_ld_wait();
              if (bx + 1 == boxes_in && h + 1 == BC / 32) release_acc();
              uint32_t w[8];
#pragma unroll
              for (int j = 0; j < 8; ++j)
                w[j] = __byte_perm(two(zr[4 * j], zr[4 * j + 1]), two(zr[4 * j + 2], zr[4 * j + 3]), 0x5410);
              if (h == 0) slot_free();
              *reinterpret_cast<uint4*>(row_base + (((uint32_t)(2 * h) ^ swz) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
              *reinterpret_cast<uint4*>(row_base + (((uint32_t)(2 * h + 1) ^ swz) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
            }
            tma_box(n0 + bx * BC, y0);
          }
        };
        if (slow) codes_and_store(std::true_type{});
        else codes_and_store(std::false_type{});
      } else if (in_range) {
      // ------------------------------------------------------------------ conversion and store, box by box
        {
          const float2 magic2 = make_float2(12582912.f, 12582912.f);
          // static scales: z is already in output steps; clip to the code range, then round (adding 1.5 * 2^23
          // leaves the integer in the low mantissa bits)
          auto quant = [&](float2 z) -> uint32_t {             // two codes in the low 16 bits
            const float2 qq = make_float2(fminf(fmaxf(z.x, -127.f), 127.f), fminf(fmaxf(z.y, -127.f), 127.f));
            const float2 m = __fadd2_rn(qq, magic2);
            return __byte_perm(__float_as_uint(m.x), __float_as_uint(m.y), 0x0040) & 0xffffu;
          };
          constexpr int LDC = BC < 32 ? BC : 32;       // columns per pair of loads inside a box
          constexpr int NB = LDC / 8;                  // 8-column blocks per load
          // byte address of (row r of the warp's 32, byte b of the box row) in the swizzled staging slot
          auto stage_at = [&](int r, int b) -> uint8_t* {
            return stg + r * BOXB + ((((uint32_t)b >> 4) ^ swizzle_xor<BOXB>(r)) << 4) + (b & 15);
          };
          // The thread's stores into the staging slot (bulk-store modes): for its row q + 8k and its column pair of an
          // 8-column block whose bytes start at a multiple of 16, the swizzled address is a per-thread constant XOR the
          // block's 16-byte chunk index -- one instruction per store instead of the whole swizzle arithmetic.
          uint32_t pre[4];
          {
            const uint32_t cb = (uint32_t)(2 * c * C::kEsz);          // byte offset of the column pair inside a block
#pragma unroll
            for (int k = 0; k < 4; ++k)
              pre[k] = ptx::smem_u32(stg) + (uint32_t)(q + 8 * k) * BOXB + (((cb >> 4) ^ swizzle_xor<BOXB>(q + 8 * k)) << 4) +
                       (cb & 15u);
          }
#pragma unroll 1
          for (int bx = 0; bx < kUnitN / BC; ++bx) {
            if (n0 + bx * BC >= p.N) break;
#pragma unroll
            for (int h = 0; h < BC / LDC; ++h) {
              const int c0 = bx * BC + h * LDC;         // first column (inside the unit) of this pair of loads
              uint32_t a0[4 * NB], a1[4 * NB];
              ptx::tmem_ld_frag<NB>(taddr + c0, a0);
              ptx::tmem_ld_frag<NB>(taddr + (16u << 16) + c0, a1);
              ptx::tmem_ld_wait();
              if (bx + 1 == boxes_in && h + 1 == BC / LDC) release_acc();
              // words of one 8-column block of the thread: 2 per row (FP32, INT32) or 1 per row (BF16)
              constexpr int WPB = C::kEsz == 4 ? 8 : 4;
              uint32_t ow[C::kTmaStore ? NB * WPB : 1];
#pragma unroll
              for (int i = 0; i < NB; ++i) {
                const int colb = h * LDC + 8 * i;      // first column of the block inside the box
                if (ASYM) asym_fix(a0 + 4 * i, a1 + 4 * i, c0 + 8 * i);
                if constexpr (OUT == QWT_OUT_INT32_ACC) {
                  // W4: every term is a multiple of 16, the shift is exact
                  const bool sixteenfold = W4 || p.w4_res != 0;
                  auto fix = [&](uint32_t v) { return sixteenfold ? (uint32_t)((int)v >> 4) : v; };
#pragma unroll
                  for (int k = 0; k < 4; ++k) {
                    ow[i * WPB + 2 * k] = fix(k < 2 ? a0[4 * i + 2 * k] : a1[4 * i + 2 * k - 4]);
                    ow[i * WPB + 2 * k + 1] = fix(k < 2 ? a0[4 * i + 2 * k + 1] : a1[4 * i + 2 * k - 3]);
                  }
                } else {
                  float2 z[4];
                  z_block(a0 + 4 * i, a1 + 4 * i, c0 + 8 * i, z);
                  if constexpr (OUT == QWT_OUT_FP32) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                      ow[i * WPB + 2 * k] = __float_as_uint(z[k].x);
                      ow[i * WPB + 2 * k + 1] = __float_as_uint(z[k].y);
                    }
                  } else if constexpr (OUT == QWT_OUT_BF16) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) ow[i * WPB + k] = pack_bf16x2(z[k].x, z[k].y);
                  } else {
                    // INT8: neighbouring lanes (c even / odd) swap halves so that each ends up with 4 consecutive
                    // codes of two rows: the even lane keeps rows q, q + 16, the odd lane rows q + 8, q + 24
                    const uint32_t h0 = quant(z[0]), h1 = quant(z[1]), h2 = quant(z[2]), h3 = quant(z[3]);
                    const bool odd = (c & 1) != 0;
                    const uint32_t send = odd ? (h0 | (h2 << 16)) : (h1 | (h3 << 16));
                    const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 1);
                    const uint32_t wa = odd ? ((recv & 0xffffu) | (h1 << 16)) : (h0 | (recv << 16));
                    const uint32_t wb = odd ? ((recv >> 16) | (h3 << 16)) : (h2 | (recv & 0xffff0000u));
                    // One store covers rows q (even lanes) and q + 8 (odd lanes): 16 rows x 8 bytes.  The odd
                    // lanes' rows use the other 8-byte half of the chunk (undone in store_box), which spreads the
                    // 16 pieces over all banks.
                    const int b = (colb + 2 * (c & ~1)) ^ (odd ? 8 : 0);
                    *reinterpret_cast<uint32_t*>(stage_at(odd ? q + 8 : q, b)) = wa;
                    *reinterpret_cast<uint32_t*>(stage_at(odd ? q + 24 : q + 16, b)) = wb;
                  }
                }
              }
              if constexpr (C::kTmaStore) {
                // the slot is written only now: the copy of the previous box has had this box's TMEM load and
                // arithmetic to finish reading it
                if (h == 0) slot_free();
#pragma unroll
                for (int i = 0; i < NB; ++i) {
                  const uint32_t chunk = (uint32_t)((h * LDC + 8 * i) * C::kEsz) & ~15u;   // 16-byte chunk of the block
#pragma unroll
                  for (int k = 0; k < 4; ++k) {
                    if constexpr (C::kEsz == 4)
                      ptx::st_shared_v2(pre[k] ^ chunk, ow[i * WPB + 2 * k], ow[i * WPB + 2 * k + 1]);
                    else
                      ptx::st_shared_b32(pre[k] ^ chunk, ow[i * WPB + k]);
                  }
                }
              }
            }
            if (C::kTmaStore) tma_box((n0 + bx * BC) * ESZ, y0);
            else store_box((n0 + bx * BC) * ESZ, y0);
          }
        }
      }
      // the group's parameter slice is free again (and the accumulator buffer, if nothing of the unit was read)
      if (!released) release_acc();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&gdone[g]);
    }
    if (C::kTmaStore && lane == 0) ptx::bulk_wait_all();     // the stores of this warp's boxes are complete
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  ptx::tc_fence_before();
  __syncthreads();
  if (PAIR) {       // neither CTA leaves (or frees tensor memory) while the other may still signal it or read its tiles
    ptx::cluster_arrive();
    ptx::cluster_wait();
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    if (PAIR) ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
    else ptx::tmem_dealloc(tmem_base, kTmemCols);
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

// NHWC byte tensor [B, H, W, row_bytes] -> rank-4 map with a box of {box_bytes, box_w (every `stride`-th position),
// box_h (likewise), box_b}.
bool make_nhwc_map(CUtensorMap* tm, const void* base, uint64_t B, uint64_t H, uint64_t W, uint64_t row_bytes,
                   uint32_t box_bytes, uint32_t box_w, uint32_t box_h, uint32_t box_b, uint32_t stride,
                   CUtensorMapSwizzle swz) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[4] = {row_bytes, W, H, B};
  cuuint64_t strides[3] = {row_bytes, row_bytes * W, row_bytes * W * H};
  cuuint32_t box[4] = {box_bytes, box_w * stride, box_h * stride, box_b};
  cuuint32_t estr[4] = {1, stride, stride, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Convolution: the output map is rank 4 as well; its box depends on the instantiation's staging box, so the
// launcher builds it from this description (set by launch_qconv2d around its launch, per thread).
struct ConvOutSpec {
  bool on;
  uint64_t B, Ho, Wo, row_bytes;
  uint32_t sub_w, sub_h, sub_b;
};
thread_local ConvOutSpec tl_conv_out = {};

// Programmatic dependent launch of the non-cooperative forward kernels (QWT_PDL=1; off by default).  In a single
// stream it takes about 1 us off every call that follows another kernel (DeiT-S shapes, BF16 out, graph replay:
// 13.1 -> 12.1, 8.5 -> 7.6, 15.3 -> 14.1, 17.3 -> 16.2 us).  With several streams it can cost more than it gives: a
// dependent kernel's CTAs take SMs as they fall free and then wait there, which keeps a cooperative kernel of another
// stream (the per-token INT8 exchange needs its whole grid resident) from starting (DeiT-S stack over two streams:
// 787 -> 652 TOPS).
bool programmatic_launch_enabled() {
  static const bool on = [] {
    const char* e = getenv("QWT_PDL");
    return e != nullptr && e[0] == '1';
  }();
  return on;
}

unsigned long long timeout_ns_from_env() {
  const unsigned long long forced = test_hooks().wait_limit_ns.load(std::memory_order_relaxed);
  if (forced != 0ull) return forced;
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

template <int BN, int OUT, bool W4, int WIDE, bool ASYM = false, bool PAIR = false>
qwt_status launch_cfg(const CUtensorMap& tmA, const CUtensorMap& tmB, QlParams prm, int grid, int res_kb,
                      cudaStream_t st) {
  using C = Cfg<BN, OUT, W4, WIDE, ASYM, PAIR>;
  constexpr int kThreads = C::kThreads;
  auto kern = qlinear_cwac_kernel<BN, OUT, W4, WIDE, ASYM, PAIR>;
  // output map: Y as a byte matrix, one staging box (32 rows x kBoxBytes, in the box's own swizzle) per copy
  CUtensorMap tmY = tmA;
  if (C::kTmaStore) {
    constexpr CUtensorMapSwizzle swz = C::kBoxBytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
                                       : (C::kBoxBytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B);
    const ConvOutSpec& co = tl_conv_out;
    const bool ok = co.on ? make_nhwc_map(&tmY, prm.Y, co.B, co.Ho, co.Wo, co.row_bytes, C::kBoxBytes, co.sub_w, co.sub_h,
                                          co.sub_b, 1, swz)
                          : make_byte_map(&tmY, prm.Y, (uint64_t)prm.M, (uint64_t)prm.N * C::kEsz, C::kBoxBytes, 32, swz);
    if (!ok) {
      set_cuda_error((int)cudaErrorInvalidValue);
      return QWT_ERR_CUDA;
    }
  }
  prm.res_kb = res_kb;
  prm.stages = C::stages_for(res_kb);
  const int smem_bytes = C::dynamic_bytes(prm.stages, res_kb);
  // the opt-in shared-memory size is a per-device attribute of the function: set once per device
  // (setting it twice is harmless, so concurrent first calls need no lock, only an atomic flag)
  static std::atomic<bool> attr_set[64];
  int dev = 0;
  QWT_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
    QWT_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448));
    if (dev >= 0 && dev < 64) attr_set[dev].store(true, std::memory_order_release);
  }
  const bool cooperative = C::kInt8Out && prm.counter_target > 1u && !prm.local_pair && !prm.own_strips;
  if (PAIR) {
    // clusters of two CTAs (and, for the row-maximum exchange, every CTA of the grid resident)
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attrs[2];
    attrs[0].id = cudaLaunchAttributeClusterDimension;
    attrs[0].val.clusterDim.x = 2;
    attrs[0].val.clusterDim.y = 1;
    attrs[0].val.clusterDim.z = 1;
    if (cooperative) {
      attrs[1].id = cudaLaunchAttributeCooperative;
      attrs[1].val.cooperative = 1;
    } else {
      attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attrs[1].val.programmaticStreamSerializationAllowed = 1;
    }
    cfg.attrs = attrs;
    cfg.numAttrs = (cooperative || programmatic_launch_enabled()) ? 2 : 1;
    QWT_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmY, prm));
    count_launch();
  } else if (cooperative) {
    // the row-maximum exchange needs every CTA of the grid resident
    void* args[] = {(void*)&tmA, (void*)&tmB, (void*)&tmY, (void*)&prm};
    QWT_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)kern, dim3(grid), dim3(kThreads), args, smem_bytes, st));
    count_launch();
  } else {
    // plain launch, allowed to begin (barrier set-up, tensor-memory allocation) while the kernel before it in the stream
    // is still finishing; the kernel itself waits for that kernel before it touches global memory
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic_launch_enabled() ? 1 : 0;
    QWT_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmY, prm));
    count_launch();
  }
  return QWT_OK;
}

// Operand ring: the resident-W layout (with the wider output staging that short-K layers want) when the plan
// asks for it and at least 4 X stages remain, else the streaming layout.
template <int BN, int OUT, bool W4>
qwt_status launch_inst(const CUtensorMap& tmA, const CUtensorMap& tmB, const QlParams& prm, int grid,
                       bool want_resident, bool pair, cudaStream_t st) {
  if constexpr (BN == 256 && OUT != kOutCalibStats) {
    if (pair) {
      if constexpr (!W4) {
        // short K: each CTA of a pair keeps its half of the W tile for the whole call; the ring then carries X only
        // (64-byte staging boxes while at least four X stages remain, else 32-byte ones)
        if (want_resident && Cfg<BN, OUT, false, 1, false, true>::stages_for(prm.num_kb) >= 4)
          return launch_cfg<BN, OUT, false, 1, false, true>(tmA, tmB, prm, grid, prm.num_kb, st);
        if (want_resident && Cfg<BN, OUT, false, 0, false, true>::stages_for(prm.num_kb) >= 4)
          return launch_cfg<BN, OUT, false, 0, false, true>(tmA, tmB, prm, grid, prm.num_kb, st);
        if (prm.w4_res) return QWT_ERR_UNSUPPORTED;     // (the plan checks the same conditions: not reached)
      }
      return launch_cfg<BN, OUT, W4, 0, false, true>(tmA, tmB, prm, grid, 0, st);
    }
  }
  if (!W4) {
    constexpr int kWide = BN == 256 ? 1 : 0;
    using CW = Cfg<BN, OUT, false, kWide>;
    if (want_resident && CW::stages_for(prm.num_kb) >= 4)
      return launch_cfg<BN, OUT, false, kWide>(tmA, tmB, prm, grid, prm.num_kb, st);
  }
  return launch_cfg<BN, OUT, W4, 0>(tmA, tmB, prm, grid, 0, st);
}

// Asymmetric (unsigned) codes: int8 weights only, streaming operand ring.
template <int BN>
qwt_status launch_asym(int out_mode, const CUtensorMap& tmA, const CUtensorMap& tmB, const QlParams& prm, int grid,
                       cudaStream_t st) {
  switch (out_mode) {
    case QWT_OUT_INT8_PER_TOKEN:
      return launch_cfg<BN, QWT_OUT_INT8_PER_TOKEN, false, false, true>(tmA, tmB, prm, grid, 0, st);
    case QWT_OUT_BF16:
      return launch_cfg<BN, QWT_OUT_BF16, false, false, true>(tmA, tmB, prm, grid, 0, st);
    case QWT_OUT_FP32:
      return launch_cfg<BN, QWT_OUT_FP32, false, false, true>(tmA, tmB, prm, grid, 0, st);
    case QWT_OUT_INT32_ACC:
      return launch_cfg<BN, QWT_OUT_INT32_ACC, false, false, true>(tmA, tmB, prm, grid, 0, st);
  }
  return QWT_ERR_UNSUPPORTED;
}

template <int BN, bool W4>
qwt_status launch_bn(int out_mode, const CUtensorMap& tmA, const CUtensorMap& tmB, const QlParams& prm, int grid,
                     bool want_resident, bool pair, cudaStream_t st) {
  if (prm.w_terms != nullptr) {
    if (W4) return QWT_ERR_UNSUPPORTED;
    return launch_asym<BN>(out_mode, tmA, tmB, prm, grid, st);
  }
  switch (out_mode) {
    case QWT_OUT_INT8_PER_TOKEN:
      return launch_inst<BN, QWT_OUT_INT8_PER_TOKEN, W4>(tmA, tmB, prm, grid, want_resident, pair, st);
    case QWT_OUT_BF16:
      return launch_inst<BN, QWT_OUT_BF16, W4>(tmA, tmB, prm, grid, want_resident, pair, st);
    case QWT_OUT_FP32:
      return launch_inst<BN, QWT_OUT_FP32, W4>(tmA, tmB, prm, grid, want_resident, pair, st);
    case QWT_OUT_INT32_ACC:
      return launch_inst<BN, QWT_OUT_INT32_ACC, W4>(tmA, tmB, prm, grid, want_resident, pair, st);
    case QWT_OUT_INT8_STATIC:
      return launch_inst<BN, QWT_OUT_INT8_STATIC, W4>(tmA, tmB, prm, grid, want_resident, pair, st);
    case kOutCalibStats:
      // packed weights with 256-wide tiles leave no room for the per-warp sums: the plan picks 128 there
      if constexpr (W4 && BN == 256) return QWT_ERR_UNSUPPORTED;
      else return launch_inst<BN, kOutCalibStats, W4>(tmA, tmB, prm, grid, want_resident, false, st);
  }
  return QWT_ERR_UNSUPPORTED;
}

}  // namespace

void qconv_tiling(int B, int Ho, int Wo, int stride, QconvArgs* out) {
  long best_tiles = -1;
  for (int bwl = 7; bwl >= 0; --bwl) {
    for (int bhl = 0; bwl + bhl <= 7; ++bhl) {
      const int bw = 1 << bwl, bh = 1 << bhl, bb = 128 >> (bwl + bhl);
      if (bw * stride > 256 || bh * stride > 256) continue;      // a box side covers at most 256 positions
      const long tw = (Wo + bw - 1) / bw, th = (Ho + bh - 1) / bh, tb = (B + bb - 1) / bb;
      const long tiles = tw * th * tb;
      if (best_tiles < 0 || tiles < best_tiles) {
        best_tiles = tiles;
        out->bw_log = bwl;
        out->bh_log = bhl;
        out->tiles_w = (int)tw;
        out->tiles_h = (int)th;
        out->tiles_b = (int)tb;
      }
    }
  }
}

namespace {
// Whether the pair kernel with resident W halves has room for its X ring (the conditions launch_inst applies).
template <int OUT>
constexpr bool pair_resident_has_room(int num_kb) {
  return Cfg<256, OUT, false, 1, false, true>::stages_for(num_kb) >= 4 ||
         Cfg<256, OUT, false, 0, false, true>::stages_for(num_kb) >= 4;
}
bool pair_resident_fits(int out_mode, int num_kb) {
  switch (out_mode) {
    case QWT_OUT_INT8_PER_TOKEN: return pair_resident_has_room<QWT_OUT_INT8_PER_TOKEN>(num_kb);
    case QWT_OUT_BF16: return pair_resident_has_room<QWT_OUT_BF16>(num_kb);
    case QWT_OUT_FP32: return pair_resident_has_room<QWT_OUT_FP32>(num_kb);
    case QWT_OUT_INT32_ACC: return pair_resident_has_room<QWT_OUT_INT32_ACC>(num_kb);
    case QWT_OUT_INT8_STATIC: return pair_resident_has_room<QWT_OUT_INT8_STATIC>(num_kb);
  }
  return false;
}
qwt_status qlinear_plan_impl(int32_t M, int32_t N, int32_t K, int32_t wfmt, int32_t out_mode, const DeviceInfo& dev,
                             QlinearPlan* plan, bool plain);
}  // namespace

qwt_status qlinear_plan(int32_t M, int32_t N, int32_t K, int32_t wfmt, int32_t out_mode, const DeviceInfo& dev,
                        QlinearPlan* plan, bool plain) {
  // Packed int4 weights: where the int8 kernel would run as CTA pairs with resident W halves, the packed tile is
  // expanded on chip, once per CTA, into that resident buffer -- the weights cross HBM as N K / 2 bytes and no
  // workspace copy is made.  QWT_W4_EXPAND=1 keeps the workspace expansion.
  // Measured on the ViT-B shapes at 25 216 rows (BF16 out) against the workspace expansion in front of the same pair
  // kernel: 2304 x 768 43.6 -> 42.4 us, 3072 x 768 55.3 -> 52.8 us; level over the 48-layer stack on two streams (there the
  // expansion kernels of one stream hide under the other stream's GEMMs).
  const char* e = getenv("QWT_W4_EXPAND");
  if (wfmt == QWT_W_INT4_PACKED && !plain && out_mode != kOutCalibStats && !(e != nullptr && e[0] == '1')) {
    QlinearPlan t{};
    const qwt_status s = qlinear_plan_impl(M, N, K, QWT_W_INT8, out_mode, dev, &t, plain);
    if (s == QWT_OK && t.pair && t.w_resident && pair_resident_fits(out_mode, (K + kBK - 1) / kBK)) {
      t.w4_res = true;
      *plan = t;
      return QWT_OK;
    }
  }
  return qlinear_plan_impl(M, N, K, wfmt, out_mode, dev, plan, plain);
}

namespace {
qwt_status qlinear_plan_impl(int32_t M, int32_t N, int32_t K, int32_t wfmt, int32_t out_mode, const DeviceInfo& dev,
                             QlinearPlan* plan, bool plain) {
  QlinearPlan pl{};
  pl.tiles_m = (M + kBM - 1) / kBM;
  // Packed int4 weights are expanded to int8 on chip, tile by tile, by four converter warps; with CTA pairs each CTA
  // expands only its half of the W tile (128 rows per k-block) and loads 24 KB per k-block instead of 48.  With many
  // rows the layer is compute-bound and the converting mainloop still trails the int8 one (ViT-B shapes at 25 216 rows,
  // BF16 out: 0.86-0.98 of it for K = 768, 0.85 for K = 3072; single CTAs: 0.65-0.75), so by default the weights are
  // then expanded once per call into the workspace (1.5 N K bytes of traffic) and the int8 kernel runs; with few rows
  // (weight-bandwidth-bound) the packed tile is streamed and converted on chip.  QWT_W4_EXPAND=0 / 1 forces either.
  const int sms = dev.sm_count > 0 ? dev.sm_count : kPlanSMs;
  {
    const char* e = getenv("QWT_W4_EXPAND");
    const bool many_rows = M >= 1024;
    pl.w4_expand = wfmt == QWT_W_INT4_PACKED && (e != nullptr ? e[0] == '1' : many_rows);
  }
  // on chip: pairs wherever they can be formed and fill the GPU
  bool w4_pair = false;
  if (wfmt == QWT_W_INT4_PACKED && !pl.w4_expand && out_mode != kOutCalibStats && N > 128 && pl.tiles_m >= 2) {
    const char* e = getenv("QWT_PAIR");
    const int tn = (N + 255) / 256;
    const int pair_tiles = ((pl.tiles_m + 1) / 2) * tn;
    const int pairs = pair_tiles < sms / 2 ? pair_tiles : sms / 2;
    w4_pair = tn <= pairs && pair_tiles >= sms / 2 && !(e != nullptr && e[0] == '0');
  }
  if (pl.w4_expand) wfmt = QWT_W_INT8;        // everything below plans the int8 kernel
  // 256-wide tiles keep the tensor pipe ahead of shared-memory bandwidth and are used when the mainloop
  // dominates (long K); short-K layers are bound by the epilogue, which is organised around 128-wide tiles
  // (four accumulator buffers, so the INT8 row-maximum exchange can trail by two tiles).
  const int phantom = out_mode == QWT_OUT_INT8_PER_TOKEN ? test_hooks().phantom_units.load(std::memory_order_relaxed) : 0;
  auto score = [&](int bn) {
    const long tn = (N + bn - 1) / bn;
    const long tiles = (long)pl.tiles_m * tn;
    const long waves = (tiles + sms - 1) / sms;
    const double wave_eff = (double)tiles / (double)(waves * sms);   // SMs busy in the last round
    const double pad_eff = (double)N / (double)(tn * bn);            // useful columns of the tiles
    return wave_eff * pad_eff;
  };
  // 256-wide whenever the grid can still be filled; for small problems the narrower tile spreads over more SMs
  const long tiles256 = (long)pl.tiles_m * ((N + 255) / 256);
  pl.bn = (N > 128 && (tiles256 >= sms || score(256) + 0.15 >= score(128))) ? 256 : 128;
  if (out_mode == kOutCalibStats && wfmt == QWT_W_INT4_PACKED) pl.bn = 128;
  if (w4_pair) pl.bn = 256;
  const char* force = getenv("QWT_FORCE_BN");
  if (force != nullptr) {
    const int f = atoi(force);
    if ((f == 128 || f == 256) && !(out_mode == kOutCalibStats && wfmt == QWT_W_INT4_PACKED)) pl.bn = f;
  }
  pl.tiles_n = (N + pl.bn - 1) / pl.bn;
  const long tiles = (long)pl.tiles_m * pl.tiles_n;
  pl.grid = (int)(tiles < sms ? tiles : sms);
  // Short K: a CTA keeps its W tile (K x bn bytes, at most 96 KB) in shared memory for the whole call.  That
  // needs every tile of a CTA in the same column tile, i.e. a grid that is a multiple of tiles_n.
  const bool w4 = wfmt == QWT_W_INT4_PACKED;
  const long w_tile_bytes = (long)((K + kBK - 1) / kBK) * kBK * pl.bn;
  const char* nores = getenv("QWT_NO_RESIDENT_W");
  pl.w_resident = !plain && !w4 && w_tile_bytes <= 96 * 1024 && pl.tiles_n <= sms && tiles > sms &&
                  !(nores != nullptr && nores[0] == '1');
  if (pl.w_resident) pl.grid = (sms / pl.tiles_n) * pl.tiles_n;
  // Per-token INT8 whose rows span exactly two 256-wide tiles, with at least half a grid of strips: a CTA takes
  // whole strips (both tiles, one after the other in its two accumulator buffers), so that the row maxima are
  // settled inside the CTA: no workspace clearing, no cooperative launch, no L2 round trips.
  {
    const char* e = getenv("QWT_OWN_STRIPS");
    const bool want = e != nullptr ? e[0] == '1' : true;
    pl.own_strips = !plain && want && out_mode == QWT_OUT_INT8_PER_TOKEN && pl.tiles_n == 2 && pl.bn == 256 && !w4 &&
                    pl.tiles_m >= sms / 2 && phantom == 0;
    if (pl.own_strips) {
      pl.w_resident = false;
      pl.grid = pl.tiles_m < sms ? pl.tiles_m : sms;
    }
  }
  // Long K, 256-wide tiles, int8 weights: CTA pairs (clusters of two) on two row strips of the same column tile, the
  // MMAs of M = 256 issued by the even CTA; each CTA then loads half of the W tile per k-block (a third less through
  // its load port and out of its shared memory per MMA), which is what the mainloop of the long-K layers waits for.
  {
    const char* e = getenv("QWT_PAIR");
    const int pair_tiles = ((pl.tiles_m + 1) / 2) * pl.tiles_n;
    const int pairs = pair_tiles < sms / 2 ? pair_tiles : sms / 2;
    const bool fits = !plain && pl.bn == 256 && !pl.w_resident && !pl.own_strips && out_mode != kOutCalibStats &&
                      pl.tiles_m >= 2 && pl.tiles_n <= pairs;
    // (measured: ahead by up to 7 % on layers 4096 and 11008 wide with K = 4096 and 11008, behind by 4 % on a layer
    // 768 wide with K = 3072, whose three column tiles leave the pairs little to share)
    const bool want = e != nullptr ? e[0] == '1'
                                   : (w4 ? w4_pair : (K >= 2048 && pl.tiles_n >= 8 && pair_tiles >= sms / 2));
    pl.pair = fits && want;
    if (pl.pair) pl.grid = 2 * pairs;
    // Short K whose 256-wide W tile is too large to stay in one CTA's shared memory: as a pair, with half of the tile
    // resident in each CTA (at most 8 k-blocks = 128 KB) and a number of pairs that is a multiple of tiles_n, so that
    // every tile of a pair has the same column tile.  What a CTA then moves per tile is its X tile and the output: the
    // W tile no longer goes through its port to L2 once per tile.  Measured at 25 216 rows, K = 768 (BF16 / FP32 /
    // static INT8 / raw accumulators out): 2304 wide 47.1 -> 43.4, 64.0 -> 55.1, 47.9 -> 46.9, 62.2 -> 53.4 us; 3072
    // wide 61.8 -> 55.1, 84.0 -> 71.0, 62.9 -> 59.4, 81.4 -> 68.3 us; 16 % at 50 432 rows, 14 % at K = 512, 2 % at
    // K = 1024; a layer 768 wide (three column tiles, 72 of 74 pairs used) loses 1-10 %, and per-token INT8 output,
    // whose pace the row-maximum exchange sets, gains nothing: both keep the single-CTA streaming kernel.
    const char* pr = getenv("QWT_PAIR_RESIDENT");
    const int num_kb = (K + kBK - 1) / kBK;
    const int res_pairs = pl.tiles_n > 0 ? (sms / 2 / pl.tiles_n) * pl.tiles_n : 0;
    const bool res_fits = !plain && !w4 && pl.bn == 256 && !pl.w_resident && !pl.own_strips &&
                          out_mode != kOutCalibStats && pl.tiles_m >= 2 && num_kb <= 8 && res_pairs > 0 &&
                          pair_tiles >= 2 * res_pairs;
    const bool res_want = pr != nullptr ? pr[0] == '1'
                                        : (pl.tiles_n >= 6 && out_mode != QWT_OUT_INT8_PER_TOKEN);
    if (res_fits && res_want) {
      pl.pair = true;
      pl.w_resident = true;
      pl.grid = 2 * res_pairs;
    }
  }
  pl.fused_requant = (out_mode == QWT_OUT_INT8_PER_TOKEN) && (pl.tiles_n <= (pl.pair ? pl.grid / 2 : pl.grid));
  size_t off = 0;
  pl.ws_status_off = off;
  off += 256;
  pl.ws_partial_off = off;      // (tag, row maximum) per strip row and 128-column unit
  // (test hook: phantom units are expected by the exchange but never published, so that its bounded wait runs out)
  const int strip_units = (N + unit_cols(out_mode) - 1) / unit_cols(out_mode) + phantom;
  pl.strip_units = strip_units;
  // tagged words for strips of up to 16 units, and up to 32 when K is short enough for the exchange to show; with a
  // long mainloop the units of a strip finish far apart and the one-flag-per-strip protocol polls far less
  pl.gather_words = (strip_units <= 16 || (strip_units <= kMaxGatherWords && K <= 4096)) ? strip_units : 0;
  if (out_mode == QWT_OUT_INT8_PER_TOKEN) {
    if (pl.gather_words > 0) {
      off += (size_t)pl.tiles_m * kBM * pl.gather_words * sizeof(unsigned long long);
    } else {     // rowmax[tiles_m * 128] | counters[tiles_m] | flags[tiles_m]
      off += ((size_t)pl.tiles_m * kBM * 4 + 2 * (size_t)pl.tiles_m * 4 + 255) / 256 * 256;
    }
  }
  pl.ws_z_off = off;
  if (out_mode == QWT_OUT_INT8_PER_TOKEN && !pl.fused_requant) off += (size_t)M * N * 4;
  off = (off + 255) / 256 * 256;
  pl.ws_w_off = off;
  if (pl.w4_expand) off += (size_t)N * (size_t)K;
  pl.ws_total = off;
  *plan = pl;
  return QWT_OK;
}
}  // namespace

qwt_status launch_qlinear(const int8_t* X, const float* x_scale, const void* W, int32_t wfmt, const float* fscale,
                          const float* fbias, int32_t M, int32_t N, int32_t K, int32_t out_mode, void* Y,
                          float* y_scale, void* workspace, const QlinearPlan& plan, cudaStream_t st,
                          const int32_t* x_zero, const int32_t* x_rowsum, const int32_t* w_terms,
                          const QlinearStatsArgs* stats, const QconvArgs* conv) {
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  if (plan.w4_expand) {
    int8_t* w8 = reinterpret_cast<int8_t*>(ws + plan.ws_w_off);
    qwt_status su = launch_unpack_int4(W, N, K, w8, st);
    if (su != QWT_OK) return su;
    W = w8;
    wfmt = QWT_W_INT8;
  }
  const bool w4 = wfmt == QWT_W_INT4_PACKED;
  // (the packed resident tile exists for the symmetric pair kernel only; the plan asks for it for nothing else)
  if (plan.w4_res && (!w4 || w_terms != nullptr || stats != nullptr || conv != nullptr)) return QWT_ERR_UNSUPPORTED;
  CUtensorMap tmA, tmB;
  // convolution: X is the NHWC activation tensor and a tile's A operand a block of its pixels (one filter tap, 128
  // channels); M is then the number of tile rows (128 x row strips), K = kh * kw * C
  const bool okA = conv != nullptr
                       ? make_nhwc_map(&tmA, X, (uint64_t)conv->B, (uint64_t)conv->H, (uint64_t)conv->W, (uint64_t)conv->C,
                                       kBK, 1u << conv->bw_log, 1u << conv->bh_log,
                                       128u >> (conv->bw_log + conv->bh_log), (uint32_t)conv->stride,
                                       CU_TENSOR_MAP_SWIZZLE_128B)
                       : make_byte_map(&tmA, X, (uint64_t)M, (uint64_t)K, kBK, kBM, CU_TENSOR_MAP_SWIZZLE_128B);
  // (asymmetric codes and the statistics epilogue have no pair instantiation: the same grid then walks single tiles)
  const bool pair = plan.pair && w_terms == nullptr && stats == nullptr;
  const bool okB = w4 ? make_byte_map(&tmB, W, (uint64_t)N, (uint64_t)K / 2, kBK / 2,
                                      (uint32_t)(pair ? plan.bn / 2 : plan.bn), CU_TENSOR_MAP_SWIZZLE_NONE)
                      : make_byte_map(&tmB, W, (uint64_t)N, (uint64_t)K, kBK, (uint32_t)(pair ? plan.bn / 2 : plan.bn),
                                      CU_TENSOR_MAP_SWIZZLE_128B);
  if (!okA || !okB) {
    set_cuda_error((int)cudaErrorInvalidValue);
    return QWT_ERR_CUDA;
  }
  // per-token INT8 output: the status word and the exchanged row maxima start at zero.  The other output
  // modes use only the status word, which their kernel clears itself (one launch less per call).
  // (a layer of at most one unit per strip, N <= 128, exchanges nothing: its kernel clears the status word itself)
  const bool local_pair = out_mode == QWT_OUT_INT8_PER_TOKEN && plan.fused_requant && plan.tiles_n == 1 &&
                          plan.bn == 256 && plan.strip_units == 2;
  const bool exchanges = out_mode == QWT_OUT_INT8_PER_TOKEN && plan.fused_requant && plan.strip_units > 1 &&
                         !local_pair && !plan.own_strips;
  if (exchanges) QWT_CUDA_TRY(cudaMemsetAsync(ws, 0, plan.ws_z_off, st));

  QlParams prm{};
  prm.x_scale = x_scale;
  prm.fscale = fscale;
  prm.fbias = fbias;
  prm.y_scale = y_scale;
  prm.M = M;
  prm.N = N;
  prm.K = K;
  prm.tiles_n = plan.tiles_n;
  prm.num_tiles = plan.tiles_m * plan.tiles_n;
  prm.num_kb = (K + kBK - 1) / kBK;
  if (plan.own_strips) {       // strips b, b + G, ...: every CTA takes tiles_n tiles of each of its strips
    prm.nl_base = plan.tiles_m / plan.grid;
    prm.nl_rem = plan.tiles_m % plan.grid;
    prm.nl_mul = plan.tiles_n;
    prm.step_q = prm.step_r = 0;
  } else if (pair) {           // pairs of CTAs take pair tiles (two row strips x one column tile) b, b + G / 2, ...
    const int pair_tiles = ((plan.tiles_m + 1) / 2) * plan.tiles_n, pairs = plan.grid / 2;
    prm.nl_base = pair_tiles / pairs;
    prm.nl_rem = pair_tiles % pairs;
    prm.nl_mul = 1;
    prm.step_q = pairs / plan.tiles_n;
    prm.step_r = pairs % plan.tiles_n;
  } else {                     // tiles b, b + G, ...
    prm.nl_base = prm.num_tiles / plan.grid;
    prm.nl_rem = prm.num_tiles % plan.grid;
    prm.nl_mul = 1;
    prm.step_q = plan.grid / plan.tiles_n;
    prm.step_r = plan.grid % plan.tiles_n;
  }
  prm.status = reinterpret_cast<uint32_t*>(ws + plan.ws_status_off);
  prm.partial = reinterpret_cast<unsigned long long*>(ws + plan.ws_partial_off);
  // units of a row strip that lie inside the matrix
  prm.counter_target = (uint32_t)plan.strip_units;
  prm.gather_words = plan.gather_words;
  prm.local_pair = local_pair ? 1 : 0;
  prm.own_strips = plan.own_strips ? 1 : 0;
  prm.x_zero = x_zero;
  prm.x_rowsum = x_rowsum;
  prm.w_terms = w_terms;
  prm.rowmax = reinterpret_cast<uint32_t*>(ws + plan.ws_partial_off);
  prm.counters = prm.rowmax + (size_t)plan.tiles_m * kBM;
  prm.flags = prm.counters + plan.tiles_m;
  prm.timeout_ns = timeout_ns_from_env();
  prm.w4_res = plan.w4_res ? 1 : 0;
  prm.w4_mul = plan.w4_res ? 0.0625f : 1.0f;
  if (conv != nullptr) {
    prm.cv.on = 1;
    prm.cv.bw_log = conv->bw_log;
    prm.cv.bh_log = conv->bh_log;
    prm.cv.tiles_w = conv->tiles_w;
    prm.cv.tiles_h = conv->tiles_h;
    prm.cv.Wo = conv->Wo;
    prm.cv.Ho = conv->Ho;
    prm.cv.B = conv->B;
    prm.cv.stride = conv->stride;
    prm.cv.pad = conv->pad;
    prm.cv.kw = conv->kw;
    prm.cv.cpb = conv->C / kBK;
    prm.cv.x_scale = conv->x_scale;
    const int bw = 1 << conv->bw_log, bh = 1 << conv->bh_log;
    prm.cv.sub_w = bw < 32 ? bw : 32;
    prm.cv.sub_h = bh < 32 / prm.cv.sub_w ? bh : 32 / prm.cv.sub_w;
    const size_t esz = out_mode == QWT_OUT_INT8_PER_TOKEN ? 1 : (out_mode == QWT_OUT_BF16 ? 2 : 4);
    tl_conv_out = ConvOutSpec{true, (uint64_t)conv->B, (uint64_t)conv->Ho, (uint64_t)conv->Wo, (uint64_t)N * esz,
                              (uint32_t)prm.cv.sub_w, (uint32_t)prm.cv.sub_h,
                              (uint32_t)(32 / (prm.cv.sub_w * prm.cv.sub_h))};
  }
  struct ConvOutReset {       // the description applies to this launch only
    ~ConvOutReset() { tl_conv_out.on = false; }
  } conv_out_reset;
  if (stats != nullptr) {
    prm.F = stats->F;
    prm.ldf = stats->ldf;
    prm.sums = stats->sums;
    prm.cpad = stats->cpad;
  }

  int mode = out_mode;
  prm.Y = Y;
  if (out_mode == QWT_OUT_INT8_PER_TOKEN && !plan.fused_requant) {
    // very wide layers (more column tiles than CTAs): z goes through FP32 scratch and a row quantizer
    mode = QWT_OUT_FP32;
    prm.Y = ws + plan.ws_z_off;
  }
  qwt_status s;
  if (w4 && !plan.w4_res) s = plan.bn == 256 ? launch_bn<256, true>(mode, tmA, tmB, prm, plan.grid, plan.w_resident, pair, st)
                             : launch_bn<128, true>(mode, tmA, tmB, prm, plan.grid, plan.w_resident, false, st);
  else s = plan.bn == 256 ? launch_bn<256, false>(mode, tmA, tmB, prm, plan.grid, plan.w_resident, pair, st)
                          : launch_bn<128, false>(mode, tmA, tmB, prm, plan.grid, plan.w_resident, false, st);
  if (s != QWT_OK) return s;
  if (mode != out_mode)
    return launch_quantize_rows(reinterpret_cast<const float*>(ws + plan.ws_z_off), M, N, N, 127,
                                static_cast<int8_t*>(Y), y_scale, st);
  return QWT_OK;
}

}  // namespace qwt
