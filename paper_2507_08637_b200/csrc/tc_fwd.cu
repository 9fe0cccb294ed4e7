// bf16 tensor-core (tcgen05 + TMEM + TMA) forward kernels of the WERSA attention path, sm_100a.
// Each kernel reads its raw bf16 operands once with TMA (rings of 128-token tiles), applies the
// multi-level Haar filter (Sec. 3.1 steps 3, 5, 6; Algorithm 2) in shared memory to 256-token blocks
// (two ring tiles, not necessarily adjacent), and feeds the filtered tiles straight to the tensor
// cores: the filtered tensors never reach global memory.  A ring slot is released tile by tile.
//
// Key side  (Eq. 7, key summary):  S' = ReLU(K_F W)^T V,  z' = ReLU(K_F W)^T 1  per sequence chunk.
//   MMA1: D1[128 features x 128 tokens] = W^T (smem, K-major) * K_F^T (smem, K-major)   -> TMEM fp32
//   ReLU warps: TMEM -> registers -> max(.,0) -> bf16 -> back into the same TMEM columns; the row sums
//   z' come from a tree of packed bf16 adds over the rounded values
//   MMA2: S'[128 features x 64] += Phi^T (TMEM operand, K = tokens) * V (smem, N-major)  -> TMEM fp32
// Query side (Eq. 7, output):  O = ReLU(Q_F W) S' / (ReLU(Q_F W) z' + eps')
//   MMA1: D1[128 tokens x 128 features] = Q_F (smem, K-major) * W (as W^T, K-major)
//   ReLU warps: TMEM -> registers -> max(.,0) -> bf16 -> TMEM, nothing else
//   MMA2: [N' | D'][128 tokens x 80] (+)= Phi (TMEM operand, K = features) * [S' | z' | 0] (smem bf16
//   image, K-major): column 64 of the accumulator is the denominator
//   epilogue warps: TMEM -> registers -> * 1/(D' + eps') -> bf16 -> swizzled smem -> TMA store
//
// Work unit of the MMA pipeline: one 128-token tile times one 128-feature half ("unit").  Three D1
// accumulators rotate, so the ReLU pass of a unit overlaps four MMAs of its neighbours.
// Issuing an MMA blocks the thread for about as long as the tensor pipe takes to accept it, so the pipe
// only stays busy when several threads issue: the waits and commits of one overlap the MMAs of another.
// Warp roles, key side (640 threads): warp 0 TMA producer (K and V rings), warp 1 issues every MMA1 and
// runs up to three units ahead, warps 2 and 3 issue the MMA2 of feature half 0 and 1 (separate
// accumulators, so the order between them does not matter), warps 4-11 two ReLU warpgroups that
// alternate over the units, warps 12-19 Haar filter.  Query side (768 threads): warp 0 TMA producer,
// warp 1 MMA1, warp 3 MMA2 (both halves add into one accumulator, hence one thread), warps 4-11 ReLU,
// warps 12-15 epilogue, warps 16-23 Haar filter.  All operand tiles use the 128-byte swizzle.
// Every wait on an mbarrier is bounded; a role whose wait expires keeps its control flow (so that
// group barriers stay balanced) but skips all further work, and the host sees the status word.
#include "common.cuh"
#include "tc_common.cuh"

namespace wersa {
using namespace tc;

namespace {

constexpr int kTile = 128;                        // tokens per MMA tile
constexpr int kBlk = 256;                         // tokens per Haar block = one pipeline stage
constexpr uint32_t kTileBytes = kTile * kD * 2;   // 128 x 64 bf16
constexpr int kNXK = 7, kNV = 4;                  // key side: ring of K tiles, ring of V tiles
constexpr int kNXQ = 7;                           // query side: ring of Q tiles
constexpr int kNF = 4;                            // "block filtered" barriers (block b uses b % 4)
constexpr int kND1 = 3;                           // D1 accumulators in TMEM (columns 0, 128, 256)
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kAccCol = 384;                 // S' halves (key side) / [N' | D'] of the current tile (query side)
constexpr uint32_t kIdesc1 = make_idesc_bf16(128, 128, false, false);  // both operands K-major
constexpr uint32_t kIdesc2 = make_idesc_bf16(128, 64, false, true);    // key side: B = V, N-major
constexpr uint32_t kIdesc2Q = make_idesc_bf16(128, 80, false, false);  // query side: B = [S' | z' | 0]^T, K-major
// Query side: one MMA1 covers a 128-token tile and all m = 128 NH features (N = m), into one of two
// 256-column TMEM buffers.  The ReLU pass packs the bf16 features of 32-column chunks [0, CH) to the front
// of the buffer and those of chunks [CH, 4 NH) to the front of their own span, which leaves 80 free
// columns in between (m = 256) for the [N' | D'] accumulator of the same tile.
constexpr uint32_t kQBufCols = 256;
template <int NH> struct QTmem {
  static constexpr int kChunks = 4 * NH;                 // 32-column fp32 chunks of D1
  static constexpr int kHeavy = NH == 2 ? 5 : 2;         // chunks packed by the first warp of a lane quarter
  static constexpr uint32_t kLightCol = 32 * kHeavy;     // where the second warp's span starts (input and output)
  static constexpr uint32_t kAcc = NH == 2 ? 80 : 128;   // first column of [N' | D'] inside the buffer
  // first TMEM column (inside the buffer) of the 8 columns that hold features 16 k .. 16 k + 15 as bf16 pairs
  __host__ __device__ static constexpr uint32_t phi_col(int k) {
    return (k >> 1) < kHeavy ? 8u * k : kLightCol + 8u * (k - 2 * kHeavy);
  }
};
static_assert(QTmem<2>::phi_col(9) + 8 <= QTmem<2>::kAcc && QTmem<2>::kAcc + 80 <= QTmem<2>::kLightCol,
              "accumulator must sit between the two packed spans");
constexpr uint32_t kSztBlockBytes = 80 * 128;      // one 64-feature K block of that operand: 80 rows of 128 bytes

constexpr int kWarpTma = 0, kWarpMma = 1, kWarpMma2 = 2;   // key side: warps 2 and 3 issue MMA2 (one per half)
constexpr int kWarpMma2Q = 3;                               // query side
constexpr int kReluWarp0 = 4, kAuxWarp0 = 12;       // 8 ReLU warps, 8 Haar warps
constexpr int kThreads = 32 * (kAuxWarp0 + 8);      // 640 threads, 96 registers each at launch
// Registers per thread after the roles have traded: the Haar step holds a 256 x 64 block in registers
// and gets what the producer / MMA warpgroup gives up.
constexpr int kRegsCtl = 40, kRegsAux = 120;
// Query side: four more warps (12-15) form the epilogue, the Haar warps follow (16-23).  768 threads
// start with kRegsLaunchQ registers each; the roles re-split exactly that pool (an increase waits
// until other warps of the CTA have released enough, so the split must never exceed it).
constexpr int kEpiWarp0Q = 12, kAuxWarp0Q = 16;
constexpr int kThreadsQ = 32 * (kAuxWarp0Q + 8);
constexpr int kRegsLaunchQ = 80;   // 65536 / 768 rounded down to a multiple of 8
constexpr int kRegsCtlQ = 40, kRegsReluQ = 56, kRegsEpiQ = 88;
static_assert(4 * kRegsCtlQ + 8 * kRegsReluQ + 4 * kRegsEpiQ + 8 * kRegsAux <= (kThreadsQ / 32) * kRegsLaunchQ,
              "roles may not claim more registers than the CTA was launched with");
// Key side: 640 threads start with 96 registers each.
static_assert(4 * kRegsCtl + 8 * 96 + 8 * kRegsAux <= (kThreads / 32) * 96, "key-side register split");

// Named barriers (id 0 is __syncthreads).
enum { kBarZsum = 1, kBarCoef = 3, kBarHaar = 4, kBarOut0 = 5 };
enum { kErrProducer = 11, kErrMma = 12, kErrRelu = 13, kErrEpilogue = 14, kErrHaar = 15 };

struct alignas(8) KsideBars {
  uint64_t x_full[kNXK], x_empty[kNXK], xf_ready[kNF], v_full[kNV], v_empty[kNV];
  uint64_t d1_full[6], phi_ready[kND1], d1_free[kND1], acc_done, acc_free, w_full;
  uint32_t tmem_base;
  int abort_flag;
};
struct alignas(8) QsideBars {
  uint64_t x_full[kNXQ], x_empty[kNXQ], xf_ready[kNF];
  uint64_t d1_full[2], phi_ready[2], d2_full[2], buf_free[2], simg_ready, simg_next, w_full;
  uint32_t tmem_base;
  int abort_flag;
};

template <int NH> struct KsideSmem {
  static constexpr uint32_t wt = 0;
  static constexpr uint32_t x = wt + NH * kTileBytes;
  static constexpr uint32_t v = x + kNXK * kTileBytes;
  static constexpr uint32_t xch = v + kNV * kTileBytes;           // 2 x 8 x 64 floats
  static constexpr uint32_t hcoef = xch + 4096;                  // kHaarCoefs floats
  static constexpr uint32_t zx = hcoef + 1024;                   // 128 floats
  static constexpr uint32_t bars = zx + 512;
  static constexpr uint32_t total = bars + 512 + 1024;           // + alignment slack
};
template <int NH> struct QsideSmem {
  static constexpr uint32_t wt = 0;
  static constexpr uint32_t simg = wt + NH * kTileBytes;          // 2 NH K blocks of [S' | z' | 0]^T
  static constexpr uint32_t simg_bytes = 2 * NH * kSztBlockBytes;
  // with m = 128 there is room for a second image: a CTA that walks several items builds the next item's
  // image while the current one is in use
  static constexpr bool two_images = NH == 1;
  static constexpr uint32_t x = simg + (two_images ? 2 : 1) * simg_bytes;
  static constexpr uint32_t ost = x + kNXQ * kTileBytes;           // 2 output staging tiles
  static constexpr uint32_t xch = ost + 2 * kTileBytes;          // 2 x 8 x 64 floats
  static constexpr uint32_t hcoef = xch + 4096;                  // kHaarCoefs floats
  static constexpr uint32_t bars = hcoef + 1024;
  static constexpr uint32_t total = bars + 512 + 1024;
};

// Ties the 32 registers of an asynchronous TMEM load to the point behind its wait, so that no use
// of them is scheduled ahead of the wait.
__device__ __forceinline__ void reg_fence32(uint32_t (&r)[32]) {
  asm volatile(""
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]),
                 "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]),
                 "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]),
                 "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}

// One arrival per warp: every lane has finished (and fenced) its part, the warp converges, lane 0
// arrives.  The barriers that collect these arrivals count warps, not threads.
__device__ __forceinline__ void warp_arrive(uint64_t* bar) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}

// Register budget per role (all warps of a warpgroup execute the same one).
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// Two fp32 values in one 64-bit register: the packed add / multiply / fma of sm_100 issue one
// instruction for both halves.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pk2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void upk2(f32x2 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint32_t pack2_bf16(f32x2 v) {
  float lo, hi;
  upk2(v, lo, hi);
  return pack_bf16x2(lo, hi);
}

// ReLU of 32 fp32 accumulator columns -> 16 packed bf16 pairs (one fused relu + round + pack per
// pair).  Returns the sum of the 16 pairs as one bf16 pair (a tree of packed bf16 adds): the row sums
// z' are taken over the same rounded values that MMA2 multiplies, and the rounding of the short tree
// (relative 2^-9 per add, independent from tile to tile) averages out over the sequence.
__device__ __forceinline__ uint32_t add_bf16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ uint32_t relu_chunk(const uint32_t (&r)[32], uint32_t (&p)[16]) {
#pragma unroll
  for (int j = 0; j < 16; ++j) p[j] = relu_pack_bf16x2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
  uint32_t t[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) t[j] = add_bf16x2(p[2 * j], p[2 * j + 1]);
#pragma unroll
  for (int j = 0; j < 4; ++j) t[j] = add_bf16x2(t[2 * j], t[2 * j + 1]);
  return add_bf16x2(add_bf16x2(t[0], t[1]), add_bf16x2(t[2], t[3]));
}

// ReLU pass over one 128-column D1 accumulator: fp32 TMEM -> bf16 pairs back into columns [0, 64)
// of the same accumulator.  The next 32 columns are in flight while the current 32 are processed.
// Returns the row sum of the (rounded) ReLU values, accumulated in fp32 from the four chunk sums.
__device__ __forceinline__ float relu_unit(uint32_t taddr) {
  uint32_t a[32], b[32], p[16];
  tmem_ld32(taddr, a);
  tmem_ld_wait();
  reg_fence32(a);
  tmem_ld32(taddr + 32, b);
  const uint32_t s0 = relu_chunk(a, p);
  tmem_st16(taddr, p);
  tmem_ld_wait();
  reg_fence32(b);
  tmem_ld32(taddr + 64, a);
  const uint32_t s1 = relu_chunk(b, p);
  tmem_st16(taddr + 16, p);
  tmem_ld_wait();
  reg_fence32(a);
  tmem_ld32(taddr + 96, b);
  const uint32_t s2 = relu_chunk(a, p);
  tmem_st16(taddr + 32, p);
  tmem_ld_wait();
  reg_fence32(b);
  const uint32_t s3 = relu_chunk(b, p);
  tmem_st16(taddr + 48, p);
  tmem_st_wait();
  float sum = 0.f;
  const uint32_t cs[4] = {s0, s1, s2, s3};
#pragma unroll
  for (int i = 0; i < 4; ++i) sum += __uint_as_float(cs[i] << 16) + __uint_as_float(cs[i] & 0xFFFF0000u);
  return sum;
}

// ---- Haar filter of one 256-token block in shared memory ------------------------------------------
// T_f x = f_0 x + sum_{i=1..L} (f_i - f_{i-1}) * blockmean_{2^i}(x): the detail projector of level l
// is blockmean_{2^(l-1)} - blockmean_{2^l} and the approximation projector of level L is
// blockmean_{2^L}, so only aligned block sums of 2, 4, ..., 2^L rows are needed.
//
// The block is filtered on packed bf16 pairs wherever that costs no accuracy that matters: the sums of
// row pairs (level 1) are packed bf16 adds, everything coarser is fp32 on those 32 sums per thread, and
// the last step, f_0 x + c, is one packed bf16 fma per two elements (one rounding, like a conversion of
// the fp32 result) with c rounded to bf16 first.  A packed fma needs f_0 as a bf16 value; instead of
// rounding the coefficient (a systematic error), the stage computes r T_f x with r = bf16(f_0) / f_0: the
// coefficient of x is then exact and every other coefficient is scaled by r in fp32.  ReLU is positively
// homogeneous and r > 0, so the features come out scaled by r as well and the kernels take the factor
// out again where they leave results (S', z': divided by r; output: eps' scaled by r).
//
// Coefficient table in shared memory, written once per CTA by the Haar warps:
//   hc[0] = bf16(f_0) in both halves (bit pattern), hc[i] = r k_i = r (f_i - f_{i-1}) / 2^i for i = 1..5
//   (0 beyond L), hc[8 + 8 hw + w] = weight of warp w's 32-row sum in warp hw's levels 6-8 term
//                                  = r (k_8 + [same 128-row group] k_7 + [same 64-row group] k_6).
constexpr int kHaarCoefs = 8 + 64;
static_assert(kHaarCoefs * 4 <= 1024, "coefficient table must fit its shared-memory slot");

// r = bf16(f_0) / f_0 (1 when f_0 = 0): the factor by which the filtered block, and with it the features, come
// out scaled.  Every role that needs it computes it from f_0 with these same operations.
__device__ __forceinline__ float haar_scale(float f0) {
  const float f0b = __uint_as_float(pack_bf16x2(f0, f0) << 16);
  return f0 != 0.f ? f0b / f0 : 1.f;
}

__device__ __forceinline__ void haar_coef_init(float* hc, const float* __restrict__ f, int L, int ht) {
  const float r = haar_scale(f[0]);
  float k[kMaxLevels + 1];
  k[0] = f[0];
  float scale = 0.5f * r;
#pragma unroll
  for (int i = 1; i <= kMaxLevels; ++i) {
    k[i] = (i <= L) ? (f[i] - f[i - 1]) * scale : 0.f;
    scale *= 0.5f;
  }
  if (ht == 0) hc[0] = __uint_as_float(pack_bf16x2(k[0], k[0]));
  if (ht >= 1 && ht < 6) {
    float v = k[1];
#pragma unroll
    for (int i = 2; i < 6; ++i) v = (ht == i) ? k[i] : v;
    hc[ht] = v;
  }
  if (ht < 64) {
    const int hw = ht >> 3, w = ht & 7;
    hc[8 + ht] = k[8] + ((w >> 2) == (hw >> 2) ? k[7] : 0.f) + ((w >> 1) == (hw >> 1) ? k[6] : 0.f);
  }
}

__device__ __forceinline__ uint32_t fma_bf16x2(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}

// 256 threads (ht = 0..255) filter the block (two 128-row tiles) in place.  Thread (c = ht & 7, rg = ht >> 3) owns rows
// 8 rg .. 8 rg + 7 of 16-byte chunk c: levels 1-3 in registers, levels 4-5 through warp shuffles
// (a warp covers 32 consecutive rows), levels 6-8 through the 32-row sums the eight warps leave in
// `xch` (8 x 64 floats, double-buffered by the caller) around one named barrier of the 256 threads.
// The barrier is executed whether or not `ok` holds, so that a role that gave up on a wait keeps the
// barrier balanced; with ok = false no memory is touched.  Rows >= valid_rows lie past the end of the
// sequence: they arrive as zeros (the zero padding of Algorithm 2) and leave as zeros (the trim
// before the feature map).
__device__ __forceinline__ void haar_block_inplace(uint8_t* tile0, uint8_t* tile1, const float* hc, bool cross,
                                                   float* xch, int ht, int valid_rows, bool ok) {
  const int c = ht & 7, rg = ht >> 3, lane = ht & 31, hw = ht >> 5;
  uint8_t* base = (rg < 16 ? tile0 : tile1) + (rg & 15) * 1024;   // rows 0-127 / 128-255 of the block
  uint32_t u[8][4];   // 8 rows x 4 column pairs, as loaded
  float a[4][8];      // sums of row pairs, then the additive term c of each row pair
  float hi[8], s5[8];
  if (ok) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {   // row 8 rg + j has swizzle phase j
      const uint4 raw = *reinterpret_cast<const uint4*>(base + j * 128 + ((c ^ j) << 4));
      u[j][0] = raw.x; u[j][1] = raw.y; u[j][2] = raw.z; u[j][3] = raw.w;
    }
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t s = add_bf16x2(u[2 * p][i], u[2 * p + 1][i]);
        a[p][2 * i] = __uint_as_float(s << 16);
        a[p][2 * i + 1] = __uint_as_float(s & 0xFFFF0000u);
      }
    const float k3 = hc[3], k4 = hc[4], k5 = hc[5];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float s3 = (a[0][q] + a[1][q]) + (a[2][q] + a[3][q]);
      const float s4 = s3 + __shfl_xor_sync(0xffffffffu, s3, 8);
      s5[q] = s4 + __shfl_xor_sync(0xffffffffu, s4, 16);
      hi[q] = fmaf(k3, s3, fmaf(k4, s4, k5 * s5[q]));
    }
  }
  if (cross) {   // uniform over the kernel: L > 5
    if (ok && (lane >> 3) == 0) {
      float4* dst = reinterpret_cast<float4*>(xch + hw * kD + c * 8);
      dst[0] = make_float4(s5[0], s5[1], s5[2], s5[3]);
      dst[1] = make_float4(s5[4], s5[5], s5[6], s5[7]);
    }
    named_bar_sync(kBarHaar, 256);
    if (ok) {
      // lane (c, q = lane >> 3) combines the eight warps' sums of columns 2 q, 2 q + 1 of chunk c (two
      // independent chains of four), then the four lanes that share a chunk swap their pairs
      const int qq = lane >> 3;
      const float2* src = reinterpret_cast<const float2*>(xch + c * 8 + 2 * qq);
      const float* cf = hc + 8 + 8 * hw;
      float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;
#pragma unroll
      for (int w = 0; w < 8; w += 2) {
        const float2 v0 = src[w * (kD / 2)], v1 = src[(w + 1) * (kD / 2)];
        a0 = fmaf(cf[w], v0.x, a0);
        a1 = fmaf(cf[w], v0.y, a1);
        b0 = fmaf(cf[w + 1], v1.x, b0);
        b1 = fmaf(cf[w + 1], v1.y, b1);
      }
      const float lo = a0 + b0, hi_ = a1 + b1;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int sl = (q << 3) | c;
        hi[2 * q] += __shfl_sync(0xffffffffu, lo, sl);
        hi[2 * q + 1] += __shfl_sync(0xffffffffu, hi_, sl);
      }
    }
  }
  if (ok) {
    const float k1 = hc[1], k2 = hc[2];
    const uint32_t f0 = __float_as_uint(hc[0]);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float c20 = fmaf(k2, a[0][q] + a[1][q], hi[q]), c21 = fmaf(k2, a[2][q] + a[3][q], hi[q]);
      a[0][q] = fmaf(k1, a[0][q], c20);
      a[1][q] = fmaf(k1, a[1][q], c20);
      a[2][q] = fmaf(k1, a[2][q], c21);
      a[3][q] = fmaf(k1, a[3][q], c21);
    }
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t cp = pack_bf16x2(a[p][2 * i], a[p][2 * i + 1]);
        u[2 * p][i] = fma_bf16x2(f0, u[2 * p][i], cp);
        u[2 * p + 1][i] = fma_bf16x2(f0, u[2 * p + 1][i], cp);
      }
    if (rg * 8 + 8 <= valid_rows) {   // the usual case: every row of this thread lies inside the sequence
#pragma unroll
      for (int j = 0; j < 8; ++j)
        *reinterpret_cast<uint4*>(base + j * 128 + ((c ^ j) << 4)) = make_uint4(u[j][0], u[j][1], u[j][2], u[j][3]);
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        uint4 out = make_uint4(u[j][0], u[j][1], u[j][2], u[j][3]);
        if (rg * 8 + j >= valid_rows) out = make_uint4(0u, 0u, 0u, 0u);
        *reinterpret_cast<uint4*>(base + j * 128 + ((c ^ j) << 4)) = out;
      }
    }
  }
}

// One Haar step: wait for the two raw tiles of block b (counted over all the work items of the CTA, like
// the ring slots and barrier phases), filter them in place, hand the block to the MMA issuer.  NX = number
// of tile slots in the ring; valid_rows = rows of the block that lie inside the sequence.
template <int NX, typename Bars>
__device__ __forceinline__ bool haar_step(uint8_t* xring, Bars* bars, float* xch, const float* hcoef, bool cross,
                                          int b, int valid_rows, int ht, bool ok, volatile int* abort_flag,
                                          int* status) {
  const int t0 = 2 * b, t1 = 2 * b + 1;
  const int s0 = t0 % NX, s1 = t1 % NX;
  if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bars->x_full[s0], (t0 / NX) & 1, abort_flag, status, kErrHaar));
  if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bars->x_full[s1], (t1 / NX) & 1, abort_flag, status, kErrHaar));
  haar_block_inplace(xring + s0 * kTileBytes, xring + s1 * kTileBytes, hcoef, cross, xch + (b & 1) * 8 * kD, ht,
                     valid_rows, ok);
  if (ok) {
    fence_proxy_async_smem();   // generic-proxy writes -> visible to the tensor core's reads
    warp_arrive(&bars->xf_ready[b & (kNF - 1)]);
  }
  return ok;
}

// ---- work items ---------------------------------------------------------------------------------
// Both kernels run one CTA per SM that walks work items: item = slab * chunks + chunk is one sequence
// chunk of one slab, CTA c takes items c, c + gridDim.x, c + 2 gridDim.x, ...  Ring slots, accumulator
// buffers and barrier phases count on across items, so the copies and the filter stage of the next item
// run while the current one is still in the tensor pipe; only what belongs to a slab (filter
// coefficients, accumulators, the S' image) is renewed at an item boundary.
__device__ __forceinline__ int item_blocks(int item, int chunks, int chunk_blocks, int n) {
  return min(chunk_blocks, (n + kBlk - 1) / kBlk - (item % chunks) * chunk_blocks);
}

// ---- key side -----------------------------------------------------------------------------------
// grid (chunks, slabs) when every CTA has one item, else (min(SMs, items)); block 640.  TMEM: D1[3] at columns 0 / 128 / 256, S' half h at 384 + 64 h.
// kMulti = false: every CTA has exactly one work item (the item loops run once and the code of the item
// boundaries drops out).
template <int NH, bool kMulti>
__global__ void __launch_bounds__(kThreads, 1)
k_tc_kside(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
           const __grid_constant__ CUtensorMap map_w, const float* __restrict__ f, float* __restrict__ spart,
           float* __restrict__ zpart, __nv_bfloat16* __restrict__ sbf, uint8_t* __restrict__ simg_out, int n, int L,
           int chunk_blocks, int chunks, int items, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  using SL = KsideSmem<NH>;
  KsideBars* bars = reinterpret_cast<KsideBars*>(smem + SL::bars);
  float* zx = reinterpret_cast<float*>(smem + SL::zx);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // item0 < items: the grid never exceeds the item count.  Without kMulti the step is a constant that ends
  // every item loop after one pass, so that the compiler sees straight-line code.
  const int item0 = blockIdx.y * gridDim.x + blockIdx.x, item_step = kMulti ? (int)gridDim.x : (1 << 30);
  if (!kMulti) items = item0 + 1;
  const int nblk0 = item_blocks(item0, chunks, chunk_blocks, n);
  constexpr bool single_item = !kMulti;
  constexpr int m = NH * 128;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kNXK; ++s) {
      mbar_init(&bars->x_full[s], 1);
      mbar_init(&bars->x_empty[s], 1);
    }
    for (int s = 0; s < kNF; ++s) mbar_init(&bars->xf_ready[s], 8);
    for (int s = 0; s < kNV; ++s) {
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_empty[s], NH);
    }
    for (int b = 0; b < 6; ++b) mbar_init(&bars->d1_full[b], 1);
    for (int b = 0; b < kND1; ++b) {
      mbar_init(&bars->phi_ready[b], 4);
      mbar_init(&bars->d1_free[b], 1);
    }
    mbar_init(&bars->acc_done, NH);
    mbar_init(&bars->acc_free, 8);
    mbar_init(&bars->w_full, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
    // K and V are inputs: the first copies of both rings (tiles of the first item) go out before the
    // dependency wait below.  K, V and the output are touched once per forward: their copies carry the
    // evict-first L2 policy (measured: 1-5 us per forward over the default policy; the same hint on the
    // query side's Q tiles cost 4 us and is not used).
    const int slab = item0 / chunks, row0 = (item0 % chunks) * chunk_blocks * kBlk;
    for (int b = 0; b < min(2 * nblk0, kNXK); ++b) {
      mbar_arrive_expect_tx(&bars->x_full[b], kTileBytes);
      tma_load_3d_hint(smem + SL::x + b * kTileBytes, &map_k, 0, row0 + b * kTile, slab, &bars->x_full[b], policy_evict_first());
    }
    for (int b = 0; b < min(2 * nblk0, kNV); ++b) {
      mbar_arrive_expect_tx(&bars->v_full[b], kTileBytes);
      tma_load_3d_hint(smem + SL::v + b * kTileBytes, &map_v, 0, row0 + b * kTile, slab, &bars->v_full[b], policy_evict_first());
    }
  }
  if (warp == kWarpMma) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  // Programmatic dependent launch: this kernel may have started while the mean-pool / gate kernel was
  // still running, and W^T and the gate coefficients f are that kernel's results.  Only then may the
  // kernels after this one be staged: the reduction waits for this grid itself, but it lets the query
  // side start in turn, whose set-up reads W^T and f without a wait of its own.
  griddep_wait();
  griddep_launch();
  if (threadIdx.x == 0) {   // the W^T image (m rows of 64 bf16) arrives by TMA; only the MMA1 issuer waits for it
    mbar_arrive_expect_tx(&bars->w_full, NH * kTileBytes);
#pragma unroll
    for (int h = 0; h < NH; ++h) tma_load_3d(smem + SL::wt + h * kTileBytes, &map_w, 0, h * kTile, 0, &bars->w_full);
  }
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bars->tmem_base;
  volatile int* abort_flag = &bars->abort_flag;

  if (warp < kReluWarp0) {
    reg_dec<kRegsCtl>();
    if (warp == kWarpTma && lane == 0) {
      // One producer for both rings: whichever ring has a free slot gets its next tile, so that a full
      // V ring never holds back the K tiles (and the other way round).  Each ring walks the tiles of this
      // CTA's items on its own: (ik, tk) / (iv, tv) = item and tile of the next K / V copy, kb / vb = tiles
      // sent so far (slot and phase of the ring).
      int kb = min(2 * nblk0, kNXK), vb = min(2 * nblk0, kNV);   // the first ring of each went out during set-up
      int ik = item0, tk = kb, iv = item0, tv = vb;
      int nk = 2 * nblk0, nv = 2 * nblk0;                         // tiles of item ik / iv
      if (tk == nk) {
        ik += item_step;
        tk = 0;
        if (ik < items) nk = 2 * item_blocks(ik, chunks, chunk_blocks, n);
      }
      if (tv == nv) {
        iv += item_step;
        tv = 0;
        if (iv < items) nv = 2 * item_blocks(iv, chunks, chunk_blocks, n);
      }
      unsigned long long t0 = global_timer_ns();
      uint32_t spins = 0;
      bool ok = true;
      while (ok && (ik < items || iv < items)) {
        bool progress = false;
        if (ik < items && mbar_try_wait(&bars->x_empty[kb % kNXK], ((kb / kNXK) & 1) ^ 1)) {
          const int s = kb % kNXK;
          mbar_arrive_expect_tx(&bars->x_full[s], kTileBytes);
          tma_load_3d_hint(smem + SL::x + s * kTileBytes, &map_k, 0, (ik % chunks) * chunk_blocks * kBlk + tk * kTile,
                      ik / chunks, &bars->x_full[s], policy_evict_first());
          ++kb;
          if (++tk == nk) {
            ik += item_step;
            tk = 0;
            if (ik < items) nk = 2 * item_blocks(ik, chunks, chunk_blocks, n);
          }
          progress = true;
        }
        if (iv < items && mbar_try_wait(&bars->v_empty[vb % kNV], ((vb / kNV) & 1) ^ 1)) {
          const int s = vb % kNV;
          mbar_arrive_expect_tx(&bars->v_full[s], kTileBytes);
          tma_load_3d_hint(smem + SL::v + s * kTileBytes, &map_v, 0, (iv % chunks) * chunk_blocks * kBlk + tv * kTile,
                      iv / chunks, &bars->v_full[s], policy_evict_first());
          ++vb;
          if (++tv == nv) {
            iv += item_step;
            tv = 0;
            if (iv < items) nv = 2 * item_blocks(iv, chunks, chunk_blocks, n);
          }
          progress = true;
        }
        if (progress) {
          t0 = global_timer_ns();   // the limit bounds the time without progress
        } else if ((++spins & 255u) == 0) {
          if (*abort_flag != 0) ok = false;
          else if (global_timer_ns() - t0 > kWaitLimitNs * 2) {
            *abort_flag = 1;
            atomicCAS(status, 0, kErrProducer);
            ok = false;
          }
        }
      }
      if (*abort_flag != 0) {   // let copies in flight land before the CTA's shared memory goes away
        for (int b = max(0, kb - kNXK); b < kb; ++b) mbar_wait_drain(&bars->x_full[b % kNXK], (b / kNXK) & 1);
        for (int b = max(0, vb - kNV); b < vb; ++b) mbar_wait_drain(&bars->v_full[b % kNV], (b / kNV) & 1);
        mbar_wait_drain(&bars->w_full, 0);
      }
    } else if (warp == kWarpMma && lane == 0) {
      // MMA1 of every unit.  Ring slots, D1 buffers and barrier phases are running counters, and the
      // descriptors only add to their start-address word.
      constexpr uint32_t kTileStep = kTileBytes >> 4;
      const uint32_t hi = smem_desc_hi(1024);
      const uint32_t wt_lo = smem_desc_lo(smem_u32(smem + SL::wt), 16);
      const uint32_t x_lo = smem_desc_lo(smem_u32(smem + SL::x), 16);
      uint32_t xs = 0, fs = 0, fpar = 0;               // K ring slot; "block filtered" barrier and phase
      uint32_t c3 = 0, c6 = 0, round = 0;              // D1 buffer, d1_full barrier, uses of buffer 0 so far
      bool ok = mbar_wait(&bars->w_full, 0, abort_flag, status, kErrMma);
      int blocks_all = 0;                              // blocks of all items of this CTA
      for (int it = item0; it < items; it += item_step) blocks_all += item_blocks(it, chunks, chunk_blocks, n);
      for (int b = 0; b < blocks_all && ok; ++b) {
        ok = mbar_wait(&bars->xf_ready[fs], fpar, abort_flag, status, kErrMma);
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll
        for (int j = 0; j < 2 * NH; ++j) {
          const int h = j % NH;
          if (round > 0) {   // the MMA2 that read this D1 buffer three units ago must have completed
            ok = mbar_wait(&bars->d1_free[c3], (round - 1) & 1, abort_flag, status, kErrMma);
            if (!ok) break;
            tc_fence_after_sync();
          }
          const uint32_t a_lo = wt_lo + h * kTileStep, b_lo = x_lo + xs * kTileStep;
          const uint32_t d1 = tmem + c3 * 128;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_ss(d1, smem_desc_join(a_lo + 2 * k, hi), smem_desc_join(b_lo + 2 * k, hi), kIdesc1, k > 0);
          mma_commit(&bars->d1_full[c6]);
          if (h == NH - 1) {   // last MMA1 that reads this tile
            mma_commit(&bars->x_empty[xs]);
            xs = xs == kNXK - 1 ? 0 : xs + 1;
          }
          c3 = c3 == kND1 - 1 ? 0 : c3 + 1;
          round += (c3 == 0);
          c6 = c6 == 5 ? 0 : c6 + 1;
        }
        fs = (fs + 1) & (kNF - 1);
        fpar ^= (fs == 0);
      }
    } else if (warp >= kWarpMma2 && warp - kWarpMma2 < NH && lane == 0) {
      // MMA2 of the units of feature half h (one issuing thread per half, each with its own
      // accumulator): S'[half h] += Phi^T (the unit's D1 buffer, bf16 pairs) * V tile.
      const int h = warp - kWarpMma2;
      constexpr uint32_t kTileStep = kTileBytes >> 4;
      const uint32_t hi = smem_desc_hi(1024);
      const uint32_t v_lo = smem_desc_lo(smem_u32(smem + SL::v), 1024);
      const uint32_t acc = tmem + kAccCol + h * 64;
      uint32_t vs = 0, vpar = 0;                       // V ring slot / phase
      int gt = 0, ic = 0;                              // tiles and items so far
      bool ok = true;
      for (int it = item0; it < items && ok; it += item_step, ++ic) {
        const int ntl = 2 * item_blocks(it, chunks, chunk_blocks, n);
        if (ic > 0) {   // the accumulators of the item before must have been read out
          ok = mbar_wait(&bars->acc_free, (ic - 1) & 1, abort_flag, status, kErrMma);
          if (!ok) break;
          tc_fence_after_sync();
        }
        for (int t = 0; t < ntl && ok; ++t, ++gt) {
          const int u = gt * NH + h, p3 = u % kND1;
          ok = mbar_wait(&bars->v_full[vs], vpar, abort_flag, status, kErrMma);
          if (!ok) break;
          ok = mbar_wait(&bars->phi_ready[p3], (u / kND1) & 1, abort_flag, status, kErrMma);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t a_tm = tmem + p3 * 128;
          const uint32_t b_lo = v_lo + vs * kTileStep;
#pragma unroll
          for (int k = 0; k < 8; ++k)
            mma_ts(acc, a_tm + k * 8, smem_desc_join(b_lo + 128 * k, hi), kIdesc2, (t > 0 || k > 0) ? 1u : 0u);
          mma_commit(&bars->d1_free[p3]);
          mma_commit(&bars->v_empty[vs]);   // one arrival per half
          vs = vs == kNV - 1 ? 0 : vs + 1;
          vpar ^= (vs == 0);
        }
        if (ok) mma_commit(&bars->acc_done);   // one phase per item
      }
    }
  } else if (warp >= kReluWarp0 && warp < kAuxWarp0) {
    const int g = (warp - kReluWarp0) >> 2;         // ReLU warpgroup 0 / 1
    const uint32_t lane_base = 32u * (warp & 3);
    const int row = lane_base + lane;               // feature within the half = TMEM lane
    bool ok = true;
    int gu0 = 0, ic = 0;                            // units and items so far (an item has an even number of units)
    for (int it = item0; it < items; it += item_step, ++ic) {
      const int slab = it / chunks;
      const int units = item_blocks(it, chunks, chunk_blocks, n) * 2 * NH;
      float zacc = 0.f;
      for (int u = g; u < units; u += 2) {
        const int gu = gu0 + u;
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bars->d1_full[gu % 6], (gu / 6) & 1, abort_flag, status, kErrRelu));
        if (ok) {
          tc_fence_after_sync();
          zacc += relu_unit(tmem + (lane_base << 16) + (gu % kND1) * 128);
          tc_fence_before_sync();
          warp_arrive(&bars->phi_ready[gu % kND1]);
        }
      }
      gu0 += units;
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bars->acc_done, ic & 1, abort_flag, status, kErrRelu));
      if (ok) tc_fence_after_sync();
      const size_t pidx = (size_t)it;                 // = slab * chunks + chunk
      if (NH == 1) {   // both warpgroups saw the same 128 features on alternating tiles
        if (ic > 0) named_bar_sync(kBarZsum, 256);    // the sums of the item before have been read
        if (g == 1) zx[row] = zacc;
        named_bar_sync(kBarZsum, 256);
        if (g == 0) zacc += zx[row];
      }
      if (ok && (NH == 2 || g == 0)) {
        const int feat0 = (NH == 2 ? g * 128 : 0) + (int)lane_base;   // first feature of this warp
        // the filter stage left K_F, and with it the features, scaled by r (see haar_block_inplace)
        const float inv_r = 1.f / haar_scale(f[(size_t)slab * (L + 1)]);
        const uint32_t acc_addr = tmem + (lane_base << 16) + kAccCol + (NH == 2 ? g * 64 : 0);
        if (single_item) {
          // The accumulator row of a thread is one feature's 64 values; written straight from the registers
          // a warp would touch 32 different 256-byte rows per store.  With one item per CTA the K ring is
          // idle by now: each warp turns its 32 x 32 chunk around in it (rows padded to 33 floats) and
          // writes whole 128-byte row segments.
          float* stage = reinterpret_cast<float*>(smem + SL::x) + (warp - kReluWarp0) * (32 * 33);
          float* dst = spart + (pidx * m + feat0) * kD;
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            uint32_t r[32];
            tmem_ld32(acc_addr + 32 * c, r);
            tmem_ld_wait();
            reg_fence32(r);
#pragma unroll
            for (int j = 0; j < 32; ++j) stage[lane * 33 + j] = __uint_as_float(r[j]) * inv_r;
            if (sbf != nullptr) {   // ... and the operand image of the query side (features along a row)
              uint8_t* img = simg_out + pidx * simg_bytes(m);
#pragma unroll
              for (int j = 0; j < 32; ++j)
                *reinterpret_cast<__nv_bfloat16*>(img + simg_offset(feat0 + lane, 32 * c + j)) =
                    __float2bfloat16_rn(__uint_as_float(r[j]) * inv_r);
            }
            __syncwarp();
#pragma unroll 8
            for (int rr = 0; rr < 32; ++rr) dst[(size_t)rr * kD + 32 * c + lane] = stage[rr * 33 + lane];
            if (sbf != nullptr) {   // one chunk per slab: this is S' itself, leave its bf16 image as well
              __nv_bfloat16* bdst = sbf + (pidx * m + feat0) * kD + 32 * c;
#pragma unroll 8
              for (int rr = 0; rr < 32; rr += 2) {   // two rows per instruction, a pair of columns per lane
                const int rw = rr + (lane >> 4), cc = 2 * (lane & 15);
                *reinterpret_cast<uint32_t*>(bdst + (size_t)rw * kD + cc) =
                    pack_bf16x2(stage[rw * 33 + cc], stage[rw * 33 + cc + 1]);
              }
            }
            __syncwarp();
          }
        } else {
          // More items follow and the rings already hold their tiles: every thread writes its own row
          // (16-byte stores; half-used sectors, but the accumulators are free again sooner).
          float* dst = spart + (pidx * m + feat0 + lane) * kD;
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            uint32_t r[32];
            tmem_ld32(acc_addr + 32 * c, r);
            tmem_ld_wait();
            reg_fence32(r);
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * inv_r);
#pragma unroll
            for (int q = 0; q < 8; ++q)
              *reinterpret_cast<uint4*>(dst + 32 * c + 4 * q) = make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
            if (sbf != nullptr) {
              uint8_t* img = simg_out + pidx * simg_bytes(m);
#pragma unroll
              for (int j = 0; j < 32; ++j)
                *reinterpret_cast<__nv_bfloat16*>(img + simg_offset(feat0 + lane, 32 * c + j)) =
                    __float2bfloat16_rn(__uint_as_float(r[j]));
              __nv_bfloat16* bdst = sbf + (pidx * m + feat0 + lane) * kD + 32 * c;
#pragma unroll
              for (int q = 0; q < 4; ++q)
                *reinterpret_cast<uint4*>(bdst + 8 * q) =
                    make_uint4(pack_bf16x2(__uint_as_float(r[8 * q]), __uint_as_float(r[8 * q + 1])),
                               pack_bf16x2(__uint_as_float(r[8 * q + 2]), __uint_as_float(r[8 * q + 3])),
                               pack_bf16x2(__uint_as_float(r[8 * q + 4]), __uint_as_float(r[8 * q + 5])),
                               pack_bf16x2(__uint_as_float(r[8 * q + 6]), __uint_as_float(r[8 * q + 7])));
            }
          }
        }
        zpart[pidx * m + feat0 + lane] = zacc * inv_r;
        if (sbf != nullptr) {   // z' is row 64 of the image, rows 65-79 are zero
          uint8_t* img = simg_out + pidx * simg_bytes(m);
          *reinterpret_cast<__nv_bfloat16*>(img + simg_offset(feat0 + lane, kD)) = __float2bfloat16_rn(zacc * inv_r);
#pragma unroll
          for (int row = kD + 1; row < kSimgRows; ++row)
            *reinterpret_cast<uint16_t*>(img + simg_offset(feat0 + lane, row)) = 0;
        }
      }
      // the accumulators may be overwritten by the next item
      tc_fence_before_sync();
      if (ok) warp_arrive(&bars->acc_free);
    }
  } else {
    reg_inc<kRegsAux>();
    const int ht = threadIdx.x - 32 * kAuxWarp0;
    float* hcoef = reinterpret_cast<float*>(smem + SL::hcoef);
    bool ok = true;
    int gb0 = 0;                                      // blocks of the items before
    for (int it = item0; it < items; it += item_step) {
      const int slab = it / chunks, blk0 = (it % chunks) * chunk_blocks;
      const int nblk = item_blocks(it, chunks, chunk_blocks, n);
      named_bar_sync(kBarCoef, 256);                  // nobody reads the coefficients of the item before any more
      haar_coef_init(hcoef, f + (size_t)slab * (L + 1), L, ht);
      named_bar_sync(kBarCoef, 256);
      for (int b = 0; b < nblk; ++b)
        ok = haar_step<kNXK>(smem + SL::x, bars, reinterpret_cast<float*>(smem + SL::xch), hcoef, L > 5, gb0 + b,
                             n - (blk0 + b) * kBlk, ht, ok, abort_flag, status);
      gb0 += nblk;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kWarpMma) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, kTmemCols);
  }
}

// ---- query side ---------------------------------------------------------------------------------
// The denominator rides on the tensor core: the B operand of MMA2 is the K-major image of
// [S' | z' | 0]^T (80 rows of m features), so that column 64 of the accumulator is D' = Phi z'.
//
// The image comes from global memory, where the kernel that produced S' and z' left it in the byte order of
// the shared-memory operand (simg_offset): 64-feature K blocks of 80 rows x 128 bytes (rows 0-63 = columns of
// S', row 64 = z', rows 65-79 = 0), 128-byte swizzle.  One bulk copy per work item fetches it.

// ReLU pass in 16-column steps (a smaller register footprint than relu_unit): fp32 TMEM columns -> bf16
// pairs in half as many columns.
__device__ __forceinline__ void reg_fence16(uint32_t (&r)[16]) {
  asm volatile(""
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]),
                 "+r"(r[15])
               :
               : "memory");
}
__device__ __forceinline__ void relu_pack16(const uint32_t (&r)[16], uint32_t (&p)[8]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) p[j] = relu_pack_bf16x2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
}
// STEPS steps of 16 fp32 columns starting at `in` -> 8 columns of bf16 pairs each starting at `out`
// (out <= in: a step's store lands at or below columns that were read before it was issued).
template <int STEPS>
__device__ __forceinline__ void relu_span(uint32_t in, uint32_t out) {
  static_assert(STEPS % 2 == 0, "two steps per iteration");
  uint32_t a[16], b[16], p[8];
  tmem_ld16(in, a);
#pragma unroll
  for (int c = 0; c < STEPS; c += 2) {
    tmem_ld_wait();
    reg_fence16(a);
    tmem_ld16(in + 16 * (c + 1), b);
    relu_pack16(a, p);
    tmem_st8(out + 8 * c, p);
    tmem_ld_wait();
    reg_fence16(b);
    if (c + 2 < STEPS) tmem_ld16(in + 16 * (c + 2), a);
    relu_pack16(b, p);
    tmem_st8(out + 8 * (c + 1), p);
  }
  tmem_st_wait();
}

// grid (min(SMs, items)), block 768; the CTA walks its work items as on the key side (tiles, buffers and
// barrier phases count on across items; the S' image and the filter coefficients are renewed when an item
// begins: one thread of the epilogue warps sends the bulk copy of an item's image once the last MMA2 that
// reads the buffer it goes to has completed).
// TMEM: two buffers of 256 columns; tile t uses buffer t & 1 for its D1
// (128 tokens x m features, fp32), then for the packed bf16 features and the [N' | D'] accumulator (see
// QTmem).  Per tile: MMA1 (warp 1) -> ReLU pass (warps 4-11, two warps per lane quarter that split the
// feature columns) -> MMA2 (warp 3) -> epilogue (warps 12-15: drain the accumulator, which frees the buffer
// for tile t + 2, scale by 1 / (D' + eps'), round to bf16 into one of two staging tiles, TMA store).
// kDen: the kernel also leaves every token's denominator D' + eps' (as it divides by it, i.e. carrying the
// filter stage's factor r) in den_out[slab * n + token]: a caller that splits the features into groups
// combines the groups' outputs with these weights.
template <int NH, bool kMulti, bool kDen = false>
__global__ void __launch_bounds__(kThreadsQ, 1)
k_tc_qside(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_o,
           const __grid_constant__ CUtensorMap map_w, const uint8_t* __restrict__ simg_g,
           const float* __restrict__ f, const float* __restrict__ beta, float eps,
           float bw_floor, int n, int L, int chunk_blocks, int chunks, int items, int* __restrict__ status,
           float* __restrict__ den_out) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  using SL = QsideSmem<NH>;
  using TM = QTmem<NH>;
  QsideBars* bars = reinterpret_cast<QsideBars*>(smem + SL::bars);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int item0 = blockIdx.y * gridDim.x + blockIdx.x, item_step = kMulti ? (int)gridDim.x : (1 << 30);   // as on the key side
  if (!kMulti) items = item0 + 1;
  constexpr int m = NH * 128;
  constexpr uint32_t kIdesc1Q = make_idesc_bf16(128, m, false, false);   // Q_F tile x all features

  if (threadIdx.x == 0) {
    for (int s = 0; s < kNXQ; ++s) {
      mbar_init(&bars->x_full[s], 1);
      mbar_init(&bars->x_empty[s], 1);
    }
    for (int s = 0; s < kNF; ++s) mbar_init(&bars->xf_ready[s], 8);
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->d1_full[b], 1);
      mbar_init(&bars->phi_ready[b], 8);
      mbar_init(&bars->d2_full[b], 1);
      mbar_init(&bars->buf_free[b], 4);
    }
    mbar_init(&bars->simg_ready, 1);
    mbar_init(&bars->simg_next, 1);
    mbar_init(&bars->w_full, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
    // W^T was complete before the kernel ahead of this one started: its image can be fetched at once
    mbar_arrive_expect_tx(&bars->w_full, NH * kTileBytes);
#pragma unroll
    for (int h = 0; h < NH; ++h) tma_load_3d(smem + SL::wt + h * kTileBytes, &map_w, 0, h * kTile, 0, &bars->w_full);
  }
  if (warp == kWarpMma) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bars->tmem_base;
  volatile int* abort_flag = &bars->abort_flag;

  if (warp < kReluWarp0) {
    reg_dec<kRegsCtlQ>();
    if (warp == kWarpTma && lane == 0) {
      int issued = 0;   // tiles sent so far, over all items (slot and phase of the ring)
      bool ok = true;
      for (int it = item0; it < items && ok; it += item_step) {
        const int slab = it / chunks, row0 = (it % chunks) * chunk_blocks * kBlk;
        const int ntl = 2 * item_blocks(it, chunks, chunk_blocks, n);
        for (int b = 0; b < ntl; ++b) {   // b counts 128-token tiles here
          const int s = issued % kNXQ;
          ok = mbar_wait(&bars->x_empty[s], ((issued / kNXQ) & 1) ^ 1, abort_flag, status, kErrProducer);
          if (!ok) break;
          mbar_arrive_expect_tx(&bars->x_full[s], kTileBytes);
          tma_load_3d(smem + SL::x + s * kTileBytes, &map_q, 0, row0 + b * kTile, slab, &bars->x_full[s]);
          ++issued;
        }
      }
      if (*abort_flag != 0) {
        for (int b = max(0, issued - kNXQ); b < issued; ++b) mbar_wait_drain(&bars->x_full[b % kNXQ], (b / kNXQ) & 1);
        mbar_wait_drain(&bars->w_full, 0);
      }
    } else if (warp == kWarpMma && lane == 0) {
      // MMA1 of every tile: D1[128 tokens x m] = Q_F tile (K-major) * W (as W^T rows, K-major), one
      // instruction per 16 columns of the head dimension.  The W^T image is m contiguous 128-byte rows.
      constexpr uint32_t kTileStep = kTileBytes >> 4;
      const uint32_t hi = smem_desc_hi(1024);
      const uint32_t wt_lo = smem_desc_lo(smem_u32(smem + SL::wt), 16);
      const uint32_t x_lo = smem_desc_lo(smem_u32(smem + SL::x), 16);
      uint32_t xs = 0, fs = 0, fpar = 0;
      int t = 0;
      bool ok = mbar_wait(&bars->w_full, 0, abort_flag, status, kErrMma);
      int blocks_all = 0;   // blocks of all items of this CTA
      for (int it = item0; it < items; it += item_step) blocks_all += item_blocks(it, chunks, chunk_blocks, n);
      for (int b = 0; b < blocks_all && ok; ++b) {
        ok = mbar_wait(&bars->xf_ready[fs], fpar, abort_flag, status, kErrMma);
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll
        for (int j = 0; j < 2; ++j, ++t) {
          const int buf = t & 1;
          if (t >= 2) {   // the epilogue must have drained the accumulator of tile t - 2 (same buffer)
            ok = mbar_wait(&bars->buf_free[buf], ((t >> 1) - 1) & 1, abort_flag, status, kErrMma);
            if (!ok) break;
            tc_fence_after_sync();
          }
          const uint32_t a_lo = x_lo + xs * kTileStep;
          const uint32_t d1 = tmem + buf * kQBufCols;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_ss(d1, smem_desc_join(a_lo + 2 * k, hi), smem_desc_join(wt_lo + 2 * k, hi), kIdesc1Q, k > 0);
          mma_commit(&bars->d1_full[buf]);
          mma_commit(&bars->x_empty[xs]);
          xs = xs == kNXQ - 1 ? 0 : xs + 1;
        }
        fs = (fs + 1) & (kNF - 1);
        fpar ^= (fs == 0);
      }
    } else if (warp == kWarpMma2Q && lane == 0) {
      // MMA2 of every tile: [N' | D'] = Phi (bf16 pairs in the tile's buffer) * [S' | z' | 0].
      const uint32_t hi = smem_desc_hi(1024);
      const uint32_t s_lo0 = smem_desc_lo(smem_u32(smem + SL::simg), 16);
      bool ok = true;
      int t = 0, ic = 0;   // tiles and items so far
      for (int it = item0; it < items && ok; it += item_step, ++ic) {
        const int ntl = 2 * item_blocks(it, chunks, chunk_blocks, n);
        // the [S' | z' | 0]^T image of this item's slab is in place (items alternate between two images
        // where there are two)
        ok = ic == 0 ? mbar_wait(&bars->simg_ready, 0, abort_flag, status, kErrMma)
                     : mbar_wait(&bars->simg_next, (ic - 1) & 1, abort_flag, status, kErrMma);
        const uint32_t s_lo = s_lo0 + ((kMulti && SL::two_images && (ic & 1)) ? (SL::simg_bytes >> 4) : 0u);
        for (int tt = 0; tt < ntl && ok; ++tt, ++t) {
          const int buf = t & 1;
          ok = mbar_wait(&bars->phi_ready[buf], (t >> 1) & 1, abort_flag, status, kErrMma);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t base = tmem + buf * kQBufCols;
#pragma unroll
          for (int k = 0; k < 8 * NH; ++k) {   // K block k / 4 of the image, 32 bytes per step of 16 features inside it
            const uint32_t b_lo = s_lo + (k >> 2) * (kSztBlockBytes >> 4) + 2 * (k & 3);
            mma_ts(base + TM::kAcc, base + TM::phi_col(k), smem_desc_join(b_lo, hi), kIdesc2Q, k > 0 ? 1u : 0u);
          }
          mma_commit(&bars->d2_full[buf]);
        }
      }
    }
  } else if (warp < kEpiWarp0Q) {
    reg_dec<kRegsReluQ>();
    const int g = (warp - kReluWarp0) >> 2;
    const uint32_t lane_base = 32u * (warp & 3);
    bool ok = true;
    int tiles_all = 0;   // tiles of all items of this CTA
    for (int it = item0; it < items; it += item_step) tiles_all += 2 * item_blocks(it, chunks, chunk_blocks, n);
    for (int t = 0; t < tiles_all; ++t) {
      const int buf = t & 1;
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bars->d1_full[buf], (t >> 1) & 1, abort_flag, status, kErrRelu));
      if (ok) {
        tc_fence_after_sync();
        const uint32_t base = tmem + (lane_base << 16) + buf * kQBufCols;
        // the two warps of a lane quarter split the columns (5 : 3 chunks with m = 256) and swap parts from
        // tile to tile
        if (((g ^ t) & 1) == 0) relu_span<2 * TM::kHeavy>(base, base);
        else relu_span<2 * (TM::kChunks - TM::kHeavy)>(base + TM::kLightCol, base + TM::kLightCol);
        tc_fence_before_sync();
        warp_arrive(&bars->phi_ready[buf]);
      }
    }
  } else if (warp < kAuxWarp0Q) {
    reg_inc<kRegsEpiQ>();
    const int et = threadIdx.x - 32 * kEpiWarp0Q;     // 0..127 = token row of the tile = TMEM lane
    int img_sent = 0;                                 // bulk copies of images sent by thread 0 (first one included)
    if (et == 0) {
      // S' and z', and with them the image, come from the kernel before this one in the stream, which may
      // still be running (programmatic dependent launch); everything else this kernel reads was complete
      // before that kernel started.
      griddep_wait();
      mbar_arrive_expect_tx(&bars->simg_ready, SL::simg_bytes);
      bulk_load_1d(smem + SL::simg, simg_g + (size_t)(item0 / chunks) * SL::simg_bytes, SL::simg_bytes, &bars->simg_ready);
      img_sent = 1;
    }
    const uint32_t lane_base = 32u * (warp & 3);
    const float bw = fmaxf(beta[0], bw_floor);
    bool ok = true;
    int t = 0, ic = 0;   // tiles and items so far
    float f0 = f[(size_t)(item0 / chunks) * (L + 1)];   // f_0 of the item's slab, fetched one item ahead
    for (int it = item0; it < items; it += item_step, ++ic) {
    const int slab = it / chunks, blk0 = (it % chunks) * chunk_blocks;
    const int ntl = 2 * item_blocks(it, chunks, chunk_blocks, n);
    const int nxt = it + item_step;
    if (kMulti && et == 0 && ok) {
      if (SL::two_images) {
        // Two images: the one of the next item is fetched now, into the buffer that the item before this one
        // used (every MMA2 of that item has completed: its last accumulator was drained above).
        if (nxt < items) {
          mbar_arrive_expect_tx(&bars->simg_next, SL::simg_bytes);
          bulk_load_1d(smem + SL::simg + ((ic + 1) & 1) * SL::simg_bytes, simg_g + (size_t)(nxt / chunks) * SL::simg_bytes,
                       SL::simg_bytes, &bars->simg_next);
          ++img_sent;
        }
      } else if (ic > 0) {
        // One image: every MMA2 of the item before has completed, this item's image takes its place.
        mbar_arrive_expect_tx(&bars->simg_next, SL::simg_bytes);
        bulk_load_1d(smem + SL::simg, simg_g + (size_t)slab * SL::simg_bytes, SL::simg_bytes, &bars->simg_next);
        ++img_sent;
      }
    }
    // the filter stage left Q_F, and with it N' and D', scaled by r (see haar_block_inplace): eps' follows
    const float epsp = eps * (float)m * bw * bw * haar_scale(f0);
    if (kMulti && nxt < items) f0 = f[(size_t)(nxt / chunks) * (L + 1)];
    for (int tt = 0; tt < ntl; ++tt, ++t) {
      const int buf = t & 1;
      const uint32_t base = tmem + (lane_base << 16) + buf * kQBufCols + TM::kAcc;
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bars->d2_full[buf], (t >> 1) & 1, abort_flag, status, kErrEpilogue));
      uint32_t r0[32], r1[32], dd = 0;
      if (ok) {
        tc_fence_after_sync();
        tmem_ld32(base, r0);
        tmem_ld32(base + 32, r1);
        tmem_ld1(base + 64, dd);
        tmem_ld_wait();
        reg_fence32(r0);
        reg_fence32(r1);
        tc_fence_before_sync();
        warp_arrive(&bars->buf_free[buf]);
      }
      // the staging tile was last used by tile t - 2: its TMA store must have finished reading
      if (et == 0) bulk_wait_group_read1();
      named_bar_sync(kBarOut0, 128);
      uint8_t* ost = smem + SL::ost + (t & 1) * kTileBytes;
      if (ok) {
        const float inv = 1.f / (__uint_as_float(dd) + epsp);
        if constexpr (kDen) {
          const int row = blk0 * kBlk + tt * kTile + et;
          if (row < n) den_out[(size_t)slab * n + row] = __uint_as_float(dd) + epsp;
        }
        const f32x2 inv2 = pk2(inv, inv);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint4 v;
          v.x = pack2_bf16(mul2(pk2(__uint_as_float(r0[8 * c]), __uint_as_float(r0[8 * c + 1])), inv2));
          v.y = pack2_bf16(mul2(pk2(__uint_as_float(r0[8 * c + 2]), __uint_as_float(r0[8 * c + 3])), inv2));
          v.z = pack2_bf16(mul2(pk2(__uint_as_float(r0[8 * c + 4]), __uint_as_float(r0[8 * c + 5])), inv2));
          v.w = pack2_bf16(mul2(pk2(__uint_as_float(r0[8 * c + 6]), __uint_as_float(r0[8 * c + 7])), inv2));
          *reinterpret_cast<uint4*>(ost + swz128(et, c)) = v;
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint4 v;
          v.x = pack2_bf16(mul2(pk2(__uint_as_float(r1[8 * c]), __uint_as_float(r1[8 * c + 1])), inv2));
          v.y = pack2_bf16(mul2(pk2(__uint_as_float(r1[8 * c + 2]), __uint_as_float(r1[8 * c + 3])), inv2));
          v.z = pack2_bf16(mul2(pk2(__uint_as_float(r1[8 * c + 4]), __uint_as_float(r1[8 * c + 5])), inv2));
          v.w = pack2_bf16(mul2(pk2(__uint_as_float(r1[8 * c + 6]), __uint_as_float(r1[8 * c + 7])), inv2));
          *reinterpret_cast<uint4*>(ost + swz128(et, 4 + c)) = v;
        }
        fence_proxy_async_smem();
      }
      named_bar_sync(kBarOut0, 128);
      const int row0 = blk0 * kBlk + tt * kTile;
      if (et == 0 && ok && row0 < n) {   // rows past n are clipped by the store
        tma_store_3d_hint(&map_o, ost, 0, row0, slab, policy_evict_first());
        bulk_commit_group();
      }
    }
    }
    if (et == 0 && *abort_flag != 0) {   // an image copy may still be in flight
      if (img_sent >= 1) mbar_wait_drain(&bars->simg_ready, 0);
      if (img_sent >= 2) mbar_wait_drain(&bars->simg_next, (img_sent - 2) & 1);
    }
    if (et == 0) bulk_wait_group0();
  } else {
    reg_inc<kRegsAux>();
    const int ht = threadIdx.x - 32 * kAuxWarp0Q;
    float* hcoef = reinterpret_cast<float*>(smem + SL::hcoef);
    bool ok = true;
    int gb0 = 0;                                      // blocks of the items before
    for (int it = item0; it < items; it += item_step) {
      const int slab = it / chunks, blk0 = (it % chunks) * chunk_blocks;
      const int nblk = item_blocks(it, chunks, chunk_blocks, n);
      named_bar_sync(kBarCoef, 256);                  // nobody reads the coefficients of the item before any more
      haar_coef_init(hcoef, f + (size_t)slab * (L + 1), L, ht);
      named_bar_sync(kBarCoef, 256);
      for (int b = 0; b < nblk; ++b)
        ok = haar_step<kNXQ>(smem + SL::x, bars, reinterpret_cast<float*>(smem + SL::xch), hcoef, L > 5, gb0 + b,
                             n - (blk0 + b) * kBlk, ht, ok, abort_flag, status);
      gb0 += nblk;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kWarpMma) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, kTmemCols);
  }
}

// ---- host side: tensor maps ---------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// (slabs x n x 64) bf16 row-major tensor, boxes of `box_rows` rows x 64 columns of one slab, 128-byte
// swizzle.  Rows past the end of a slab read as zeros and are not written.
// Rows of `cols` bf16 values (a multiple of 8: row pitches are multiples of 16 bytes); the box is always 64
// columns wide, so that a narrower tensor arrives zero-filled up to column 63 and is stored clipped.
cudaError_t make_tile_map(const void* base, int slabs, int n, int box_rows, CUtensorMap* out, int cols = kD) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return cudaErrorNotSupported;
  const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)n, (cuuint64_t)slabs};
  const cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)n * cols * 2};
  const cuuint32_t box[3] = {kD, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

}  // namespace

// (the head dimension does not enter: the tensor maps zero-fill narrower heads up to 64 columns, and feature
// maps wider than 256 run as groups of 256)
bool tc_supported(const wersa_config& cfg) {
  return cfg.dtype == WERSA_BF16 &&
         (cfg.features == 128 || cfg.features == 256 ||
          (cfg.features > kGroupFeatures && cfg.features % kGroupFeatures == 0));
}

// Both tensor-core kernels are launched as programmatic dependents of the kernel before them.
template <typename... Args>
static cudaError_t launch_pdl(void (*k)(Args...), dim3 grid, int threads, size_t smem, cudaStream_t st, Args... args) {
  cudaError_t err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k, args...);
}

cudaError_t launch_tc_kside(const Plan& p, const Ws& w, const void* K, const void* V, cudaStream_t st,
                            int* launches) {
  CUtensorMap map_k, map_v;
  cudaError_t err;
  if ((err = make_tile_map(K, p.slabs, p.cfg.seq_len, kTile, &map_k, p.fwd_cols)) != cudaSuccess) return err;
  if ((err = make_tile_map(V, p.slabs, p.cfg.seq_len, kTile, &map_v, p.fwd_cols)) != cudaSuccess) return err;
  CUtensorMap map_w;   // W^T (m x 64) as one slab of m rows
  if ((err = make_tile_map(w.Wt, 1, p.cfg.features, kTile, &map_w)) != cudaSuccess) return err;
  const int items = p.tchunks * p.slabs;   // (slab, chunk) pairs; one CTA per SM walks them
  dim3 grid(items < p.sms ? items : p.sms);
  // With one chunk per slab the "partial" is the result: the kernel writes S', z' and the bf16 image
  // itself and no reduction follows.
  const bool single = p.tchunks == 1;
  float* sp = single ? w.S : w.spart;
  float* zp = single ? w.z : w.zpart;
  __nv_bfloat16* sb = single ? w.Sbf : nullptr;
  uint8_t* si = single ? w.Simg : nullptr;
  const bool multi = items > (int)grid.x;   // some CTA walks more than one item
  // One item per CTA: a (chunks, slabs) grid (item = blockIdx.y * gridDim.x + blockIdx.x either way; other
  // shapes with the same number of CTAs measured the same).
  if (!multi) grid = dim3(p.tchunks, p.slabs);
  auto launch = [&](auto kernel, size_t smem_bytes) {
    return launch_pdl(kernel, grid, kThreads, smem_bytes, st, map_k, map_v, map_w, (const float*)w.f, sp, zp, sb, si,
                      p.cfg.seq_len, p.cfg.levels, p.tchunk_blocks, p.tchunks, items, w.status);
  };
  if (p.cfg.features == 256)
    err = multi ? launch(k_tc_kside<2, true>, KsideSmem<2>::total) : launch(k_tc_kside<2, false>, KsideSmem<2>::total);
  else
    err = multi ? launch(k_tc_kside<1, true>, KsideSmem<1>::total) : launch(k_tc_kside<1, false>, KsideSmem<1>::total);
  *launches += 1;
  return err != cudaSuccess ? err : cudaGetLastError();
}

cudaError_t launch_tc_qside(const Plan& p, const Ws& w, const void* Q, const float* beta, void* O, float* den,
                            cudaStream_t st, int* launches) {
  CUtensorMap map_q, map_o;
  cudaError_t err;
  // (with feature groups O is a 64-wide buffer of the workspace, else the caller's tensor)
  if ((err = make_tile_map(Q, p.slabs, p.cfg.seq_len, kTile, &map_q, p.fwd_cols)) != cudaSuccess) return err;
  if ((err = make_tile_map(O, p.slabs, p.cfg.seq_len, kTile, &map_o, den != nullptr ? kD : p.fwd_cols)) != cudaSuccess)
    return err;
  // (the query side may start while the reduction that produces S', z' is still running; it waits for
  // that kernel where it first needs its results)
  CUtensorMap map_w;
  if ((err = make_tile_map(w.Wt, 1, p.cfg.features, kTile, &map_w)) != cudaSuccess) return err;
  const int items = p.tchunks * p.slabs;
  dim3 grid(items < p.sms ? items : p.sms);
  const bool multi = items > (int)grid.x;
  if (!multi) grid = dim3(p.tchunks, p.slabs);   // see launch_tc_kside
  auto launch = [&](auto kernel, size_t smem_bytes) {
    return launch_pdl(kernel, grid, kThreadsQ, smem_bytes, st, map_q, map_o, map_w, (const uint8_t*)w.Simg,
                      (const float*)w.f, beta, p.cfg.eps, p.cfg.bw_floor, p.cfg.seq_len, p.cfg.levels,
                      p.tchunk_blocks, p.tchunks, items, w.status, den);
  };
  if (den != nullptr) {   // one group of 256 features of a wider feature map
    if (p.cfg.features != 256) return cudaErrorInvalidValue;
    err = multi ? launch(k_tc_qside<2, true, true>, QsideSmem<2>::total)
                : launch(k_tc_qside<2, false, true>, QsideSmem<2>::total);
  } else if (p.cfg.features == 256)
    err = multi ? launch(k_tc_qside<2, true>, QsideSmem<2>::total) : launch(k_tc_qside<2, false>, QsideSmem<2>::total);
  else
    err = multi ? launch(k_tc_qside<1, true>, QsideSmem<1>::total) : launch(k_tc_qside<1, false>, QsideSmem<1>::total);
  *launches += 1;
  return err != cudaSuccess ? err : cudaGetLastError();
}

}  // namespace wersa
