// bf16 tensor-core (tcgen05 + TMEM + TMA) backward kernels of the WERSA attention path, sm_100a.
// The paper does not write the backward pass; these are the chain rule through Eq. 6 / Eq. 7 with
// dReLU(a)/da = 1[a > 0], on the same unscaled quantities the forward kernels use.
//
// Key side, per 128-token tile (token = TMEM lane, one thread per token):
//   MMA1: B_h = K_F (smem, K-major; three bf16 planes hi + mid + lo that add up to the fp32 K_F, so
//         that the mask below does not flip through rounding) * W_h (as W^T, K-major) -> TMEM fp32
//   threads: mask = 1[B_h > 0] (bits in registers), Phi_h = ReLU(B_h) -> bf16 pairs in place
//   MMA2: dV = sum_h Phi_h (TMEM operand) * dS'_h (smem bf16, N-major) -> TMEM fp32 -> smem -> TMA store
//   MMA3: G_h = V (smem, K-major) * dS'_h^T (same image, K-major)      -> TMEM fp32
//   threads: dB_h = (G_h + dz'_h) (.) mask                              -> bf16 pairs in place
//   MMA4: dK_F = sum_h dB_h (TMEM operand) * W_h^T (W^T image, N-major) -> TMEM fp32 -> smem -> TMA store
// Query side, per 128-token tile:
//   MMA1: A_h = Q_F (three planes) * W_h                                -> TMEM fp32 (token = lane)
//   threads: mask, Phi_h -> bf16 in place, D' = sum_h Phi_h . z'_h + eps'
//   MMA2: N' = sum_h Phi_h * S'_h (smem bf16 image, N-major)            -> TMEM fp32
//   threads: O = N'/D', dN' = dO/D' -> bf16 tile in smem, dD' = -sum_c dO O / D' -> smem
//   MMA1t: A_h^T = W_h^T * Q_F^T (hi plane)                             -> TMEM fp32 (feature = lane)
//   threads: Phi_h^T -> bf16 in place, dz'_h += Phi_h^T dD'
//   MMA5: dS'_h += Phi_h^T (TMEM operand) * dN' (smem tile, N-major)    -> TMEM fp32, kept for the chunk
//   MMA3: G_h = dN' (smem, K-major) * S'_h^T (same image, K-major)      -> TMEM fp32 (token = lane)
//   threads: dA_h = (G_h + dD' z'_h) (.) mask                           -> bf16 in place
//   MMA4: dQ_F = sum_h dA_h * W_h^T (W^T image, N-major)                -> TMEM fp32 -> smem -> TMA store
// and at the end of the chunk the partial dS', dz' and sum of dD' go to the split-sequence buffers.
// One CTA of 256 threads per SM walks a chunk of tiles one step at a time (thread 0 issues the copies
// and the MMAs, everybody waits on one mbarrier); the copies of the next tile are in flight meanwhile.
// The two warpgroups see the same 128 TMEM lanes and share every elementwise pass by columns: of the
// 4 NH chunks of 32 accumulator columns, warpgroup g takes chunks 2 NH g .. 2 NH g + 2 NH - 1 (with
// m = 256 that is feature half g), and of a 64-column result it takes columns 32 g .. 32 g + 31.
// TMEM per CTA: 128 columns per feature half; the two 64-column results (dV, dK_F) reuse the upper
// half of the first accumulator.  Every mbarrier wait is bounded; after an expired wait the CTA
// leaves its loop (the decision is taken CTA-wide, so barriers stay balanced) and the host sees the
// status word.
#include "common.cuh"
#include "tc_common.cuh"

namespace wersa {
using namespace tc;

namespace {

constexpr int kTile = 128;
constexpr uint32_t kTileBytes = kTile * kD * 2;   // 128 x 64 bf16
constexpr uint32_t kIdescP = make_idesc_bf16(128, 128, false, false);  // projections: both operands K-major
constexpr uint32_t kIdescC = make_idesc_bf16(128, 64, false, true);    // contractions over features: B N-major
enum { kErrBwdCopy = 21, kErrBwdMma = 22 };

struct alignas(8) BwdBars {
  uint64_t full[2], mma, slo;
  uint32_t tmem_base;
  int abort_flag;
};

template <int NH> struct BwdKSmem {
  static constexpr uint32_t wt = 0;                          // W^T image, NH x (128 x 64) bf16
  static constexpr uint32_t ds = wt + NH * kTileBytes;       // dS' image, same shape
  static constexpr uint32_t stage = ds + NH * kTileBytes;    // 2 stages x (3 K_F planes + V) tiles
  static constexpr uint32_t stage_bytes = 4 * kTileBytes;
  static constexpr uint32_t dz = stage + 2 * stage_bytes;    // NH x 128 floats
  static constexpr uint32_t bars = dz + NH * 512;
  static constexpr uint32_t total = bars + 64 + 1024;        // + alignment slack
};

__device__ __forceinline__ void load_rows_swizzled(uint8_t* dst, const __nv_bfloat16* src, int rows) {
  for (int i = threadIdx.x; i < rows * 8; i += blockDim.x) {
    const int r = i >> 3, c = i & 7;
    const uint4 val = *reinterpret_cast<const uint4*>(src + (size_t)r * kD + c * 8);
    *reinterpret_cast<uint4*>(dst + swz128(r, c)) = val;
  }
}

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

// CTA-wide wait: every thread waits (bounded) on the barrier; the outcome is made uniform.
__device__ __forceinline__ bool cta_wait(uint64_t* bar, uint32_t parity, BwdBars* bars, int* status, int code) {
  const bool ok = mbar_wait(bar, parity, &bars->abort_flag, status, code);
  return __syncthreads_and(ok) != 0;
}

__device__ __forceinline__ void store_row32(float* dst, const uint32_t (&r)[32]) {
#pragma unroll
  for (int j = 0; j < 8; ++j)
    *reinterpret_cast<uint4*>(dst + 4 * j) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
}

// A 128 x 64 result tile leaves through shared memory and a TMA store: written straight from the
// registers (one token row per lane) every store instruction of a warp would touch 32 different
// 128-byte lines, and the load/store unit stays busy with them for about 2,000 cycles per tile, during
// which the barrier polls and MMA issues of the next step queue behind them.
// stage_row32: columns 32 wg .. 32 wg + 31 of row tl into the staging image, in the 128-byte-swizzled
// layout the store's tensor map describes: fp32 = two boxes of 128 rows x 32 columns (16 KB each, box
// wg), bf16 = one box of 128 rows x 64 columns (16-byte chunks 4 wg .. 4 wg + 3 of the row).
template <typename TG>
__device__ __forceinline__ void stage_row32(uint8_t* stage, int tl, int wg, const uint32_t (&r)[32]);
template <> __device__ __forceinline__ void stage_row32<float>(uint8_t* stage, int tl, int wg, const uint32_t (&r)[32]) {
  uint8_t* box = stage + wg * kTileBytes;
#pragma unroll
  for (int j = 0; j < 8; ++j)
    *reinterpret_cast<uint4*>(box + swz128(tl, j)) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
}
template <>
__device__ __forceinline__ void stage_row32<__nv_bfloat16>(uint8_t* stage, int tl, int wg, const uint32_t (&r)[32]) {
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint4 v;
    v.x = pack_bf16x2(__uint_as_float(r[8 * j]), __uint_as_float(r[8 * j + 1]));
    v.y = pack_bf16x2(__uint_as_float(r[8 * j + 2]), __uint_as_float(r[8 * j + 3]));
    v.z = pack_bf16x2(__uint_as_float(r[8 * j + 4]), __uint_as_float(r[8 * j + 5]));
    v.w = pack_bf16x2(__uint_as_float(r[8 * j + 6]), __uint_as_float(r[8 * j + 7]));
    *reinterpret_cast<uint4*>(stage + swz128(tl, 4 * wg + j)) = v;
  }
}
// Issued by one thread after the CTA barrier that follows the staging writes (each writer has fenced its
// writes for the async proxy).  Rows past the end of the slab are clipped by the tensor map.
// kAdd: the tile is added to what the tensor holds (feature groups after the first accumulate their share).
template <typename TG, bool kAdd = false>
__device__ __forceinline__ void store_tile(const CUtensorMap* map, const uint8_t* stage, int row0, int slab) {
  if constexpr (kAdd) {
    tma_reduce_add_3d(map, stage, 0, row0, slab);
    if (sizeof(TG) == 4) tma_reduce_add_3d(map, stage + kTileBytes, 32, row0, slab);
  } else {
    tma_store_3d(map, stage, 0, row0, slab);
    if (sizeof(TG) == 4) tma_store_3d(map, stage + kTileBytes, 32, row0, slab);
  }
  bulk_commit_group();
}

// bf16 hi + lo split of a pair of fp32 values: hi = bf16(x), lo = bf16(x - hi).  Feeding both to the
// tensor core keeps 16 mantissa bits of an operand that would otherwise be rounded to 8.
__device__ __forceinline__ void split_pack(float g0, float g1, uint32_t& p_hi, uint32_t& p_lo) {
  p_hi = pack_bf16x2(g0, g1);
  p_lo = pack_bf16x2(g0 - __uint_as_float(p_hi << 16), g1 - __uint_as_float(p_hi & 0xFFFF0000u));
}

// ReLU pass over this warpgroup's 2 NH chunks of 32 fp32 accumulator columns: chunk (h, c) = columns
// 128 h + 32 c .. + 31 becomes 16 bf16 pairs in columns 128 h + 16 c .. + 15 of the same accumulator.
// `side(ii, h, c, r)` sees the 32 raw values of the warpgroup's ii-th chunk (mask bits, row sums).
// With NH = 2 a warpgroup owns its accumulator and a chunk's pairs land in columns it has already
// read; with NH = 1 the two warpgroups share one accumulator, so all pairs are held back until both
// have read their columns (one CTA barrier).
template <int NH, typename F>
__device__ __forceinline__ void relu_pass(uint32_t trow, int wg, F&& side) {
  uint32_t pp[NH == 1 ? 2 : 1][16];
#pragma unroll
  for (int ii = 0; ii < 2 * NH; ++ii) {
    const int i = wg * 2 * NH + ii, h = i >> 2, c = i & 3;
    uint32_t r[32];
    tmem_ld32(trow + h * 128 + 32 * c, r);
    tmem_ld_wait();
    reg_fence32(r);
    side(ii, h, c, r);
    uint32_t(&p)[16] = pp[NH == 1 ? ii : 0];
#pragma unroll
    for (int j = 0; j < 16; ++j) p[j] = relu_pack_bf16x2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
    if (NH != 1) tmem_st16(trow + h * 128 + 16 * c, p);
  }
  if (NH == 1) {
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
#pragma unroll
    for (int ii = 0; ii < 2; ++ii) tmem_st16(trow + 16 * (wg * 2 + ii), pp[ii]);
  }
  tmem_st_wait();
}

// Gradient through the ReLU for this warpgroup's 2 NH chunks of 32 accumulator columns (token = lane):
// x_j = (G_j + s * zr_j) where mask bit j is set, else 0; written back as bf16 hi pairs in columns
// [0, 64) and lo pairs in columns [64, 128) of the same accumulator.  All columns are read before the
// first one is overwritten; with NH = 1 the two warpgroups share one accumulator, so a CTA barrier
// separates the reads from the writes.  `zr` points at the m values z'_f (or dz'_f).
template <int NH>
__device__ __forceinline__ void relu_grad_split(uint32_t trow, int wg, const uint32_t (&mask)[2 * NH], float s,
                                                const float* __restrict__ zr) {
  uint32_t r[2 * NH][32];
#pragma unroll
  for (int ii = 0; ii < 2 * NH; ++ii) {
    const int i = wg * 2 * NH + ii;
    tmem_ld32(trow + (i >> 2) * 128 + 32 * (i & 3), r[ii]);
  }
  tmem_ld_wait();
#pragma unroll
  for (int ii = 0; ii < 2 * NH; ++ii) reg_fence32(r[ii]);
  if (NH == 1) {
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
  }
#pragma unroll
  for (int ii = 0; ii < 2 * NH; ++ii) {
    const int i = wg * 2 * NH + ii, h = i >> 2, c = i & 3;
    uint32_t ph[16], pl[16];
    const uint32_t bits = mask[ii];
    const float* z = zr + h * 128 + 32 * c;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const float g0 = ((bits >> (2 * j)) & 1u) ? fmaf(s, z[2 * j], __uint_as_float(r[ii][2 * j])) : 0.f;
      const float g1 = ((bits >> (2 * j + 1)) & 1u) ? fmaf(s, z[2 * j + 1], __uint_as_float(r[ii][2 * j + 1])) : 0.f;
      split_pack(g0, g1, ph[j], pl[j]);
    }
    tmem_st16(trow + h * 128 + 16 * c, ph);
    tmem_st16(trow + h * 128 + 64 + 16 * c, pl);
  }
  tmem_st_wait();
}

// ---- key side -----------------------------------------------------------------------------------
// grid (chunks, slabs), block 256.
template <int NH, typename TG, bool kAdd = false>
__global__ void __launch_bounds__(256, 1)
k_tc_bwd_kside(const __grid_constant__ CUtensorMap map_kf, const __grid_constant__ CUtensorMap map_v,
               const __nv_bfloat16* __restrict__ Wt, const __nv_bfloat16* __restrict__ dSbf,
               const float* __restrict__ dzg, const __grid_constant__ CUtensorMap map_dv,
               const __grid_constant__ CUtensorMap map_dkf, int n, int slabs, int* __restrict__ status) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  using SL = BwdKSmem<NH>;
  BwdBars* bars = reinterpret_cast<BwdBars*>(smem + SL::bars);
  float* dzs = reinterpret_cast<float*>(smem + SL::dz);
  const int warp = threadIdx.x >> 5;
  // The tiles of all slabs form one list (slab-major) that the CTAs share evenly: a tile of this side
  // depends on no other tile, only on the dS' image and dz' of its slab, which are reloaded when the
  // CTA's range crosses into the next slab.
  const int tiles_per_slab = (n + kTile - 1) / kTile;
  const long long tiles_all = (long long)tiles_per_slab * slabs;
  const int g0 = (int)(tiles_all * blockIdx.x / gridDim.x);
  const int ntiles = (int)(tiles_all * (blockIdx.x + 1) / gridDim.x) - g0;
  int cur_slab = g0 / tiles_per_slab;
  constexpr int m = NH * 128;
  constexpr uint32_t kCols = NH * 256;            // TMEM columns: NH accumulators of 128, then dV / dK_F (64)

  if (threadIdx.x == 0) {
    mbar_init(&bars->full[0], 1);
    mbar_init(&bars->full[1], 1);
    mbar_init(&bars->mma, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&bars->tmem_base, kCols);
    tmem_relinquish();
  }
  load_rows_swizzled(smem + SL::wt, Wt, m);
  load_rows_swizzled(smem + SL::ds, dSbf + (size_t)cur_slab * m * kD, m);
  for (int i = threadIdx.x; i < m; i += blockDim.x) dzs[i] = dzg[(size_t)cur_slab * m + i];
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bars->tmem_base;
  const int wg = warp >> 2, tl = threadIdx.x & 127;      // warpgroup; token of this thread = TMEM lane
  const uint32_t trow = tmem + ((32u * (warp & 3)) << 16);   // this warp's lane quarter
  const uint32_t acc = NH * 128;                         // dV / dK_F

  const uint32_t hi = smem_desc_hi(1024);
  const uint32_t wt_k = smem_desc_lo(smem_u32(smem + SL::wt), 16), wt_n = smem_desc_lo(smem_u32(smem + SL::wt), 1024);
  const uint32_t ds_k = smem_desc_lo(smem_u32(smem + SL::ds), 16), ds_n = smem_desc_lo(smem_u32(smem + SL::ds), 1024);
  const uint32_t stage_k = smem_desc_lo(smem_u32(smem + SL::stage), 16);
  constexpr uint32_t kTileStep = kTileBytes >> 4, kStageStep = SL::stage_bytes >> 4;
  uint32_t mma_par = 0;
  int issued = 0;
  bool ok = true;

  // copies of tile t into stage t & 1: the three K_F planes (plane p of slab s is slab p * slabs + s of
  // the stacked tensor) and V
  auto issue_copies = [&](int t) {
    uint8_t* dst = smem + SL::stage + (t & 1) * SL::stage_bytes;
    uint64_t* bar = &bars->full[t & 1];
    const int slab = (g0 + t) / tiles_per_slab;
    const int r0 = ((g0 + t) - slab * tiles_per_slab) * kTile;
    mbar_arrive_expect_tx(bar, 4 * kTileBytes);
#pragma unroll
    for (int pl = 0; pl < 3; ++pl) tma_load_3d(dst + pl * kTileBytes, &map_kf, 0, r0, pl * slabs + slab, bar);
    tma_load_3d(dst + 3 * kTileBytes, &map_v, 0, r0, slab, bar);
  };
  if (threadIdx.x == 0 && ntiles > 0) {
    issue_copies(0);
    issued = 1;
  }

  for (int ti = 0; ti < ntiles && ok; ++ti) {
    const int slab = (g0 + ti) / tiles_per_slab;
    const int row0 = ((g0 + ti) - slab * tiles_per_slab) * kTile;
    const uint32_t x_k = stage_k + (ti & 1) * kStageStep, v_k = x_k + 3 * kTileStep;
    // results leave through this tile's own stage: dV over planes 0-1 (read for the last time by MMA1),
    // dK_F over plane 2 and the V tile (read for the last time by MMA3)
    uint8_t* out_stage = smem + SL::stage + (ti & 1) * SL::stage_bytes;
    if (slab != cur_slab) {   // uniform over the CTA; every MMA of the previous tile has completed
      cur_slab = slab;
      load_rows_swizzled(smem + SL::ds, dSbf + (size_t)slab * m * kD, m);
      for (int i = threadIdx.x; i < m; i += blockDim.x) dzs[i] = dzg[(size_t)slab * m + i];
      fence_proxy_async_smem();
      __syncthreads();
    }
    // ---- MMA1, then the copies of the next tile: its stage is the one tile ti - 1 left its results in,
    // so the stores of that tile must have read it first
    ok = cta_wait(&bars->full[ti & 1], (ti >> 1) & 1, bars, status, kErrBwdCopy);
    if (!ok) break;
    if (threadIdx.x == 0) {
      tc_fence_after_sync();
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int pl = 0; pl < 3; ++pl)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_ss(tmem + h * 128, smem_desc_join(x_k + pl * kTileStep + 2 * k, hi),
                   smem_desc_join(wt_k + h * kTileStep + 2 * k, hi), kIdescP, (pl > 0 || k > 0) ? 1u : 0u);
      mma_commit(&bars->mma);
      if (ti + 1 < ntiles) {
        bulk_wait_group_read0();
        issue_copies(ti + 1);
        issued = ti + 2;
      }
    }
    ok = cta_wait(&bars->mma, mma_par, bars, status, kErrBwdMma);
    mma_par ^= 1;
    if (!ok) break;
    tc_fence_after_sync();
    // ---- mask and Phi
    uint32_t mask[2 * NH];
    relu_pass<NH>(trow, wg, [&](int ii, int, int, const uint32_t(&r)[32]) {
      uint32_t bits = 0;
#pragma unroll
      for (int j = 0; j < 32; ++j) bits |= (__uint_as_float(r[j]) > 0.f ? 1u : 0u) << j;
      mask[ii] = bits;
    });
    tc_fence_before_sync();
    __syncthreads();
    // ---- MMA2: dV
    if (threadIdx.x == 0) {
      tc_fence_after_sync();
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int k = 0; k < 8; ++k)
          mma_ts(tmem + acc, tmem + h * 128 + k * 8, smem_desc_join(ds_n + h * kTileStep + 128 * k, hi), kIdescC,
                 (h > 0 || k > 0) ? 1u : 0u);
      mma_commit(&bars->mma);
    }
    ok = cta_wait(&bars->mma, mma_par, bars, status, kErrBwdMma);
    mma_par ^= 1;
    if (!ok) break;
    tc_fence_after_sync();
    {
      uint32_t r[32];
      tmem_ld32(trow + acc + 32 * wg, r);
      tmem_ld_wait();
      reg_fence32(r);
      stage_row32<TG>(out_stage, tl, wg, r);
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    // ---- MMA3: G_h = V dS'_h^T
    if (threadIdx.x == 0) {
      store_tile<TG, kAdd>(&map_dv, out_stage, row0, slab);
      tc_fence_after_sync();
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int k = 0; k < 4; ++k)
          mma_ss(tmem + h * 128, smem_desc_join(v_k + 2 * k, hi), smem_desc_join(ds_k + h * kTileStep + 2 * k, hi),
                 kIdescP, k > 0);
      mma_commit(&bars->mma);
    }
    ok = cta_wait(&bars->mma, mma_par, bars, status, kErrBwdMma);
    mma_par ^= 1;
    if (!ok) break;
    tc_fence_after_sync();
    // ---- dB_h = (G_h + dz'_h) (.) mask, as bf16 hi + lo
    relu_grad_split<NH>(trow, wg, mask, 1.f, dzs);
    tc_fence_before_sync();
    __syncthreads();
    // ---- MMA4: dK_F
    if (threadIdx.x == 0) {
      tc_fence_after_sync();
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int k = 0; k < 8; ++k)
#pragma unroll
          for (int part = 0; part < 2; ++part)   // hi pairs at columns 0..63, lo pairs at 64..127
            mma_ts(tmem + acc, tmem + h * 128 + 64 * part + k * 8, smem_desc_join(wt_n + h * kTileStep + 128 * k, hi),
                   kIdescC, (h > 0 || k > 0 || part > 0) ? 1u : 0u);
      mma_commit(&bars->mma);
    }
    ok = cta_wait(&bars->mma, mma_par, bars, status, kErrBwdMma);
    mma_par ^= 1;
    if (!ok) break;
    tc_fence_after_sync();
    {
      uint32_t r[32];
      tmem_ld32(trow + acc + 32 * wg, r);
      tmem_ld_wait();
      reg_fence32(r);
      stage_row32<float>(out_stage + 2 * kTileBytes, tl, wg, r);
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();   // the next tile's MMA1 overwrites what this tile read
    if (threadIdx.x == 0) store_tile<float, kAdd>(&map_dkf, out_stage + 2 * kTileBytes, row0, slab);
  }
  if (threadIdx.x == 0) {
    if (!ok)   // copies may still be in flight
      for (int t = max(0, issued - 2); t < issued; ++t) mbar_wait_drain(&bars->full[t & 1], (t >> 1) & 1);
    bulk_wait_group0();   // the result stores read this CTA's shared memory
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, kCols);
  }
}

// ---- query side ---------------------------------------------------------------------------------
template <int NH> struct BwdQSmem {
  static constexpr uint32_t wt = 0;                          // W^T image
  static constexpr uint32_t simg = wt + NH * kTileBytes;     // S' image
  static constexpr uint32_t stage = simg + NH * kTileBytes;  // 2 stages x (3 Q_F planes + dO) tiles
  static constexpr uint32_t stage_bytes = 4 * kTileBytes;
  static constexpr uint32_t dn = stage + 2 * stage_bytes;    // dN' tiles, bf16 hi and lo
  static constexpr uint32_t zs = dn + 2 * kTileBytes;        // NH x 128 floats
  static constexpr uint32_t dd = zs + NH * 512;              // 128 floats
  static constexpr uint32_t red = dd + 512;                  // 4 floats
  static constexpr uint32_t bars = red + 64;
  static constexpr uint32_t total = bars + 64 + 1024;
};

// grid (chunks, slabs), block 256.  TMEM: accumulator h at columns 128 h (A_h, A_h^T, G_h in turn; the
// 64-column results N' and dQ_F sit at 384), dS'_h at 256 + 64 h.  Row quantities that both
// warpgroups contribute to (D', dD', and with m = 128 dz') meet in the 128-float array `dds`:
// warpgroup 1 leaves its part there, warpgroup 0 adds its own (always in this order) and leaves the
// total there for everybody, with the CTA barriers of the step sequence in between.
// kGroup: the launch handles one group of 256 features of a wider feature map.  The denominator of Eq. 7 and
// dD' then belong to the whole map and come from den_ext / dd_ext (one float per token), and with kAdd the
// group's share of dQ_F is added to what the groups before it left.
template <int NH, bool kGroup = false, bool kAdd = false>
__global__ void __launch_bounds__(256, 1)
k_tc_bwd_qside(const __grid_constant__ CUtensorMap map_qf, const __grid_constant__ CUtensorMap map_do,
               const __grid_constant__ CUtensorMap map_slo, const __nv_bfloat16* __restrict__ Wt,
               const __nv_bfloat16* __restrict__ Sbf,
               const float* __restrict__ zg, const float* __restrict__ beta, float eps, float bw_floor,
               const __grid_constant__ CUtensorMap map_dqf, float* __restrict__ dspart,
               float* __restrict__ dzpart, float* __restrict__ sumdD, int n, int chunk_tiles,
               int* __restrict__ status, const float* __restrict__ den_ext, const float* __restrict__ dd_ext) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  using SL = BwdQSmem<NH>;
  BwdBars* bars = reinterpret_cast<BwdBars*>(smem + SL::bars);
  float* zs = reinterpret_cast<float*>(smem + SL::zs);
  float* dds = reinterpret_cast<float*>(smem + SL::dd);
  float* red = reinterpret_cast<float*>(smem + SL::red);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x, slab = blockIdx.y;
  const int tiles_total = (n + kTile - 1) / kTile;
  const int tile0 = chunk * chunk_tiles;
  const int ntiles = min(chunk_tiles, tiles_total - tile0);
  constexpr int m = NH * 128;
  constexpr uint32_t kCols = 512;
  constexpr uint32_t kAccS = 256;                 // dS'_h accumulators

  if (threadIdx.x == 0) {
    mbar_init(&bars->full[0], 1);
    mbar_init(&bars->full[1], 1);
    mbar_init(&bars->mma, 1);
    mbar_init(&bars->slo, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&bars->tmem_base, kCols);
    tmem_relinquish();
  }
  load_rows_swizzled(smem + SL::wt, Wt, m);
  load_rows_swizzled(smem + SL::simg, Sbf + (size_t)slab * m * kD, m);
  for (int i = threadIdx.x; i < m; i += blockDim.x) zs[i] = zg[(size_t)slab * m + i];
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bars->tmem_base;
  const int wg = warp >> 2, tl = threadIdx.x & 127;      // warpgroup; token / feature of this thread = TMEM lane
  const uint32_t trow = tmem + ((32u * (warp & 3)) << 16);
  const uint32_t acc = 384;
  const float bw = fmaxf(beta[0], bw_floor);
  const float epsp = eps * (float)m * bw * bw;

  const uint32_t hi = smem_desc_hi(1024);
  const uint32_t wt_k = smem_desc_lo(smem_u32(smem + SL::wt), 16), wt_n = smem_desc_lo(smem_u32(smem + SL::wt), 1024);
  const uint32_t s_k = smem_desc_lo(smem_u32(smem + SL::simg), 16), s_n = smem_desc_lo(smem_u32(smem + SL::simg), 1024);
  const uint32_t dn_k = smem_desc_lo(smem_u32(smem + SL::dn), 16), dn_n = smem_desc_lo(smem_u32(smem + SL::dn), 1024);
  const uint32_t stage_k = smem_desc_lo(smem_u32(smem + SL::stage), 16);
  constexpr uint32_t kTileStep = kTileBytes >> 4, kStageStep = SL::stage_bytes >> 4;
  const int slabs = gridDim.y;
  uint32_t mma_par = 0;
  int issued = 0, slo_issued = 0;
  bool ok = true;
  float dzacc[NH];                                // feature = thread: dz'_h partial of this chunk
#pragma unroll
  for (int h = 0; h < NH; ++h) dzacc[h] = 0.f;
  float sum_dd = 0.f;                             // token = thread: sum of dD' over this thread's tokens

  auto issue_copies = [&](int t) {
    uint8_t* dst = smem + SL::stage + (t & 1) * SL::stage_bytes;
    uint64_t* bar = &bars->full[t & 1];
    const int r0 = (tile0 + t) * kTile;
    mbar_arrive_expect_tx(bar, 4 * kTileBytes);
#pragma unroll
    for (int pl = 0; pl < 3; ++pl) tma_load_3d(dst + pl * kTileBytes, &map_qf, 0, r0, pl * slabs + slab, bar);
    tma_load_3d(dst + 3 * kTileBytes, &map_do, 0, r0, slab, bar);
  };
  auto wait_mma = [&]() {
    const bool r = cta_wait(&bars->mma, mma_par, bars, status, kErrBwdMma);
    mma_par ^= 1;
    if (r) tc_fence_after_sync();
    return r;
  };
  if (threadIdx.x == 0 && ntiles > 0) {
    issue_copies(0);
    issued = 1;
  }

  for (int ti = 0; ti < ntiles && ok; ++ti) {
    const int row0 = (tile0 + ti) * kTile;
    const int row = row0 + tl;
    const uint32_t x_k = stage_k + (ti & 1) * kStageStep;
    const uint8_t* do_tile = smem + SL::stage + (ti & 1) * SL::stage_bytes + 3 * kTileBytes;
    if (threadIdx.x == 0 && ti + 1 < ntiles) {
      issue_copies(ti + 1);
      issued = ti + 2;
    }
    ok = cta_wait(&bars->full[ti & 1], (ti >> 1) & 1, bars, status, kErrBwdCopy);
    if (!ok) break;
    // ---- MMA1: A_h (three planes)
    if (threadIdx.x == 0) {
      tc_fence_after_sync();
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int pl = 0; pl < 3; ++pl)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_ss(tmem + h * 128, smem_desc_join(x_k + pl * kTileStep + 2 * k, hi),
                   smem_desc_join(wt_k + h * kTileStep + 2 * k, hi), kIdescP, (pl > 0 || k > 0) ? 1u : 0u);
      mma_commit(&bars->mma);
    }
    if (!(ok = wait_mma())) break;
    // The mid and lo planes of this tile's stage are dead from here on (MMA1 has read them; the transposed
    // projection below takes the hi plane only): the low-order image of S' of this slab, bf16(S' - bf16(S')),
    // is fetched into their place for MMA3.  (Shared memory has no room to hold it for the whole chunk.)
    if (threadIdx.x == 0) {
      uint8_t* dst = smem + SL::stage + (ti & 1) * SL::stage_bytes + kTileBytes;
      mbar_arrive_expect_tx(&bars->slo, NH * kTileBytes);
#pragma unroll
      for (int h = 0; h < NH; ++h) tma_load_3d(dst + h * kTileBytes, &map_slo, 0, h * kTile, slab, &bars->slo);
      slo_issued = ti + 1;
    }
    // ---- mask, Phi, denominator
    uint32_t mask[2 * NH];
    float den = 0.f;
    relu_pass<NH>(trow, wg, [&](int ii, int h, int c, const uint32_t(&r)[32]) {
      uint32_t bits = 0;
      const float* zr = zs + h * 128 + 32 * c;
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const float a = __uint_as_float(r[j]);
        bits |= (a > 0.f ? 1u : 0u) << j;
        den = fmaf(fmaxf(a, 0.f), zr[j], den);
      }
      mask[ii] = bits;
    });
    if (wg == 1) dds[tl] = den;
    tc_fence_before_sync();
    __syncthreads();
    if (wg == 0) {
      if constexpr (kGroup) den = row < n ? den_ext[(size_t)slab * n + row] : 1.f;
      else den = epsp + (den + dds[tl]);
      dds[tl] = den;
    }
    // ---- MMA2: N'
    if (threadIdx.x == 0) {
      bulk_wait_group_read0();   // dQ_F of the previous tile has left the dN' tiles, which are written next
      tc_fence_after_sync();
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int k = 0; k < 8; ++k)
          mma_ts(tmem + acc, tmem + h * 128 + k * 8, smem_desc_join(s_n + h * kTileStep + 128 * k, hi), kIdescC,
                 (h > 0 || k > 0) ? 1u : 0u);
      mma_commit(&bars->mma);
    }
    if (!(ok = wait_mma())) break;
    // ---- O, dN' (-> smem tile, bf16), dD': warpgroup g takes columns 32 g .. 32 g + 31
    if (wg == 1) den = dds[tl];                    // the total left by warpgroup 0 before the last barrier
    const float inv = row < n ? 1.f / den : 0.f;   // rows past the end contribute nothing
    float dd = 0.f;
    {
      uint8_t* dn_tile = smem + SL::dn;
      uint32_t r[32];
      tmem_ld32(trow + acc + 32 * wg, r);
      tmem_ld_wait();
      reg_fence32(r);
#pragma unroll
      for (int q = 0; q < 4; ++q) {   // 16-byte chunk 4 g + q of this token's row: 8 columns
        const uint4 raw = *reinterpret_cast<const uint4*>(do_tile + swz128(tl, 4 * wg + q));
        const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
        uint32_t oh[4], ol[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float g0 = __uint_as_float(u[i] << 16), g1 = __uint_as_float(u[i] & 0xFFFF0000u);
          const float o0 = __uint_as_float(r[8 * q + 2 * i]) * inv, o1 = __uint_as_float(r[8 * q + 2 * i + 1]) * inv;
          dd = fmaf(g0, o0, dd);
          dd = fmaf(g1, o1, dd);
          split_pack(g0 * inv, g1 * inv, oh[i], ol[i]);
        }
        *reinterpret_cast<uint4*>(dn_tile + swz128(tl, 4 * wg + q)) = make_uint4(oh[0], oh[1], oh[2], oh[3]);
        *reinterpret_cast<uint4*>(dn_tile + kTileBytes + swz128(tl, 4 * wg + q)) =
            make_uint4(ol[0], ol[1], ol[2], ol[3]);
      }
    }
    if (wg == 1) dds[tl] = dd;                     // (the same thread has read D' from this slot above)
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (wg == 0) {
      if constexpr (kGroup) dd = row < n ? dd_ext[(size_t)slab * n + row] : 0.f;
      else dd = -(dd + dds[tl]) * inv;
      dds[tl] = dd;
      sum_dd += dd;
    }
    // ---- MMA1t: A_h^T (feature = lane), hi plane only
    if (threadIdx.x == 0) {
      tc_fence_after_sync();
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int k = 0; k < 4; ++k)
          mma_ss(tmem + h * 128, smem_desc_join(wt_k + h * kTileStep + 2 * k, hi), smem_desc_join(x_k + 2 * k, hi),
                 kIdescP, k > 0);
      mma_commit(&bars->mma);
    }
    if (!(ok = wait_mma())) break;
    // ---- Phi^T, dz' partial (the barrier that ended the MMA wait also published dD')
    if (wg == 1) dd = dds[tl];
    relu_pass<NH>(trow, wg, [&](int, int h, int c, const uint32_t(&r)[32]) {
      const float* ddr = dds + 32 * c;
      float part = 0.f;
#pragma unroll
      for (int j = 0; j < 32; ++j) part = fmaf(fmaxf(__uint_as_float(r[j]), 0.f), ddr[j], part);
      dzacc[h] += part;
    });
    tc_fence_before_sync();
    __syncthreads();
    // ---- MMA5: dS'_h += Phi_h^T dN'   and   MMA3: G_h = dN' S'_h^T (after MMA5 has read Phi_h^T)
    if (threadIdx.x == 0) {
      tc_fence_after_sync();
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int k = 0; k < 8; ++k)
#pragma unroll
          for (int part = 0; part < 2; ++part)   // dN' hi tile, then lo tile
            mma_ts(tmem + kAccS + h * 64, tmem + h * 128 + k * 8, smem_desc_join(dn_n + part * kTileStep + 128 * k, hi),
                   kIdescC, (ti > 0 || k > 0 || part > 0) ? 1u : 0u);
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int part = 0; part < 2; ++part)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_ss(tmem + h * 128, smem_desc_join(dn_k + part * kTileStep + 2 * k, hi),
                   smem_desc_join(s_k + h * kTileStep + 2 * k, hi), kIdescP, (part > 0 || k > 0) ? 1u : 0u);
      // + dN'(hi) S'(lo)^T: the single bf16 rounding of S' was the largest error of dQ_F
      if (mbar_wait(&bars->slo, ti & 1, &bars->abort_flag, status, kErrBwdCopy)) {
        const uint32_t slo_k = x_k + kTileStep;
#pragma unroll
        for (int h = 0; h < NH; ++h)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_ss(tmem + h * 128, smem_desc_join(dn_k + 2 * k, hi), smem_desc_join(slo_k + h * kTileStep + 2 * k, hi),
                   kIdescP, 1u);
      }
      mma_commit(&bars->mma);
    }
    if (!(ok = wait_mma())) break;
    // ---- dA_h = (G_h + dD' z'_h) (.) mask, as bf16 hi + lo
    relu_grad_split<NH>(trow, wg, mask, dd, zs);
    tc_fence_before_sync();
    __syncthreads();
    // ---- MMA4: dQ_F
    if (threadIdx.x == 0) {
      tc_fence_after_sync();
#pragma unroll
      for (int h = 0; h < NH; ++h)
#pragma unroll
        for (int k = 0; k < 8; ++k)
#pragma unroll
          for (int part = 0; part < 2; ++part)
            mma_ts(tmem + acc, tmem + h * 128 + 64 * part + k * 8, smem_desc_join(wt_n + h * kTileStep + 128 * k, hi),
                   kIdescC, (h > 0 || k > 0 || part > 0) ? 1u : 0u);
      mma_commit(&bars->mma);
    }
    if (!(ok = wait_mma())) break;
    {
      uint32_t r[32];
      tmem_ld32(trow + acc + 32 * wg, r);
      tmem_ld_wait();
      reg_fence32(r);
      stage_row32<float>(smem + SL::dn, tl, wg, r);   // the dN' tiles are free: MMA5 and MMA3 have completed
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) store_tile<float, kAdd>(&map_dqf, smem + SL::dn, row0, slab);
  }
  // ---- partial dS', dz', sum dD' of this chunk (zeros if the chunk gave up)
  const size_t pidx = (size_t)slab * gridDim.x + chunk;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum_dd += __shfl_xor_sync(0xffffffffu, sum_dd, o);
  if (lane == 0 && wg == 0) red[warp] = sum_dd;
  if (NH == 1 && wg == 1) dds[tl] = dzacc[0];      // with one feature half both warpgroups hold a part of dz'
  __syncthreads();
  if (threadIdx.x == 0) sumdD[pidx] = ok ? (red[0] + red[1]) + (red[2] + red[3]) : 0.f;
  if (ok && ntiles > 0) {
    tc_fence_after_sync();
    // dS': of the 2 NH chunks of 32 columns (half h, columns 32 c ..), warpgroup g takes NH g .. NH g + NH - 1
#pragma unroll
    for (int ii = 0; ii < NH; ++ii) {
      const int i = wg * NH + ii, h = i >> 1, c = i & 1;
      uint32_t r[32];
      tmem_ld32(trow + kAccS + h * 64 + 32 * c, r);
      tmem_ld_wait();
      reg_fence32(r);
      store_row32(dspart + (pidx * m + h * 128 + tl) * kD + 32 * c, r);
    }
    if (NH == 1) {
      if (wg == 0) dzpart[pidx * m + tl] = dzacc[0] + dds[tl];
    } else {
      dzpart[pidx * m + wg * 128 + tl] = dzacc[NH - 1 < wg ? 0 : wg];
    }
  }
  if (threadIdx.x == 0) {
    if (!ok) {
      for (int t = max(0, issued - 2); t < issued; ++t) mbar_wait_drain(&bars->full[t & 1], (t >> 1) & 1);
      if (slo_issued > 0) mbar_wait_drain(&bars->slo, (slo_issued - 1) & 1);
    }
    bulk_wait_group0();   // the dQ_F stores read this CTA's shared memory
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, kCols);
  }
}

// lo = bf16(x - hi) for hi = bf16(x) as the forward left it: the second half of a hi + lo pair for S'.
__global__ void __launch_bounds__(256) k_split_lo(const float* __restrict__ x, const __nv_bfloat16* __restrict__ hi_img,
                                                   __nv_bfloat16* __restrict__ lo_img, size_t count) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (i < count) lo_img[i] = __float2bfloat16_rn(x[i] - __bfloat162float(hi_img[i]));
}

// ---- host side ----------------------------------------------------------------------------------
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

// (slabs x n x 64) bf16 tensor, boxes of 128 rows x 64 columns of one slab, 128-byte swizzle; rows past
// the end of a slab read as zeros.
cudaError_t make_tile_map(const void* base, int slabs, int n, CUtensorMap* out) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return cudaErrorNotSupported;
  const cuuint64_t dims[3] = {kD, (cuuint64_t)n, (cuuint64_t)slabs};
  const cuuint64_t strides[2] = {kD * 2, (cuuint64_t)n * kD * 2};
  const cuuint32_t box[3] = {kD, kTile, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// Store map of a (slabs x n x 64) result tensor: fp32 in boxes of 128 rows x 32 columns (128 bytes, the
// widest a 128-byte swizzle takes), bf16 in boxes of 128 rows x 64 columns; rows past n are not written.
cudaError_t make_out_map(void* base, int slabs, int n, bool bf16, CUtensorMap* out) {
  if (bf16) return make_tile_map(base, slabs, n, out);
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return cudaErrorNotSupported;
  const cuuint64_t dims[3] = {kD, (cuuint64_t)n, (cuuint64_t)slabs};
  const cuuint64_t strides[2] = {kD * 4, (cuuint64_t)n * kD * 4};
  const cuuint32_t box[3] = {32, kTile, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int NH, typename TG, bool kAdd = false>
cudaError_t launch_kside(const Plan& p, const Ws& w, const CUtensorMap& map_kf, const CUtensorMap& map_v, void* dV,
                         cudaStream_t st) {
  CUtensorMap map_dv, map_dkf;
  cudaError_t merr;
  if ((merr = make_out_map(dV, p.slabs, p.cfg.seq_len, sizeof(TG) == 2, &map_dv)) != cudaSuccess) return merr;
  if ((merr = make_out_map(w.dKF, p.slabs, p.cfg.seq_len, false, &map_dkf)) != cudaSuccess) return merr;
  auto k = k_tc_bwd_kside<NH, TG, kAdd>;
  cudaError_t err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdKSmem<NH>::total);
  if (err != cudaSuccess) return err;
  const long long tiles_all = (long long)((p.cfg.seq_len + kTile - 1) / kTile) * p.slabs;
  const unsigned grid = (unsigned)(tiles_all < p.sms ? tiles_all : p.sms);   // one CTA per SM, one wave
  launch_after(k, dim3(grid), dim3(256), BwdKSmem<NH>::total, st, map_kf, map_v, w.Wt, w.dSbf, w.dz, map_dv, map_dkf, p.cfg.seq_len, p.slabs,
                                            w.status);
  return cudaGetLastError();
}

template <int NH, bool kGroup = false, bool kAdd = false>
cudaError_t launch_qside(const Plan& p, const Ws& w, const CUtensorMap& map_qf, const CUtensorMap& map_do,
                         const float* beta, cudaStream_t st, const float* den_ext = nullptr,
                         const float* dd_ext = nullptr) {
  // low-order bf16 image of S' (rows = features of a slab), fetched tile by tile by the kernel
  const size_t count = (size_t)p.slabs * p.cfg.features * kD;
  launch_after(k_split_lo, dim3((unsigned)((count + 255) / 256)), dim3(256), 0, st, w.S, w.Sbf, w.Slo, count);
  CUtensorMap map_slo;
  cudaError_t merr;
  if ((merr = make_tile_map(w.Slo, p.slabs, p.cfg.features, &map_slo)) != cudaSuccess) return merr;
  auto k = k_tc_bwd_qside<NH, kGroup, kAdd>;
  cudaError_t err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdQSmem<NH>::total);
  if (err != cudaSuccess) return err;
  CUtensorMap map_dqf;
  if ((err = make_out_map(w.dQF, p.slabs, p.cfg.seq_len, false, &map_dqf)) != cudaSuccess) return err;
  dim3 grid(p.bchunks, p.slabs);
  launch_after(k, dim3(grid), dim3(256), BwdQSmem<NH>::total, st, map_qf, map_do, map_slo, w.Wt, w.Sbf, w.z, beta, p.cfg.eps, p.cfg.bw_floor, map_dqf,
                                            w.spart, w.zpart, w.sumdD, p.cfg.seq_len, p.bchunk_tiles, w.status, den_ext,
                                            dd_ext);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_tc_bwd_qside(const Plan& p, const Ws& w, const void* QF3, const float* beta, const void* dO,
                                const float* den_ext, const float* dd_ext, bool add, cudaStream_t st, int* launches) {
  CUtensorMap map_qf, map_do;
  cudaError_t err;
  if ((err = make_tile_map(QF3, 3 * p.slabs, p.cfg.seq_len, &map_qf)) != cudaSuccess) return err;
  if ((err = make_tile_map(dO, p.slabs, p.cfg.seq_len, &map_do)) != cudaSuccess) return err;
  *launches += 2;   // the low-order image of S', then the kernel
  if (den_ext != nullptr) {   // one group of 256 features of a wider map
    if (p.cfg.features != 256 || dd_ext == nullptr) return cudaErrorInvalidValue;
    return add ? launch_qside<2, true, true>(p, w, map_qf, map_do, beta, st, den_ext, dd_ext)
               : launch_qside<2, true, false>(p, w, map_qf, map_do, beta, st, den_ext, dd_ext);
  }
  return p.cfg.features == 256 ? launch_qside<2>(p, w, map_qf, map_do, beta, st)
                               : launch_qside<1>(p, w, map_qf, map_do, beta, st);
}

cudaError_t launch_tc_bwd_kside(const Plan& p, const Ws& w, const void* KF3, const void* V, void* dV, bool add,
                                cudaStream_t st, int* launches) {
  CUtensorMap map_kf, map_v;
  cudaError_t err;
  if ((err = make_tile_map(KF3, 3 * p.slabs, p.cfg.seq_len, &map_kf)) != cudaSuccess) return err;
  if ((err = make_tile_map(V, p.slabs, p.cfg.seq_len, &map_v)) != cudaSuccess) return err;
  *launches += 1;
  if (add) {   // a feature group after the first: dV and dK_F accumulate
    if (p.cfg.features != 256) return cudaErrorInvalidValue;
    return p.grad_bf16 ? launch_kside<2, __nv_bfloat16, true>(p, w, map_kf, map_v, dV, st)
                       : launch_kside<2, float, true>(p, w, map_kf, map_v, dV, st);
  }
  if (p.cfg.features == 256)
    return p.grad_bf16 ? launch_kside<2, __nv_bfloat16>(p, w, map_kf, map_v, dV, st)
                       : launch_kside<2, float>(p, w, map_kf, map_v, dV, st);
  return p.grad_bf16 ? launch_kside<1, __nv_bfloat16>(p, w, map_kf, map_v, dV, st)
                     : launch_kside<1, float>(p, w, map_kf, map_v, dV, st);
}

}  // namespace wersa
