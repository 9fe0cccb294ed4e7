// bf16 tensor-core (tcgen05 + TMEM + TMA) forward kernels of the WERSA attention path, sm_100a.
//
// Key side  (Eq. 7, key summary):  S' = ReLU(K_F W)^T V,  z' = ReLU(K_F W)^T 1  per sequence chunk.
//   MMA1: D1[128 features x 128 tokens] = W^T (smem, K-major) * K_F^T (smem, K-major)   -> TMEM fp32
//   ReLU warps: TMEM -> registers -> max(.,0) -> bf16 -> back into the same TMEM columns
//   MMA2: S'[128 features x 64] += Phi^T (TMEM operand, K = tokens) * V (smem, N-major)  -> TMEM fp32
// Query side (Eq. 7, output):  O = ReLU(Q_F W) S' / (ReLU(Q_F W) z' + eps')
//   MMA1: D1[128 tokens x 128 features] = Q_F (smem, K-major) * W (as W^T, K-major)
//   ReLU warps as above, plus the row dot product with z' (denominator)
//   MMA2: N'[128 tokens x 64] (+)= Phi (TMEM operand, K = features) * S' (smem bf16, N-major)
//   epilogue warps: TMEM -> registers -> * 1/(D' + eps') -> bf16 -> swizzled smem -> TMA store
// Warp roles: warp 0 TMA producer, warp 1 MMA issuer (one thread), two ReLU warpgroups that
// alternate over the 128-column units, and (query side) one epilogue warpgroup.  All operand
// tiles use the 128-byte swizzle; every wait on an mbarrier is bounded.
#include "common.cuh"
#include "tc_common.cuh"

namespace wersa {
using namespace tc;

namespace {

constexpr int kTile = 128;                       // tokens per MMA tile
constexpr int kStages = 4;                       // TMA ring depth
constexpr uint32_t kTileBytes = kTile * kD * 2;  // one 128 x 64 bf16 tile
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kIdesc1 = make_idesc_bf16(128, 128, false, false);  // both operands K-major
constexpr uint32_t kIdesc2 = make_idesc_bf16(128, 64, false, true);    // B = V or S', N-major

enum { kErrProducer = 11, kErrMma = 12, kErrRelu = 13, kErrEpilogue = 14 };

struct alignas(8) KsideBars {
  uint64_t full[kStages], empty[kStages], d1_full[2], phi_ready[2], acc_done;
  uint32_t tmem_base;
  int abort_flag;
};
struct alignas(8) QsideBars {
  uint64_t full[kStages], empty[kStages], d1_full[2], phi_ready[2], d2_full[2], d2_free[2];
  uint32_t tmem_base;
  int abort_flag;
};

template <int NH> struct KsideSmem {
  static constexpr uint32_t wt = 0;
  static constexpr uint32_t kf = wt + NH * kTileBytes;
  static constexpr uint32_t v = kf + kStages * kTileBytes;
  static constexpr uint32_t zx = v + kStages * kTileBytes;       // 128 floats
  static constexpr uint32_t bars = zx + 512;
  static constexpr uint32_t total = bars + 256 + 1024;           // + alignment slack
};
template <int NH> struct QsideSmem {
  static constexpr uint32_t wt = 0;
  static constexpr uint32_t simg = wt + NH * kTileBytes;
  static constexpr uint32_t qf = simg + NH * kTileBytes;
  static constexpr uint32_t ost = qf + kStages * kTileBytes;     // 2 output staging tiles
  static constexpr uint32_t zs = ost + 2 * kTileBytes;           // NH*128 floats
  static constexpr uint32_t bars = zs + NH * 512;
  static constexpr uint32_t total = bars + 256 + 1024;
};

// (rows x 64) bf16 row-major in global memory -> 128B-swizzled rows of 128 bytes in shared memory.
__device__ __forceinline__ void load_rows_swizzled(uint8_t* dst, const __nv_bfloat16* src, int rows) {
  for (int i = threadIdx.x; i < rows * 8; i += blockDim.x) {
    const int r = i >> 3, c = i & 7;
    const uint4 val = *reinterpret_cast<const uint4*>(src + (size_t)r * kD + c * 8);
    *reinterpret_cast<uint4*>(dst + swz128(r, c)) = val;
  }
}

// ReLU pass over one 128-column unit of D1: fp32 TMEM -> bf16 pairs back into columns [0, 64) of
// the unit.  `sum` adds up the ReLU values of the row; `dot` their dot product with zrow[0..127]
// (nullptr: skipped).
__device__ __forceinline__ void relu_unit(uint32_t taddr, const float* __restrict__ zrow, float& sum, float& dot) {
#pragma unroll 1
  for (int c = 0; c < 4; ++c) {
    uint32_t r[32];
    tmem_ld32(taddr + 32 * c, r);
    tmem_ld_wait();
    uint32_t p[16];
    if (zrow != nullptr) {
#pragma unroll
      for (int j4 = 0; j4 < 8; ++j4) {
        const float4 zv = *reinterpret_cast<const float4*>(zrow + 32 * c + 4 * j4);
        const float a0 = fmaxf(__uint_as_float(r[4 * j4]), 0.f), a1 = fmaxf(__uint_as_float(r[4 * j4 + 1]), 0.f);
        const float a2 = fmaxf(__uint_as_float(r[4 * j4 + 2]), 0.f), a3 = fmaxf(__uint_as_float(r[4 * j4 + 3]), 0.f);
        dot = fmaf(a0, zv.x, dot);
        dot = fmaf(a1, zv.y, dot);
        dot = fmaf(a2, zv.z, dot);
        dot = fmaf(a3, zv.w, dot);
        p[2 * j4] = pack_bf16x2(a0, a1);
        p[2 * j4 + 1] = pack_bf16x2(a2, a3);
      }
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float a0 = fmaxf(__uint_as_float(r[2 * j]), 0.f), a1 = fmaxf(__uint_as_float(r[2 * j + 1]), 0.f);
        sum += a0 + a1;
        p[j] = pack_bf16x2(a0, a1);
      }
    }
    tmem_st16(taddr + 16 * c, p);
  }
  tmem_st_wait();
}

// ---- key side -----------------------------------------------------------------------------------
// grid (chunks, slabs), block 320: warp 0 producer, warp 1 MMA, warps 2-5 / 6-9 ReLU warpgroups.
template <int NH>
__global__ void __launch_bounds__(320, 1)
k_tc_kside(const __grid_constant__ CUtensorMap map_kf, const __grid_constant__ CUtensorMap map_v,
           const __nv_bfloat16* __restrict__ Wt, float* __restrict__ spart, float* __restrict__ zpart, int n,
           int chunk_tiles, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  using L = KsideSmem<NH>;
  KsideBars* bars = reinterpret_cast<KsideBars*>(smem + L::bars);
  float* zx = reinterpret_cast<float*>(smem + L::zx);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x, slab = blockIdx.y;
  const int tiles_total = n / kTile;
  const int tile0 = chunk * chunk_tiles;
  const int ntiles = min(chunk_tiles, tiles_total - tile0);
  const int units = ntiles * NH;
  constexpr int m = NH * 128;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->d1_full[b], 1);
      mbar_init(&bars->phi_ready[b], 128);
    }
    mbar_init(&bars->acc_done, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  load_rows_swizzled(smem + L::wt, Wt, m);
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bars->tmem_base;
  volatile int* abort_flag = &bars->abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int t = 0; t < ntiles; ++t) {
        const int s = t % kStages;
        if (!mbar_wait(&bars->empty[s], ((t / kStages) & 1) ^ 1, abort_flag, status, kErrProducer)) break;
        const int row = slab * n + (tile0 + t) * kTile;
        mbar_arrive_expect_tx(&bars->full[s], 2 * kTileBytes);
        tma_load_2d(smem + L::kf + s * kTileBytes, &map_kf, 0, row, &bars->full[s]);
        tma_load_2d(smem + L::v + s * kTileBytes, &map_v, 0, row, &bars->full[s]);
        issued = t + 1;
      }
      if (*abort_flag != 0) {   // let copies in flight land before the CTA's shared memory goes away
        for (int t = max(0, issued - kStages); t < issued; ++t)
          mbar_wait_drain(&bars->full[t % kStages], (t / kStages) & 1);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t wt_addr = smem_u32(smem + L::wt);
      const uint32_t kf_addr = smem_u32(smem + L::kf);
      const uint32_t v_addr = smem_u32(smem + L::v);
      bool ok = true;
      for (int u = 0; u <= units && ok; ++u) {
        if (u < units) {
          const int t = u / NH, h = u % NH, s = t % kStages;
          if (h == 0) {
            ok = mbar_wait(&bars->full[s], (t / kStages) & 1, abort_flag, status, kErrMma);
            if (!ok) break;
            tc_fence_after_sync();
          }
          const uint32_t d1 = tmem + (u & 1) * 128;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_ss(d1, make_smem_desc(wt_addr + h * kTileBytes + k * 32, 16, 1024),
                   make_smem_desc(kf_addr + s * kTileBytes + k * 32, 16, 1024), kIdesc1, k > 0);
          mma_commit(&bars->d1_full[u & 1]);
        }
        if (u >= 1) {
          const int v = u - 1;
          const int t = v / NH, h = v % NH, s = t % kStages;
          ok = mbar_wait(&bars->phi_ready[v & 1], (v >> 1) & 1, abort_flag, status, kErrMma);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t acc = tmem + 256 + h * 64;
#pragma unroll
          for (int k = 0; k < 8; ++k)
            mma_ts(acc, tmem + (v & 1) * 128 + k * 8, make_smem_desc(v_addr + s * kTileBytes + k * 2048, 1024, 1024),
                   kIdesc2, (t > 0 || k > 0) ? 1u : 0u);
          if (h == NH - 1) mma_commit(&bars->empty[s]);
        }
      }
      mma_commit(&bars->acc_done);
    }
  } else {
    const int g = (warp - 2) >> 2;                 // ReLU warpgroup 0 / 1
    const uint32_t lane_base = 32u * (warp & 3);
    const int row = lane_base + lane;              // feature within the half = TMEM lane
    const uint32_t taddr = tmem + (lane_base << 16) + g * 128;
    float zacc = 0.f, unused = 0.f;
    int it = 0;
    bool ok = true;
    for (int u = g; u < units; u += 2, ++it) {
      ok = mbar_wait(&bars->d1_full[g], it & 1, abort_flag, status, kErrRelu);
      if (!ok) break;
      tc_fence_after_sync();
      relu_unit(taddr, nullptr, zacc, unused);
      tc_fence_before_sync();
      mbar_arrive(&bars->phi_ready[g]);
    }
    if (ok) ok = mbar_wait(&bars->acc_done, 0, abort_flag, status, kErrRelu);
    if (ok) {
      tc_fence_after_sync();
      const size_t pidx = (size_t)slab * gridDim.x + chunk;
      if (NH == 1) {   // both warpgroups saw the same 128 features on alternating tiles
        if (g == 1) zx[row] = zacc;
        named_bar_sync(1, 256);
        if (g == 0) zacc += zx[row];
      }
      if (NH == 2 || g == 0) {
        const int feat = (NH == 2 ? g * 128 : 0) + row;
        float* dst = spart + (pidx * m + feat) * kD;
#pragma unroll 1
        for (int c = 0; c < 2; ++c) {
          uint32_t r[32];
          tmem_ld32(tmem + (lane_base << 16) + 256 + (NH == 2 ? g * 64 : 0) + 32 * c, r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 8; ++j)
            *reinterpret_cast<uint4*>(dst + 32 * c + 4 * j) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
        }
        zpart[pidx * m + feat] = zacc;
      }
    } else if (NH == 1) {
      named_bar_sync(1, 256);   // keep the barrier count balanced on the abort path
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, kTmemCols);
  }
}

// ---- query side ---------------------------------------------------------------------------------
// grid (chunks, slabs), block 448: warp 0 producer, warp 1 MMA, warps 2-5 / 6-9 ReLU warpgroups,
// warps 10-13 epilogue.  TMEM: D1[2] at columns 0/128, N' of tile parity p at 256 + 128 p (64
// columns) followed by the NH partial denominators of the tile's rows.
template <int NH>
__global__ void __launch_bounds__(448, 1)
k_tc_qside(const __grid_constant__ CUtensorMap map_qf, const __grid_constant__ CUtensorMap map_o,
           const __nv_bfloat16* __restrict__ Wt, const __nv_bfloat16* __restrict__ Sbf,
           const float* __restrict__ zg, const float* __restrict__ beta, float eps, float bw_floor, int n,
           int chunk_tiles, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  using L = QsideSmem<NH>;
  QsideBars* bars = reinterpret_cast<QsideBars*>(smem + L::bars);
  float* zs = reinterpret_cast<float*>(smem + L::zs);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x, slab = blockIdx.y;
  const int tiles_total = n / kTile;
  const int tile0 = chunk * chunk_tiles;
  const int ntiles = min(chunk_tiles, tiles_total - tile0);
  const int units = ntiles * NH;
  constexpr int m = NH * 128;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->d1_full[b], 1);
      mbar_init(&bars->phi_ready[b], 128);
      mbar_init(&bars->d2_full[b], 1);
      mbar_init(&bars->d2_free[b], 128);
    }
    bars->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  load_rows_swizzled(smem + L::wt, Wt, m);
  load_rows_swizzled(smem + L::simg, Sbf + (size_t)slab * m * kD, m);
  for (int i = threadIdx.x; i < m; i += blockDim.x) zs[i] = zg[(size_t)slab * m + i];
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bars->tmem_base;
  volatile int* abort_flag = &bars->abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int t = 0; t < ntiles; ++t) {
        const int s = t % kStages;
        if (!mbar_wait(&bars->empty[s], ((t / kStages) & 1) ^ 1, abort_flag, status, kErrProducer)) break;
        mbar_arrive_expect_tx(&bars->full[s], kTileBytes);
        tma_load_2d(smem + L::qf + s * kTileBytes, &map_qf, 0, slab * n + (tile0 + t) * kTile, &bars->full[s]);
        issued = t + 1;
      }
      if (*abort_flag != 0) {
        for (int t = max(0, issued - kStages); t < issued; ++t)
          mbar_wait_drain(&bars->full[t % kStages], (t / kStages) & 1);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t wt_addr = smem_u32(smem + L::wt);
      const uint32_t s_addr = smem_u32(smem + L::simg);
      const uint32_t qf_addr = smem_u32(smem + L::qf);
      bool ok = true;
      for (int u = 0; u <= units && ok; ++u) {
        if (u < units) {
          const int t = u / NH, h = u % NH, s = t % kStages;
          if (h == 0) {
            ok = mbar_wait(&bars->full[s], (t / kStages) & 1, abort_flag, status, kErrMma);
            if (!ok) break;
            tc_fence_after_sync();
          }
          const uint32_t d1 = tmem + (u & 1) * 128;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            mma_ss(d1, make_smem_desc(qf_addr + s * kTileBytes + k * 32, 16, 1024),
                   make_smem_desc(wt_addr + h * kTileBytes + k * 32, 16, 1024), kIdesc1, k > 0);
          mma_commit(&bars->d1_full[u & 1]);
        }
        if (u >= 1) {
          const int v = u - 1;
          const int t = v / NH, h = v % NH, s = t % kStages;
          ok = mbar_wait(&bars->phi_ready[v & 1], (v >> 1) & 1, abort_flag, status, kErrMma);
          if (!ok) break;
          if (h == 0 && t >= 2) {
            ok = mbar_wait(&bars->d2_free[t & 1], ((t >> 1) - 1) & 1, abort_flag, status, kErrMma);
            if (!ok) break;
          }
          tc_fence_after_sync();
          const uint32_t d2 = tmem + 256 + (t & 1) * 128;
#pragma unroll
          for (int k = 0; k < 8; ++k)
            mma_ts(d2, tmem + (v & 1) * 128 + k * 8, make_smem_desc(s_addr + h * kTileBytes + k * 2048, 1024, 1024),
                   kIdesc2, (h > 0 || k > 0) ? 1u : 0u);
          if (h == NH - 1) {
            mma_commit(&bars->d2_full[t & 1]);
            mma_commit(&bars->empty[s]);
          }
        }
      }
    }
  } else if (warp < 10) {
    const int g = (warp - 2) >> 2;
    const uint32_t lane_base = 32u * (warp & 3);
    const uint32_t taddr = tmem + (lane_base << 16) + g * 128;
    int it = 0;
    for (int u = g; u < units; u += 2, ++it) {
      const int t = u / NH, h = u % NH;
      if (!mbar_wait(&bars->d1_full[g], it & 1, abort_flag, status, kErrRelu)) break;
      tc_fence_after_sync();
      float dot = 0.f, unused = 0.f;
      relu_unit(taddr, zs + h * 128, unused, dot);
      // the tile's N' columns (and the denominator slots behind them) must have been read by the
      // epilogue of tile t-2 before they are written again
      if (t >= 2) {
        if (!mbar_wait(&bars->d2_free[t & 1], ((t >> 1) - 1) & 1, abort_flag, status, kErrRelu)) break;
        tc_fence_after_sync();
      }
      tmem_st1(tmem + (lane_base << 16) + 256 + (t & 1) * 128 + 64 + h, __float_as_uint(dot));
      tmem_st_wait();
      tc_fence_before_sync();
      mbar_arrive(&bars->phi_ready[g]);
    }
  } else {
    const uint32_t lane_base = 32u * (warp & 3);
    const int row = lane_base + lane;              // token within the tile = TMEM lane
    const int et = threadIdx.x - 320;              // 0..127 inside the epilogue warpgroup
    const float bw = fmaxf(beta[0], bw_floor);
    const float epsp = eps * (float)m * bw * bw;
    for (int t = 0; t < ntiles; ++t) {
      const int p = t & 1;
      if (!mbar_wait(&bars->d2_full[p], (t >> 1) & 1, abort_flag, status, kErrEpilogue)) break;
      tc_fence_after_sync();
      const uint32_t base = tmem + (lane_base << 16) + 256 + p * 128;
      uint32_t r0[32], r1[32], dd[NH];
      tmem_ld32(base, r0);
      tmem_ld32(base + 32, r1);
#pragma unroll
      for (int h = 0; h < NH; ++h) tmem_ld1(base + 64 + h, dd[h]);
      tmem_ld_wait();
      tc_fence_before_sync();
      mbar_arrive(&bars->d2_free[p]);
      float den = epsp;
#pragma unroll
      for (int h = 0; h < NH; ++h) den += __uint_as_float(dd[h]);
      const float inv = 1.f / den;
      // staging buffer p was last used by tile t-2: its TMA store must have finished reading
      if (et == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      named_bar_sync(2, 128);
      uint8_t* ost = smem + L::ost + p * kTileBytes;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint4 v;
        v.x = pack_bf16x2(__uint_as_float(r0[8 * c]) * inv, __uint_as_float(r0[8 * c + 1]) * inv);
        v.y = pack_bf16x2(__uint_as_float(r0[8 * c + 2]) * inv, __uint_as_float(r0[8 * c + 3]) * inv);
        v.z = pack_bf16x2(__uint_as_float(r0[8 * c + 4]) * inv, __uint_as_float(r0[8 * c + 5]) * inv);
        v.w = pack_bf16x2(__uint_as_float(r0[8 * c + 6]) * inv, __uint_as_float(r0[8 * c + 7]) * inv);
        *reinterpret_cast<uint4*>(ost + swz128(row, c)) = v;
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint4 v;
        v.x = pack_bf16x2(__uint_as_float(r1[8 * c]) * inv, __uint_as_float(r1[8 * c + 1]) * inv);
        v.y = pack_bf16x2(__uint_as_float(r1[8 * c + 2]) * inv, __uint_as_float(r1[8 * c + 3]) * inv);
        v.z = pack_bf16x2(__uint_as_float(r1[8 * c + 4]) * inv, __uint_as_float(r1[8 * c + 5]) * inv);
        v.w = pack_bf16x2(__uint_as_float(r1[8 * c + 6]) * inv, __uint_as_float(r1[8 * c + 7]) * inv);
        *reinterpret_cast<uint4*>(ost + swz128(row, 4 + c)) = v;
      }
      fence_proxy_async_smem();
      named_bar_sync(2, 128);
      if (et == 0) {
        tma_store_2d(&map_o, ost, 0, slab * n + (tile0 + t) * kTile);
        bulk_commit_group();
      }
    }
    if (et == 0) bulk_wait_group0();
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, kTmemCols);
  }
}

// W (64 x m) -> Wt (m x 64), bf16.
__global__ void k_transpose_w(const __nv_bfloat16* __restrict__ W, __nv_bfloat16* __restrict__ Wt, int m) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < m * kD) {
    const int r = i / kD, c = i - r * kD;
    Wt[i] = W[(size_t)c * m + r];
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

// (rows x 64) bf16 row-major tensor, boxes of 128 rows x 64 columns, 128-byte swizzle.
cudaError_t make_tile_map(const void* base, size_t rows, CUtensorMap* out) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return cudaErrorNotSupported;
  const cuuint64_t dims[2] = {kD, rows};
  const cuuint64_t strides[1] = {kD * 2};
  const cuuint32_t box[2] = {kD, kTile};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

}  // namespace

bool tc_supported(const wersa_config& cfg) {
  return cfg.dtype == WERSA_BF16 && (cfg.features == 128 || cfg.features == 256) && cfg.seq_len % kTile == 0 &&
         cfg.head_dim == kD;
}

cudaError_t launch_tc_prepare_w(const Plan& p, const Ws& w, const void* W, cudaStream_t st, int* launches) {
  const int m = p.cfg.features;
  k_transpose_w<<<(m * kD + 255) / 256, 256, 0, st>>>((const __nv_bfloat16*)W, w.Wt, m);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_tc_kside(const Plan& p, const Ws& w, const void* KFb, const void* V, cudaStream_t st,
                            int* launches) {
  CUtensorMap map_kf, map_v;
  const size_t rows = (size_t)p.slabs * p.cfg.seq_len;
  cudaError_t err;
  if ((err = make_tile_map(KFb, rows, &map_kf)) != cudaSuccess) return err;
  if ((err = make_tile_map(V, rows, &map_v)) != cudaSuccess) return err;
  dim3 grid(p.tchunks, p.slabs);
  if (p.cfg.features == 256) {
    auto k = k_tc_kside<2>;
    if ((err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, KsideSmem<2>::total)) != cudaSuccess)
      return err;
    k<<<grid, 320, KsideSmem<2>::total, st>>>(map_kf, map_v, w.Wt, w.spart, w.zpart, p.cfg.seq_len, p.tchunk_tiles,
                                              w.status);
  } else {
    auto k = k_tc_kside<1>;
    if ((err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, KsideSmem<1>::total)) != cudaSuccess)
      return err;
    k<<<grid, 320, KsideSmem<1>::total, st>>>(map_kf, map_v, w.Wt, w.spart, w.zpart, p.cfg.seq_len, p.tchunk_tiles,
                                              w.status);
  }
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_tc_qside(const Plan& p, const Ws& w, const void* QFb, const float* beta, void* O, cudaStream_t st,
                            int* launches) {
  CUtensorMap map_qf, map_o;
  const size_t rows = (size_t)p.slabs * p.cfg.seq_len;
  cudaError_t err;
  if ((err = make_tile_map(QFb, rows, &map_qf)) != cudaSuccess) return err;
  if ((err = make_tile_map(O, rows, &map_o)) != cudaSuccess) return err;
  dim3 grid(p.tchunks, p.slabs);
  if (p.cfg.features == 256) {
    auto k = k_tc_qside<2>;
    if ((err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, QsideSmem<2>::total)) != cudaSuccess)
      return err;
    k<<<grid, 448, QsideSmem<2>::total, st>>>(map_qf, map_o, w.Wt, w.Sbf, w.z, beta, p.cfg.eps, p.cfg.bw_floor,
                                              p.cfg.seq_len, p.tchunk_tiles, w.status);
  } else {
    auto k = k_tc_qside<1>;
    if ((err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, QsideSmem<1>::total)) != cudaSuccess)
      return err;
    k<<<grid, 448, QsideSmem<1>::total, st>>>(map_qf, map_o, w.Wt, w.Sbf, w.z, beta, p.cfg.eps, p.cfg.bw_floor,
                                              p.cfg.seq_len, p.tchunk_tiles, w.status);
  }
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace wersa
