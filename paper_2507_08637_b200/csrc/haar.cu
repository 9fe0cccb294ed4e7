// Multi-level Haar analysis -> per-scale gating -> synthesis along the sequence, as one on-chip
// pass over tiles of 256 tokens (Sec. 3.1 steps 3, 5, 6 and Algorithm 2 of the WERSA paper).
//
// Because the Haar detail projector of level l equals blockmean_{2^(l-1)} - blockmean_{2^l} and
// the approximation projector of level L equals blockmean_{2^L}, the filtered signal is
//   T_f x = f_0 x + sum_{i=1..L} (f_i - f_{i-1}) * blockmean_{2^i}(x),
// so one pass needs only the aligned block sums of 2, 4, ..., 2^L rows.  A thread holds 8
// consecutive rows x 8 columns in registers (levels 1-3), partner lanes give levels 4-5 through
// warp shuffles and the eight warps exchange their 32-row sums through shared memory (levels 6-8).
// Rows past the end of the sequence read as zero, which is the zero padding of Algorithm 2.
#include "common.cuh"

namespace wersa {
namespace {

struct LevelCoef {
  float f0;
  float k[kMaxLevels + 1];   // k[i] = (f_i - f_{i-1}) / 2^i for 1 <= i <= L, else 0
};

__device__ __forceinline__ LevelCoef level_coef(const float* __restrict__ f, int L) {
  LevelCoef c;
  c.f0 = f[0];
  float scale = 0.5f;
#pragma unroll
  for (int i = 1; i <= kMaxLevels; ++i) {
    c.k[i] = (i <= L) ? (f[i] - f[i - 1]) * scale : 0.f;
    scale *= 0.5f;
  }
  c.k[0] = 0.f;
  return c;
}

template <typename T>
__device__ __forceinline__ void load_tile(const T* __restrict__ X, int n, int row0, float (&x)[8][8]) {
  const int cg = threadIdx.x & 7;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int r = row0 + j;
    if (r < n) {
      load8(X + (size_t)r * kD + cg * 8, x[j]);
    } else {
#pragma unroll
      for (int c = 0; c < 8; ++c) x[j][c] = 0.f;
    }
  }
}

constexpr int kPyr = 63;    // 32 + 16 + 8 + 4 + 2 + 1 block sums per column
constexpr int kHalfD = kD / 2;
__device__ __forceinline__ int pyr_base(int l) { return 64 - (64 >> (l - 3)); }   // level 3 -> 0, 4 -> 32, 5 -> 48 ...

__device__ __forceinline__ void load4(const float* p, float (&v)[4]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&v)[4]) {
  const uint2 raw = *reinterpret_cast<const uint2*>(p);
  v[0] = __uint_as_float(raw.x << 16);
  v[1] = __uint_as_float(raw.x & 0xFFFF0000u);
  v[2] = __uint_as_float(raw.y << 16);
  v[3] = __uint_as_float(raw.y & 0xFFFF0000u);
}
__device__ __forceinline__ void store4(float* p, const float (&v)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void store4(__nv_bfloat16* p, const float (&v)[4]) {
  const __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b2 = __floats2bfloat162_rn(v[2], v[3]);
  uint2 raw;
  raw.x = *reinterpret_cast<const uint32_t*>(&a);
  raw.y = *reinterpret_cast<const uint32_t*>(&b2);
  *reinterpret_cast<uint2*>(p) = raw;
}


// Stand-alone filter pass, XF = T_f(X).  The transform acts on every column separately, so one CTA takes
// 256 rows x 32 columns (half of the head dimension), 8 rows x 4 columns per thread: a register tile of
// 32 values lets several CTAs share an SM, so that the loads of one overlap the arithmetic and stores of
// the others (the pass is bound by memory bandwidth).  Levels 1-3 come from the register tile; the 8-row
// sums go to a pyramid in shared memory (per column 32 sums of level 3, then 16, 8, 4, 2, 1 of levels
// 4-8), from which every thread takes the coarse part of its output rows.
// With kAddVec every output row of slab s also gets vec[s][:] * vec_scale added (the mean-pool term of dQ).
// grid (2 * htiles, slabs): blockIdx.x = 2 * tile + column half; block 256.
template <typename Tin, typename Tout, bool kAddVec>
__global__ void __launch_bounds__(256, 4) k_haar_filter(const Tin* __restrict__ X, const float* __restrict__ f,
                                                     Tout* __restrict__ XF, int n, int L,
                                                     const float* __restrict__ vec, float vec_scale) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  __shared__ float pyr[kPyr][kHalfD];
  __shared__ float hit[32][kHalfD];   // sum_{l=3..8} k_l * s_l(block of row group r), per column
  const int slab = blockIdx.y, half = blockIdx.x & 1;
  const int cg = threadIdx.x & 7, rg = threadIdx.x >> 3;
  const int row0 = (blockIdx.x >> 1) * kHaarTile + rg * 8;
  const int col0 = half * kHalfD + cg * 4;   // first of this thread's four columns
  const LevelCoef k = level_coef(f + (size_t)slab * (L + 1), L);
  float x[8][4];
  {
    const Tin* xp = X + (size_t)slab * n * kD + col0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (row0 + j < n) {
        load4(xp + (size_t)(row0 + j) * kD, x[j]);
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) x[j][c] = 0.f;
      }
    }
  }
#pragma unroll
  for (int c = 0; c < 4; ++c)
    pyr[rg][cg * 4 + c] = ((x[0][c] + x[1][c]) + (x[2][c] + x[3][c])) + ((x[4][c] + x[5][c]) + (x[6][c] + x[7][c]));
  __syncthreads();
  if (threadIdx.x < kHalfD) {   // levels 4-8 of the pyramid, one thread per column
    const int col = threadIdx.x;
#pragma unroll
    for (int l = 4; l <= 8; ++l) {
      const int src = pyr_base(l - 1), dst = pyr_base(l), cnt = 256 >> l;
      for (int b2 = 0; b2 < cnt; ++b2) pyr[dst + b2][col] = pyr[src + 2 * b2][col] + pyr[src + 2 * b2 + 1][col];
    }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int e = threadIdx.x + 256 * i, r = e >> 5, col = e & 31;
    float v = k.k[3] * pyr[r][col];
#pragma unroll
    for (int l = 4; l <= 8; ++l) v += k.k[l] * pyr[pyr_base(l) + (r >> (l - 3))][col];
    hit[r][col] = v;
  }
  __syncthreads();
  Tout* dst = XF + (size_t)slab * n * kD + col0;
#pragma unroll
  for (int j = 0; j < 8; j += 4) {   // four rows (one level-2 block) at a time
    float y[4][4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float a0 = x[j][c] + x[j + 1][c], a1 = x[j + 2][c] + x[j + 3][c];
      float c2 = fmaf(k.k[2], a0 + a1, hit[rg][cg * 4 + c]);
      if constexpr (kAddVec) c2 = fmaf(vec[(size_t)slab * kD + col0 + c], vec_scale, c2);
      const float c10 = fmaf(k.k[1], a0, c2), c11 = fmaf(k.k[1], a1, c2);
      y[0][c] = fmaf(k.f0, x[j][c], c10);
      y[1][c] = fmaf(k.f0, x[j + 1][c], c10);
      y[2][c] = fmaf(k.f0, x[j + 2][c], c11);
      y[3][c] = fmaf(k.f0, x[j + 3][c], c11);
    }
#pragma unroll
    for (int jj = 0; jj < 4; ++jj)
      if (row0 + j + jj < n) store4(dst + (size_t)(row0 + j + jj) * kD, y[jj]);
  }
}

// The same pass for bf16 input: a thread keeps its 8 rows x 8 columns as the 32 packed words it loaded
// (16-byte loads; unpacked where they are used, twice), so that three CTAs of 256 rows x 64 columns share an
// SM with 16-byte accesses in flight.  grid (htiles, slabs), block 256.
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

template <typename Tout>
__global__ void __launch_bounds__(256, 3) k_haar_filter_bf16(const __nv_bfloat16* __restrict__ X,
                                                             const float* __restrict__ f, Tout* __restrict__ XF,
                                                             int n, int L) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  __shared__ float pyr[kPyr][kD];
  __shared__ float hit[32][kD];   // sum_{l=3..8} k_l * s_l(block of row group r), per column
  const int slab = blockIdx.y;
  const int cg = threadIdx.x & 7, rg = threadIdx.x >> 3;
  const int row0 = blockIdx.x * kHaarTile + rg * 8;
  const LevelCoef k = level_coef(f + (size_t)slab * (L + 1), L);
  uint32_t u[8][4];
  {
    const __nv_bfloat16* xp = X + (size_t)slab * n * kD + cg * 8;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      uint4 raw = make_uint4(0u, 0u, 0u, 0u);
      if (row0 + j < n) raw = *reinterpret_cast<const uint4*>(xp + (size_t)(row0 + j) * kD);
      u[j][0] = raw.x; u[j][1] = raw.y; u[j][2] = raw.z; u[j][3] = raw.w;
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float lo = 0.f, hi = 0.f;
#pragma unroll
    for (int j = 0; j < 8; j += 2) {   // pairs first, as the other kernels add them
      lo += bf_lo(u[j][i]) + bf_lo(u[j + 1][i]);
      hi += bf_hi(u[j][i]) + bf_hi(u[j + 1][i]);
    }
    pyr[rg][cg * 8 + 2 * i] = lo;
    pyr[rg][cg * 8 + 2 * i + 1] = hi;
  }
  __syncthreads();
  if (threadIdx.x < kD) {   // levels 4-8 of the pyramid, one thread per column
    const int col = threadIdx.x;
#pragma unroll
    for (int l = 4; l <= 8; ++l) {
      const int src = pyr_base(l - 1), dst = pyr_base(l), cnt = 256 >> l;
      for (int b2 = 0; b2 < cnt; ++b2) pyr[dst + b2][col] = pyr[src + 2 * b2][col] + pyr[src + 2 * b2 + 1][col];
    }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int e = threadIdx.x + 256 * i, r = e >> 6, col = e & 63;
    float v = k.k[3] * pyr[r][col];
#pragma unroll
    for (int l = 4; l <= 8; ++l) v += k.k[l] * pyr[pyr_base(l) + (r >> (l - 3))][col];
    hit[r][col] = v;
  }
  __syncthreads();
  Tout* dst = XF + (size_t)slab * n * kD + cg * 8;
  if constexpr (sizeof(Tout) == 2) {
    // bf16 out: the results replace the packed inputs column pair by column pair, rows are stored whole
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float h0 = hit[rg][cg * 8 + 2 * i], h1 = hit[rg][cg * 8 + 2 * i + 1];
#pragma unroll
      for (int j = 0; j < 8; j += 4) {
        float y[4][2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float x0 = h ? bf_hi(u[j][i]) : bf_lo(u[j][i]), x1 = h ? bf_hi(u[j + 1][i]) : bf_lo(u[j + 1][i]);
          const float x2 = h ? bf_hi(u[j + 2][i]) : bf_lo(u[j + 2][i]), x3 = h ? bf_hi(u[j + 3][i]) : bf_lo(u[j + 3][i]);
          const float a0 = x0 + x1, a1 = x2 + x3;
          const float c2 = fmaf(k.k[2], a0 + a1, h ? h1 : h0);
          const float c10 = fmaf(k.k[1], a0, c2), c11 = fmaf(k.k[1], a1, c2);
          y[0][h] = fmaf(k.f0, x0, c10);
          y[1][h] = fmaf(k.f0, x1, c10);
          y[2][h] = fmaf(k.f0, x2, c11);
          y[3][h] = fmaf(k.f0, x3, c11);
        }
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const __nv_bfloat162 pk = __floats2bfloat162_rn(y[jj][0], y[jj][1]);
          u[j + jj][i] = *reinterpret_cast<const uint32_t*>(&pk);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (row0 + j < n)
        *reinterpret_cast<uint4*>(dst + (size_t)(row0 + j) * kD) = make_uint4(u[j][0], u[j][1], u[j][2], u[j][3]);
  } else {
#pragma unroll
    for (int j = 0; j < 8; j += 4) {   // four rows (one level-2 block) at a time
      float y[4][8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int c = 2 * i + h;
          const float x0 = h ? bf_hi(u[j][i]) : bf_lo(u[j][i]), x1 = h ? bf_hi(u[j + 1][i]) : bf_lo(u[j + 1][i]);
          const float x2 = h ? bf_hi(u[j + 2][i]) : bf_lo(u[j + 2][i]), x3 = h ? bf_hi(u[j + 3][i]) : bf_lo(u[j + 3][i]);
          const float a0 = x0 + x1, a1 = x2 + x3;
          const float c2 = fmaf(k.k[2], a0 + a1, hit[rg][cg * 8 + c]);
          const float c10 = fmaf(k.k[1], a0, c2), c11 = fmaf(k.k[1], a1, c2);
          y[0][c] = fmaf(k.f0, x0, c10);
          y[1][c] = fmaf(k.f0, x1, c10);
          y[2][c] = fmaf(k.f0, x2, c11);
          y[3][c] = fmaf(k.f0, x3, c11);
        }
      }
#pragma unroll
      for (int jj = 0; jj < 4; ++jj)
        if (row0 + j + jj < n) store8(dst + (size_t)(row0 + j + jj) * kD, y[jj]);
    }
  }
}

// The same filter with the result written as three bf16 planes hi + mid + lo (each slabs x n x 64):
// hi = bf16(x), mid = bf16(x - hi), lo = bf16(x - hi - mid), so that their sum carries the fp32
// value (24 mantissa bits) into bf16 tensor-core products.  The backward kernels need that: the
// ReLU mask 1[a > 0] of a = X_F W must not flip through the rounding of X_F.
template <typename Tin>
__global__ void __launch_bounds__(256, 2) k_haar_filter_split3(const Tin* __restrict__ X, const float* __restrict__ f,
                                                            __nv_bfloat16* __restrict__ XF3, size_t plane, int n,
                                                            int L) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  // levels 4-8 through a pyramid of the 8-row sums in shared memory (per column: 32 sums of level 3,
  // then 16, 8, 4, 2, 1), as in k_haar_backward
  __shared__ float pyr[63][kD];
  __shared__ float hit[32][kD];   // sum_{l=3..8} k_l * s_l(block of row group r), per column
  const int slab = blockIdx.y;
  const int cg = threadIdx.x & 7, rg = threadIdx.x >> 3;
  const int row0 = blockIdx.x * kHaarTile + rg * 8;
  const LevelCoef k = level_coef(f + (size_t)slab * (L + 1), L);
  float x[8][8];
  load_tile(X + (size_t)slab * n * kD, n, row0, x);
#pragma unroll
  for (int c = 0; c < 8; ++c)
    pyr[rg][cg * 8 + c] = ((x[0][c] + x[1][c]) + (x[2][c] + x[3][c])) + ((x[4][c] + x[5][c]) + (x[6][c] + x[7][c]));
  __syncthreads();
  if (threadIdx.x < kD) {
    const int col = threadIdx.x;
    int src = 0, cnt = 16;
#pragma unroll
    for (int l = 4; l <= 8; ++l) {
      const int dst = src + 2 * cnt;
      for (int b2 = 0; b2 < cnt; ++b2) pyr[dst + b2][col] = pyr[src + 2 * b2][col] + pyr[src + 2 * b2 + 1][col];
      src = dst;
      cnt >>= 1;
    }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int e = threadIdx.x + 256 * i, r = e >> 6, col = e & 63;
    float v = k.k[3] * pyr[r][col];
    int base = 32;
#pragma unroll
    for (int l = 4; l <= 8; ++l) {
      v += k.k[l] * pyr[base + (r >> (l - 3))][col];
      base += 256 >> l;
    }
    hit[r][col] = v;
  }
  __syncthreads();
  __nv_bfloat16* dst = XF3 + (size_t)slab * n * kD + cg * 8;
  float hi_c[8], s1[4][8], s2[2][8];
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    hi_c[c] = hit[rg][cg * 8 + c];
#pragma unroll
    for (int p = 0; p < 4; ++p) s1[p][c] = x[2 * p][c] + x[2 * p + 1][c];
    s2[0][c] = s1[0][c] + s1[1][c];
    s2[1][c] = s1[2][c] + s1[3][c];
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if (row0 + j >= n) continue;
    float hi[8], mid[8], lo[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const float y = k.f0 * x[j][c] + k.k[1] * s1[j >> 1][c] + k.k[2] * s2[j >> 2][c] + hi_c[c];
      hi[c] = __bfloat162float(__float2bfloat16_rn(y));
      const float r1 = y - hi[c];
      mid[c] = __bfloat162float(__float2bfloat16_rn(r1));
      lo[c] = r1 - mid[c];
    }
    __nv_bfloat16* row = dst + (size_t)(row0 + j) * kD;
    store8(row, hi);
    store8(row + plane, mid);
    store8(row + 2 * plane, lo);
  }
}

// Backward of the filter for one tile: dX = T_f(G) (the operator is symmetric) and the band
// inner products of (G, X) that give df:
//   slot l-1 (l = 1..8): sum over blocks of Delta_l(G) * Delta_l(X) / 2^l, the product of the
//                        level-l detail coefficients (Delta_l = left half sum - right half sum);
//   slot 8+l-1:          sum over blocks of s_l(G) * s_l(X) / 2^l, the product of the level-l
//                        approximation coefficients.
// The transform acts on every column separately, so one CTA takes 256 rows x 32 columns (half of the
// head dimension): 8 rows x 4 columns per thread, a small register tile (several CTAs per SM keep loads,
// arithmetic and stores of different tiles overlapped).  G and X are loaded together.  Levels 1-3 live
// in the register tiles; the 8-row sums go to a pyramid in shared memory (per tensor and column: 32
// sums of level 3, then 16, 8, 4, 2, 1 of levels 4-8), from which one thread per column takes the level
// 4-8 products and every thread the coarse part of its output rows.
// grid (2 * htiles, slabs): blockIdx.x = 2 * tile + column half; one band partial per CTA.
// kWrite = false leaves dX unwritten (only the band inner products are wanted).  Two CTAs per SM with the
// output (at three the 85-register limit spilled the register tiles: 77 -> 69 us per pass on config 5), four
// without it.
template <typename Tin, typename Tout, bool kWrite>
__global__ void __launch_bounds__(256, kWrite ? 2 : 4) k_haar_backward(const Tin* __restrict__ X, const float* __restrict__ G,
                                                          const float* __restrict__ f, Tout* __restrict__ dX,
                                                          float* __restrict__ bands, int n, int L) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  __shared__ float pyr[2][kPyr][kHalfD];   // [0] = G, [1] = X
  __shared__ float hit[32][kHalfD];        // coarse part of the output of row group rg, per column
  __shared__ float red[8][kBandVals];
  const int slab = blockIdx.y, half = blockIdx.x & 1;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int cg = threadIdx.x & 7, rg = threadIdx.x >> 3;
  const int row0 = (blockIdx.x >> 1) * kHaarTile + rg * 8;
  const int col0 = half * kHalfD + cg * 4;   // first of this thread's four columns
  const LevelCoef k = level_coef(f + (size_t)slab * (L + 1), L);
  float acc[kBandVals];
#pragma unroll
  for (int i = 0; i < kBandVals; ++i) acc[i] = 0.f;
  float g[8][4], x[8][4];
  {
    const float* gp = G + (size_t)slab * n * kD + col0;
    const Tin* xp = X + (size_t)slab * n * kD + col0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (row0 + j < n) {
        load4(gp + (size_t)(row0 + j) * kD, g[j]);
        load4(xp + (size_t)(row0 + j) * kD, x[j]);
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) g[j][c] = x[j][c] = 0.f;
      }
    }
  }
  // levels 1-3: products from the register tiles, 8-row sums into the pyramid
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    float g1[4], x1[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      g1[p] = g[2 * p][c] + g[2 * p + 1][c];
      x1[p] = x[2 * p][c] + x[2 * p + 1][c];
      acc[0] += (g[2 * p][c] - g[2 * p + 1][c]) * (x[2 * p][c] - x[2 * p + 1][c]);
      acc[8] += g1[p] * x1[p];
    }
    const float g20 = g1[0] + g1[1], g21 = g1[2] + g1[3], x20 = x1[0] + x1[1], x21 = x1[2] + x1[3];
    acc[1] += (g1[0] - g1[1]) * (x1[0] - x1[1]) + (g1[2] - g1[3]) * (x1[2] - x1[3]);
    acc[9] += g20 * x20 + g21 * x21;
    const float g3 = g20 + g21, x3 = x20 + x21;
    acc[2] += (g20 - g21) * (x20 - x21);
    acc[10] += g3 * x3;
    pyr[0][rg][cg * 4 + c] = g3;
    pyr[1][rg][cg * 4 + c] = x3;
  }
  __syncthreads();
  // levels 4-8 of the pyramid: thread (tensor = tid >> 5, column = tid & 31), tid < 64
  if (threadIdx.x < 2 * kHalfD) {
    float(*py)[kHalfD] = pyr[threadIdx.x >> 5];
    const int col = threadIdx.x & 31;
#pragma unroll
    for (int l = 4; l <= 8; ++l) {
      const int src = pyr_base(l - 1), dst = pyr_base(l), cnt = 256 >> l;
      for (int b2 = 0; b2 < cnt; ++b2) py[dst + b2][col] = py[src + 2 * b2][col] + py[src + 2 * b2 + 1][col];
    }
  }
  __syncthreads();
  // level 4-8 products: one thread per column
  if (threadIdx.x < kHalfD) {
    const int col = threadIdx.x;
#pragma unroll
    for (int l = 4; l <= 8; ++l) {
      const int src = pyr_base(l - 1), dst = pyr_base(l), cnt = 256 >> l;
      float dsum = 0.f, asum = 0.f;
      for (int b2 = 0; b2 < cnt; ++b2) {
        dsum += (pyr[0][src + 2 * b2][col] - pyr[0][src + 2 * b2 + 1][col]) *
                (pyr[1][src + 2 * b2][col] - pyr[1][src + 2 * b2 + 1][col]);
        asum += pyr[0][dst + b2][col] * pyr[1][dst + b2][col];
      }
      acc[l - 1] = dsum;
      acc[8 + l - 1] = asum;
    }
  }
  // coarse part of the output rows: hit[r][col] = sum_{l=3..8} k_l * s_l(block of row group r)
  if constexpr (kWrite) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = threadIdx.x + 256 * i, r = e >> 5, col = e & 31;
      float v = k.k[3] * pyr[0][r][col];
#pragma unroll
      for (int l = 4; l <= 8; ++l) v += k.k[l] * pyr[0][pyr_base(l) + (r >> (l - 3))][col];
      hit[r][col] = v;
    }
    __syncthreads();
  }
  if constexpr (kWrite) {
    Tout* dst = dX + (size_t)slab * n * kD + col0;
    float hi[4], s1[4][4], s2[2][4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      hi[c] = hit[rg][cg * 4 + c];
#pragma unroll
      for (int p = 0; p < 4; ++p) s1[p][c] = g[2 * p][c] + g[2 * p + 1][c];
      s2[0][c] = s1[0][c] + s1[1][c];
      s2[1][c] = s1[2][c] + s1[3][c];
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float y[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) y[c] = k.f0 * g[j][c] + k.k[1] * s1[j >> 1][c] + k.k[2] * s2[j >> 2][c] + hi[c];
      if (row0 + j < n) store4(dst + (size_t)(row0 + j) * kD, y);
    }
  }
  // 1 / 2^l normalisation
#pragma unroll
  for (int l = 0; l < 8; ++l) {
    const float wgt = 1.f / (float)(2 << l);
    acc[l] *= wgt;
    acc[8 + l] *= wgt;
  }
#pragma unroll
  for (int i = 0; i < kBandVals; ++i) {
    float v = acc[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) red[warp][i] = v;
  }
  __syncthreads();
  if (threadIdx.x < kBandVals) {
    float v = 0.f;
#pragma unroll
    for (int wi = 0; wi < 8; ++wi) v += red[wi][threadIdx.x];
    bands[((size_t)slab * gridDim.x + blockIdx.x) * kBandVals + threadIdx.x] = v;
  }
}

}  // namespace

cudaError_t launch_haar_filter(const Plan& p, const void* X, int in_kind, const float* f, void* XF,
                               int out_kind, cudaStream_t st, int* launches) {
  dim3 grid(2 * p.htiles, p.slabs);   // fp32 input: two column halves per 256-row tile
  dim3 grid_bf(p.htiles, p.slabs);
  const int n = p.cfg.seq_len, L = p.cfg.levels;
  if (in_kind == 1 && out_kind == 1)
    launch_after(k_haar_filter_bf16<__nv_bfloat16>, dim3(grid_bf), dim3(256), 0, st, (const __nv_bfloat16*)X, f, (__nv_bfloat16*)XF, n, L);
  else if (in_kind == 1 && out_kind == 0)
    launch_after(k_haar_filter_bf16<float>, dim3(grid_bf), dim3(256), 0, st, (const __nv_bfloat16*)X, f, (float*)XF, n, L);
  else if (in_kind == 0 && out_kind == 0)
    launch_after(k_haar_filter<float, float, false>, dim3(grid), dim3(256), 0, st, (const float*)X, f, (float*)XF, n, L, nullptr, 0.f);
  else
    launch_after(k_haar_filter<float, __nv_bfloat16, false>, dim3(grid), dim3(256), 0, st, (const float*)X, f, (__nv_bfloat16*)XF, n, L,
                                                                    nullptr, 0.f);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_haar_filter_addvec(const Plan& p, const float* G, const float* f, const float* vec,
                                      float vec_scale, void* dX, int out_kind, cudaStream_t st, int* launches) {
  dim3 grid(2 * p.htiles, p.slabs);
  const int n = p.cfg.seq_len, L = p.cfg.levels;
  if (out_kind == 0)
    launch_after(k_haar_filter<float, float, true>, dim3(grid), dim3(256), 0, st, G, f, (float*)dX, n, L, vec, vec_scale);
  else
    launch_after(k_haar_filter<float, __nv_bfloat16, true>, dim3(grid), dim3(256), 0, st, G, f, (__nv_bfloat16*)dX, n, L, vec, vec_scale);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_haar_filter_split3(const Plan& p, const void* X, int in_kind, const float* f,
                                      __nv_bfloat16* XF3, cudaStream_t st, int* launches) {
  dim3 grid(p.htiles, p.slabs);
  const int n = p.cfg.seq_len, L = p.cfg.levels;
  const size_t plane = (size_t)p.slabs * n * kD;
  if (in_kind == 1)
    launch_after(k_haar_filter_split3<__nv_bfloat16>, dim3(grid), dim3(256), 0, st, (const __nv_bfloat16*)X, f, XF3, plane, n, L);
  else
    launch_after(k_haar_filter_split3<float>, dim3(grid), dim3(256), 0, st, (const float*)X, f, XF3, plane, n, L);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_haar_backward(const Plan& p, const Ws& w, const void* X, int in_kind, const float* G,
                                 void* dX, int out_kind, int which, cudaStream_t st, int* launches) {
  dim3 grid(2 * p.htiles, p.slabs);   // two column halves per 256-row tile
  const int n = p.cfg.seq_len, L = p.cfg.levels;
  float* bands = w.bands + (size_t)which * p.slabs * 2 * p.htiles * kBandVals;
  if (dX == nullptr) {   // band inner products only
    if (in_kind == 1)
      launch_after(k_haar_backward<__nv_bfloat16, float, false>, dim3(grid), dim3(256), 0, st, (const __nv_bfloat16*)X, G, w.f, nullptr,
                                                                        bands, n, L);
    else
      launch_after(k_haar_backward<float, float, false>, dim3(grid), dim3(256), 0, st, (const float*)X, G, w.f, nullptr, bands, n, L);
  } else if (in_kind == 1 && out_kind == 1)
    launch_after(k_haar_backward<__nv_bfloat16, __nv_bfloat16, true>, dim3(grid), dim3(256), 0, st, 
        (const __nv_bfloat16*)X, G, w.f, (__nv_bfloat16*)dX, bands, n, L);
  else if (in_kind == 1 && out_kind == 0)
    launch_after(k_haar_backward<__nv_bfloat16, float, true>, dim3(grid), dim3(256), 0, st, (const __nv_bfloat16*)X, G, w.f, (float*)dX,
                                                                     bands, n, L);
  else if (in_kind == 0 && out_kind == 0)
    launch_after(k_haar_backward<float, float, true>, dim3(grid), dim3(256), 0, st, (const float*)X, G, w.f, (float*)dX, bands, n, L);
  else
    launch_after(k_haar_backward<float, __nv_bfloat16, true>, dim3(grid), dim3(256), 0, st, (const float*)X, G, w.f, (__nv_bfloat16*)dX,
                                                                     bands, n, L);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace wersa
