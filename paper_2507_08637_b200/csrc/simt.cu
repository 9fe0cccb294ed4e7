// fp32 FFMA kernels of the WERSA attention path (Eqs. 6-7 of the paper and their backward):
// random projection + ReLU, key summary S' = ReLU(K_F W)^T V and z' = ReLU(K_F W)^T 1 over
// sequence chunks, output O = ReLU(Q_F W) S' / (ReLU(Q_F W) z' + eps'), and the gradient kernels.
//
// The feature-map factor c = 1/(bw sqrt(m)) is folded away: ReLU is positively homogeneous, so
// phi = c ReLU(X_F W) and O = N'/(D' + eps/c^2) with the unscaled N', D'; eps' = eps m bw^2.
//
// These kernels serve the fp32 configuration (a 1e-4 tolerance rules out 10-bit-mantissa tensor
// core inputs) and give every other path a second opinion.  Work is tiled as 32 tokens per step,
// one token per lane, eight warps splitting the other dimension of each small GEMM.
#include "common.cuh"

namespace wersa {
namespace {

constexpr int kXs = kD + 4;                 // row stride of 32 x 64 tiles in shared memory (floats)
template <int M> struct Smem {
  static constexpr int kRs = M + 4;         // row stride of the 32 x M feature tile
  static constexpr int wt = 0;                        // WT[M][64]  (W transposed)
  static constexpr int ss = wt + M * kD;              // Ss[M][64]  (S' or dS')
  static constexpr int zs = ss + M * kD;              // zs[M]
  static constexpr int xs = zs + M;                   // Xs[32][68]
  static constexpr int gs = xs + kSimtTile * kXs;     // Gs[32][68]
  static constexpr int rs = gs + kSimtTile * kXs;     // Rs[32][M+4]
  static constexpr int dd = rs + kSimtTile * kRs;     // Dd[32]
  static constexpr int dp = dd + 32;                  // Dp[8][32]
  static constexpr int total = dp + 8 * 32;
};

// W (d x m, row-major) -> WT[r][c] in shared memory as floats.
template <int M, typename T>
__device__ __forceinline__ void load_wt(const T* __restrict__ W, float* __restrict__ WT) {
  // consecutive threads take consecutive c: conflict-free shared stores, strided (cached) loads
  for (int i = threadIdx.x; i < kD * M; i += blockDim.x) {
    const int r = i / kD, c = i - r * kD;
    WT[i] = to_f32(W[(size_t)c * M + r]);
  }
}

// 32 x 64 tile of `src` (row-major, rows [row0, row0+32) of an n-row slab) -> dst[32][68].
template <typename T>
__device__ __forceinline__ void load_tile32(const T* __restrict__ src, int n, int row0,
                                            float* __restrict__ dst) {
  const int r = threadIdx.x >> 3, cg = threadIdx.x & 7;
  float v[8];
  if (row0 + r < n) {
    load8(src + (size_t)(row0 + r) * kD + cg * 8, v);
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = 0.f;
  }
  store8(dst + r * kXs + cg * 8, v);
}

// Rs[t][r] = ReLU(sum_c Xs[t][c] WT[r][c]) for the warp's share of the features.
template <int M>
__device__ __forceinline__ void gemm_project_relu(const float* __restrict__ Xs, const float* __restrict__ WT,
                                                  float* __restrict__ Rs) {
  constexpr int FW = M / 8;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float x[kD];
#pragma unroll
  for (int c4 = 0; c4 < kD / 4; ++c4) {
    const float4 v = *reinterpret_cast<const float4*>(Xs + lane * kXs + c4 * 4);
    x[c4 * 4] = v.x; x[c4 * 4 + 1] = v.y; x[c4 * 4 + 2] = v.z; x[c4 * 4 + 3] = v.w;
  }
  for (int r = warp * FW; r < (warp + 1) * FW; r += 4) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c4 = 0; c4 < kD / 4; ++c4) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4 w = *reinterpret_cast<const float4*>(WT + (r + k) * kD + c4 * 4);
        acc[k] = fmaf(x[c4 * 4], w.x, acc[k]);
        acc[k] = fmaf(x[c4 * 4 + 1], w.y, acc[k]);
        acc[k] = fmaf(x[c4 * 4 + 2], w.z, acc[k]);
        acc[k] = fmaf(x[c4 * 4 + 3], w.w, acc[k]);
      }
    }
    *reinterpret_cast<float4*>(Rs + lane * Smem<M>::kRs + r) =
        make_float4(fmaxf(acc[0], 0.f), fmaxf(acc[1], 0.f), fmaxf(acc[2], 0.f), fmaxf(acc[3], 0.f));
  }
}

// Feature ownership of the token-reduction GEMM: thread owns FR = M/32 features
// feat(j, v) = j*32*VW + lane*VW + v and the 8 columns warp*8 .. warp*8+7.
template <int M> struct Own {
  static constexpr int VW = (M >= 128) ? 4 : 2;
  static constexpr int NJ = M / (32 * VW);
  static constexpr int FR = NJ * VW;
};

// acc[f][c] += sum_t Rs[t][feat f] * Gs[t][warp*8+c];  zacc[f] += sum_t Rs[t][feat f] * Dd[t]
// (Dd == nullptr means all ones).
template <int M>
__device__ __forceinline__ void gemm_reduce_tokens(const float* __restrict__ Rs, const float* __restrict__ Gs,
                                                   const float* __restrict__ Dd,
                                                   float (&acc)[Own<M>::FR][8], float (&zacc)[Own<M>::FR]) {
  constexpr int VW = Own<M>::VW, NJ = Own<M>::NJ;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll 4
  for (int t = 0; t < kSimtTile; ++t) {
    const float4 g0 = *reinterpret_cast<const float4*>(Gs + t * kXs + warp * 8);
    const float4 g1 = *reinterpret_cast<const float4*>(Gs + t * kXs + warp * 8 + 4);
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    const float dt = Dd != nullptr ? Dd[t] : 1.f;
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      float rv[VW];
      const float* src = Rs + t * Smem<M>::kRs + j * 32 * VW + lane * VW;
      if constexpr (VW == 4) {
        const float4 v = *reinterpret_cast<const float4*>(src);
        rv[0] = v.x; rv[1] = v.y; rv[2] = v.z; rv[3] = v.w;
      } else {
        const float2 v = *reinterpret_cast<const float2*>(src);
        rv[0] = v.x; rv[1] = v.y;
      }
#pragma unroll
      for (int v = 0; v < VW; ++v) {
        zacc[j * VW + v] = fmaf(rv[v], dt, zacc[j * VW + v]);
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[j * VW + v][c] = fmaf(rv[v], g[c], acc[j * VW + v][c]);
      }
    }
  }
}

// out[c] = sum_r Rs[lane][r] * Bm[r][warp*8+c] (c < 8);  dot = sum_r Rs[lane][r] * zv[r]
// (zv == nullptr: dot = 0).  Bm is an M x 64 matrix in shared memory (S', dS' or WT).
template <int M>
__device__ __forceinline__ void gemm_contract_features(const float* __restrict__ Rs, const float* __restrict__ Bm,
                                                       const float* __restrict__ zv, float (&out)[8],
                                                       float& dot) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int c = 0; c < 8; ++c) out[c] = 0.f;
  dot = 0.f;
#pragma unroll 2
  for (int r = 0; r < M; r += 4) {
    const float4 rv4 = *reinterpret_cast<const float4*>(Rs + lane * Smem<M>::kRs + r);
    const float rv[4] = {rv4.x, rv4.y, rv4.z, rv4.w};
    if (zv != nullptr) {
      const float4 z4 = *reinterpret_cast<const float4*>(zv + r);
      dot = fmaf(rv[0], z4.x, dot);
      dot = fmaf(rv[1], z4.y, dot);
      dot = fmaf(rv[2], z4.z, dot);
      dot = fmaf(rv[3], z4.w, dot);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float4 b0 = *reinterpret_cast<const float4*>(Bm + (r + k) * kD + warp * 8);
      const float4 b1 = *reinterpret_cast<const float4*>(Bm + (r + k) * kD + warp * 8 + 4);
      out[0] = fmaf(rv[k], b0.x, out[0]); out[1] = fmaf(rv[k], b0.y, out[1]);
      out[2] = fmaf(rv[k], b0.z, out[2]); out[3] = fmaf(rv[k], b0.w, out[3]);
      out[4] = fmaf(rv[k], b1.x, out[4]); out[5] = fmaf(rv[k], b1.y, out[5]);
      out[6] = fmaf(rv[k], b1.z, out[6]); out[7] = fmaf(rv[k], b1.w, out[7]);
    }
  }
}

// Rs[t][r] <- (Rs[t][r] > 0) ? sum_c Gs[t][c] * Bm[r][c] + dd[t] * zv[r] : 0, warp's feature share.
// (Gradient with respect to the ReLU pre-activation.)  dd == nullptr means all ones.
template <int M>
__device__ __forceinline__ void gemm_feature_grad(const float* __restrict__ Gs, const float* __restrict__ Bm,
                                                  const float* __restrict__ zv, const float* __restrict__ Dd,
                                                  float* __restrict__ Rs) {
  constexpr int FW = M / 8;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float g[kD];
#pragma unroll
  for (int c4 = 0; c4 < kD / 4; ++c4) {
    const float4 v = *reinterpret_cast<const float4*>(Gs + lane * kXs + c4 * 4);
    g[c4 * 4] = v.x; g[c4 * 4 + 1] = v.y; g[c4 * 4 + 2] = v.z; g[c4 * 4 + 3] = v.w;
  }
  const float dt = Dd != nullptr ? Dd[lane] : 1.f;
  for (int r = warp * FW; r < (warp + 1) * FW; r += 4) {
    float acc[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) acc[k] = dt * zv[r + k];
#pragma unroll
    for (int c4 = 0; c4 < kD / 4; ++c4) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4 b = *reinterpret_cast<const float4*>(Bm + (r + k) * kD + c4 * 4);
        acc[k] = fmaf(g[c4 * 4], b.x, acc[k]);
        acc[k] = fmaf(g[c4 * 4 + 1], b.y, acc[k]);
        acc[k] = fmaf(g[c4 * 4 + 2], b.z, acc[k]);
        acc[k] = fmaf(g[c4 * 4 + 3], b.w, acc[k]);
      }
    }
    float4* p = reinterpret_cast<float4*>(Rs + lane * Smem<M>::kRs + r);
    const float4 act = *p;
    *p = make_float4(act.x > 0.f ? acc[0] : 0.f, act.y > 0.f ? acc[1] : 0.f, act.z > 0.f ? acc[2] : 0.f,
                     act.w > 0.f ? acc[3] : 0.f);
  }
}

template <int M>
__device__ __forceinline__ void store_partials(const float (&acc)[Own<M>::FR][8], const float (&zacc)[Own<M>::FR],
                                               float* __restrict__ sp, float* __restrict__ zp) {
  constexpr int VW = Own<M>::VW, NJ = Own<M>::NJ;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int j = 0; j < NJ; ++j)
#pragma unroll
    for (int v = 0; v < VW; ++v) {
      const int r = j * 32 * VW + lane * VW + v;
      float* dst = sp + (size_t)r * kD + warp * 8;
      *reinterpret_cast<float4*>(dst) =
          make_float4(acc[j * VW + v][0], acc[j * VW + v][1], acc[j * VW + v][2], acc[j * VW + v][3]);
      *reinterpret_cast<float4*>(dst + 4) =
          make_float4(acc[j * VW + v][4], acc[j * VW + v][5], acc[j * VW + v][6], acc[j * VW + v][7]);
      if (warp == 0) zp[r] = zacc[j * VW + v];
    }
}

// ---- forward, key side: partial S', z' of one sequence chunk.  grid (schunks, slabs) ----------
template <int M, typename T>
__global__ void __launch_bounds__(256) k_simt_kside(const float* __restrict__ KF, const T* __restrict__ V,
                                                    const T* __restrict__ W, float* __restrict__ spart,
                                                    float* __restrict__ zpart, int n, int chunk_tiles) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  extern __shared__ __align__(16) float sm[];
  using S = Smem<M>;
  float* WT = sm + S::wt;
  float* Xs = sm + S::xs;
  float* Gs = sm + S::gs;
  float* Rs = sm + S::rs;
  const int chunk = blockIdx.x, slab = blockIdx.y;
  load_wt<M>(W, WT);
  float acc[Own<M>::FR][8], zacc[Own<M>::FR];
#pragma unroll
  for (int f = 0; f < Own<M>::FR; ++f) {
    zacc[f] = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[f][c] = 0.f;
  }
  const float* kf = KF + (size_t)slab * n * kD;
  const T* v = V + (size_t)slab * n * kD;
  const int tile0 = chunk * chunk_tiles;
  for (int ti = 0; ti < chunk_tiles; ++ti) {
    const int row0 = (tile0 + ti) * kSimtTile;
    if (row0 >= n) break;
    __syncthreads();
    load_tile32(kf, n, row0, Xs);
    load_tile32(v, n, row0, Gs);
    __syncthreads();
    gemm_project_relu<M>(Xs, WT, Rs);
    __syncthreads();
    gemm_reduce_tokens<M>(Rs, Gs, nullptr, acc, zacc);
  }
  const size_t pidx = (size_t)slab * gridDim.x + chunk;
  store_partials<M>(acc, zacc, spart + pidx * M * kD, zpart + pidx * M);
}

// ---- forward, query side.  grid (schunks, slabs) --------------------------------------------------
template <int M, typename T>
__global__ void __launch_bounds__(256) k_simt_qside(const float* __restrict__ QF, const T* __restrict__ W,
                                                    const float* __restrict__ Sg, const float* __restrict__ zg,
                                                    const float* __restrict__ beta, float eps, float bw_floor,
                                                    T* __restrict__ O, int n, int chunk_tiles) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  extern __shared__ __align__(16) float sm[];
  using S = Smem<M>;
  float* WT = sm + S::wt;
  float* Ss = sm + S::ss;
  float* zs = sm + S::zs;
  float* Xs = sm + S::xs;
  float* Rs = sm + S::rs;
  const int chunk = blockIdx.x, slab = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  load_wt<M>(W, WT);
  for (int i = threadIdx.x; i < M * kD; i += blockDim.x) Ss[i] = Sg[(size_t)slab * M * kD + i];
  for (int i = threadIdx.x; i < M; i += blockDim.x) zs[i] = zg[(size_t)slab * M + i];
  const float bw = fmaxf(beta[0], bw_floor);
  const float epsp = eps * (float)M * bw * bw;
  const float* qf = QF + (size_t)slab * n * kD;
  T* o = O + (size_t)slab * n * kD;
  const int tile0 = chunk * chunk_tiles;
  for (int ti = 0; ti < chunk_tiles; ++ti) {
    const int row0 = (tile0 + ti) * kSimtTile;
    if (row0 >= n) break;
    __syncthreads();
    load_tile32(qf, n, row0, Xs);
    __syncthreads();
    gemm_project_relu<M>(Xs, WT, Rs);
    __syncthreads();
    float num[8], den;
    gemm_contract_features<M>(Rs, Ss, zs, num, den);
    const float inv = 1.f / (den + epsp);
#pragma unroll
    for (int c = 0; c < 8; ++c) num[c] *= inv;
    if (row0 + lane < n) store8(o + (size_t)(row0 + lane) * kD + warp * 8, num);
  }
}

// ---- backward, query side.  grid (schunks, slabs) ------------------------------------------------
// Per tile: recompute R = ReLU(Q_F W), N', Dh = D' + eps', O; dN' = dO/Dh; dDh = -sum_c dO O / Dh;
// dS' += R^T dN'; dz' += R^T dDh; dA = (dN' S'^T + dDh z'^T) (.) 1[R > 0]; dQ_F = dA W^T.
template <int M, typename T>
__global__ void __launch_bounds__(256) k_simt_bwd_qside(
    const float* __restrict__ QF, const T* __restrict__ W, const float* __restrict__ Sg,
    const float* __restrict__ zg, const float* __restrict__ beta, float eps, float bw_floor,
    const T* __restrict__ dO, float* __restrict__ dQF, float* __restrict__ dspart, float* __restrict__ dzpart,
    float* __restrict__ sumdD, int n, int chunk_tiles) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  extern __shared__ __align__(16) float sm[];
  using S = Smem<M>;
  float* WT = sm + S::wt;
  float* Ss = sm + S::ss;
  float* zs = sm + S::zs;
  float* Xs = sm + S::xs;
  float* Gs = sm + S::gs;
  float* Rs = sm + S::rs;
  float* Dd = sm + S::dd;
  float* Dp = sm + S::dp;
  const int chunk = blockIdx.x, slab = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  load_wt<M>(W, WT);
  for (int i = threadIdx.x; i < M * kD; i += blockDim.x) Ss[i] = Sg[(size_t)slab * M * kD + i];
  for (int i = threadIdx.x; i < M; i += blockDim.x) zs[i] = zg[(size_t)slab * M + i];
  const float bw = fmaxf(beta[0], bw_floor);
  const float epsp = eps * (float)M * bw * bw;
  float acc[Own<M>::FR][8], zacc[Own<M>::FR];
#pragma unroll
  for (int f = 0; f < Own<M>::FR; ++f) {
    zacc[f] = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[f][c] = 0.f;
  }
  float sum_dd = 0.f;   // warp 0, lane t: sum over tiles of dDh of token t
  const float* qf = QF + (size_t)slab * n * kD;
  const T* go = dO + (size_t)slab * n * kD;
  float* dqf = dQF + (size_t)slab * n * kD;
  const int tile0 = chunk * chunk_tiles;
  for (int ti = 0; ti < chunk_tiles; ++ti) {
    const int row0 = (tile0 + ti) * kSimtTile;
    if (row0 >= n) break;
    __syncthreads();
    load_tile32(qf, n, row0, Xs);
    load_tile32(go, n, row0, Gs);
    __syncthreads();
    gemm_project_relu<M>(Xs, WT, Rs);
    __syncthreads();
    float num[8], den;
    gemm_contract_features<M>(Rs, Ss, zs, num, den);
    const float inv = 1.f / (den + epsp);
    float part = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const float g = Gs[lane * kXs + warp * 8 + c];
      part = fmaf(g, num[c] * inv, part);
      Gs[lane * kXs + warp * 8 + c] = g * inv;    // dN'
    }
    Dp[warp * 32 + lane] = part;
    __syncthreads();
    if (warp == 0) {
      float tot = 0.f;
#pragma unroll
      for (int wi = 0; wi < 8; ++wi) tot += Dp[wi * 32 + lane];
      const float dd = -tot * inv;               // every warp computed the same `inv` for this token
      Dd[lane] = dd;
      sum_dd += dd;
    }
    __syncthreads();
    gemm_reduce_tokens<M>(Rs, Gs, Dd, acc, zacc);
    __syncthreads();
    gemm_feature_grad<M>(Gs, Ss, zs, Dd, Rs);
    __syncthreads();
    float gx[8], unused;
    gemm_contract_features<M>(Rs, WT, nullptr, gx, unused);
    if (row0 + lane < n) store8(dqf + (size_t)(row0 + lane) * kD + warp * 8, gx);
  }
  const size_t pidx = (size_t)slab * gridDim.x + chunk;
  store_partials<M>(acc, zacc, dspart + pidx * M * kD, dzpart + pidx * M);
  if (warp == 0) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum_dd += __shfl_xor_sync(0xffffffffu, sum_dd, o);
    if (lane == 0) sumdD[pidx] = sum_dd;
  }
}

// ---- backward, key side.  grid (schunks, slabs) ---------------------------------------------------
// Per tile: R = ReLU(K_F W); dV = R dS'; dB = (V dS'^T + 1 dz'^T) (.) 1[R > 0]; dK_F = dB W^T.
template <int M, typename T, typename TG>
__global__ void __launch_bounds__(256) k_simt_bwd_kside(const float* __restrict__ KF, const T* __restrict__ V,
                                                        const T* __restrict__ W, const float* __restrict__ dSg,
                                                        const float* __restrict__ dzg, TG* __restrict__ dV,
                                                        float* __restrict__ dKF, int n, int chunk_tiles) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  extern __shared__ __align__(16) float sm[];
  using S = Smem<M>;
  float* WT = sm + S::wt;
  float* Ss = sm + S::ss;
  float* zs = sm + S::zs;
  float* Xs = sm + S::xs;
  float* Gs = sm + S::gs;
  float* Rs = sm + S::rs;
  const int chunk = blockIdx.x, slab = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  load_wt<M>(W, WT);
  for (int i = threadIdx.x; i < M * kD; i += blockDim.x) Ss[i] = dSg[(size_t)slab * M * kD + i];
  for (int i = threadIdx.x; i < M; i += blockDim.x) zs[i] = dzg[(size_t)slab * M + i];
  const float* kf = KF + (size_t)slab * n * kD;
  const T* v = V + (size_t)slab * n * kD;
  TG* dv = dV + (size_t)slab * n * kD;
  float* dkf = dKF + (size_t)slab * n * kD;
  const int tile0 = chunk * chunk_tiles;
  for (int ti = 0; ti < chunk_tiles; ++ti) {
    const int row0 = (tile0 + ti) * kSimtTile;
    if (row0 >= n) break;
    __syncthreads();
    load_tile32(kf, n, row0, Xs);
    load_tile32(v, n, row0, Gs);
    __syncthreads();
    gemm_project_relu<M>(Xs, WT, Rs);
    __syncthreads();
    float out[8], unused;
    gemm_contract_features<M>(Rs, Ss, nullptr, out, unused);
    if (row0 + lane < n) store8(dv + (size_t)(row0 + lane) * kD + warp * 8, out);
    __syncthreads();
    gemm_feature_grad<M>(Gs, Ss, zs, nullptr, Rs);
    __syncthreads();
    gemm_contract_features<M>(Rs, WT, nullptr, out, unused);
    if (row0 + lane < n) store8(dkf + (size_t)(row0 + lane) * kD + warp * 8, out);
  }
}

// S[slab][i] = sum over chunks of part[slab][chunk][i], always in the same order: four running sums
// take the chunks k = 0, 1, 2, 3 (mod 4) in increasing k (four loads in flight instead of one) and are
// added as (a0 + a1) + (a2 + a3).  One thread per element of [S | z].
__device__ __forceinline__ float sum_chunks4(const float* __restrict__ p, size_t stride, int chunks) {
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
  int k = 0;
  for (; k + 4 <= chunks; k += 4) {
    a0 += p[(size_t)k * stride];
    a1 += p[(size_t)(k + 1) * stride];
    a2 += p[(size_t)(k + 2) * stride];
    a3 += p[(size_t)(k + 3) * stride];
  }
  if (k < chunks) a0 += p[(size_t)k * stride];
  if (k + 1 < chunks) a1 += p[(size_t)(k + 1) * stride];
  if (k + 2 < chunks) a2 += p[(size_t)(k + 2) * stride];
  return (a0 + a1) + (a2 + a3);
}

// grid (m / 8, slabs), block 512: one CTA adds the partials of eight consecutive features (512 elements of
// S', one per thread, and their eight entries of z') in chunk order.  With Sbf it also leaves the bf16 copy
// of S', with Simg the operand image of the query-side kernel (see simg_offset): eight consecutive features
// are one 16-byte chunk of an image row, so the 80 rows of the CTA's part go out as one 16-byte store each.
__global__ void __launch_bounds__(512) k_reduce_partials(const float* __restrict__ spart,
                                                         const float* __restrict__ zpart, int chunks, int m,
                                                         float* __restrict__ S, float* __restrict__ z,
                                                         __nv_bfloat16* __restrict__ Sbf, uint8_t* __restrict__ Simg) {
  // Programmatic dependent launch: the kernel after this one may be staged now (it waits for this grid
  // before it reads S, z, Sbf, Simg), and this kernel may itself have been staged early: the partials are
  // complete once the kernel before it has finished.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  __shared__ __align__(16) __nv_bfloat16 tile[kSimgRows][8];   // [image row][feature - f0]
  const int slab = blockIdx.y, f0 = blockIdx.x * 8;
  const int ns = m * kD;
  {
    const int e = threadIdx.x;                    // element of the CTA's 8 x 64 part
    const int i = f0 * kD + e;                    // element of S' (feature i / 64, column i % 64)
    const float s = sum_chunks4(spart + (size_t)slab * chunks * ns + i, ns, chunks);
    S[(size_t)slab * ns + i] = s;
    const __nv_bfloat16 sb = __float2bfloat16_rn(s);
    if (Sbf != nullptr) Sbf[(size_t)slab * ns + i] = sb;
    tile[e & (kD - 1)][e >> 6] = sb;
  }
  if (threadIdx.x < 8) {
    const int r = f0 + threadIdx.x;
    const float zr = sum_chunks4(zpart + (size_t)slab * chunks * m + r, m, chunks);
    z[(size_t)slab * m + r] = zr;
    tile[kD][threadIdx.x] = __float2bfloat16_rn(zr);   // z' is row 64 of the image
  } else if (threadIdx.x < 8 * (kSimgRows - kD)) {
    tile[kD + (threadIdx.x >> 3)][threadIdx.x & 7] = __float2bfloat16_rn(0.f);   // rows 65-79 are zero
  }
  if (Simg == nullptr) return;
  __syncthreads();
  if (threadIdx.x < kSimgRows)
    *reinterpret_cast<uint4*>(Simg + (size_t)slab * simg_bytes(m) + simg_offset(f0, threadIdx.x)) =
        *reinterpret_cast<const uint4*>(&tile[threadIdx.x][0]);
}

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

#define WERSA_DISPATCH_M(m, ...)                             \
  switch (m) {                                               \
    case 64: { constexpr int MM = 64; __VA_ARGS__; } break;   \
    case 128: { constexpr int MM = 128; __VA_ARGS__; } break; \
    case 256: { constexpr int MM = 256; __VA_ARGS__; } break; \
    default: return cudaErrorInvalidValue;                   \
  }

}  // namespace

cudaError_t launch_simt_kside(const Plan& p, const Ws& w, const void* V, const void* W, cudaStream_t st,
                              int* launches) {
  dim3 grid(p.schunks, p.slabs);
  const int n = p.cfg.seq_len;
  cudaError_t err = cudaSuccess;
  WERSA_DISPATCH_M(p.cfg.features, {
    const size_t bytes = sizeof(float) * Smem<MM>::total;
    if (p.bf16) {
      auto k = k_simt_kside<MM, __nv_bfloat16>;
      if ((err = set_smem(k, bytes)) != cudaSuccess) return err;
      launch_after(k, dim3(grid), dim3(256), bytes, st, w.KF, (const __nv_bfloat16*)V, (const __nv_bfloat16*)W, w.spart, w.zpart, n,
                                  p.schunk_tiles);
    } else {
      auto k = k_simt_kside<MM, float>;
      if ((err = set_smem(k, bytes)) != cudaSuccess) return err;
      launch_after(k, dim3(grid), dim3(256), bytes, st, w.KF, (const float*)V, (const float*)W, w.spart, w.zpart, n, p.schunk_tiles);
    }
  });
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_reduce_partials(const Plan& p, const float* spart, const float* zpart, int chunks, float* S,
                                   float* z, __nv_bfloat16* Sbf, uint8_t* Simg, cudaStream_t st, int* launches) {
  const int m = p.cfg.features;
  dim3 grid(m / 8, p.slabs);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(512);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t err = cudaLaunchKernelEx(&cfg, k_reduce_partials, spart, zpart, chunks, m, S, z, Sbf, Simg);
  *launches += 1;
  return err != cudaSuccess ? err : cudaGetLastError();
}

cudaError_t launch_simt_qside(const Plan& p, const Ws& w, const void* W, const float* beta, void* O,
                              cudaStream_t st, int* launches) {
  dim3 grid(p.schunks, p.slabs);
  const int n = p.cfg.seq_len;
  cudaError_t err = cudaSuccess;
  WERSA_DISPATCH_M(p.cfg.features, {
    const size_t bytes = sizeof(float) * Smem<MM>::total;
    if (p.bf16) {
      auto k = k_simt_qside<MM, __nv_bfloat16>;
      if ((err = set_smem(k, bytes)) != cudaSuccess) return err;
      launch_after(k, dim3(grid), dim3(256), bytes, st, w.QF, (const __nv_bfloat16*)W, w.S, w.z, beta, p.cfg.eps, p.cfg.bw_floor,
                                  (__nv_bfloat16*)O, n, p.schunk_tiles);
    } else {
      auto k = k_simt_qside<MM, float>;
      if ((err = set_smem(k, bytes)) != cudaSuccess) return err;
      launch_after(k, dim3(grid), dim3(256), bytes, st, w.QF, (const float*)W, w.S, w.z, beta, p.cfg.eps, p.cfg.bw_floor, (float*)O, n,
                                  p.schunk_tiles);
    }
  });
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_simt_bwd_qside(const Plan& p, const Ws& w, const void* W, const float* beta, const void* dO,
                                  cudaStream_t st, int* launches) {
  dim3 grid(p.schunks, p.slabs);
  const int n = p.cfg.seq_len;
  cudaError_t err = cudaSuccess;
  WERSA_DISPATCH_M(p.cfg.features, {
    const size_t bytes = sizeof(float) * Smem<MM>::total;
    if (p.bf16) {
      auto k = k_simt_bwd_qside<MM, __nv_bfloat16>;
      if ((err = set_smem(k, bytes)) != cudaSuccess) return err;
      launch_after(k, dim3(grid), dim3(256), bytes, st, w.QF, (const __nv_bfloat16*)W, w.S, w.z, beta, p.cfg.eps, p.cfg.bw_floor,
                                  (const __nv_bfloat16*)dO, w.dQF, w.spart, w.zpart, w.sumdD, n, p.schunk_tiles);
    } else {
      auto k = k_simt_bwd_qside<MM, float>;
      if ((err = set_smem(k, bytes)) != cudaSuccess) return err;
      launch_after(k, dim3(grid), dim3(256), bytes, st, w.QF, (const float*)W, w.S, w.z, beta, p.cfg.eps, p.cfg.bw_floor,
                                  (const float*)dO, w.dQF, w.spart, w.zpart, w.sumdD, n, p.schunk_tiles);
    }
  });
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_simt_bwd_kside(const Plan& p, const Ws& w, const void* V, const void* W, void* dV,
                                  cudaStream_t st, int* launches) {
  dim3 grid(p.schunks, p.slabs);
  const int n = p.cfg.seq_len;
  cudaError_t err = cudaSuccess;
  WERSA_DISPATCH_M(p.cfg.features, {
    const size_t bytes = sizeof(float) * Smem<MM>::total;
    if (p.bf16 && p.grad_bf16) {
      auto k = k_simt_bwd_kside<MM, __nv_bfloat16, __nv_bfloat16>;
      if ((err = set_smem(k, bytes)) != cudaSuccess) return err;
      launch_after(k, dim3(grid), dim3(256), bytes, st, w.KF, (const __nv_bfloat16*)V, (const __nv_bfloat16*)W, w.dS, w.dz,
                                  (__nv_bfloat16*)dV, w.dKF, n, p.schunk_tiles);
    } else if (p.bf16) {
      auto k = k_simt_bwd_kside<MM, __nv_bfloat16, float>;
      if ((err = set_smem(k, bytes)) != cudaSuccess) return err;
      launch_after(k, dim3(grid), dim3(256), bytes, st, w.KF, (const __nv_bfloat16*)V, (const __nv_bfloat16*)W, w.dS, w.dz, (float*)dV,
                                  w.dKF, n, p.schunk_tiles);
    } else if (p.grad_bf16) {
      auto k = k_simt_bwd_kside<MM, float, __nv_bfloat16>;
      if ((err = set_smem(k, bytes)) != cudaSuccess) return err;
      launch_after(k, dim3(grid), dim3(256), bytes, st, w.KF, (const float*)V, (const float*)W, w.dS, w.dz, (__nv_bfloat16*)dV, w.dKF,
                                  n, p.schunk_tiles);
    } else {
      auto k = k_simt_bwd_kside<MM, float, float>;
      if ((err = set_smem(k, bytes)) != cudaSuccess) return err;
      launch_after(k, dim3(grid), dim3(256), bytes, st, w.KF, (const float*)V, (const float*)W, w.dS, w.dz, (float*)dV, w.dKF, n,
                                  p.schunk_tiles);
    }
  });
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace wersa
