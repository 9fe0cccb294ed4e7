// Layout kernels around the 64-wide, at most 256-feature kernels:
//  * head dimensions below 64 run as the zero-padded 64-wide problem (zero columns of Q, K, V and zero rows of
//    W change nothing in Eqs. 1-7: the projections, the pooled logits and the first d columns of the output
//    are those of the narrow problem, the other output columns are zero);
//  * feature maps wider than 256 run as groups of 256 features.  With N'_g, D'_g the numerator and
//    denominator of group g (Eq. 7 restricted to the group's features) and eps' shared out evenly,
//    O = sum_g N'_g / sum_g (D'_g + eps'/G) = sum_g O_g den_g / sum_g den_g, where O_g = N'_g / den_g is what
//    the query-side kernel writes for the group and den_g = D'_g + eps'/G is the denominator it leaves beside it.
#include "common.cuh"

namespace wersa {
namespace {

// dst[row][0..63] = src[row][0..d) followed by zeros.  One thread per 8 elements of dst.
template <typename T>
__global__ void __launch_bounds__(256) k_pad_cols(const T* __restrict__ src, T* __restrict__ dst, size_t rows, int d) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
  const size_t row = idx >> 3;
  const int c0 = (int)(idx & 7) * 8;
  if (row >= rows) return;
  float v[8];
  if (c0 < d) {
    load8(src + row * d + c0, v);
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = 0.f;
  }
  store8(dst + row * kD + c0, v);
}

// dst[row][0..d) = src[row][0..d) of a 64-wide source.
template <typename T>
__global__ void __launch_bounds__(256) k_unpad_cols(const T* __restrict__ src, T* __restrict__ dst, size_t rows, int d) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
  const size_t row = idx >> 3;
  const int c0 = (int)(idx & 7) * 8;
  if (row >= rows || c0 >= d) return;
  float v[8];
  load8(src + row * kD + c0, v);
  store8(dst + row * d + c0, v);
}

// O[tok][:] = sum_g Og[g][tok][:] * den[g][tok] / sum_g den[g][tok], groups in a fixed order.  Og is 64 wide,
// O has `cols` columns.  One thread per 8 columns of a token; tokens = slabs * n.
template <typename T>
__global__ void __launch_bounds__(256) k_combine_groups(const T* __restrict__ Og, const float* __restrict__ den,
                                                        T* __restrict__ O, size_t tokens, int groups, int cols) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
  const size_t tok = idx >> 3;
  const int c0 = (int)(idx & 7) * 8;
  if (tok >= tokens || c0 >= cols) return;
  float acc[8], dsum = 0.f;
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  for (int g = 0; g < groups; ++g) {
    const float dg = den[(size_t)g * tokens + tok];
    float v[8];
    load8(Og + ((size_t)g * tokens + tok) * kD + c0, v);
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = fmaf(v[j], dg, acc[j]);
    dsum += dg;
  }
  const float inv = 1.f / dsum;
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] *= inv;
  store8(O + tok * cols + c0, acc);
}

// One token per 8 threads (8 columns each): O = sum_g Og den_g / sum_g den_g, D = sum_g den_g / r,
// dD' = -(dO . O) / D.  The forward's denominators carry the factor r = bf16(f_0) / f_0 of its filter stage,
// which the backward's filtered planes do not.
template <typename T>
__global__ void __launch_bounds__(256) k_group_bwd_prep(const T* __restrict__ Og, const float* __restrict__ den,
                                                        const T* __restrict__ dO, const float* __restrict__ f, int n,
                                                        int L1, size_t tokens, int groups, float* __restrict__ Dtot,
                                                        float* __restrict__ dDtot) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
  const size_t tok = idx >> 3;
  const int c0 = (int)(idx & 7) * 8;
  const bool live = tok < tokens;
  float acc[8], dsum = 0.f;
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  float dot = 0.f;
  if (live) {
    for (int g = 0; g < groups; ++g) {
      const float dg = den[(size_t)g * tokens + tok];
      float v[8];
      load8(Og + ((size_t)g * tokens + tok) * kD + c0, v);
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = fmaf(v[j], dg, acc[j]);
      dsum += dg;
    }
    float g8[8];
    load8(dO + tok * kD + c0, g8);
#pragma unroll
    for (int j = 0; j < 8; ++j) dot = fmaf(g8[j], acc[j], dot);
  }
#pragma unroll
  for (int o = 4; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);   // the 8 threads of a token
  if (live && c0 == 0) {
    const float f0 = f[(tok / n) * L1];
    const float f0b = __bfloat162float(__float2bfloat16_rn(f0));
    const float r = f0 != 0.f ? f0b / f0 : 1.f;
    const float D = dsum / r;
    // dot = sum_c dO_c (sum_g Og_c den_g); O = that / dsum
    Dtot[tok] = D;
    dDtot[tok] = -(dot / dsum) / D;
  }
}

// Group-major S' and z' (as the kernels leave them: [group][slab][256][...]) -> slab-major [slab][m][...].
__global__ void __launch_bounds__(256) k_gather_groups(const float* __restrict__ Sg, const float* __restrict__ zg,
                                                       float* __restrict__ S, float* __restrict__ z, int slabs,
                                                       int groups, int mg) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;   // one float4 of S
  const size_t total4 = (size_t)slabs * groups * mg * (kD / 4);
  if (idx >= total4) return;
  const int c4 = (int)(idx % (kD / 4));
  const size_t row = idx / (kD / 4);            // slab-major row: slab * m + g * mg + r
  const int m = groups * mg;
  const int slab = (int)(row / m), f = (int)(row % m), g = f / mg, r = f % mg;
  const size_t src_row = ((size_t)g * slabs + slab) * mg + r;
  reinterpret_cast<float4*>(S)[row * (kD / 4) + c4] = reinterpret_cast<const float4*>(Sg)[src_row * (kD / 4) + c4];
  if (c4 == 0) z[row] = zg[src_row];
}

unsigned blocks_for(size_t threads) { return (unsigned)((threads + 255) / 256); }

}  // namespace

cudaError_t launch_pad_cols(const void* src, void* dst, size_t rows, int d, int kind, cudaStream_t st, int* launches) {
  if (kind == 1)
    launch_after(k_pad_cols<__nv_bfloat16>, dim3(blocks_for(rows * 8)), dim3(256), 0, st, (const __nv_bfloat16*)src, (__nv_bfloat16*)dst, rows, d);
  else
    launch_after(k_pad_cols<float>, dim3(blocks_for(rows * 8)), dim3(256), 0, st, (const float*)src, (float*)dst, rows, d);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_unpad_cols(const void* src, void* dst, size_t rows, int d, int kind, cudaStream_t st,
                              int* launches) {
  if (kind == 1)
    launch_after(k_unpad_cols<__nv_bfloat16>, dim3(blocks_for(rows * 8)), dim3(256), 0, st, (const __nv_bfloat16*)src, (__nv_bfloat16*)dst, rows,
                                                                     d);
  else
    launch_after(k_unpad_cols<float>, dim3(blocks_for(rows * 8)), dim3(256), 0, st, (const float*)src, (float*)dst, rows, d);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_combine_groups(const void* Og, const float* den, void* O, size_t tokens, int groups, int cols,
                                  int kind, cudaStream_t st, int* launches) {
  if (kind == 1)
    launch_after(k_combine_groups<__nv_bfloat16>, dim3(blocks_for(tokens * 8)), dim3(256), 0, st, (const __nv_bfloat16*)Og, den,
                                                                           (__nv_bfloat16*)O, tokens, groups, cols);
  else
    launch_after(k_combine_groups<float>, dim3(blocks_for(tokens * 8)), dim3(256), 0, st, (const float*)Og, den, (float*)O, tokens, groups,
                                                                   cols);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_group_bwd_prep(const void* Og, const float* den, const void* dO, const float* f, int n, int L1,
                                  size_t tokens, int groups, int kind, float* Dtot, float* dDtot, cudaStream_t st,
                                  int* launches) {
  if (kind == 1)
    launch_after(k_group_bwd_prep<__nv_bfloat16>, dim3(blocks_for(tokens * 8)), dim3(256), 0, st, 
        (const __nv_bfloat16*)Og, den, (const __nv_bfloat16*)dO, f, n, L1, tokens, groups, Dtot, dDtot);
  else
    launch_after(k_group_bwd_prep<float>, dim3(blocks_for(tokens * 8)), dim3(256), 0, st, (const float*)Og, den, (const float*)dO, f, n, L1,
                                                                   tokens, groups, Dtot, dDtot);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_gather_groups(const float* Sg, const float* zg, float* S, float* z, int slabs, int groups, int mg,
                                 cudaStream_t st, int* launches) {
  const size_t total4 = (size_t)slabs * groups * mg * (kD / 4);
  launch_after(k_gather_groups, dim3(blocks_for(total4)), dim3(256), 0, st, Sg, zg, S, z, slabs, groups, mg);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace wersa
