// Mean-pooled query, content-adaptive gate (Eqs. 1-3 of the WERSA paper) and its backward pass.
#include <mutex>

#include "common.cuh"

namespace wersa {
namespace {

// Scratch of wersa_gate_static: lives in the library image of every GPU that loads it.  The last
// kStaticCounterInts elements are reserved for the arrival counters, at a place that does not depend on
// the problem, so that no float of any call's layout can ever land on them.
constexpr size_t kStaticScratchFloats = 262144;   // 1 MiB
constexpr size_t kStaticCounterInts = 8192;       // slab counters, then batch counters
static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];
constexpr int kMaxDevices = 64;
float* g_static_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_static_scratch_mutex;

// Finish of one slab by the last CTA of that slab to arrive (256 threads): qbar = sum of the chunk
// partials in chunk order / n (Eq. 1), the head's logits u = gate_w[h]^T qbar (Eq. 2) and, for the
// per-head gate, sigmoid(u + gate_b[h]) and f = sigmoid * omega (Eq. 3).  For the batch-wide gate the
// bias-free logits are parked in f for batch_gate.
__device__ __forceinline__ void slab_gate(const float* __restrict__ qpart, int qchunks, int slab, int H, int n, int L1,
                                          int per_head, const float* __restrict__ gate_w,
                                          const float* __restrict__ gate_b, const float* __restrict__ omega,
                                          float* __restrict__ qbar, float* __restrict__ sg, float* __restrict__ f,
                                          float (*red)[kD], float* qs, int dcols) {
  const int h = slab % H;
  const int c = threadIdx.x & (kD - 1), part = threadIdx.x >> 6;   // 4 interleaved partial sums per column
  float s = 0.f;
  const float* src = qpart + (size_t)slab * qchunks * kD + c;
  int k = part;
  for (; k + 12 < qchunks; k += 16) {
    const float v0 = __ldcg(src + (size_t)k * kD), v1 = __ldcg(src + (size_t)(k + 4) * kD);
    const float v2 = __ldcg(src + (size_t)(k + 8) * kD), v3 = __ldcg(src + (size_t)(k + 12) * kD);
    s += (v0 + v1) + (v2 + v3);
  }
  for (; k < qchunks; k += 4) s += __ldcg(src + (size_t)k * kD);
  red[part][c] = s;
  __syncthreads();
  if (threadIdx.x < kD) {
    const float q = ((red[0][c] + red[1][c]) + (red[2][c] + red[3][c])) / (float)n;
    qbar[(size_t)slab * kD + c] = q;
    qs[c] = q;
  }
  __syncthreads();
  // logits: 16 lanes per band, four of the 64 terms each, then a fixed-order butterfly
  const int i = threadIdx.x >> 4, seg = threadIdx.x & 15;
  float u = 0.f;
  if (gate_w != nullptr && i < L1) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int kk = seg * 4 + j;   // gate_w is (heads, dcols, L1); columns >= dcols of qbar are zero padding
      if (kk < dcols) u += gate_w[((size_t)h * dcols + kk) * L1 + i] * qs[kk];
    }
  }
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) u += __shfl_xor_sync(0xffffffffu, u, o);
  if (i < L1 && seg == 0) {
    if (per_head) {
      if (gate_b != nullptr) u += gate_b[h * L1 + i];
      const float sgm = 1.f / (1.f + expf(-u));
      sg[(size_t)slab * L1 + i] = sgm;
      f[(size_t)slab * L1 + i] = sgm * (omega != nullptr ? omega[i] : 1.f);
    } else {
      f[(size_t)slab * L1 + i] = u;
    }
  }
}

// Batch-wide gate (Algorithm 1, W_filter), by the last slab of a batch element to finish:
// u[b] = sum_h u[b,h] + gate_b[0], one sigmoid per batch element shared by its heads.
__device__ __forceinline__ void batch_gate(int b, int H, int L1, const float* __restrict__ gate_b,
                                           const float* __restrict__ omega, float* __restrict__ sg,
                                           float* __restrict__ f) {
  const int i = threadIdx.x;
  if (i >= L1) return;
  float u = gate_b != nullptr ? gate_b[i] : 0.f;
  for (int h = 0; h < H; ++h) u += __ldcg(f + ((size_t)b * H + h) * L1 + i);
  const float sgm = 1.f / (1.f + expf(-u));
  for (int h = 0; h < H; ++h) {
    sg[((size_t)b * H + h) * L1 + i] = sgm;
    f[((size_t)b * H + h) * L1 + i] = sgm * (omega != nullptr ? omega[i] : 1.f);
  }
}

// Mean pool and gate in one launch.  grid (qchunks, slabs [+ 1]), block 256.
// Rows y < slabs: partial column sums of one row chunk of one slab of Q -- thread (cg = tid & 7,
// rl = tid >> 3) owns 8 consecutive columns and every 32nd row, loads 16 bytes (bf16) / 32 bytes
// (fp32) per row, four rows in flight, with the streaming cache hint (Q is read once here).  The CTA that finds it is the last of its slab to finish
// (a counter per slab) then runs slab_gate, and for the batch-wide gate the last slab of a batch
// element (a counter per batch element) runs batch_gate; sums are taken in a fixed order, so the
// result does not depend on which CTA comes last.  The counters start at zero and are left at zero.
// Row y == slabs (only with W != nullptr): bf16 transpose Wt (m x 64) of W (64 x m) for the
// tensor-core kernels.
// kFull = false: Q has dcols < 64 columns (a multiple of 8), gate_w dcols rows per head and W dcols rows;
// dcols / 8 threads share a row, 256 / (dcols / 8) rows are in flight per pass, and the partial sums, q-bar
// and W^T come out 64 wide with zeros in the columns past dcols.
template <typename T, bool kFull>
__global__ void __launch_bounds__(256) k_qmean_gate(const T* __restrict__ Q, float* __restrict__ qpart, int n,
                                                    int chunk_rows, int slabs, int H, int L1, int per_head,
                                                    const float* __restrict__ gate_w, const float* __restrict__ gate_b,
                                                    const float* __restrict__ omega, float* __restrict__ qbar,
                                                    float* __restrict__ sg, float* __restrict__ f,
                                                    int* __restrict__ slab_count, int* __restrict__ batch_count,
                                                    const __nv_bfloat16* __restrict__ W, __nv_bfloat16* __restrict__ Wt,
                                                    int m, int dcols_arg) {
  const int dcols = kFull ? kD : dcols_arg;
  // This grid may have been placed while the work before it in the stream was still running: nothing is
  // read or written before that work has completed.  After that the key-side kernel may be staged
  // (programmatic dependent launch; it waits for this grid before it reads W^T or the gate).
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if ((int)blockIdx.y == slabs) {
    for (int i = blockIdx.x * 256 + threadIdx.x; i < m * kD; i += gridDim.x * 256) {
      const int r = i / kD, c = i - r * kD;
      Wt[i] = c < dcols ? W[(size_t)c * m + r] : __float2bfloat16_rn(0.f);
    }
    return;
  }
  const int chunk = blockIdx.x, slab = blockIdx.y;
  const int cgs = kFull ? 8 : dcols >> 3;      // threads across a row
  const int rp = kFull ? 32 : 256 / cgs;       // rows per pass
  const int cg = kFull ? (threadIdx.x & 7) : (int)threadIdx.x % cgs;
  const int rl = kFull ? (threadIdx.x >> 3) : (int)threadIdx.x / cgs;
  const int r0 = chunk * chunk_rows;
  const int r1 = min(n, r0 + chunk_rows);
  const T* base = Q + (size_t)slab * n * dcols + cg * 8;
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  int r = rl < rp ? r0 + rl : r1;              // (256 need not be a multiple of cgs: the last threads idle)
  for (; r + 3 * rp < r1; r += 4 * rp) {
    float v0[8], v1[8], v2[8], v3[8];
    load8_stream(base + (size_t)r * dcols, v0);
    load8_stream(base + (size_t)(r + rp) * dcols, v1);
    load8_stream(base + (size_t)(r + 2 * rp) * dcols, v2);
    load8_stream(base + (size_t)(r + 3 * rp) * dcols, v3);
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] += (v0[j] + v1[j]) + (v2[j] + v3[j]);
  }
  for (; r < r1; r += rp) {
    float v0[8];
    load8_stream(base + (size_t)r * dcols, v0);
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] += v0[j];
  }
  __shared__ float red[kFull ? 32 * (kD + 1) : 256 * 9];   // rp rows of dcols + 1 floats
  __shared__ float red4[4][kD];
  __shared__ float qs[kD];
  __shared__ int s_last;
  if (rl < rp) {
#pragma unroll
    for (int j = 0; j < 8; ++j) red[rl * (dcols + 1) + cg * 8 + j] = acc[j];
  }
  __syncthreads();
  if (threadIdx.x < kD) {
    float s = 0.f;
    if ((int)threadIdx.x < dcols) {
#pragma unroll 8
      for (int i = 0; i < rp; ++i) s += red[i * (dcols + 1) + threadIdx.x];   // fixed order
    }
    qpart[((size_t)slab * gridDim.x + chunk) * kD + threadIdx.x] = s;
    __threadfence();
  }
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(&slab_count[slab], 1) == (int)gridDim.x - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  slab_gate(qpart, gridDim.x, slab, H, n, L1, per_head, gate_w, gate_b, omega, qbar, sg, f, red4, qs, dcols);
  if (threadIdx.x == 0) slab_count[slab] = 0;
  if (per_head) return;
  __threadfence();
  __syncthreads();
  const int b = slab / H;
  if (threadIdx.x == 0) s_last = atomicAdd(&batch_count[b], 1) == H - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  batch_gate(b, H, L1, gate_b, omega, sg, f);
  if (threadIdx.x == 0) batch_count[b] = 0;
}

// Gate from column sums that are already complete (sequence shards: the sums of all shards were added by the
// caller): one CTA of 256 threads per slab runs slab_gate on a single "partial" with the whole sequence's
// length, then, for the batch-wide gate, a second launch runs batch_gate per batch element.
// qbar_scale: q-bar of a shard times its length gives the shard's column sums back.
__global__ void __launch_bounds__(256) k_scale_qbar(const float* __restrict__ qbar, float scale,
                                                    float* __restrict__ qsum, int count) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i < count) qsum[i] = qbar[i] * scale;
}
__global__ void __launch_bounds__(256) k_gate_from_sums(const float* __restrict__ qsum, int H, int n_total, int L1,
                                                        int per_head, const float* __restrict__ gate_w,
                                                        const float* __restrict__ gate_b,
                                                        const float* __restrict__ omega, float* __restrict__ qbar,
                                                        float* __restrict__ sg, float* __restrict__ f, int dcols) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  __shared__ float red4[4][kD];
  __shared__ float qs[kD];
  slab_gate(qsum, 1, blockIdx.x, H, n_total, L1, per_head, gate_w, gate_b, omega, qbar, sg, f, red4, qs, dcols);
}
__global__ void __launch_bounds__(32) k_batch_gate(int H, int L1, const float* __restrict__ gate_b,
                                                   const float* __restrict__ omega, float* __restrict__ sg,
                                                   float* __restrict__ f) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  batch_gate(blockIdx.x, H, L1, gate_b, omega, sg, f);
}

// Sum the per-tile band inner products of both filtered tensors and turn them into df[slab][i]: i < L takes
// the detail-band product of level i+1, i = L the approximation product of level L.  One CTA of 256 threads
// per slab: thread (j = tid & 15, part = tid >> 4) adds every 16th partial of band slot j in tile order
// (four loads in flight), the 16 parts are added in a fixed order: the result repeats bit for bit.
__global__ void __launch_bounds__(256) k_band_reduce(const float* __restrict__ bands, int slabs, int htiles,
                                                     int L, float* __restrict__ df) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  __shared__ float part[16][kBandVals];
  const int slab = blockIdx.x, j = threadIdx.x & (kBandVals - 1), pt = threadIdx.x >> 4;
  float s = 0.f;
  for (int which = 0; which < 2; ++which) {
    const float* src = bands + (((size_t)which * slabs + slab) * htiles) * kBandVals + j;
    int t = pt;
    for (; t + 48 < htiles; t += 64) {
      const float v0 = src[(size_t)t * kBandVals], v1 = src[(size_t)(t + 16) * kBandVals];
      const float v2 = src[(size_t)(t + 32) * kBandVals], v3 = src[(size_t)(t + 48) * kBandVals];
      s += (v0 + v1) + (v2 + v3);
    }
    for (; t < htiles; t += 16) s += src[(size_t)t * kBandVals];
  }
  part[pt][j] = s;
  __syncthreads();
  if (threadIdx.x < kBandVals) {
    float tot = 0.f;
#pragma unroll
    for (int q = 0; q < 16; ++q) tot += part[q][j];
    // slots 0..7: detail products of levels 1..8; slots 8..15: approximation products of levels 1..8
    if (j < L) df[(size_t)slab * kBandVals + j] = tot;
    if (j == 8 + L - 1) df[(size_t)slab * kBandVals + L] = tot;
  }
}

// out[0] = sum of x[0..n) in a fixed order (64 threads, strided partial sums, then a tree).
__global__ void __launch_bounds__(kD) k_sum_floats(const float* __restrict__ x, int n, float* __restrict__ out) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  __shared__ float part[kD];
  const int c = threadIdx.x;
  float tot = 0.f;
  for (int i = c; i < n; i += kD) tot += x[i];
  part[c] = tot;
  __syncthreads();
  for (int o = kD / 2; o > 0; o >>= 1) {
    if (c < o) part[c] += part[c + o];
    __syncthreads();
  }
  if (c == 0) out[0] = part[0];
}

// Chain rule through f = sigmoid(u) * omega, u = gate(qbar): domega, dgate_b, dgate_w, dqbar; and the
// bandwidth gradient dbeta = 2 eps m bw * sum_t dDh_t (ReLU is positively homogeneous, so beta only
// acts through eps).  Grid H + 2, 64 threads: CTA h < H handles head h (thread c = column of q-bar,
// loop over the batch), CTA H sums domega, CTA H + 1 sums dbeta; every sum has a fixed order.
__global__ void __launch_bounds__(kD) k_gate_backward(
    const float* __restrict__ df, const float* __restrict__ sg, const float* __restrict__ qbar,
    const float* __restrict__ gate_w, const float* __restrict__ omega, const float* __restrict__ sumdD,
    int n_sumdD, const float* __restrict__ beta, float eps, float bw_floor, int m, int B, int H, int L1,
    int per_head, float* __restrict__ dbeta, float* __restrict__ dgate_w, float* __restrict__ dgate_b,
    float* __restrict__ domega, float* __restrict__ dqbar) {
  wait_for_stream_predecessor();   // (launched as a programmatic dependent: see launch_after)
  const int c = threadIdx.x;
  __shared__ float du[kMaxLevels + 1];
  __shared__ float part[kD];
  if ((int)blockIdx.x < H) {
    const int h = blockIdx.x;
    float gw_acc[kMaxLevels + 1], gb_acc = 0.f;
#pragma unroll
    for (int i = 0; i <= kMaxLevels; ++i) gw_acc[i] = 0.f;
    for (int b = 0; b < B; ++b) {
      const int slab = b * H + h;
      __syncthreads();
      if (c < L1) {
        float dfi = 0.f;
        if (per_head) {
          dfi = df[(size_t)slab * kBandVals + c];
        } else {
          for (int hh = 0; hh < H; ++hh) dfi += df[((size_t)b * H + hh) * kBandVals + c];
        }
        float s = sg[(size_t)slab * L1 + c];
        du[c] = dfi * omega[c] * s * (1.f - s);
        if (per_head || h == 0) gb_acc += du[c];
      }
      __syncthreads();
      float dq = 0.f;
      const float qb = qbar[(size_t)slab * kD + c];
#pragma unroll
      for (int i = 0; i <= kMaxLevels; ++i)
        if (i < L1) {
          gw_acc[i] += qb * du[i];
          if (gate_w != nullptr) dq += gate_w[((size_t)h * kD + c) * L1 + i] * du[i];
        }
      dqbar[(size_t)slab * kD + c] = dq;
    }
    if (dgate_w != nullptr) {
#pragma unroll
      for (int i = 0; i <= kMaxLevels; ++i)
        if (i < L1) dgate_w[((size_t)h * kD + c) * L1 + i] = gw_acc[i];
    }
    if (dgate_b != nullptr && c < L1) dgate_b[h * L1 + c] = (per_head || h == 0) ? gb_acc : 0.f;
  } else if ((int)blockIdx.x == H) {
    // domega[i] = sum over slabs of df_i * sigmoid(u_i): thread (i = c & 15, q = c >> 4) takes the
    // batch elements b = q, q + 4, ..., then the four parts are added in order
    const int i = c & 15, q = c >> 4;
    float acc = 0.f;
    if (domega != nullptr && i < L1) {
      for (int b = q; b < B; b += 4) {
        if (per_head) {
          for (int h = 0; h < H; ++h) {
            const int slab = b * H + h;
            acc += df[(size_t)slab * kBandVals + i] * sg[(size_t)slab * L1 + i];
          }
        } else {
          float dfi = 0.f;
          for (int h = 0; h < H; ++h) dfi += df[((size_t)b * H + h) * kBandVals + i];
          acc += dfi * sg[((size_t)b * H) * L1 + i];
        }
      }
    }
    part[c] = acc;
    __syncthreads();
    if (domega != nullptr && c < L1) domega[c] = (part[c] + part[16 + c]) + (part[32 + c] + part[48 + c]);
  } else {
    float tot = 0.f;
    for (int i = c; i < n_sumdD; i += kD) tot += sumdD[i];
    part[c] = tot;
    __syncthreads();
    for (int o = kD / 2; o > 0; o >>= 1) {
      if (c < o) part[c] += part[c + o];
      __syncthreads();
    }
    if (dbeta != nullptr && c == 0) {
      const float bt = beta[0];
      const float bw = fmaxf(bt, bw_floor);
      dbeta[0] = bt > bw_floor ? 2.f * eps * (float)m * bw * part[0] : 0.f;
    }
  }
}

}  // namespace

// The launch shared by the workspace and the static-scratch variants.
static cudaError_t launch_qmean_gate_impl(const Plan& p, const void* Q, float* qpart, const float* gate_w,
                                          const float* gate_b, const float* omega, float* qbar, float* sg, float* f,
                                          int* counters, const void* W, __nv_bfloat16* Wt, int cols,
                                          cudaStream_t st) {
  dim3 grid(p.qchunks, p.slabs + (W != nullptr ? 1 : 0));
  int* slab_count = counters;
  int* batch_count = counters + p.slabs;
  cudaError_t launch_err = cudaSuccess;
  auto launch = [&](auto kernel, auto* q) {
    // Launched as a programmatic dependent of whatever precedes it in the stream: the kernel's first
    // instruction waits for that work to complete, so ordering and visibility are those of a plain launch,
    // but its CTAs are already placed when the wait ends (2 us per forward in a sequence of steps).
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid;
    lc.blockDim = dim3(256);
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    launch_err = cudaLaunchKernelEx(&lc, kernel, q, qpart, p.cfg.seq_len, p.qchunk_rows, p.slabs, p.cfg.heads, p.L1,
                                    p.cfg.gate_per_head, gate_w, gate_b, omega, qbar, sg, f, slab_count, batch_count,
                                    (const __nv_bfloat16*)W, Wt, p.cfg.features, cols);
  };
  if (p.bf16) {
    if (cols == kD) launch(k_qmean_gate<__nv_bfloat16, true>, (const __nv_bfloat16*)Q);
    else launch(k_qmean_gate<__nv_bfloat16, false>, (const __nv_bfloat16*)Q);
  } else {
    if (cols == kD) launch(k_qmean_gate<float, true>, (const float*)Q);
    else launch(k_qmean_gate<float, false>, (const float*)Q);
  }
  return launch_err != cudaSuccess ? launch_err : cudaGetLastError();
}

cudaError_t launch_qmean_gate(const Plan& p, const Ws& w, const void* Q, const float* gate_w,
                              const float* gate_b, const float* omega, const void* W, int cols, cudaStream_t st,
                              int* launches) {
  *launches += 1;
  return launch_qmean_gate_impl(p, Q, w.qpart, gate_w, gate_b, omega, w.qbar, w.sg, w.f, w.counters, W, w.Wt, cols, st);
}

cudaError_t launch_shard_qsum(const Plan& p, const Ws& w, float* qsum, cudaStream_t st, int* launches) {
  const int count = p.slabs * kD;
  launch_after(k_scale_qbar, dim3((count + 255) / 256), dim3(256), 0, st, w.qbar, (float)p.cfg.seq_len, qsum, count);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_gate_from_sums(const Plan& p, const Ws& w, const float* qsum, long long n_total,
                                  const float* gate_w, const float* gate_b, const float* omega, int cols,
                                  cudaStream_t st, int* launches) {
  launch_after(k_gate_from_sums, dim3(p.slabs), dim3(256), 0, st, qsum, p.cfg.heads, (int)n_total, p.L1, p.cfg.gate_per_head, gate_w, gate_b,
                                           omega, w.qbar, w.sg, w.f, cols);
  *launches += 1;
  if (!p.cfg.gate_per_head) {
    launch_after(k_batch_gate, dim3(p.cfg.batch), dim3(32), 0, st, p.cfg.heads, p.L1, gate_b, omega, w.sg, w.f);
    *launches += 1;
  }
  return cudaGetLastError();
}

// Device address of the static scratch array on the current device, resolved once per device.
// In host code the array's name is only a handle: the kernels need the address this returns.
cudaError_t static_scratch_address(int device, float** out) {
  if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (g_static_scratch_addr[device] == nullptr) {
    void* ptr = nullptr;
    cudaError_t err = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (err != cudaSuccess) return err;
    g_static_scratch_addr[device] = static_cast<float*>(ptr);
  }
  *out = g_static_scratch_addr[device];
  return cudaSuccess;
}

size_t static_scratch_capacity_floats() { return kStaticScratchFloats - kStaticCounterInts; }
size_t static_scratch_counter_capacity() { return kStaticCounterInts; }

cudaError_t launch_qmean_gate_static(const Plan& p, float* scratch, const void* Q, const float* gate_w,
                                     const float* gate_b, const float* omega, float* qbar, float* f,
                                     cudaStream_t st) {
  // scratch = [ partial column sums: slabs x qchunks x 64 | sigmoid(u): slabs x (L+1) | unused ...
  //             | arrival counters in the last kStaticCounterInts elements: slabs, then batch ints ]
  // The counters this call uses are cleared on the stream first (a memset allocates nothing): a call
  // then starts from zero whatever an earlier call of another shape, or one that failed half way, left.
  float* qpart = scratch;
  float* sg = scratch + (size_t)p.slabs * p.qchunks * kD;
  int* counters = reinterpret_cast<int*>(scratch + (kStaticScratchFloats - kStaticCounterInts));
  cudaError_t err = cudaMemsetAsync(counters, 0, sizeof(int) * ((size_t)p.slabs + (size_t)p.cfg.batch), st);
  if (err != cudaSuccess) return err;
  return launch_qmean_gate_impl(p, Q, qpart, gate_w, gate_b, omega, qbar, sg, f, counters, nullptr, nullptr, kD, st);
}

size_t static_scratch_floats_needed(const Plan& p) {
  return (size_t)p.slabs * p.qchunks * kD + (size_t)p.slabs * p.L1;
}
size_t static_scratch_counters_needed(const Plan& p) { return (size_t)p.slabs + (size_t)p.cfg.batch; }

// The two halves of launch_gate_backward, for sequence shards: this shard's band inner products (df, slabs x 16)
// and its sum of dD'; then, from the sums over all shards, the parameter gradients and d(qbar).
cudaError_t launch_band_sums(const Plan& p, const Ws& w, int n_sumdD, float* df, float* sumdD_total, cudaStream_t st,
                             int* launches) {
  launch_after(k_band_reduce, dim3(p.slabs), dim3(256), 0, st, w.bands, p.slabs, 2 * p.htiles, p.cfg.levels, df);
  launch_after(k_sum_floats, dim3(1), dim3(kD), 0, st, w.sumdD, n_sumdD, sumdD_total);
  *launches += 2;
  return cudaGetLastError();
}
cudaError_t launch_gate_backward_from(const Plan& p, const Ws& w, const float* df, const float* sumdD_total,
                                      const float* beta, const float* gate_w, const float* omega, float* dbeta,
                                      float* dgate_w, float* dgate_b, float* domega, cudaStream_t st, int* launches) {
  launch_after(k_gate_backward, dim3(p.cfg.heads + 2), dim3(kD), 0, st, df, w.sg, w.qbar, gate_w, omega, sumdD_total, 1,
               beta, p.cfg.eps, p.cfg.bw_floor, p.cfg.features, p.cfg.batch, p.cfg.heads, p.L1, p.cfg.gate_per_head,
               dbeta, dgate_w, dgate_b, domega, w.dqbar);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_gate_backward(const Plan& p, const Ws& w, const float* beta, const float* gate_w,
                                 const float* omega, int n_sumdD, float* dbeta, float* dgate_w, float* dgate_b,
                                 float* domega, cudaStream_t st, int* launches) {
  float* df = w.dqbar + (size_t)p.slabs * kD;   // df lives behind dqbar in the same region
  launch_after(k_band_reduce, dim3(p.slabs), dim3(256), 0, st, w.bands, p.slabs, 2 * p.htiles, p.cfg.levels, df);   // two partials per tile
  launch_after(k_gate_backward, dim3(p.cfg.heads + 2), dim3(kD), 0, st, df, w.sg, w.qbar, gate_w, omega, w.sumdD, n_sumdD, beta,
                                    p.cfg.eps, p.cfg.bw_floor, p.cfg.features, p.cfg.batch, p.cfg.heads,
                                    p.L1, p.cfg.gate_per_head, dbeta, dgate_w, dgate_b, domega, w.dqbar);
  *launches += 2;
  return cudaGetLastError();
}

}  // namespace wersa
