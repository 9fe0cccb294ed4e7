// Shared declarations of the WERSA CUDA library: the host-side plan, the workspace layout and
// the launch functions each translation unit exports to the C-ABI layer (api.cu).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/wersa.h"

namespace wersa {

constexpr int kD = 64;           // head dim the kernels work on (narrower heads are zero-padded to it)
constexpr int kGroupFeatures = 256;   // widest feature map of one kernel launch; wider maps run in groups
constexpr int kMaxLevels = 8;    // Haar levels supported: block of 2^8 = 256 tokens
constexpr int kHaarTile = 256;   // tokens per Haar tile (>= 2^kMaxLevels)
constexpr int kSimtTile = 32;    // tokens per tile in the fp32 FFMA kernels
constexpr int kBandVals = 16;    // per-tile band inner products kept by the Haar backward

// Host-side plan: problem sizes, chunking and byte offsets into the caller's workspace.
struct Plan {
  wersa_config cfg;
  int slabs;          // B*H
  int sms;            // streaming multiprocessors of cfg.device
  int L1;             // levels + 1
  bool bf16;          // storage type of Q,K,V,W,O,dO
  bool grad_bf16;     // storage type of dQ,dK,dV
  bool use_tc;        // bf16 tcgen05 forward kernels
  bool with_backward;
  bool dpad;          // cfg.head_dim < 64: tensors pass through zero-padded 64-wide copies in the workspace
  int groups;         // feature groups of kGroupFeatures (1 when cfg.features <= 256)
  int fwd_cols;       // columns of Q, K, V, O as the forward kernels see them: head_dim on the tensor-core path
                      // (the tensor maps zero-fill up to 64), 64 on the fp32 path (padded copies)
  // mean pool
  int qchunks, qchunk_rows;
  // haar tiles
  int htiles;
  // fp32 FFMA key-side / backward query-side split of the sequence
  int schunks, schunk_tiles;   // chunks per slab, 32-token tiles per chunk
  // tcgen05 key-side split
  int tchunks, tchunk_blocks;  // chunks per slab, 256-token blocks per chunk
  // tcgen05 backward: chunks per slab, 128-token tiles per chunk
  int bchunks, bchunk_tiles;
  // workspace offsets (bytes)
  size_t off_status, off_counters, status_bytes, off_qpart, off_qbar, off_sg, off_f, off_spart, off_zpart, off_S, off_z,
      off_Sbf, off_Wt, off_dS, off_dz, off_sumdD, off_bands, off_dqbar, off_QF, off_KF, off_dQF,
      off_dKF, off_dSbf, off_KF3, off_QF3, off_Slo, off_Simg, off_Qp, off_Kp, off_Vp, off_Op, off_Wp, off_gwp,
      off_dOp, off_dQp, off_dKp, off_dVp, off_dgwp, off_Og, off_den, off_Sout, off_zout, off_Dtot, off_shardtot, total;
  int part_chunks;    // max(schunks, tchunks): leading extent of the partial buffers
};

// Fills `p` from `cfg`; returns WERSA_OK, WERSA_ERR_INVALID_ARG or WERSA_ERR_UNSUPPORTED.
wersa_status make_plan(const wersa_config& cfg, Plan* p);

struct Ws {   // resolved workspace pointers
  int* status;
  int* counters;   // arrival counters (slabs + batch + slabs ints), zero between launches
  float *qpart, *qbar, *sg, *f, *spart, *zpart, *S, *z, *dS, *dz, *sumdD, *bands, *dqbar;
  __nv_bfloat16 *Sbf, *Wt, *dSbf, *KF3, *QF3, *Slo;   // Slo = bf16(S' - bf16(S')), built by the backward
  uint8_t* Simg;   // [S' | z' | 0]^T operand images of the query-side kernel, one per slab (see simg_offset)
  float *QF, *KF, *dQF, *dKF;
  // head_dim < 64: padded copies of the inputs and outputs (storage / gradient type), of W and of the gate weights
  void *Qp, *Kp, *Vp, *Op, *Wp, *dOp, *dQp, *dKp, *dVp;
  float *gwp, *dgwp;
  // features > 256: per-group outputs and denominators, and the slab-major S', z' handed out by wersa_saved
  void* Og;
  float *den, *Sout, *zout;
  float* shardtot;   // sequence shards, backward: this shard's sum of dD' (one float)
  float* Dtot;   // backward with feature groups: the whole map's denominator per token, then dD' per token
};
Ws resolve(const Plan& p, void* workspace);

// ---- gate.cu -------------------------------------------------------------------------------
// Partial column sums of Q over row chunks, then qbar, sigmoid(u) and f per slab (Eqs. 1-3).
// With W != nullptr the second launch also leaves the bf16 transpose of W (m x 64) in w.Wt.
// cols: columns of Q as stored (64, or the head dimension when Q comes unpadded; then gate_w has cols rows
// per head and W cols rows).
cudaError_t launch_qmean_gate(const Plan& p, const Ws& w, const void* Q, const float* gate_w,
                              const float* gate_b, const float* omega, const void* W, int cols, cudaStream_t st,
                              int* launches);
// Sequence shards: column sums of this shard's Q (q-bar times the shard's length), and the gate from the
// sums of all shards and the whole sequence's length (writes w.qbar, w.sg, w.f).
cudaError_t launch_shard_qsum(const Plan& p, const Ws& w, float* qsum, cudaStream_t st, int* launches);
cudaError_t launch_gate_from_sums(const Plan& p, const Ws& w, const float* qsum, long long n_total,
                                  const float* gate_w, const float* gate_b, const float* omega, int cols,
                                  cudaStream_t st, int* launches);
cudaError_t launch_band_sums(const Plan& p, const Ws& w, int n_sumdD, float* df, float* sumdD_total, cudaStream_t st,
                             int* launches);
cudaError_t launch_gate_backward_from(const Plan& p, const Ws& w, const float* df, const float* sumdD_total,
                                      const float* beta, const float* gate_w, const float* omega, float* dbeta,
                                      float* dgate_w, float* dgate_b, float* domega, cudaStream_t st, int* launches);
// Gate backward: band inner products -> df -> domega, dgate_b, dgate_w, dqbar; dbeta.
cudaError_t launch_gate_backward(const Plan& p, const Ws& w, const float* beta, const float* gate_w,
                                 const float* omega, int n_sumdD, float* dbeta, float* dgate_w, float* dgate_b,
                                 float* domega, cudaStream_t st, int* launches);

// Mean pool + gate with their scratch in a file-scope device array (no caller workspace).
cudaError_t static_scratch_address(int device, float** out);
size_t static_scratch_capacity_floats();      // floats available to the partial sums and sigmoids
size_t static_scratch_counter_capacity();     // ints reserved for the arrival counters
size_t static_scratch_floats_needed(const Plan& p);
size_t static_scratch_counters_needed(const Plan& p);
cudaError_t launch_qmean_gate_static(const Plan& p, float* scratch, const void* Q, const float* gate_w,
                                     const float* gate_b, const float* omega, float* qbar, float* f,
                                     cudaStream_t st);

// ---- haar.cu -------------------------------------------------------------------------------
// XF = T_f(X).  in_kind/out_kind: 0 = float, 1 = bf16.
cudaError_t launch_haar_filter(const Plan& p, const void* X, int in_kind, const float* f, void* XF,
                               int out_kind, cudaStream_t st, int* launches);
// XF3 = T_f(X) as three bf16 planes hi, mid, lo (each slabs x n x 64) whose sum is the fp32 result.
cudaError_t launch_haar_filter_split3(const Plan& p, const void* X, int in_kind, const float* f,
                                      __nv_bfloat16* XF3, cudaStream_t st, int* launches);
// dX = T_f(G) + vec[slab] * vec_scale on every row (G fp32, vec = slabs x 64 floats).
cudaError_t launch_haar_filter_addvec(const Plan& p, const float* G, const float* f, const float* vec,
                                      float vec_scale, void* dX, int out_kind, cudaStream_t st, int* launches);
// dX = T_f(G) (G fp32) and per-tile band inner products of (G, X) into bands[which]; dX == nullptr: only
// the band inner products.
cudaError_t launch_haar_backward(const Plan& p, const Ws& w, const void* X, int in_kind,
                                 const float* G, void* dX, int out_kind, int which, cudaStream_t st,
                                 int* launches);

// ---- simt.cu -------------------------------------------------------------------------------
cudaError_t launch_simt_kside(const Plan& p, const Ws& w, const void* V, const void* W,
                              cudaStream_t st, int* launches);
// S = sum_chunks spart, z = sum_chunks zpart in chunk order (also used for dS, dz).
cudaError_t launch_reduce_partials(const Plan& p, const float* spart, const float* zpart, int chunks,
                                   float* S, float* z, __nv_bfloat16* Sbf, uint8_t* Simg, cudaStream_t st,
                                   int* launches);
cudaError_t launch_simt_qside(const Plan& p, const Ws& w, const void* W, const float* beta, void* O,
                              cudaStream_t st, int* launches);
cudaError_t launch_simt_bwd_qside(const Plan& p, const Ws& w, const void* W, const float* beta,
                                  const void* dO, cudaStream_t st, int* launches);
cudaError_t launch_simt_bwd_kside(const Plan& p, const Ws& w, const void* V, const void* W, void* dV,
                                  cudaStream_t st, int* launches);

// ---- tc_fwd.cu -----------------------------------------------------------------------------
// Both read the raw bf16 tensors and apply the Haar filter (coefficients from w.f) on chip.
cudaError_t launch_tc_kside(const Plan& p, const Ws& w, const void* K, const void* V, cudaStream_t st,
                            int* launches);
// den != nullptr (features == 256 only): also leaves every token's denominator in den[slab * n + token].
cudaError_t launch_tc_qside(const Plan& p, const Ws& w, const void* Q, const float* beta, void* O, float* den,
                            cudaStream_t st, int* launches);

// ---- tc_bwd.cu -----------------------------------------------------------------------------
// Key-side backward on the tensor cores: dV and dK_F from K_F as three bf16 planes, V, the bf16 dS' image
// (w.dSbf), dz' (w.dz) and the bf16 W^T image (w.Wt).
// Query-side backward on the tensor cores: dQ_F, and the split-sequence partials of dS', dz' and
// sum dD' (w.spart, w.zpart, w.sumdD; p.bchunks chunks per slab), from Q_F as three bf16 planes, dO,
// the bf16 S' image (w.Sbf), z' (w.z) and the bf16 W^T image.
// Feature groups (p.cfg.features == 256 as one group of a wider map): den_ext / dd_ext hold the whole map's
// denominator and dD' per token (slabs x n floats each), `add` makes dQ_F (dV, dK_F) accumulate.
cudaError_t launch_tc_bwd_qside(const Plan& p, const Ws& w, const void* QF3, const float* beta, const void* dO,
                                const float* den_ext, const float* dd_ext, bool add, cudaStream_t st, int* launches);
cudaError_t launch_tc_bwd_kside(const Plan& p, const Ws& w, const void* KF3, const void* V, void* dV, bool add,
                                cudaStream_t st, int* launches);


// ---- glue.cu -------------------------------------------------------------------------------
// kind: 0 = float, 1 = bf16.  rows x d <-> rows x 64 (zero-filled); d is a multiple of 8.
cudaError_t launch_pad_cols(const void* src, void* dst, size_t rows, int d, int kind, cudaStream_t st, int* launches);
cudaError_t launch_unpad_cols(const void* src, void* dst, size_t rows, int d, int kind, cudaStream_t st, int* launches);
// O = sum_g Og[g] * den[g] / sum_g den[g] per token (Og: groups x tokens x 64, den: groups x tokens).
// O has `cols` columns (the first `cols` of the 64 are written).
cudaError_t launch_combine_groups(const void* Og, const float* den, void* O, size_t tokens, int groups, int cols,
                                  int kind, cudaStream_t st, int* launches);
// Backward of the combination: per token the whole map's denominator D = sum_g den_g / r (r = the filter
// stage's factor carried by the forward's denominators, from f) and dD' = -(dO . O) / D with
// O = sum_g Og den_g / sum_g den_g.  dO and Og are 64 wide.
cudaError_t launch_group_bwd_prep(const void* Og, const float* den, const void* dO, const float* f, int n, int L1,
                                  size_t tokens, int groups, int kind, float* Dtot, float* dDtot, cudaStream_t st,
                                  int* launches);
// Group-major S', z' ([group][slab][mg][...]) -> slab-major ([slab][groups * mg][...]).
cudaError_t launch_gather_groups(const float* Sg, const float* zg, float* S, float* z, int slabs, int groups, int mg,
                                 cudaStream_t st, int* launches);

// ---- selftest.cu ---------------------------------------------------------------------------
// One CTA whose bounded wait runs out after limit_ns: sets the status word; observed[0] = abort flag,
// observed[1], observed[2] = whether the two roles' waits succeeded (both must read 0).
cudaError_t launch_selftest_wait(const Ws& w, unsigned long long limit_ns, int* observed, cudaStream_t st);

// ---- operand image of the query-side second contraction --------------------------------------
// The query-side kernel multiplies the features by [S' | z' | 0] (m x 80) as a K-major bf16 operand: per
// slab, m / 64 blocks of 80 rows x 128 bytes -- rows 0-63 are the columns of S', row 64 is z', rows 65-79
// are zero, and a row holds 64 consecutive features in the 128-byte swizzle the tensor core reads (16-byte
// chunk j of row r sits at chunk j ^ (r & 7)).  Whoever produces S' and z' leaves this image in global
// memory in exactly that byte order, so that the kernel fetches it with one bulk copy.
constexpr int kSimgRows = 80;
constexpr size_t kSimgBlockBytes = kSimgRows * 128;
__host__ __device__ inline size_t simg_bytes(int m) { return (size_t)(m / 64) * kSimgBlockBytes; }
// byte offset of (feature f, row r) inside a slab's image
__device__ __forceinline__ size_t simg_offset(int f, int r) {
  return (size_t)(f >> 6) * kSimgBlockBytes + (size_t)r * 128 + (size_t)((((f & 63) >> 3) ^ (r & 7)) << 4) + (f & 7) * 2;
}

// Launch as a programmatic dependent of the work before it in the stream.  The kernel's first instruction
// must be griddepcontrol.wait (nothing is read or written before that work has completed), so ordering and
// visibility are those of a plain launch; only the placement of the CTAs overlaps the end of that work.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_after(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}
__device__ __forceinline__ void wait_for_stream_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- device helpers ------------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}

// Loads 8 consecutive elements (16-byte aligned for bf16, 32-byte for float) as floats.
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  float4 a = *reinterpret_cast<const float4*>(p);
  float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
  uint4 raw = *reinterpret_cast<const uint4*>(p);
  const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(u[i] << 16);
    v[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
  }
}
// The same loads with the streaming (evict-first) cache hint, for data that is read once: the lines make room
// for themselves in L2 instead of pushing out what other kernels left there (dirty output lines of the step
// before are then written back later, under kernels that do not need the DRAM bandwidth).
__device__ __forceinline__ void load8_stream(const float* p, float (&v)[8]) {
  const float4 a = __ldcs(reinterpret_cast<const float4*>(p));
  const float4 b = __ldcs(reinterpret_cast<const float4*>(p + 4));
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8_stream(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(p));
  const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(u[i] << 16);
    v[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ void store8(float* p, const float (&v)[8]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  *reinterpret_cast<float4*>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void store8(__nv_bfloat16* p, const float (&v)[8]) {
  uint4 raw;
  uint32_t* u = reinterpret_cast<uint32_t*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    u[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  *reinterpret_cast<uint4*>(p) = raw;
}

}  // namespace wersa
