// C-ABI layer of the WERSA library: configuration checks, workspace planning and the launch
// sequences of the forward and backward passes.  All arithmetic lives in the kernels.
#include <new>

#include "common.cuh"

namespace wersa {

bool tc_supported(const wersa_config& cfg);   // tc_fwd.cu

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
int ceil_div(int a, int b) { return (a + b - 1) / b; }
int next_pow2(int n) {
  int p = 1;
  while (p < n) p <<= 1;
  return p;
}
// Streaming multiprocessors of the device the plan is made for: the chunk counts below aim at whole
// waves of CTAs.  Without a device (host-only sizing queries) the count of a B200 is assumed.
int device_sm_count(int device) {
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1) {
    cudaGetLastError();   // a failed query leaves no sticky error behind
    sms = 148;
  }
  return sms;
}

}  // namespace

wersa_status make_plan(const wersa_config& c, Plan* p) {
  if (c.batch < 1 || c.heads < 1 || c.seq_len < 2 || c.head_dim < 1 || c.levels < 1 || c.features < 1)
    return WERSA_ERR_INVALID_ARG;
  if (c.dtype != WERSA_F32 && c.dtype != WERSA_BF16) return WERSA_ERR_INVALID_ARG;
  if (c.grad_dtype != WERSA_F32 && c.grad_dtype != WERSA_BF16) return WERSA_ERR_INVALID_ARG;
  if (!(c.eps >= 0.f) || !(c.bw_floor > 0.f)) return WERSA_ERR_INVALID_ARG;
  if (c.device < 0) return WERSA_ERR_INVALID_ARG;
  if (c.levels <= 30 && (1LL << c.levels) > (long long)next_pow2(c.seq_len)) return WERSA_ERR_INVALID_ARG;
  // head dimensions 8, 16, ... 64 (narrower ones run zero-padded to 64 columns)
  if (c.head_dim > kD || c.head_dim < 8 || c.head_dim % 8 != 0) return WERSA_ERR_UNSUPPORTED;
  if (c.levels > kMaxLevels) return WERSA_ERR_UNSUPPORTED;
  // feature maps of 64, 128 or 256, and (bf16 tensor-core path) 512, 768, 1024 in groups of 256
  const bool grouped = c.features > kGroupFeatures;
  if (grouped) {
    if (c.features % kGroupFeatures != 0 || c.features > 4 * kGroupFeatures) return WERSA_ERR_UNSUPPORTED;
    if (c.dtype != WERSA_BF16 || (c.flags & WERSA_FLAG_SIMT_ONLY)) return WERSA_ERR_UNSUPPORTED;
  } else if (c.features != 64 && c.features != 128 && c.features != 256) {
    return WERSA_ERR_UNSUPPORTED;
  }
  if ((long long)c.batch * c.heads > 65535) return WERSA_ERR_UNSUPPORTED;   // gridDim.y

  p->cfg = c;
  p->slabs = c.batch * c.heads;
  p->L1 = c.levels + 1;
  p->bf16 = c.dtype == WERSA_BF16;
  p->grad_bf16 = c.grad_dtype == WERSA_BF16;
  p->with_backward = !(c.flags & WERSA_FLAG_FORWARD_ONLY);
  p->dpad = c.head_dim < kD;
  p->groups = grouped ? c.features / kGroupFeatures : 1;
  p->use_tc = p->bf16 && !(c.flags & WERSA_FLAG_SIMT_ONLY) && tc_supported(c);
  p->fwd_cols = p->use_tc ? c.head_dim : kD;
  const int n = c.seq_len, m = c.features;
  p->sms = device_sm_count(c.device);

  p->qchunks = ceil_div(4 * p->sms, p->slabs);
  if (p->qchunks > ceil_div(n, 128)) p->qchunks = ceil_div(n, 128);
  if (p->qchunks < 1) p->qchunks = 1;
  p->qchunk_rows = ceil_div(ceil_div(n, p->qchunks), 32) * 32;
  p->qchunks = ceil_div(n, p->qchunk_rows);

  p->htiles = ceil_div(n, kHaarTile);

  const int tiles32 = ceil_div(n, kSimtTile);
  p->schunks = ceil_div(2 * p->sms, p->slabs);
  if (p->schunks > tiles32) p->schunks = tiles32;
  p->schunk_tiles = ceil_div(tiles32, p->schunks);
  p->schunks = ceil_div(tiles32, p->schunk_tiles);

  p->tchunks = 0;
  p->tchunk_blocks = 0;
  if (p->use_tc) {
    const int blocks = ceil_div(n, 256);
    p->tchunks = p->sms / p->slabs;
    if (p->tchunks < 1) p->tchunks = 1;
    if (p->tchunks > blocks) p->tchunks = blocks;
    p->tchunk_blocks = ceil_div(blocks, p->tchunks);
    p->tchunks = ceil_div(blocks, p->tchunk_blocks);
  }
  {
    const int tiles128 = ceil_div(n, 128);
    p->bchunks = p->sms / p->slabs;   // one CTA per SM, a single wave
    if (p->bchunks < 1) p->bchunks = 1;
    if (p->bchunks > tiles128) p->bchunks = tiles128;
    p->bchunk_tiles = ceil_div(tiles128, p->bchunks);
    p->bchunks = ceil_div(tiles128, p->bchunk_tiles);
  }
  p->part_chunks = p->schunks > p->tchunks ? p->schunks : p->tchunks;

  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  const size_t slabs = (size_t)p->slabs;
  // status word (256 bytes) followed by the arrival counters; cleared together before the first launch
  p->off_status = off;
  p->off_counters = off + 256;
  p->status_bytes = align_up(256 + sizeof(int) * (2 * slabs + (size_t)c.batch), 256);
  take(p->status_bytes);
  p->off_qpart = take(sizeof(float) * slabs * p->qchunks * kD);
  p->off_qbar = take(sizeof(float) * slabs * kD);
  p->off_sg = take(sizeof(float) * slabs * p->L1);
  p->off_f = take(sizeof(float) * slabs * p->L1);
  p->off_spart = take(sizeof(float) * slabs * p->part_chunks * m * kD);
  p->off_zpart = take(sizeof(float) * slabs * p->part_chunks * m);
  p->off_S = take(sizeof(float) * slabs * m * kD);
  p->off_z = take(sizeof(float) * slabs * m);
  p->off_Sbf = take(sizeof(__nv_bfloat16) * slabs * m * kD);
  p->off_Wt = take(sizeof(__nv_bfloat16) * (size_t)m * kD);
  p->off_Simg = take(p->use_tc ? slabs * simg_bytes(m) : 0);
  const size_t slab_elems = slabs * (size_t)n * kD;
  const size_t io_bytes = p->bf16 ? 2 : 4, grad_bytes = p->grad_bf16 ? 2 : 4;
  p->off_Qp = take(p->dpad ? io_bytes * slab_elems : 0);
  p->off_Kp = take(p->dpad ? io_bytes * slab_elems : 0);
  p->off_Vp = take(p->dpad ? io_bytes * slab_elems : 0);
  p->off_Op = take(p->dpad ? io_bytes * slab_elems : 0);
  p->off_Wp = take(p->dpad ? io_bytes * (size_t)kD * m : 0);
  p->off_gwp = take(p->dpad ? sizeof(float) * (size_t)c.heads * kD * p->L1 : 0);
  p->off_Og = take(grouped ? io_bytes * slab_elems * p->groups : 0);
  p->off_den = take(grouped ? sizeof(float) * slabs * n * p->groups : 0);
  p->off_Sout = take(grouped ? sizeof(float) * slabs * m * kD : 0);
  p->off_zout = take(grouped ? sizeof(float) * slabs * m : 0);
  const bool need_xf = !p->use_tc;   // the tensor-core kernels filter on chip (forward) or read bf16 planes (backward)
  p->off_QF = take(need_xf ? sizeof(float) * slab_elems : 0);
  p->off_KF = take(need_xf ? sizeof(float) * slab_elems : 0);
  if (p->with_backward) {
    p->off_dS = take(sizeof(float) * slabs * m * kD);
    p->off_dz = take(sizeof(float) * slabs * m);
    p->off_sumdD = take(sizeof(float) * slabs * p->schunks);
    p->off_bands = take(sizeof(float) * 2 * slabs * 2 * p->htiles * kBandVals);   // Q and K; two column halves per tile
    p->off_dqbar = take(sizeof(float) * slabs * (kD + kBandVals));
    p->off_dQF = take(sizeof(float) * slab_elems);
    p->off_dKF = take(sizeof(float) * slab_elems);
    p->off_dSbf = take(sizeof(__nv_bfloat16) * slabs * m * kD);
    p->off_KF3 = take(p->use_tc ? 3 * sizeof(__nv_bfloat16) * slab_elems : 0);
    p->off_QF3 = take(p->use_tc ? 3 * sizeof(__nv_bfloat16) * slab_elems : 0);
    p->off_Slo = take(p->use_tc ? sizeof(__nv_bfloat16) * slabs * m * kD : 0);
    p->off_dOp = take(p->dpad ? io_bytes * slab_elems : 0);
    p->off_dQp = take(p->dpad ? grad_bytes * slab_elems : 0);
    p->off_dKp = take(p->dpad ? grad_bytes * slab_elems : 0);
    p->off_dVp = take(p->dpad ? grad_bytes * slab_elems : 0);
    p->off_dgwp = take(p->dpad ? sizeof(float) * (size_t)c.heads * kD * p->L1 : 0);
    p->off_Dtot = take(grouped ? sizeof(float) * 2 * slabs * n : 0);
    p->off_shardtot = take(256);
  } else {
    p->off_Dtot = p->off_shardtot = 0;
    p->off_dS = p->off_dz = p->off_sumdD = p->off_bands = p->off_dqbar = p->off_dQF = p->off_dKF = p->off_dSbf = p->off_KF3 = p->off_QF3 = p->off_Slo = 0;
    p->off_dOp = p->off_dQp = p->off_dKp = p->off_dVp = p->off_dgwp = 0;
  }
  p->total = off;
  return WERSA_OK;
}

Ws resolve(const Plan& p, void* workspace) {
  char* b = static_cast<char*>(workspace);
  Ws w;
  w.status = reinterpret_cast<int*>(b + p.off_status);
  w.counters = reinterpret_cast<int*>(b + p.off_counters);
  w.qpart = reinterpret_cast<float*>(b + p.off_qpart);
  w.qbar = reinterpret_cast<float*>(b + p.off_qbar);
  w.sg = reinterpret_cast<float*>(b + p.off_sg);
  w.f = reinterpret_cast<float*>(b + p.off_f);
  w.spart = reinterpret_cast<float*>(b + p.off_spart);
  w.zpart = reinterpret_cast<float*>(b + p.off_zpart);
  w.S = reinterpret_cast<float*>(b + p.off_S);
  w.z = reinterpret_cast<float*>(b + p.off_z);
  w.Sbf = reinterpret_cast<__nv_bfloat16*>(b + p.off_Sbf);
  w.Wt = reinterpret_cast<__nv_bfloat16*>(b + p.off_Wt);
  w.Simg = reinterpret_cast<uint8_t*>(b + p.off_Simg);
  w.QF = reinterpret_cast<float*>(b + p.off_QF);
  w.KF = reinterpret_cast<float*>(b + p.off_KF);
  w.dS = reinterpret_cast<float*>(b + p.off_dS);
  w.dz = reinterpret_cast<float*>(b + p.off_dz);
  w.sumdD = reinterpret_cast<float*>(b + p.off_sumdD);
  w.bands = reinterpret_cast<float*>(b + p.off_bands);
  w.dqbar = reinterpret_cast<float*>(b + p.off_dqbar);
  w.dQF = reinterpret_cast<float*>(b + p.off_dQF);
  w.dKF = reinterpret_cast<float*>(b + p.off_dKF);
  w.dSbf = reinterpret_cast<__nv_bfloat16*>(b + p.off_dSbf);
  w.KF3 = reinterpret_cast<__nv_bfloat16*>(b + p.off_KF3);
  w.QF3 = reinterpret_cast<__nv_bfloat16*>(b + p.off_QF3);
  w.Slo = reinterpret_cast<__nv_bfloat16*>(b + p.off_Slo);
  w.Qp = b + p.off_Qp;
  w.Kp = b + p.off_Kp;
  w.Vp = b + p.off_Vp;
  w.Op = b + p.off_Op;
  w.Wp = b + p.off_Wp;
  w.gwp = reinterpret_cast<float*>(b + p.off_gwp);
  w.dOp = b + p.off_dOp;
  w.dQp = b + p.off_dQp;
  w.dKp = b + p.off_dKp;
  w.dVp = b + p.off_dVp;
  w.dgwp = reinterpret_cast<float*>(b + p.off_dgwp);
  w.Og = b + p.off_Og;
  w.den = reinterpret_cast<float*>(b + p.off_den);
  w.Sout = reinterpret_cast<float*>(b + p.off_Sout);
  w.zout = reinterpret_cast<float*>(b + p.off_zout);
  w.Dtot = reinterpret_cast<float*>(b + p.off_Dtot);
  w.shardtot = reinterpret_cast<float*>(b + p.off_shardtot);
  return w;
}

}  // namespace wersa

using namespace wersa;

constexpr int kMaxSteps = 32;

// Optional per-step timing: an event before the first launch and one after every step.
struct StepTimer {
  bool enabled = false;
  cudaEvent_t ev[2][kMaxSteps + 1];
  const char* name[2][kMaxSteps];
  int count[2] = {0, 0};
};

struct wersa_ctx {
  Plan plan;
  Ws ws;
  void* workspace;
  bool forward_done;
  bool status_cleared;
  int launches_fwd, launches_bwd;
  StepTimer timer;
};

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Makes cfg.device current for the lifetime of the object and restores the caller's device.
struct DeviceGuard {
  int prev = -1;
  cudaError_t err;
  explicit DeviceGuard(int dev) {
    err = cudaGetDevice(&prev);
    if (err == cudaSuccess && prev != dev) err = cudaSetDevice(dev);
    else if (err == cudaSuccess) prev = -1;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

#define WERSA_CUDA(call)                                   \
  do {                                                     \
    cudaError_t e_ = (call);                               \
    if (e_ != cudaSuccess) return WERSA_ERR_CUDA;          \
  } while (0)

// Runs one step of a pass and, when step timing is on, records an event behind it.
#define WERSA_STEP(which, label, call)                                             \
  do {                                                                             \
    WERSA_CUDA(call);                                                              \
    StepTimer& t_ = ctx->timer;                                                    \
    if (t_.enabled && t_.count[which] < kMaxSteps) {                               \
      t_.name[which][t_.count[which]] = label;                                     \
      WERSA_CUDA(cudaEventRecord(t_.ev[which][t_.count[which] + 1], st));          \
      ++t_.count[which];                                                           \
    }                                                                              \
  } while (0)

wersa_status begin_pass(wersa_ctx* ctx, int which, cudaStream_t st) {
  StepTimer& t = ctx->timer;
  t.count[which] = 0;
  if (t.enabled) WERSA_CUDA(cudaEventRecord(t.ev[which][0], st));
  return WERSA_OK;
}

// Feature group g of a map wider than 256 features: the plan of a 256-feature problem and the workspace
// regions of that group (the kernels' buffers are kept group-major: [group][slab][...]).
Plan group_plan(const Plan& p) {
  Plan pg = p;
  pg.cfg.features = kGroupFeatures;
  return pg;
}
// `chunks`: chunks per slab of the partial sums the view is used with (forward: p.tchunks, backward: p.bchunks).
Ws group_view(const Plan& p, const Ws& w, int g, int chunks) {
  Ws v = w;
  const size_t slabs = (size_t)p.slabs, mg = kGroupFeatures;
  v.Wt = w.Wt + (size_t)g * mg * kD;
  v.spart = w.spart + (size_t)g * slabs * chunks * mg * kD;
  v.zpart = w.zpart + (size_t)g * slabs * chunks * mg;
  if (p.with_backward) {
    v.dS = w.dS + (size_t)g * slabs * mg * kD;
    v.dz = w.dz + (size_t)g * slabs * mg;
    v.dSbf = w.dSbf + (size_t)g * slabs * mg * kD;
    v.Slo = w.Slo + (size_t)g * slabs * mg * kD;
  }
  v.S = w.S + (size_t)g * slabs * mg * kD;
  v.z = w.z + (size_t)g * slabs * mg;
  v.Sbf = w.Sbf + (size_t)g * slabs * mg * kD;
  v.Simg = w.Simg + (size_t)g * slabs * simg_bytes((int)mg);
  return v;
}

// Zero-padded 64-wide copies of the gate weights (heads x d x (L+1) -> heads x 64 x (L+1)) and of W (d x m -> 64 x m).
cudaError_t pad_parameters(const Plan& p, const Ws& w, const void* W, const float* gate_w, cudaStream_t st) {
  const int d = p.cfg.head_dim, m = p.cfg.features;
  const size_t es = p.bf16 ? 2 : 4;
  cudaError_t err = cudaMemsetAsync(w.Wp, 0, es * kD * m, st);
  if (err == cudaSuccess) err = cudaMemcpyAsync(w.Wp, W, es * (size_t)d * m, cudaMemcpyDeviceToDevice, st);
  if (err == cudaSuccess && gate_w != nullptr) {
    const size_t row = sizeof(float) * p.L1;
    err = cudaMemsetAsync(w.gwp, 0, row * kD * p.cfg.heads, st);
    if (err == cudaSuccess)
      err = cudaMemcpy2DAsync(w.gwp, row * kD, gate_w, row * d, row * d, p.cfg.heads, cudaMemcpyDeviceToDevice, st);
  }
  return err;
}

wersa_status clear_status_once(wersa_ctx* ctx, cudaStream_t st) {
  if (!ctx->status_cleared) {
    WERSA_CUDA(cudaMemsetAsync(ctx->ws.status, 0, ctx->plan.status_bytes, st));
    ctx->status_cleared = true;
  }
  return WERSA_OK;
}

}  // namespace

extern "C" {

size_t wersa_workspace_bytes(const wersa_config* cfg) {
  if (cfg == nullptr) return 0;
  Plan p;
  if (make_plan(*cfg, &p) != WERSA_OK) return 0;
  return p.total;
}

wersa_status wersa_create(const wersa_config* cfg, void* workspace, size_t workspace_bytes, wersa_ctx** out) {
  if (cfg == nullptr || out == nullptr) return WERSA_ERR_INVALID_ARG;
  Plan p;
  wersa_status s = make_plan(*cfg, &p);
  if (s != WERSA_OK) return s;
  if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 || workspace_bytes < p.total)
    return WERSA_ERR_WORKSPACE;
  wersa_ctx* ctx = new (std::nothrow) wersa_ctx;
  if (ctx == nullptr) return WERSA_ERR_INVALID_ARG;
  ctx->plan = p;
  ctx->workspace = workspace;
  ctx->ws = resolve(p, workspace);
  ctx->forward_done = false;
  ctx->status_cleared = false;
  ctx->launches_fwd = ctx->launches_bwd = 0;
  *out = ctx;
  return WERSA_OK;
}

wersa_status wersa_forward(wersa_ctx* ctx, const void* Q, const void* K, const void* V, const void* W,
                           const float* beta, const float* gate_w, const float* gate_b, const float* omega,
                           void* O, void* cuda_stream) {
  if (ctx == nullptr || Q == nullptr || K == nullptr || V == nullptr || W == nullptr || beta == nullptr ||
      omega == nullptr || O == nullptr)
    return WERSA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(W) || !aligned16(O))
    return WERSA_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  const Ws& w = ctx->ws;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  wersa_status s = clear_status_once(ctx, st);
  if (s != WERSA_OK) return s;
  int launches = 0;
  const int kind = p.bf16 ? 1 : 0;
  if ((s = begin_pass(ctx, 0, st)) != WERSA_OK) return s;
  const size_t rows = (size_t)p.slabs * p.cfg.seq_len;
  // Narrow heads: the tensor-core kernels and the mean pool read and write the narrow tensors themselves (the
  // tensor maps zero-fill the missing columns); the fp32 path runs on zero-padded copies (see glue.cu).
  const bool padded = p.dpad && p.fwd_cols == kD;
  if (padded) {
    WERSA_STEP(0, "pad_q", launch_pad_cols(Q, w.Qp, rows, p.cfg.head_dim, kind, st, &launches));
    WERSA_STEP(0, "pad_k", launch_pad_cols(K, w.Kp, rows, p.cfg.head_dim, kind, st, &launches));
    WERSA_STEP(0, "pad_v", launch_pad_cols(V, w.Vp, rows, p.cfg.head_dim, kind, st, &launches));
    WERSA_CUDA(pad_parameters(p, w, W, gate_w, st));
    Q = w.Qp;
    K = w.Kp;
    V = w.Vp;
    W = w.Wp;
    if (gate_w != nullptr) gate_w = w.gwp;
  }
  void* Ocore = padded ? w.Op : O;
  WERSA_STEP(0, "qmean_gate",
             launch_qmean_gate(p, w, Q, gate_w, gate_b, omega, p.use_tc ? W : nullptr, p.fwd_cols, st, &launches));
  if (p.groups > 1) {
    // feature groups of 256 (tensor-core path): every group runs the key side and the query side on its own
    // rows of W^T; the query side leaves O_g and the denominators, which the last launch combines
    const Plan pg = group_plan(p);
    const size_t es = p.bf16 ? 2 : 4;
    for (int g = 0; g < p.groups; ++g) {
      const Ws wg = group_view(p, w, g, p.tchunks);
      WERSA_STEP(0, "tc_kside", launch_tc_kside(pg, wg, K, V, st, &launches));
      if (p.tchunks > 1)
        WERSA_STEP(0, "reduce_partials",
                   launch_reduce_partials(pg, wg.spart, wg.zpart, p.tchunks, wg.S, wg.z, wg.Sbf, wg.Simg, st, &launches));
      WERSA_STEP(0, "tc_qside",
                 launch_tc_qside(pg, wg, Q, beta, static_cast<char*>(w.Og) + (size_t)g * rows * kD * es,
                                 w.den + (size_t)g * rows, st, &launches));
    }
    WERSA_STEP(0, "combine_groups",
               launch_combine_groups(w.Og, w.den, Ocore, rows, p.groups, p.fwd_cols, kind, st, &launches));
    WERSA_STEP(0, "gather_groups",
               launch_gather_groups(w.S, w.z, w.Sout, w.zout, p.slabs, p.groups, kGroupFeatures, st, &launches));
  } else if (p.use_tc) {
    WERSA_STEP(0, "tc_kside", launch_tc_kside(p, w, K, V, st, &launches));
    if (p.tchunks > 1)   // with one chunk per slab the key-side kernel has written S', z' and the image itself
      WERSA_STEP(0, "reduce_partials",
                 launch_reduce_partials(p, w.spart, w.zpart, p.tchunks, w.S, w.z, w.Sbf, w.Simg, st, &launches));
    WERSA_STEP(0, "tc_qside", launch_tc_qside(p, w, Q, beta, Ocore, nullptr, st, &launches));
  } else {
    WERSA_STEP(0, "haar_filter_q", launch_haar_filter(p, Q, kind, w.f, w.QF, 0, st, &launches));
    WERSA_STEP(0, "haar_filter_k", launch_haar_filter(p, K, kind, w.f, w.KF, 0, st, &launches));
    WERSA_STEP(0, "simt_kside", launch_simt_kside(p, w, V, W, st, &launches));
    WERSA_STEP(0, "reduce_partials",
               launch_reduce_partials(p, w.spart, w.zpart, p.schunks, w.S, w.z, nullptr, nullptr, st, &launches));
    WERSA_STEP(0, "simt_qside", launch_simt_qside(p, w, W, beta, Ocore, st, &launches));
  }
  if (padded) WERSA_STEP(0, "unpad_o", launch_unpad_cols(w.Op, O, rows, p.cfg.head_dim, kind, st, &launches));
  ctx->launches_fwd = launches;
  ctx->forward_done = true;
  return WERSA_OK;
}

// ---- sequence-sharded forward ------------------------------------------------------------------------
// The four steps of wersa_forward with the two places opened where shards of one sequence have to exchange
// sums: after the mean pool (column sums of Q) and after the key side (S', z').  Tensor-core path, one feature
// group; the context is created with the shard's own length.
static bool shardable(const Plan& p) { return p.use_tc && p.groups == 1; }

wersa_status wersa_shard_pool(wersa_ctx* ctx, const void* Q, const void* W, float* qsum, void* cuda_stream) {
  if (ctx == nullptr || Q == nullptr || W == nullptr || qsum == nullptr) return WERSA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(W)) return WERSA_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  if (!shardable(p)) return WERSA_ERR_UNSUPPORTED;
  const Ws& w = ctx->ws;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  wersa_status s = clear_status_once(ctx, st);
  if (s != WERSA_OK) return s;
  int launches = 0;
  // (the gate this launch also computes belongs to the shard alone and is replaced by wersa_shard_gate)
  WERSA_CUDA(launch_qmean_gate(p, w, Q, nullptr, nullptr, nullptr, W, p.fwd_cols, st, &launches));
  WERSA_CUDA(launch_shard_qsum(p, w, qsum, st, &launches));
  ctx->launches_fwd = launches;
  ctx->forward_done = false;
  return WERSA_OK;
}

wersa_status wersa_shard_gate(wersa_ctx* ctx, const float* qsum_total, int64_t n_total, const float* gate_w,
                              const float* gate_b, const float* omega, void* cuda_stream) {
  if (ctx == nullptr || qsum_total == nullptr || omega == nullptr || n_total < 1 || n_total > 0x7fffffffLL)
    return WERSA_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  if (!shardable(p)) return WERSA_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  int launches = 0;
  WERSA_CUDA(launch_gate_from_sums(p, ctx->ws, qsum_total, n_total, gate_w, gate_b, omega, p.fwd_cols, st, &launches));
  ctx->launches_fwd += launches;
  return WERSA_OK;
}

wersa_status wersa_shard_keys(wersa_ctx* ctx, const void* K, const void* V, void* cuda_stream) {
  if (ctx == nullptr || K == nullptr || V == nullptr) return WERSA_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V)) return WERSA_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  if (!shardable(p)) return WERSA_ERR_UNSUPPORTED;
  const Ws& w = ctx->ws;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  int launches = 0;
  WERSA_CUDA(launch_tc_kside(p, w, K, V, st, &launches));
  if (p.tchunks > 1)
    WERSA_CUDA(launch_reduce_partials(p, w.spart, w.zpart, p.tchunks, w.S, w.z, w.Sbf, w.Simg, st, &launches));
  ctx->launches_fwd += launches;
  ctx->forward_done = true;   // S', z' of this shard can be read with wersa_saved
  return WERSA_OK;
}

wersa_status wersa_shard_output(wersa_ctx* ctx, const void* Q, const float* S_total, const float* z_total,
                                const float* beta, void* O, void* cuda_stream) {
  if (ctx == nullptr || Q == nullptr || S_total == nullptr || z_total == nullptr || beta == nullptr || O == nullptr)
    return WERSA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(O)) return WERSA_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  if (!shardable(p)) return WERSA_ERR_UNSUPPORTED;
  const Ws& w = ctx->ws;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  int launches = 0;
  // the totals take the place of a single partial: the reduction copies them and writes the operand images
  WERSA_CUDA(launch_reduce_partials(p, S_total, z_total, 1, w.S, w.z, w.Sbf, w.Simg, st, &launches));
  WERSA_CUDA(launch_tc_qside(p, w, Q, beta, O, nullptr, st, &launches));
  ctx->launches_fwd += launches;
  return WERSA_OK;
}

// ---- sequence-sharded backward: three steps with the sums of dS', dz' and of (df, sum dD') taken by the caller
static bool shardable_bwd(const Plan& p) { return shardable(p) && p.with_backward && !p.dpad; }

wersa_status wersa_shard_backward_queries(wersa_ctx* ctx, const void* Q, const float* beta, const void* dO,
                                          void* cuda_stream) {
  if (ctx == nullptr || Q == nullptr || beta == nullptr || dO == nullptr) return WERSA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(dO)) return WERSA_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  if (!shardable_bwd(p)) return WERSA_ERR_UNSUPPORTED;
  if (!ctx->forward_done) return WERSA_ERR_STATE;
  const Ws& w = ctx->ws;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  int launches = 0;
  const int kind = 1, gkind = p.grad_bf16 ? 1 : 0;
  WERSA_CUDA(launch_haar_filter_split3(p, Q, kind, w.f, w.QF3, st, &launches));
  WERSA_CUDA(launch_tc_bwd_qside(p, w, w.QF3, beta, dO, nullptr, nullptr, false, st, &launches));
  WERSA_CUDA(launch_reduce_partials(p, w.spart, w.zpart, p.bchunks, w.dS, w.dz, w.dSbf, nullptr, st, &launches));
  WERSA_CUDA(launch_haar_backward(p, w, Q, kind, w.dQF, nullptr, gkind, 0, st, &launches));   // band inner products
  ctx->launches_bwd = launches;
  return WERSA_OK;
}

wersa_status wersa_shard_backward_keys(wersa_ctx* ctx, const void* K, const void* V, const float* dS_total,
                                       const float* dz_total, void* dK, void* dV, void* cuda_stream) {
  if (ctx == nullptr || K == nullptr || V == nullptr || dS_total == nullptr || dz_total == nullptr || dK == nullptr ||
      dV == nullptr)
    return WERSA_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(dK) || !aligned16(dV)) return WERSA_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  if (!shardable_bwd(p)) return WERSA_ERR_UNSUPPORTED;
  if (!ctx->forward_done) return WERSA_ERR_STATE;
  const Ws& w = ctx->ws;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  int launches = 0;
  const int kind = 1, gkind = p.grad_bf16 ? 1 : 0;
  // the totals take the place of a single partial: the reduction copies them and writes the bf16 image of dS'
  WERSA_CUDA(launch_reduce_partials(p, dS_total, dz_total, 1, w.dS, w.dz, w.dSbf, nullptr, st, &launches));
  WERSA_CUDA(launch_haar_filter_split3(p, K, kind, w.f, w.KF3, st, &launches));
  WERSA_CUDA(launch_tc_bwd_kside(p, w, w.KF3, V, dV, false, st, &launches));
  WERSA_CUDA(launch_haar_backward(p, w, K, kind, w.dKF, dK, gkind, 1, st, &launches));
  float* df = w.dqbar + (size_t)p.slabs * kD;
  WERSA_CUDA(launch_band_sums(p, w, p.slabs * p.bchunks, df, w.shardtot, st, &launches));
  ctx->launches_bwd += launches;
  return WERSA_OK;
}

wersa_status wersa_shard_backward_gate(wersa_ctx* ctx, const float* df_total, const float* sumdD_total, int64_t n_total,
                                       const float* beta, const float* gate_w, const float* omega, float* dbeta,
                                       float* dgate_w, float* dgate_b, float* domega, void* dQ, void* cuda_stream) {
  if (ctx == nullptr || df_total == nullptr || sumdD_total == nullptr || beta == nullptr || omega == nullptr ||
      dQ == nullptr || n_total < 1)
    return WERSA_ERR_INVALID_ARG;
  if (!aligned16(dQ)) return WERSA_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  if (!shardable_bwd(p)) return WERSA_ERR_UNSUPPORTED;
  if (!ctx->forward_done) return WERSA_ERR_STATE;
  const Ws& w = ctx->ws;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  int launches = 0;
  WERSA_CUDA(launch_gate_backward_from(p, w, df_total, sumdD_total, beta, gate_w, omega, dbeta, dgate_w, dgate_b, domega,
                                       st, &launches));
  WERSA_CUDA(launch_haar_filter_addvec(p, w.dQF, w.f, w.dqbar, 1.f / (float)n_total, dQ, p.grad_bf16 ? 1 : 0, st,
                                       &launches));
  ctx->launches_bwd += launches;
  return WERSA_OK;
}

wersa_status wersa_forward_host(wersa_ctx* ctx, const void* hQ, const void* hK, const void* hV, void* dQ,
                                void* dK, void* dV, const void* W, const float* beta, const float* gate_w,
                                const float* gate_b, const float* omega, void* dO, void* hO, void* cuda_stream) {
  if (ctx == nullptr || hQ == nullptr || hK == nullptr || hV == nullptr || hO == nullptr || dQ == nullptr ||
      dK == nullptr || dV == nullptr || dO == nullptr || W == nullptr || beta == nullptr || omega == nullptr)
    return WERSA_ERR_INVALID_ARG;
  if (!aligned16(dQ) || !aligned16(dK) || !aligned16(dV) || !aligned16(dO) || !aligned16(W))
    return WERSA_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t bytes = (size_t)p.slabs * p.cfg.seq_len * p.cfg.head_dim * (p.bf16 ? 2 : 4);
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  WERSA_CUDA(cudaMemcpyAsync(dQ, hQ, bytes, cudaMemcpyHostToDevice, st));
  WERSA_CUDA(cudaMemcpyAsync(dK, hK, bytes, cudaMemcpyHostToDevice, st));
  WERSA_CUDA(cudaMemcpyAsync(dV, hV, bytes, cudaMemcpyHostToDevice, st));
  const wersa_status s = wersa_forward(ctx, dQ, dK, dV, W, beta, gate_w, gate_b, omega, dO, cuda_stream);
  if (s != WERSA_OK) return s;
  WERSA_CUDA(cudaMemcpyAsync(hO, dO, bytes, cudaMemcpyDeviceToHost, st));
  return WERSA_OK;
}

wersa_status wersa_backward(wersa_ctx* ctx, const void* Q, const void* K, const void* V, const void* W,
                            const float* beta, const float* gate_w, const float* gate_b, const float* omega,
                            const void* dO, void* dQ, void* dK, void* dV, float* dbeta, float* dgate_w,
                            float* dgate_b, float* domega, void* cuda_stream) {
  (void)gate_b;
  if (ctx == nullptr || Q == nullptr || K == nullptr || V == nullptr || W == nullptr || beta == nullptr ||
      omega == nullptr || dO == nullptr || dQ == nullptr || dK == nullptr || dV == nullptr)
    return WERSA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(W) || !aligned16(dO) || !aligned16(dQ) ||
      !aligned16(dK) || !aligned16(dV))
    return WERSA_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  if (!p.with_backward) return WERSA_ERR_UNSUPPORTED;
  if (!ctx->forward_done) return WERSA_ERR_STATE;
  const Ws& w = ctx->ws;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  int launches = 0;
  const int kind = p.bf16 ? 1 : 0, gkind = p.grad_bf16 ? 1 : 0;
  wersa_status s = begin_pass(ctx, 1, st);
  if (s != WERSA_OK) return s;
  const int bwd_chunks = p.use_tc ? p.bchunks : p.schunks;   // chunks per slab of the dS', dz', sum dD' partials
  const size_t rows = (size_t)p.slabs * p.cfg.seq_len;
  void *dQ_out = dQ, *dK_out = dK, *dV_out = dV;
  float* dgate_w_out = dgate_w;
  if (p.dpad) {   // the zero-padded 64-wide problem: gradients come back 64 wide and are cut to head_dim columns
    WERSA_STEP(1, "pad_q", launch_pad_cols(Q, w.Qp, rows, p.cfg.head_dim, kind, st, &launches));
    WERSA_STEP(1, "pad_k", launch_pad_cols(K, w.Kp, rows, p.cfg.head_dim, kind, st, &launches));
    WERSA_STEP(1, "pad_v", launch_pad_cols(V, w.Vp, rows, p.cfg.head_dim, kind, st, &launches));
    WERSA_STEP(1, "pad_do", launch_pad_cols(dO, w.dOp, rows, p.cfg.head_dim, kind, st, &launches));
    WERSA_CUDA(pad_parameters(p, w, W, gate_w, st));
    Q = w.Qp;
    K = w.Kp;
    V = w.Vp;
    W = w.Wp;
    dO = w.dOp;
    dQ = w.dQp;
    dK = w.dKp;
    dV = w.dVp;
    if (gate_w != nullptr) gate_w = w.gwp;
    if (dgate_w != nullptr) dgate_w = w.dgwp;
  }
  if (p.groups > 1) {
    // Feature groups: the denominator and dD' of the whole map come from what the forward left (the groups'
    // outputs and denominators); every group then runs both tensor-core kernels on its own rows of W^T, S', z',
    // dS', dz', and dQ_F, dV, dK_F accumulate over the groups in launch order.
    WERSA_STEP(1, "haar_filter_q", launch_haar_filter_split3(p, Q, kind, w.f, w.QF3, st, &launches));
    WERSA_STEP(1, "haar_filter_k", launch_haar_filter_split3(p, K, kind, w.f, w.KF3, st, &launches));
    WERSA_STEP(1, "group_bwd_prep",
               launch_group_bwd_prep(w.Og, w.den, dO, w.f, p.cfg.seq_len, p.L1, rows, p.groups, kind, w.Dtot,
                                     w.Dtot + rows, st, &launches));
    const Plan pg = group_plan(p);
    for (int g = 0; g < p.groups; ++g) {
      const Ws wg = group_view(p, w, g, bwd_chunks);
      WERSA_STEP(1, "tc_bwd_qside",
                 launch_tc_bwd_qside(pg, wg, w.QF3, beta, dO, w.Dtot, w.Dtot + rows, g > 0, st, &launches));
      WERSA_STEP(1, "reduce_partials",
                 launch_reduce_partials(pg, wg.spart, wg.zpart, bwd_chunks, wg.dS, wg.dz, wg.dSbf, nullptr, st, &launches));
      WERSA_STEP(1, "tc_bwd_kside", launch_tc_bwd_kside(pg, wg, w.KF3, V, dV, g > 0, st, &launches));
    }
  } else if (p.use_tc) {
    // the tensor-core forward keeps Q_F, K_F on chip: rebuild them, as three bf16 planes each
    WERSA_STEP(1, "haar_filter_q", launch_haar_filter_split3(p, Q, kind, w.f, w.QF3, st, &launches));
    WERSA_STEP(1, "haar_filter_k", launch_haar_filter_split3(p, K, kind, w.f, w.KF3, st, &launches));
    WERSA_STEP(1, "tc_bwd_qside", launch_tc_bwd_qside(p, w, w.QF3, beta, dO, nullptr, nullptr, false, st, &launches));
  } else {
    WERSA_STEP(1, "simt_bwd_qside", launch_simt_bwd_qside(p, w, W, beta, dO, st, &launches));
  }
  if (p.groups == 1)
    WERSA_STEP(1, "reduce_partials",
               launch_reduce_partials(p, w.spart, w.zpart, bwd_chunks, w.dS, w.dz, p.use_tc ? w.dSbf : nullptr, nullptr,
                                      st, &launches));
  if (p.groups > 1) {
    // (done group by group above)
  } else if (p.use_tc) {
    WERSA_STEP(1, "tc_bwd_kside", launch_tc_bwd_kside(p, w, w.KF3, V, dV, false, st, &launches));
  } else {
    WERSA_STEP(1, "simt_bwd_kside", launch_simt_bwd_kside(p, w, V, W, dV, st, &launches));
  }
  // With gate weights dQ has a second term, d(qbar) / n on every row (Eq. 1), which is known only after the
  // gate backward: the first pass over dQ_F then takes the band inner products alone, and dQ is written
  // once, by a filter pass that adds the row vector.
  const bool pooled_term = gate_w != nullptr;
  WERSA_STEP(1, "haar_backward_q",
             launch_haar_backward(p, w, Q, kind, w.dQF, pooled_term ? nullptr : dQ, gkind, 0, st, &launches));
  WERSA_STEP(1, "haar_backward_k", launch_haar_backward(p, w, K, kind, w.dKF, dK, gkind, 1, st, &launches));
  WERSA_STEP(1, "gate_backward",
             launch_gate_backward(p, w, beta, gate_w, omega, p.slabs * bwd_chunks, dbeta, dgate_w, dgate_b, domega, st,
                                  &launches));
  if (pooled_term)
    WERSA_STEP(1, "haar_filter_dq",
               launch_haar_filter_addvec(p, w.dQF, w.f, w.dqbar, 1.f / (float)p.cfg.seq_len, dQ, gkind, st, &launches));
  if (p.dpad) {
    WERSA_STEP(1, "unpad_dq", launch_unpad_cols(w.dQp, dQ_out, rows, p.cfg.head_dim, gkind, st, &launches));
    WERSA_STEP(1, "unpad_dk", launch_unpad_cols(w.dKp, dK_out, rows, p.cfg.head_dim, gkind, st, &launches));
    WERSA_STEP(1, "unpad_dv", launch_unpad_cols(w.dVp, dV_out, rows, p.cfg.head_dim, gkind, st, &launches));
    if (dgate_w_out != nullptr) {
      const size_t row = sizeof(float) * p.L1;
      WERSA_CUDA(cudaMemcpy2DAsync(dgate_w_out, row * p.cfg.head_dim, w.dgwp, row * kD, row * p.cfg.head_dim,
                                   p.cfg.heads, cudaMemcpyDeviceToDevice, st));
    }
  }
  ctx->launches_bwd = launches;
  return WERSA_OK;
}

wersa_status wersa_haar_filter(wersa_ctx* ctx, const void* X, const float* f, void* XF, void* cuda_stream) {
  if (ctx == nullptr || X == nullptr || f == nullptr || XF == nullptr) return WERSA_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(XF)) return WERSA_ERR_INVALID_ARG;
  const Plan& p = ctx->plan;
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  int launches = 0;
  const int kind = p.bf16 ? 1 : 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (p.dpad) {
    const size_t rows = (size_t)p.slabs * p.cfg.seq_len;
    WERSA_CUDA(launch_pad_cols(X, ctx->ws.Qp, rows, p.cfg.head_dim, kind, st, &launches));
    WERSA_CUDA(launch_haar_filter(p, ctx->ws.Qp, kind, f, ctx->ws.Op, kind, st, &launches));
    WERSA_CUDA(launch_unpad_cols(ctx->ws.Op, XF, rows, p.cfg.head_dim, kind, st, &launches));
    return WERSA_OK;
  }
  WERSA_CUDA(launch_haar_filter(p, X, kind, f, XF, kind, st, &launches));
  return WERSA_OK;
}

wersa_status wersa_gate_static(const wersa_config* cfg, const void* Q, const float* gate_w, const float* gate_b,
                               const float* omega, float* qbar, float* f, void* cuda_stream) {
  if (cfg == nullptr || Q == nullptr || omega == nullptr || qbar == nullptr || f == nullptr)
    return WERSA_ERR_INVALID_ARG;
  if (!aligned16(Q)) return WERSA_ERR_INVALID_ARG;
  Plan p;
  wersa_status s = make_plan(*cfg, &p);
  if (s != WERSA_OK) return s;
  if (p.dpad) return WERSA_ERR_UNSUPPORTED;   // no workspace to pad into
  if (static_scratch_floats_needed(p) > static_scratch_capacity_floats() ||
      static_scratch_counters_needed(p) > static_scratch_counter_capacity())
    return WERSA_ERR_TOO_LARGE;
  DeviceGuard guard(p.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  float* scratch = nullptr;
  WERSA_CUDA(static_scratch_address(p.cfg.device, &scratch));
  WERSA_CUDA(launch_qmean_gate_static(p, scratch, Q, gate_w, gate_b, omega, qbar, f,
                                      static_cast<cudaStream_t>(cuda_stream)));
  return WERSA_OK;
}

wersa_status wersa_saved(wersa_ctx* ctx, int which, const float** device_ptr, size_t* count) {
  if (ctx == nullptr || device_ptr == nullptr || count == nullptr) return WERSA_ERR_INVALID_ARG;
  if (!ctx->forward_done) return WERSA_ERR_STATE;
  const Plan& p = ctx->plan;
  const size_t slabs = (size_t)p.slabs;
  switch (which) {
    case 0: *device_ptr = ctx->ws.f; *count = slabs * p.L1; break;
    case 1: *device_ptr = ctx->ws.qbar; *count = slabs * kD; break;
    case 2: *device_ptr = p.groups > 1 ? ctx->ws.Sout : ctx->ws.S; *count = slabs * p.cfg.features * kD; break;
    case 3: *device_ptr = p.groups > 1 ? ctx->ws.zout : ctx->ws.z; *count = slabs * p.cfg.features; break;
    // sequence-sharded backward: this shard's dS', dz', band inner products and sum of dD'
    case 4: if (!p.with_backward) return WERSA_ERR_UNSUPPORTED; *device_ptr = ctx->ws.dS; *count = slabs * p.cfg.features * kD; break;
    case 5: if (!p.with_backward) return WERSA_ERR_UNSUPPORTED; *device_ptr = ctx->ws.dz; *count = slabs * p.cfg.features; break;
    case 6: if (!p.with_backward) return WERSA_ERR_UNSUPPORTED; *device_ptr = ctx->ws.dqbar + slabs * kD; *count = slabs * kBandVals; break;
    case 7: if (!p.with_backward) return WERSA_ERR_UNSUPPORTED; *device_ptr = ctx->ws.shardtot; *count = 1; break;
    default: return WERSA_ERR_INVALID_ARG;
  }
  return WERSA_OK;
}

wersa_status wersa_query_status(wersa_ctx* ctx, void* cuda_stream) {
  if (ctx == nullptr) return WERSA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(ctx->plan.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  WERSA_CUDA(cudaStreamSynchronize(st));
  if (!ctx->status_cleared) return WERSA_OK;   // nothing has run yet
  int word = 0;
  WERSA_CUDA(cudaMemcpyAsync(&word, ctx->ws.status, sizeof(int), cudaMemcpyDeviceToHost, st));
  WERSA_CUDA(cudaStreamSynchronize(st));
  if (word != 0) {
    WERSA_CUDA(cudaMemsetAsync(ctx->ws.status, 0, 256, st));
    WERSA_CUDA(cudaStreamSynchronize(st));
    return WERSA_ERR_TIMEOUT;
  }
  return WERSA_OK;
}

wersa_status wersa_selftest_wait_timeout(wersa_ctx* ctx, uint32_t limit_us, int32_t* observed, void* cuda_stream) {
  if (ctx == nullptr || observed == nullptr || limit_us == 0 || limit_us > 100000) return WERSA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(ctx->plan.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  wersa_status s = clear_status_once(ctx, st);
  if (s != WERSA_OK) return s;
  WERSA_CUDA(launch_selftest_wait(ctx->ws, 1000ull * limit_us, observed, st));
  return WERSA_OK;
}

wersa_status wersa_set_step_timing(wersa_ctx* ctx, int enable) {
  if (ctx == nullptr) return WERSA_ERR_INVALID_ARG;
  StepTimer& t = ctx->timer;
  if ((enable != 0) == t.enabled) return WERSA_OK;
  DeviceGuard guard(ctx->plan.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  if (enable) {
    for (int wch = 0; wch < 2; ++wch)
      for (int i = 0; i <= kMaxSteps; ++i) WERSA_CUDA(cudaEventCreate(&t.ev[wch][i]));
    t.count[0] = t.count[1] = 0;
    t.enabled = true;
  } else {
    t.enabled = false;
    for (int wch = 0; wch < 2; ++wch)
      for (int i = 0; i <= kMaxSteps; ++i) cudaEventDestroy(t.ev[wch][i]);
  }
  return WERSA_OK;
}

wersa_status wersa_step_times(wersa_ctx* ctx, int which, int capacity, float* ms, const char** names,
                              int* count) {
  if (ctx == nullptr || count == nullptr || which < 0 || which > 1) return WERSA_ERR_INVALID_ARG;
  StepTimer& t = ctx->timer;
  if (!t.enabled) return WERSA_ERR_STATE;
  DeviceGuard guard(ctx->plan.cfg.device);
  if (guard.err != cudaSuccess) return WERSA_ERR_CUDA;
  const int n = t.count[which];
  *count = n;
  if (n == 0) return WERSA_OK;
  WERSA_CUDA(cudaEventSynchronize(t.ev[which][n]));
  for (int i = 0; i < n && i < capacity; ++i) {
    if (ms != nullptr) WERSA_CUDA(cudaEventElapsedTime(&ms[i], t.ev[which][i], t.ev[which][i + 1]));
    if (names != nullptr) names[i] = t.name[which][i];
  }
  return WERSA_OK;
}

wersa_status wersa_destroy(wersa_ctx* ctx) {
  if (ctx != nullptr && ctx->timer.enabled) wersa_set_step_timing(ctx, 0);
  delete ctx;
  return WERSA_OK;
}

const char* wersa_status_string(wersa_status status) {
  switch (status) {
    case WERSA_OK: return "ok";
    case WERSA_ERR_INVALID_ARG: return "invalid argument";
    case WERSA_ERR_UNSUPPORTED: return "unsupported configuration";
    case WERSA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case WERSA_ERR_CUDA: return "CUDA runtime error";
    case WERSA_ERR_TIMEOUT: return "bounded device wait expired";
    case WERSA_ERR_STATE: return "backward or saved-tensor query without a preceding forward";
    case WERSA_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of wersa_gate_static (253952 floats + 8192 counters)";
  }
  return "unknown status";
}

int32_t wersa_uses_tensor_cores(const wersa_ctx* ctx) { return ctx != nullptr && ctx->plan.use_tc ? 1 : 0; }

int32_t wersa_launch_count(const wersa_ctx* ctx, int which) {
  if (ctx == nullptr) return 0;
  return which == 0 ? ctx->launches_fwd : ctx->launches_bwd;
}

}  // extern "C"
