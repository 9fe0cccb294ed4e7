/*
 * wersa.h -- C ABI of the B200 (sm_100a) implementation of the per-head WERSA attention
 * operator (Wavelet-Enhanced Random Spectral Attention, arXiv 2507.08637).
 *
 * The operator, per (batch, head) slab, with Q, K, V in R^{n x d} (Sec. 3.1, problem
 * statement) stored as (batch, heads, seq, head_dim) row-major (Algorithm 1, SplitHeads):
 *
 *   qbar = mean_t Q[t,:]                                   (Eq. 1)
 *   u    = gate_w^T qbar + gate_b ;  f_i = sigmoid(u_i) * omega_i, i = 0..L   (Eqs. 2-3)
 *   X_F  = IDWT_L( f (.) DWT_L(X) )  for X in {Q, K}, Haar wavelet along the sequence,
 *          coefficient order [d_1, ..., d_L, a_L]          (Sec. 3.1 steps 3,5,6; Algorithm 2)
 *   phi(x) = ReLU(x W / max(beta, bw_floor)) / sqrt(m)     (Eq. 6; Algorithm 1 scalings)
 *   S = phi(K_F)^T V,  z = phi(K_F)^T 1                    (Eq. 7, key summary / normaliser)
 *   O = phi(Q_F) S / (phi(Q_F) z + eps)                    (Eq. 7 / Sec. 3.1 step 8)
 *
 * Non-causal, unmasked.  One random matrix W (d x m) is shared by queries, keys and all
 * heads.  Everything runs on one GPU in hand-written CUDA kernels; there is no CPU path:
 * without a CUDA device every compute entry point returns WERSA_ERR_CUDA.
 *
 * Conventions
 *   - All tensor pointers are DEVICE pointers, dense, row-major, 16-byte aligned.
 *   - Q, K, V, O, dO, dQ, dK, dV: (batch, heads, seq_len, head_dim), head_dim contiguous.
 *   - W: (head_dim, features).  beta: 1 float.  gate_w: (heads, head_dim, levels+1) float.
 *     gate_b: (heads, levels+1) float.  omega: (levels+1) float; index i of the last axis
 *     addresses the wavelet band: 0 = finest detail d_1, ..., L-1 = d_L, L = approximation a_L.
 *   - The caller owns every tensor and the workspace; the library allocates no device memory.
 *   - forward/backward enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL =
 *     default stream) and return without synchronising.  A context is not thread-safe and
 *     carries one forward/backward at a time.
 *   - Errors are return codes; nothing is thrown, nothing aborts, no device trap is used.
 */
#ifndef WERSA_H_
#define WERSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct wersa_ctx wersa_ctx; /* opaque, host memory, owned by the library */

typedef enum {
  WERSA_OK = 0,
  WERSA_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, misaligned pointer      */
  WERSA_ERR_UNSUPPORTED = 2, /* valid problem outside the compiled set of shapes / types */
  WERSA_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small               */
  WERSA_ERR_CUDA = 4,        /* a CUDA runtime call failed (no device, launch error)     */
  WERSA_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired                       */
  WERSA_ERR_STATE = 6,       /* backward called without a preceding forward              */
  WERSA_ERR_TOO_LARGE = 7    /* problem exceeds the fixed scratch of wersa_gate_static   */
} wersa_status;

typedef enum { WERSA_F32 = 0, WERSA_BF16 = 1 } wersa_dtype;

/* Flags for wersa_config.flags. */
enum {
  WERSA_FLAG_SIMT_ONLY = 1,    /* bf16 storage but fp32 FFMA arithmetic everywhere (no tensor
                                  cores); the fp32 dtype always computes this way        */
  WERSA_FLAG_FORWARD_ONLY = 2  /* the context will never run wersa_backward: its workspace
                                  omits the gradient scratch buffers                     */
};

typedef struct wersa_config {
  int32_t batch;         /* B >= 1                                                      */
  int32_t heads;         /* H >= 1                                                      */
  int32_t seq_len;       /* n >= 2; 2^levels must not exceed the next power of two >= n */
  int32_t head_dim;      /* d: 8, 16, ... 64.  Below 64 the problem runs as its zero-padded
                            64-wide equivalent, which leaves Eqs. 1-7 unchanged: the bf16
                            tensor-core forward reads and writes the narrow tensors directly,
                            the fp32 path and the backward use padded copies in the workspace */
  int32_t levels;        /* L, Haar levels, 1..8                                        */
  int32_t features;      /* m, random features: 64, 128 or 256; with dtype bf16 and without
                            WERSA_FLAG_SIMT_ONLY also 512, 768 and 1024 (Sec. 3.3 uses 1024):
                            the features then run in groups of 256 whose outputs are combined
                            by their denominators (the cost grows with the number of groups) */
  int32_t dtype;         /* wersa_dtype of Q, K, V, W, O, dO; accumulation is fp32      */
  int32_t grad_dtype;    /* wersa_dtype of dQ, dK, dV                                   */
  float eps;             /* denominator epsilon of Eq. 7 (paper: "small constant")      */
  float bw_floor;        /* bw = max(beta, bw_floor) as in Algorithm 1                  */
  int32_t gate_per_head; /* 1: u[b,h] = gate_w[h]^T qbar[b,h] + gate_b[h]  (Sec. 3.1)
                            0: u[b] = sum_h gate_w[h]^T qbar[b,h] + gate_b[0], shared by
                               all heads of a batch element (Algorithm 1, W_filter)     */
  int32_t device;        /* CUDA device ordinal                                         */
  int32_t flags;         /* WERSA_FLAG_*                                                */
} wersa_config;

/* Bytes of device workspace a context of this configuration needs (a multiple of 256);
 * 0 if the configuration is invalid or unsupported.  Pure host arithmetic. */
size_t wersa_workspace_bytes(const wersa_config* cfg);

/* Validates cfg, records the plan (tiling, split-sequence chunking) and adopts `workspace`
 * (device memory, 256-byte aligned, >= wersa_workspace_bytes(cfg); must outlive the context
 * and must not be shared by contexts that run concurrently).  *out is set only on WERSA_OK.
 * Launches no kernel. */
wersa_status wersa_create(const wersa_config* cfg, void* workspace, size_t workspace_bytes,
                          wersa_ctx** out);

/* Forward pass of the operator defined at the top of this file (Sec. 3.1 steps 3-8, Eqs. 1-7).
 * Argument order follows the problem statement: Q, K, V, then the random projection, the
 * bandwidth and the scale-gating parameters.  gate_w may be NULL (treated as zeros).  O has the
 * dtype of the inputs.  Also leaves f, qbar, S and z in the workspace for wersa_backward and
 * wersa_saved.  Split-sequence partial sums are combined in a fixed order: results are
 * bit-identical from run to run. */
wersa_status wersa_forward(wersa_ctx* ctx, const void* Q, const void* K, const void* V,
                           const void* W, const float* beta, const float* gate_w,
                           const float* gate_b, const float* omega, void* O,
                           void* cuda_stream);

/* The same forward for tensors that live in HOST memory (the end-to-end path: Sec. 3.1 steps 3-8 with
 * the transfers a caller without device-resident activations has to pay).  Enqueues on cuda_stream, in
 * this order: copies of hQ, hK, hV (host; batch*heads*seq_len*head_dim elements of cfg.dtype each) into
 * the device staging buffers dQ, dK, dV; wersa_forward on them into the device buffer dO; a copy of dO
 * into hO (host).  The four staging buffers are caller-owned device memory of the same size, 16-byte
 * aligned; the library allocates nothing.  W, beta, gate_w, gate_b, omega are DEVICE pointers as for
 * wersa_forward (parameters stay resident).  With page-locked host buffers the call returns once the
 * work is enqueued; with pageable ones the copies may block.  hO is valid after cuda_stream has been
 * synchronised.  Errors: WERSA_ERR_INVALID_ARG on a NULL or misaligned pointer (nothing enqueued),
 * WERSA_ERR_CUDA if a copy cannot be enqueued, else wersa_forward's status. */
wersa_status wersa_forward_host(wersa_ctx* ctx, const void* hQ, const void* hK, const void* hV,
                                void* dQ, void* dK, void* dV, const void* W, const float* beta,
                                const float* gate_w, const float* gate_b, const float* omega,
                                void* dO, void* hO, void* cuda_stream);

/* Backward pass: gradients of sum(dO (.) O) with respect to Q, K, V (cfg.grad_dtype), beta
 * (1 float), gate_w (heads, head_dim, levels+1), gate_b (heads, levels+1; rows >= 1 are zero
 * when gate_per_head = 0) and omega (levels+1).  The paper does not write the backward pass;
 * it is the chain rule through Eqs. 1-7 with dReLU(a)/da = 1[a > 0].  W is a fixed random
 * matrix (Sec. 3.1 step 7) and gets no gradient.  Must follow a wersa_forward on the same
 * context with the same inputs (it reuses f, qbar, S, z).  Any of the five parameter-gradient
 * pointers may be NULL. */
wersa_status wersa_backward(wersa_ctx* ctx, const void* Q, const void* K, const void* V,
                            const void* W, const float* beta, const float* gate_w,
                            const float* gate_b, const float* omega, const void* dO, void* dQ,
                            void* dK, void* dV, float* dbeta, float* dgate_w, float* dgate_b,
                            float* domega, void* cuda_stream);

/* Stand-alone Haar filter (Sec. 3.1 steps 3, 5, 6; Algorithm 2): XF = IDWT_L(f (.) DWT_L(X))
 * for every slab of X (batch, heads, seq_len, head_dim; cfg.dtype), with f a device array
 * (batch*heads, levels+1) of floats.  XF has cfg.dtype.  Each element of X is read once. */
wersa_status wersa_haar_filter(wersa_ctx* ctx, const void* X, const float* f, void* XF,
                               void* cuda_stream);

/* Mean-pooled query and gate (Eqs. 1-3) for callers that cannot hand the library a workspace.
 * (The paper has no counterpart of this entry point; it computes what wersa_forward's first step
 * computes.)  Some callers cannot allocate device memory at the point where they need the gate:
 * code running under an allocator that is frozen or owned by someone else (an inference server's
 * pre-sized arena, a plugin inside another framework's memory plan), or a process whose device
 * memory is already fully committed.  For them this entry point needs no context and no
 * workspace: the per-chunk partial sums of Q and the sigmoid values go to a fixed 1 MiB
 * (262144 floats) array that is part of the library image on every GPU that loads it, for as
 * long as the process lives.  The entry point never calls cudaMalloc, cudaFree or any allocating
 * routine.
 *   cfg    as for wersa_create (only shapes, dtype, gate_per_head and device are used).
 *   Q      (batch, heads, seq_len, head_dim) of cfg->dtype; gate_w, gate_b may be NULL (zeros).
 *   qbar   out, (batch*heads, head_dim) floats;  f  out, (batch*heads, levels+1) floats.
 * Returns WERSA_ERR_TOO_LARGE, launching nothing, when batch*heads*(64*chunks + levels+1) exceeds the
 * 253952 floats the array leaves for sums (chunks is the number of row chunks the mean pool splits the
 * sequence into, about four per multiprocessor over all slabs -- 592/(batch*heads) on a B200 --, at least 1), or when batch*heads + batch exceeds the 8192
 * arrival counters kept in the array's last 8192 elements: all five benchmark configurations fit.
 * The first call on a device resolves the array's device address (once per device, with that
 * device made current); make that first call outside any CUDA stream capture.  The address is kept for
 * the life of the process: do not reset the device (cudaDeviceReset) while the library is loaded.
 * Every call on a device shares the one array, and the array keeps what the last call left.  The partial
 * sums and sigmoid values a call reads are written earlier in the same call.  The arrival counters live at
 * a fixed place at the end of the array, whatever the problem's shape, and every call clears the ones it
 * uses with a memset on cuda_stream ahead of its kernel: calls of different shapes may follow each other
 * in any order, and a call that failed half way does not disturb the next.  Two calls that overlap on the
 * GPU (different streams, no ordering between them) race on the array and must be serialised by the
 * caller. */
wersa_status wersa_gate_static(const wersa_config* cfg, const void* Q, const float* gate_w,
                               const float* gate_b, const float* omega, float* qbar, float* f,
                               void* cuda_stream);

/* Sequence-sharded forward.  (The paper runs one GPU; Sec. 3.2's linear cost is what makes sequences longer
 * than one device's memory worth having.)  The sequence of every slab is cut into contiguous shards, one per
 * rank, every shard but the last a multiple of 2^levels tokens long, so that no wavelet block straddles two
 * shards (all shards but the last must therefore also be at least 2^levels long).  Each rank creates its
 * context with seq_len = its shard's length and calls, on one stream and in this order:
 *   wersa_shard_pool    Q shard, W -> qsum (batch*heads, 64) floats: column sums of the shard's Q
 *                       (columns >= head_dim zero).  The caller adds the qsum of all shards.
 *   wersa_shard_gate    the added sums and the whole sequence's length n_total -> gate (Eqs. 1-3), kept in the
 *                       context.
 *   wersa_shard_keys    K, V shards -> this shard's S', z' (read them with wersa_saved, which = 2 and 3).  The
 *                       caller adds the S' and the z' of all shards (Eq. 7's sums over the tokens).
 *   wersa_shard_output  Q shard, the added S_total (batch*heads, features, 64) and z_total (batch*heads,
 *                       features), beta -> O shard.
 * The two additions are the only exchange between ranks (an all-reduce each; the library does not do them).
 * bf16 tensor-core contexts with features <= 256 only, else WERSA_ERR_UNSUPPORTED.
 *
 * Backward of the same (the chain rule through Eqs. 1-7, as wersa_backward; head_dim = 64 and a context created
 * without WERSA_FLAG_FORWARD_ONLY), after the four forward steps, again on one stream and in this order:
 *   wersa_shard_backward_queries  Q, dO shards -> this shard's dS' and dz' (wersa_saved, which = 4 and 5).  The
 *                                 caller adds them over all shards.
 *   wersa_shard_backward_keys     K, V shards and the added dS_total, dz_total -> dK, dV shards, and this shard's
 *                                 band inner products df (batch*heads, 16) and sum of dD' (1 float) (wersa_saved,
 *                                 which = 6 and 7).  The caller adds both over all shards.
 *   wersa_shard_backward_gate     the added df_total, sumdD_total and n_total -> dbeta, dgate_w, dgate_b, domega
 *                                 (the same on every rank; any may be NULL) and the dQ shard. */
wersa_status wersa_shard_pool(wersa_ctx* ctx, const void* Q, const void* W, float* qsum, void* cuda_stream);
wersa_status wersa_shard_gate(wersa_ctx* ctx, const float* qsum_total, int64_t n_total, const float* gate_w,
                              const float* gate_b, const float* omega, void* cuda_stream);
wersa_status wersa_shard_keys(wersa_ctx* ctx, const void* K, const void* V, void* cuda_stream);
wersa_status wersa_shard_output(wersa_ctx* ctx, const void* Q, const float* S_total, const float* z_total,
                                const float* beta, void* O, void* cuda_stream);

wersa_status wersa_shard_backward_queries(wersa_ctx* ctx, const void* Q, const float* beta, const void* dO,
                                          void* cuda_stream);
wersa_status wersa_shard_backward_keys(wersa_ctx* ctx, const void* K, const void* V, const float* dS_total,
                                       const float* dz_total, void* dK, void* dV, void* cuda_stream);
wersa_status wersa_shard_backward_gate(wersa_ctx* ctx, const float* df_total, const float* sumdD_total,
                                       int64_t n_total, const float* beta, const float* gate_w, const float* omega,
                                       float* dbeta, float* dgate_w, float* dgate_b, float* domega, void* dQ,
                                       void* cuda_stream);

/* Device pointers into the workspace of quantities the last forward left there.
 * which: 0 = f (batch*heads, levels+1); 1 = qbar (batch*heads, 64);
 *        2 = S' (batch*heads, features, 64); 3 = z' (batch*heads, features),
 * the last axis of qbar and S' being the padded head dimension (columns >= head_dim are zero),
 * where S' = ReLU(K_F W)^T V and z' = ReLU(K_F W)^T 1 are the key summary and normaliser of
 * Eq. 7 without the 1/(bw sqrt(m)) factor of the feature map (S = S' / (bw sqrt(m))).
 * which = 4 .. 7 are the sequence-sharded backward's exchange quantities (see wersa_shard_backward_*).
 * *count receives the number of floats. */
wersa_status wersa_saved(wersa_ctx* ctx, int which, const float** device_ptr, size_t* count);

/* Synchronises `cuda_stream`, then returns WERSA_ERR_TIMEOUT if a kernel of this context gave
 * up on a bounded wait, WERSA_ERR_CUDA on a sticky CUDA error, else WERSA_OK.  Clears the
 * device-side error word. */
wersa_status wersa_query_status(wersa_ctx* ctx, void* cuda_stream);

/* Self-test of the error path behind WERSA_ERR_TIMEOUT (the paper has no counterpart).  Every wait of the
 * tensor-core kernels on a shared-memory barrier is bounded; when one runs out, the waiting role records
 * a code in the context's device status word, raises the CTA's abort flag and every role leaves without
 * touching further data.  This call enqueues one small CTA that runs exactly that path: it waits, for at
 * most limit_us microseconds (1..100000), on a barrier that is one arrival short, while a second role
 * waits for a hand-off that therefore never comes.  Nothing faults and nothing waits longer than the
 * limit.  observed: DEVICE pointer to 3 ints, written by the kernel: [0] the abort flag (1), [1] and [2]
 * whether the two roles' waits succeeded (0 and 0).  Afterwards wersa_query_status returns
 * WERSA_ERR_TIMEOUT once and WERSA_OK from then on. */
wersa_status wersa_selftest_wait_timeout(wersa_ctx* ctx, uint32_t limit_us, int32_t* observed,
                                         void* cuda_stream);

/* Releases the host-side context.  Does not touch the workspace.  NULL is accepted. */
wersa_status wersa_destroy(wersa_ctx* ctx);

/* Static, human-readable name of a status code. */
const char* wersa_status_string(wersa_status status);

/* Number of kernels the last forward (which = 0) or backward (which = 1) on this context
 * launched; 0 before the first call. */
int32_t wersa_launch_count(const wersa_ctx* ctx, int which);

/* 1 if this context's forward runs the bf16 tcgen05 tensor-core kernels, 0 if it runs the fp32
 * FFMA kernels (fp32 storage, WERSA_FLAG_SIMT_ONLY, or a shape the tensor-core kernels do not
 * cover). */
int32_t wersa_uses_tensor_cores(const wersa_ctx* ctx);

/* Step timing (a measurement aid; the paper has no counterpart).  When enabled, forward and
 * backward record a CUDA event on `cuda_stream` before their first launch and after each step
 * (a step is one kernel, or two for the gate).  Enabling creates the events, disabling destroys
 * them; neither touches device memory. */
wersa_status wersa_set_step_timing(wersa_ctx* ctx, int enable);

/* Durations of the steps of the last forward (which = 0) or backward (which = 1), in
 * milliseconds, after waiting for that pass to finish.  Writes min(*count, capacity) entries to
 * `ms` and to `names` (static strings); either may be NULL.  WERSA_ERR_STATE if timing is off. */
wersa_status wersa_step_times(wersa_ctx* ctx, int which, int capacity, float* ms,
                              const char** names, int* count);

#ifdef __cplusplus
}
#endif
#endif /* WERSA_H_ */
