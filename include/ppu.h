/*
 * ppu.h - C ABI of the partial-parameter-update training step for one B200.
 *
 * The library runs the hot path of "Partial Parameter Updates for Efficient
 * Distributed Training": every simulated node (a "replica") runs a full
 * forward pass of a pre-LayerNorm causal decoder over all parameters,
 * back-propagates activation gradients down to its lowest trained layer,
 * forms weight gradients only for its own fixed parameter subset, applies
 * AdamW to that subset (Algorithm 1, the local step), and the replicas are
 * periodically merged by a count-normalised average of their deltas followed
 * by an outer Nesterov step (Algorithm 1, the outer step).
 *
 * Conventions
 *  - Every function returns PPU_OK (0) or a negative ppu_status.  Nothing
 *    throws across the boundary.  ppu_last_error() gives a text for the most
 *    recent failure of the calling thread.
 *  - Pointers are marked HOST or DEVICE.  The caller owns every buffer it
 *    passes, including the arena and the CUDA stream; the context owns only
 *    host-side metadata.  No call allocates device memory.
 *  - All device work is enqueued on the stream given to ppu_create and is
 *    asynchronous unless the call returns a host value.
 *  - There is no CPU fallback: without a CUDA device every compute call
 *    fails with PPU_ECUDA.
 *  - Kernel attributes and device properties are cached per device, so contexts
 *    on several devices of one process work; a context belongs to the device
 *    that was current when it was created, and that device must be current in
 *    every later call on it.
 *
 * Canonical parameter vector (fp32, length ppu_param_count): E[V,d]; then for
 * each layer ln1_g[d], ln1_b[d], W_q[d,d], W_k[d,d], W_v[d,d], W_o[d,d],
 * ln2_g[d], ln2_b[d], W_in[F,d], W_out[d,F]; then lnf_g[d], lnf_b[d].  Linear
 * weights are stored [out, in] row-major (y = x W^T): W_in and W_out are the
 * matrices W in R^{4d x d} and V in R^{d x 4d} of Section 2.2.1.  The output
 * head is tied to E.  There are no linear biases.
 */
#ifndef PPU_H_
#define PPU_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PPU_OK = 0,
  PPU_EINVAL = -1,   /* bad argument (null pointer, replica out of range, duplicate ...) */
  PPU_ESHAPE = -2,   /* model shape not supported (divisibility / alignment)            */
  PPU_ESUBSET = -3,  /* subset specification invalid                                    */
  PPU_ENOMEM = -4,   /* arena smaller than ppu_query_bytes reports                      */
  PPU_ESTATE = -5,   /* call not valid in the current state                             */
  PPU_ECUDA = -6,    /* CUDA runtime error or no device                                 */
  PPU_ETIMEOUT = -7, /* a bounded wait inside a kernel gave up                          */
  PPU_ETOKEN = -8    /* a token id outside [0, vocab) was seen (it was clamped)         */
} ppu_status;

/* Model and optimizer description.  Section 3.1 gives the paper's values
 * (AdamW beta 0.9/0.99, wd 0.1; outer Nesterov momentum 0.9). */
typedef struct {
  int32_t n_layer, d_model, n_head, d_ff, vocab;
  int32_t max_batch, max_seq;  /* largest [batch, seq] a local step will be given */
  float ln_eps;                /* LayerNorm epsilon                               */
  float rope_base;             /* rotary base (pairs (2i,2i+1), angle pos*base^(-2i/d_h)) */
  float adam_lr, adam_beta1, adam_beta2, adam_eps, adam_wd;
  float outer_lr, outer_momentum;
} ppu_model_cfg;

typedef enum {
  PPU_SUBSET_FFN_SLICE = 0,  /* Section 2.2.1 MLP-only slicing of the FFN hidden units   */
  PPU_SUBSET_FFN_LAYERS = 1, /* whole FFNs of the blocks l with l mod layer_stride == n  */
  PPU_SUBSET_EXPLICIT = 2    /* ranges[k][l] = {lo, hi} given by the caller              */
} ppu_subset_mode;

/* Which parameters replica k trains (the set I_k^train of Algorithm 1).  The set has up to
 * three parts:
 *  (a) per layer l, the rows [lo,hi) of W_in and the columns [lo,hi) of W_out (mode, n_slices,
 *      layer_stride, ranges) - the MLP slicing of Section 2.2.1.  Replica k uses slice index
 *      n = k mod n_slices; n_replicas must be a multiple of n_slices; lo and hi are multiples
 *      of 8;
 *  (b) the rows of W_q, W_k and W_v of a range of heads [h_lo,h_hi) in every layer - the
 *      columns W_{Q,K,V}[:, H_n] of the MLP + attention-head slicing of Section 2.2.1 (W_o is
 *      never sliced).  head_ranges gives the range per replica; otherwise n_head_slices > 0
 *      gives replica k the head group k mod n_head_slices (n_head a multiple of n_head_slices,
 *      n_replicas a multiple of it too); otherwise all heads when train_non_mlp is set, none
 *      when it is not;
 *  (c) with train_non_mlp = 1, every parameter Section 2.2.1 never slices: the embedding (tied
 *      to the output head), W_o and the gains and shifts of all normalisation layers.  This is
 *      what the paper's runs train on every node; 0 freezes them on every node.
 * Everything else is frozen on that replica.  The packed order of a replica's trained values
 * (ppu_subset_index) is: per trained layer the W_in rows block, then the W_out columns block;
 * then the positions of (b) and (c) in the order of the canonical vector.  AdamW's weight decay
 * applies to matrices, not to the gains and shifts of the normalisation layers. */
typedef struct {
  int32_t n_replicas;    /* K */
  int32_t mode;          /* ppu_subset_mode */
  int32_t n_slices;      /* N (FFN_SLICE: d_ff % (8 N) == 0) */
  int32_t layer_stride;  /* FFN_LAYERS only */
  const int32_t* ranges; /* HOST, EXPLICIT only: [n_replicas][n_layer][2] */
  int32_t train_non_mlp; /* part (c), and the default of part (b) */
  int32_t n_head_slices; /* part (b): 0 = not sliced */
  const int32_t* head_ranges; /* HOST, optional: [n_replicas][2] = {h_lo, h_hi} */
} ppu_subset_spec;

typedef struct ppu_ctx ppu_ctx;

/* Per-context counters filled by ppu_stats. */
typedef struct {
  int64_t param_count;         /* |theta|                                              */
  int64_t arena_bytes;         /* bytes of the arena in use                            */
  int64_t state_bytes;         /* parameters, outer momentum, replica slices and state */
  int64_t activation_bytes;    /* saved activations + backward scratch + logits        */
  int64_t launches_last_step;  /* kernels enqueued by the most recent local step       */
  int64_t launches_last_sync;  /* kernels enqueued by the most recent outer sync       */
  double flops_fwd, flops_dgrad, flops_wgrad; /* executed matmul FLOPs of the last step */
  double outer_bytes;          /* algorithmic bytes of the last outer sync             */
  int64_t saved_bytes_last_step; /* activation bytes the last step's forward pass kept for
                                    its backward pass (nothing below the lowest trained layer) */
} ppu_stats_t;

/* Bytes of device memory a context needs.  bytes: HOST out. */
int ppu_query_bytes(const ppu_model_cfg* cfg, const ppu_subset_spec* spec, size_t* bytes);

/* Builds a context inside `arena` (DEVICE, 256-byte aligned, arena_bytes >= the
 * queried size).  Parameters start at zero with LayerNorm gains at one; load
 * real values with ppu_set_params.  `cuda_stream` is a cudaStream_t (may be
 * null for the default stream).  out: HOST. */
int ppu_create(const ppu_model_cfg* cfg, const ppu_subset_spec* spec, void* arena,
               size_t arena_bytes, void* cuda_stream, ppu_ctx** out);
int ppu_destroy(ppu_ctx* ctx);

/* The local step of Algorithm 1 for one replica: forward on all parameters, restricted
 * backward (Appendix C.1), AdamW on I_k^train; the replica's step count grows by
 * one.  tokens: DEVICE int32 [batch, seq], kept alive by the caller until the
 * stream has passed the call.  Ids outside [0, vocab) are clamped and reported
 * as PPU_ETOKEN by the next call that synchronises.  Asynchronous. */
int ppu_local_step(ppu_ctx* ctx, int replica, const int32_t* tokens, int batch, int seq);

/* The same step for a caller holding tokens in HOST memory: copies them to the
 * device, runs the step, waits, and writes the step's loss to loss_out (HOST). */
int ppu_local_step_host(ppu_ctx* ctx, int replica, const int32_t* tokens_host, int batch,
                        int seq, double* loss_out);

/* The outer step of Algorithm 1 over the listed replicas (HOST array, no duplicates):
 * Delta[i] = sum_k (theta_k[i] - theta[i]) / m[i] with m counted over the list
 * and Delta = 0 where m = 0; pseudo-gradient g = -Delta; buf = mu buf + g;
 * theta -= eta (g + mu buf).  Sweeps every parameter, refreshes the bf16 working
 * copy and restarts the listed replicas from the new theta (Algorithm 1 line
 * 6).  AdamW moments and step counts are kept.  Asynchronous. */
int ppu_outer_sync(ppu_ctx* ctx, const int32_t* replicas, int n);

/* Streaming synchronisation by layers (Appendix "Streaming Synchronization", Section
 * 3.1): the same outer step, taken on one group of positions only.  The n_layer
 * layers are split in order into n_groups groups of n_layer / n_groups layers (every
 * tensor of those layers); group == n_groups is one more group holding the embeddings
 * and the final LayerNorm (the paper: 24 layers as 8 groups of 3, plus that ninth
 * group).  Outside the group nothing changes: not the global parameters, not the
 * outer momentum, not the listed replicas' own values (they keep training from where
 * they are).  The caller owns the schedule (which group after which local steps).
 * n_layer must be a multiple of n_groups and 0 <= group <= n_groups, else PPU_EINVAL.
 * replicas: HOST array, no duplicates.  Asynchronous. */
int ppu_outer_sync_group(ppu_ctx* ctx, const int32_t* replicas, int n, int group, int n_groups);

/* Loss of the replica's most recent local step: Eq. 2.2 as the mean negative
 * log-likelihood (nats) over the batch*(seq-1) predicted tokens.  Waits for the
 * stream.  loss_out: HOST. */
int ppu_loss(ppu_ctx* ctx, int replica, double* loss_out);

/* Forward pass only, with replica's parameters (replica = -1: the global
 * parameters).  tokens: DEVICE.  Waits for the stream.  loss_out: HOST. */
int ppu_eval_loss(ppu_ctx* ctx, int replica, const int32_t* tokens, int batch, int seq,
                  double* loss_out);

/* ---- accessors (tests, checkpoints); all HOST buffers, all synchronising ---- */
int ppu_param_count(const ppu_ctx* ctx, int64_t* n);
int ppu_tensor_count(const ppu_ctx* ctx, int32_t* n);
/* name: HOST buffer of name_cap bytes; shape: HOST int64[2] (unused dims = 1). */
int ppu_tensor_info(const ppu_ctx* ctx, int32_t index, char* name, int32_t name_cap,
                    int64_t* offset, int32_t* ndim, int64_t* shape);
/* replica = -1: sets the global parameters theta^(t) (canonical vector), refreshes the bf16
 * copy and restarts every replica from them.  replica >= 0: sets that replica's own values
 * theta_k on its trained positions from the canonical vector given (other positions of the
 * vector are not read); the global parameters and the other replicas are untouched.
 * Optimizer state is untouched in both forms. */
int ppu_set_params(ppu_ctx* ctx, int replica, const float* theta, int64_t n);
/* replica >= 0: theta_k (global vector with the replica's subset overlaid);
 * replica = -1: the global parameters. */
int ppu_get_params(ppu_ctx* ctx, int replica, float* theta, int64_t n);
/* bf16 working copy as the kernels currently see it (raw bf16 bits). */
int ppu_get_working_bf16(ppu_ctx* ctx, uint16_t* w, int64_t n);
int ppu_get_outer_momentum(ppu_ctx* ctx, float* buf, int64_t n);
int ppu_set_outer_momentum(ppu_ctx* ctx, const float* buf, int64_t n);
/* |I_k^train| and its flat indices in the order the packed subset arrays use:
 * per trained layer the W_in rows block, then the W_out columns block
 * (row-major over [d, hi-lo]). */
int ppu_subset_count(const ppu_ctx* ctx, int replica, int64_t* n);
int ppu_subset_index(const ppu_ctx* ctx, int replica, int64_t* index, int64_t n);
/* Gradient of the most recent local step (valid for the replica stepped last). */
int ppu_get_subset_grads(ppu_ctx* ctx, int replica, float* grads, int64_t n);
/* AdamW moments and step count of a replica; any out pointer may be null. */
int ppu_get_subset_state(ppu_ctx* ctx, int replica, float* m, float* v, int32_t* step,
                         int64_t n);
/* Restores them (checkpoint resume): m and v in the packed order, length ppu_subset_count;
 * either may be null to leave it as it is; step >= 0. */
int ppu_set_subset_state(ppu_ctx* ctx, int replica, const float* m, const float* v, int32_t step,
                         int64_t n);
/* Device address of replica k's packed trained values (fp32, ppu_subset_count elements, inside
 * the caller's arena).  For a multi-GPU exchange step: each GPU steps its own replicas, the
 * owners' packed values are copied into the same replica's buffer on the other GPUs (plain
 * device-to-device copies or a collective on these local buffers), and every GPU then runs
 * the same ppu_outer_sync.  dev_ptr: HOST out. */
int ppu_replica_values(ppu_ctx* ctx, int replica, void** dev_ptr, int64_t* n);
/* Debug aid: every sub-buffer the context carves out of the arena (parameters, each replica's
 * packed arrays, every activation and scratch buffer) is followed by a 256-byte guard block
 * filled at creation with a fixed pattern that no kernel may write.  This call waits for the
 * stream, reads all guard blocks back and reports how many were modified (n_bad: HOST out);
 * PPU_ESTATE if any was - an out-of-bounds write by one of the kernels. */
int ppu_check_guards(ppu_ctx* ctx, int64_t* n_bad);
int ppu_set_adam_lr(ppu_ctx* ctx, float lr);
int ppu_sync(ppu_ctx* ctx);   /* waits for the stream; reports PPU_ETOKEN / PPU_ETIMEOUT */
int ppu_stats(ppu_ctx* ctx, ppu_stats_t* out);
const char* ppu_last_error(void);

/* Per-kernel-class device timing.  While enabled, the launches of a local step and of an outer
 * sync are bracketed by CUDA events on the context's stream (up to a fixed pool; launches
 * beyond it are not recorded).  ppu_profile_read waits for the stream, sums the recorded
 * intervals and their algorithmic work since the last read, and empties the pool.  work is in
 * FLOPs for the GEMM and attention classes and in algorithmic bytes for the others. */
enum {
  PPU_CLS_GEMM = 0,   /* every tcgen05 (or SIMT) GEMM launch                       */
  PPU_CLS_ATTN = 1,   /* attention forward + backward                              */
  PPU_CLS_LN = 2,     /* LayerNorm forward, backward, gain/shift gradients         */
  PPU_CLS_XENT = 3,   /* fused cross-entropy                                       */
  PPU_CLS_ADAMW = 4,  /* AdamW on the subset                                       */
  PPU_CLS_OUTER = 5,  /* outer sweep                                               */
  PPU_CLS_OTHER = 6,  /* embedding gather / scatter, residency moves, reductions   */
  PPU_CLS_COUNT = 8
};
typedef struct {
  double ms[PPU_CLS_COUNT], work[PPU_CLS_COUNT];
  int64_t launches[PPU_CLS_COUNT];
  int64_t dropped;
} ppu_profile_t;
int ppu_profile_enable(ppu_ctx* ctx, int enable);
int ppu_profile_read(ppu_ctx* ctx, ppu_profile_t* out);

/* Test hook: which kernels the context's steps use.  gemm: 0 = tcgen05 tiles, 1 = plain SIMT
 * check kernel.  attention: 0 = tcgen05 kernels where the shape allows, 1 = SIMT check
 * kernels.  The default is 0, 0; production code has no reason to call this. */
int ppu_set_backends(ppu_ctx* ctx, int gemm, int attention);

/* Failure-detection self-test.  Every wait inside the tcgen05 kernels is bounded: when a
 * barrier is not signalled within the limit the kernel sets an error word, releases what it
 * holds and returns, and the next synchronising call reports PPU_ETIMEOUT.  This call exercises
 * that path without any fault: one CTA waits `limit` polls (1..65536) on a barrier nothing
 * arrives at.  Returns PPU_ETIMEOUT when the kernel gave up as designed (the expected outcome),
 * PPU_OK if the wait was somehow satisfied, PPU_ECUDA on a runtime error.  The context stays
 * usable afterwards.  Synchronises the stream. */
int ppu_wait_probe(int limit, void* cuda_stream);

/* ---- single-operator entry points (kernel-level parity tests) -------------- */

/* C[M,N] = A . B^T on bf16 operands with fp32 accumulation (the contraction of
 * every forward, input-gradient and subset weight-gradient product of Appendix
 * C.1).  A is [M,K] row-major when a_kmajor, else stored [K,M]; B is [N,K]
 * row-major when b_kmajor, else stored [K,N].  lda/ldb/ldc in elements,
 * multiples of 8.  out_f32: C is fp32, else bf16.  backend: 0 = tcgen05 tiles,
 * shape chosen from the problem size as the training step does; 1 = plain SIMT
 * check kernel; 2 = tcgen05, one CTA per 128-row tile; 3 = tcgen05, one SM pair
 * (cta_group::2) per 256 x 256 tile, a half-empty last wave of tiles worked as
 * 128-column halves; 4 = one SM pair per 256 x 128 tile; 5 = as 3 with whole
 * tiles only.  All pointers DEVICE.  Asynchronous on stream. */
int ppu_gemm(const void* A, int64_t lda, int a_kmajor, const void* B, int64_t ldb,
             int b_kmajor, void* C, int64_t ldc, int out_f32, int M, int N, int K,
             int backend, void* cuda_stream);

/* Fused causal attention on rotated q,k and v packed as qkv[T, 3d] bf16 (T =
 * batch*seq; q at column 0, k at d, v at 2d; head j at columns j*d_h).  Forward
 * writes U[T,d] bf16 and lse[batch, n_head, seq] fp32 (log-sum-exp of the scaled
 * scores).  Backward reads them plus dU[T,d] bf16 and writes dqkv[T,3d] bf16;
 * scratch is fp32 [batch*n_head*seq].  backend: 0 = tcgen05 / TMEM kernels (d_head 64 or
 * 128), 1 = plain SIMT check kernel.  All pointers DEVICE. */
int ppu_attention_fwd(const void* qkv, void* U, float* lse, int batch, int seq, int n_head,
                      int d_head, int backend, void* cuda_stream);
int ppu_attention_bwd(const void* qkv, const void* U, const float* lse, const void* dU,
                      void* dqkv, float* scratch, int batch, int seq, int n_head, int d_head,
                      int backend, void* cuda_stream);

/* No counterpart in the paper: a convenience for callers that cannot allocate device memory
 * (code running while a stream is being captured, hosts whose framework owns the allocator,
 * processes that are handed fixed buffers only).  Same computation and arguments as
 * ppu_attention_bwd, but the per-row scratch lives in a fixed array inside the library image
 * instead of being passed in; the call itself allocates nothing.
 *  - Limit: batch * n_head * seq <= PPU_STATIC_SCRATCH_FLOATS, else PPU_ESHAPE.  Each GPU that
 *    loads the library holds the array (4 MiB) until the process exits.
 *  - The first call on a device looks up the array's device address (with that device current);
 *    make that first call before starting any stream capture.
 *  - All calls share the one array.  It needs no clearing (each call writes every row it later
 *    reads), but two calls that overlap on the GPU - different streams, or different threads -
 *    race on it: keep calls to this entry point on one stream, or order them yourself. */
#define PPU_STATIC_SCRATCH_FLOATS (1 << 20)
int ppu_attention_bwd_static(const void* qkv, const void* U, const float* lse, const void* dU,
                             void* dqkv, int batch, int seq, int n_head, int d_head, int backend,
                             void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* PPU_H_ */
