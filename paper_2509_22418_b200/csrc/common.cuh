// Shared declarations of the sm_100a kernels behind the ppu C ABI.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;

// Device-side error word indices (one int32 each, in the context's flag block).
enum { PPU_FLAG_TOKEN = 0, PPU_FLAG_TIMEOUT = 1, PPU_FLAG_COUNT = 8 };

// ---- GEMM: C[M,N] (+epilogue) = A . B^T, bf16 operands, fp32 accumulation ----
enum GemmEpilogue {
  EPI_STORE_BF16 = 0,  // C bf16
  EPI_STORE_F32 = 1,   // C fp32
  EPI_GELU_DUAL = 2,   // C bf16 = acc (pre-activation), C2 bf16 = gelu(acc)
  EPI_RESID_F32 = 3,   // C fp32 = aux fp32 + acc (residual stream)
  EPI_DGELU = 4,       // C bf16 = acc * gelu'(aux bf16)
  EPI_ROPE_BF16 = 5,   // C bf16 = acc with rotary positions applied to the columns < rope_cols
  // C bf16 = acc (the attention output's gradient dU), and per (token, head)
  // C3 fp32 [batch, heads, rope_S] = sum over the head's rope_dh columns of C * aux (aux = U bf16):
  // the row term of the softmax backward, formed while dU is still in registers
  EPI_DELTA_BF16 = 6
};

struct GemmArgs {
  const bf16* A; int64_t lda; int a_kmajor;  // a_kmajor: A[m*lda+k], else A[k*lda+m]
  const bf16* B; int64_t ldb; int b_kmajor;  // b_kmajor: B[n*ldb+k], else B[k*ldb+n]
  int M, N, K;
  int epilogue;
  void* C; int64_t ldc;
  void* C2;                     // EPI_GELU_DUAL second output (ld = ldc)
  const void* aux; int64_t ldaux;
  int* flags;                   // device error words (may be null for the test entry)
  // split-K: the reduction is cut into `splits` ranges; range s writes its partial product to
  // C + s * split_stride (elements).  The consumer adds the partials in index order.
  int splits = 1; int64_t split_stride = 0;
  // EPI_GELU_DUAL: columns [c3_lo, c3_hi) of gelu(acc) are also stored, packed, to C3[m, n - c3_lo]
  // (the slice of the activation that a subset weight gradient will read); C3 may be null
  void* C3 = nullptr; int64_t ldc3 = 0; int c3_lo = 0, c3_hi = 0;
  // EPI_ROPE_BF16: aux is the (cos, sin) table [rope_S][rope_dh / 2]; row m is position m % rope_S
  int rope_S = 0, rope_dh = 0, rope_cols = 0;
  // tcgen05 tile shape: 0 chosen from the problem size, 1 one CTA per 128-row tile, 2 an SM pair
  // per 256 x 256 tile, 3 an SM pair per 256 x 128 tile (tests force each)
  int tile_shape = 0;
};

int launch_gemm_simt(const GemmArgs& g, cudaStream_t st);
int launch_gemm_tc(const GemmArgs& g, cudaStream_t st);   // tcgen05 / TMEM / TMA
// whether launch_gemm_tc accepts EPI_DELTA_BF16 for this product (tile shape and alignment allow
// a thread to own whole heads of its row); otherwise the caller runs launch_attn_delta
bool gemm_tc_fuses_delta(const GemmArgs& g);
int gemm_tc_init();                                        // resolves the tensor-map encoder

// ---- attention -------------------------------------------------------------
int launch_attn_fwd_simt(const bf16* qkv, bf16* U, float* lse, int B, int S, int h, int dh,
                         cudaStream_t st);
int launch_attn_bwd_simt(const bf16* qkv, const bf16* U, const float* lse, const bf16* dU,
                         bf16* dqkv, float* scratch, int B, int S, int h, int dh, cudaStream_t st);
int launch_attn_fwd_mma(const bf16* qkv, bf16* U, float* lse, int B, int S, int h, int dh,
                        cudaStream_t st);
int launch_attn_bwd_mma(const bf16* qkv, const bf16* U, const float* lse, const bf16* dU,
                        bf16* dqkv, float* scratch, int B, int S, int h, int dh, cudaStream_t st);
bool attn_mma_supported(int S, int dh);
// tcgen05 attention (TMEM accumulators, TMA operands); flags: device error words or null
bool attn_tc_supported(int S, int dh);
int launch_attn_fwd_tc(const bf16* qkv, bf16* U, float* lse, int B, int S, int h, int dh, int* flags,
                       cudaStream_t st);
int launch_attn_bwd_tc(const bf16* qkv, const bf16* U, const float* lse, const bf16* dU, bf16* dqkv,
                       float* scratch, int B, int S, int h, int dh, int* flags, cudaStream_t st,
                       const float2* inv_rope_cs = nullptr,    // non-null: rotate dq, dk back by -angle
                       bool delta_done = false);               // scratch already holds delta
// delta[b,h,s] = sum_e dU * U of the head's slice
void launch_attn_delta(const bf16* U, const bf16* dU, float* delta, int B, int S, int h, int dh,
                       cudaStream_t st);

// ---- bandwidth-bound kernels -------------------------------------------------
void launch_embed(const int32_t* tok, const bf16* E16, float* x, int T, int d, int V, int* flags,
                  cudaStream_t st);
// y bf16 = LN(x) * g + b ; stats[t] = {mean, rstd}
void launch_ln_fwd(const float* x, const float* g, const float* b, bf16* y, float2* stats, int T,
                   int d, float eps, cudaStream_t st);
// gout fp32 (+ bf16 copy) = (gin ? gin : 0) + LNbwd_dx(dy; x, stats, gamma)
void launch_ln_bwd(const bf16* dy, const float* x, const float2* stats, const float* gamma,
                   const float* gin, float* gout, bf16* gout16, int T, int d, cudaStream_t st);
// rotates q and k parts of qkv[T,3d] in place by the (cos, sin) table cs[S, dh/2];
// inverse (rotation by -angle) for gradients
void launch_rope(bf16* qkv, const float2* cs, int B, int S, int h, int dh, int inverse,
                 cudaStream_t st);
// logits bf16 [T,V] -> dlogits in place; row_loss[t] (0 for the last position of a sequence)
void launch_xent(bf16* logits, const int32_t* tok, float* row_loss, int B, int S, int V,
                 int write_grad, cudaStream_t st);
void launch_loss_reduce(const float* row_loss, int T, float inv_count, float* out, cudaStream_t st);
void launch_cast_bf16(const float* src, bf16* dst, int64_t n, cudaStream_t st);

// One trained block of a replica: rows [lo,hi) of W_in then columns [lo,hi) of W_out,
// packed back to back at `packed_off` of the replica's packed arrays.
struct SliceSeg {
  int64_t win_off, wout_off;   // offsets of the layer's W_in / W_out in the canonical vector
  int64_t packed_off;          // start of this layer's block in the packed arrays
  int32_t lo, hi;
};

struct AdamHyper { float lr, beta1, beta2, eps, wd, bc1, bc2; };

// AdamW over the packed subset; n_partials gradient buffers (stride grad_stride) are summed in order.
void launch_adamw(const SliceSeg* segs, int n_seg, float* master, float* m, float* v,
                  const float* grad, int n_partials, int64_t grad_stride, bf16* w16, int d, int F,
                  int64_t n_total, AdamHyper hp, cudaStream_t st);
// packed fp32 <-> canonical vectors
void launch_slices_gather(const SliceSeg* segs, int n_seg, const float* theta, float* packed,
                          int d, int F, int64_t n_total, cudaStream_t st);
// w16[subset] = bf16(src) where src is the packed master (from_packed) or theta itself
void launch_slices_to_w16(const SliceSeg* segs, int n_seg, const float* packed, const float* theta,
                          bf16* w16, int from_packed, int d, int F, int64_t n_total,
                          cudaStream_t st);
void launch_slices_scatter_f32(const SliceSeg* segs, int n_seg, const float* packed, float* dense,
                               int d, int F, int64_t n_total, cudaStream_t st);

// Outer sync tables.  Owner o is one listed replica's trained block of one layer: hidden
// units [lo,hi); its packed W_in block starts at master + in_off, its W_out block at
// master + out_off.  For every group of 8 hidden units of every layer, unit_begin/unit_owner
// (CSR) list the owners that contain the group, in the order the replicas were listed.
struct OuterOwner { float* master; int64_t in_off, out_off; int32_t lo, hi; };
struct OuterTables {
  const OuterOwner* owners;      // device
  const int32_t* unit_begin;     // device [L * F/8 + 1]
  const int32_t* unit_owner;     // device
  int64_t P, e_size, layer_size, win_rel, wout_rel;  // canonical geometry
  int32_t L, d, F;
};
// Segments of the canonical vector the outer sweep works through: 0-3 quarters of E, then three
// per layer (non-FFN block, W_in, W_out), then the final LayerNorm.  The sweep covers segments
// [seg_lo, seg_lo + seg_count).
inline int outer_segments(int n_layer) { return 4 + 3 * n_layer + 1; }
void launch_outer(const OuterTables& t, float* theta, float* buf, bf16* w16, float lr, float mu,
                  int seg_lo, int seg_count, cudaStream_t st);
