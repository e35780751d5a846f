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
  EPI_GELU_DUAL = 2,   // C bf16 = acc (pre-activation; skipped when C is null), C2 bf16 = gelu(acc)
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
  // per 256 x 256 tile, 3 an SM pair per 256 x 128 tile, 4 as 2 without cutting the tiles of a
  // half-empty last wave in two (tests force each)
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

// ---- per-device caches -------------------------------------------------------
// Kernel attributes (dynamic shared-memory limits) and device properties are per device; a
// process may hold contexts on several.  Lookups are idempotent, so two threads that race on
// the first use of a device at worst both perform the same query.
constexpr int PPU_MAX_DEVICES = 64;
int ppu_current_device();                 // index of the current device, clamped to the table
int ppu_sm_count();                       // SMs of the current device (read once per device)
struct PerDeviceFlag { bool done[PPU_MAX_DEVICES] = {}; };
template <typename Kernel>
inline bool ppu_set_smem_once(PerDeviceFlag& f, Kernel kernel, int bytes) {
  const int dev = ppu_current_device();
  if (f.done[dev]) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
    return false;
  f.done[dev] = true;
  return true;
}

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

// rows of E that a batch touches: dE[tok[t], :] += g[t, :] over all t in ascending order of t
// (one warp owns all occurrences of an id, so the sum has a fixed order and needs no atomics)
void launch_embed_grad(const int32_t* tok, const float* g, float* dE, int T, int d, int V,
                       cudaStream_t st);
// dgamma[c] = sum_t dy[t,c] * xhat[t,c], dbeta[c] = sum_t dy[t,c], in two stages with a fixed
// order; partial: fp32 scratch [2 * ln_param_partial_blocks(T) * d]
int ln_param_partial_blocks(int T);
void launch_ln_param_grad(const bf16* dy, const float* x, const float2* stats, float* dgamma,
                          float* dbeta, float* partial, int T, int d, cudaStream_t st);

// One trained FFN block of a replica: rows [lo,hi) of W_in then columns [lo,hi) of W_out,
// packed back to back at `packed_off` of the replica's packed arrays.
struct SliceSeg {
  int64_t win_off, wout_off;   // offsets of the layer's W_in / W_out in the canonical vector
  int64_t packed_off;          // start of this layer's block in the packed arrays
  int32_t lo, hi;
};
// One contiguous run of the canonical vector that a replica trains outside the FFNs (a whole
// tensor, or the rows of W_q / W_k / W_v of its heads), packed at `packed_off`.
struct DenseSeg {
  int64_t canon_off, len, packed_off;   // len is a multiple of 8
  int32_t decay;                        // 1: AdamW's weight decay applies (matrices)
  int32_t pad;
};

struct AdamHyper { float lr, beta1, beta2, eps, wd, bc1, bc2; };

// AdamW over the packed FFN blocks; n_partials gradient buffers (stride grad_stride) are summed in order.
void launch_adamw(const SliceSeg* segs, int n_seg, float* master, float* m, float* v,
                  const float* grad, int n_partials, int64_t grad_stride, bf16* w16, int d, int F,
                  int64_t n_total, AdamHyper hp, cudaStream_t st);
// AdamW over the packed dense runs; the gradient of packed element j is grad[j - grad_shift]
void launch_adamw_dense(const DenseSeg* segs, int n_seg, float* master, float* m, float* v,
                        const float* grad, int64_t grad_shift, bf16* w16, int64_t packed_base,
                        int64_t n_total, AdamHyper hp, cudaStream_t st);
// packed fp32 <-> canonical vectors
void launch_slices_gather(const SliceSeg* segs, int n_seg, const float* theta, float* packed,
                          int d, int F, int64_t n_total, cudaStream_t st);
// w16[subset] = bf16(src) where src is the packed master (from_packed) or theta itself
void launch_slices_to_w16(const SliceSeg* segs, int n_seg, const float* packed, const float* theta,
                          bf16* w16, int from_packed, int d, int F, int64_t n_total,
                          cudaStream_t st);
// the same two moves for the dense runs, which fill packed positions [packed_base, packed_base +
// n_total): mode 0 packed = theta, 1 w16 = bf16(packed), 2 w16 = bf16(theta)
void launch_dense_move(const DenseSeg* segs, int n_seg, float* packed, const float* theta, bf16* w16,
                       int mode, int64_t packed_base, int64_t n_total, cudaStream_t st);

// Outer sync tables.  The canonical vector is cut into runs ("segments") that are uniform in
// how their owners are found:
//   kind 0  a run that is contiguous in its owners' packed arrays too - anything outside the FFN
//           matrices, and the rows of a W_in between two slice boundaries; every owner in
//           [ob, oe) of `dense_owner` trains the whole run, its value of canonical position i
//           is master[i + shift];
//   kind 2  a layer's W_out, of which a replica trains columns: the owners of a hidden unit are
//           listed per group of 8 units in unit_begin / unit_owner (CSR over layer * F/8 + unit/8).
// (There is no kind 1: W_in had a kind of its own until its rows were swept as dense runs.)
// Work is dealt to blocks in chunks of OUTER_CHUNK elements of one segment.
constexpr int OUTER_CHUNK = 1 << 16;
struct OuterSeg {
  int64_t start, len;        // run of the canonical vector (multiples of 4)
  int64_t base;              // kind 2: canonical offset of the whole matrix
  int32_t kind, layer;
  int32_t ob, oe;            // kind 0: owners
};
struct OuterChunk { int32_t seg; int32_t pad; int64_t off; };   // chunk = elements [off, off + OUTER_CHUNK) of the segment
struct DenseOwner { float* master; int64_t shift; };
// a listed replica's trained block of one layer: hidden units [lo,hi); packed W_in block at
// master + in_off, W_out block at master + out_off
struct OuterOwner { float* master; int64_t in_off, out_off; int32_t lo, hi; };
// Division by a fixed divisor d < 2^16 as multiply-high and shift: with 2^shift < d <= 2^(shift+1)
// and mul = floor(2^(32 + shift) / d) + 1, floor(n / d) = (n * mul) >> (32 + shift) for every
// n < 2^28 (the sweep divides element offsets inside one weight matrix).
struct FastDiv { uint32_t mul, shift; };
inline FastDiv make_fast_div(uint32_t d) {
  FastDiv f; f.shift = 0;
  while ((1u << f.shift) < d) ++f.shift;          // 2^shift >= d
  if (f.shift > 0) --f.shift;                     // 2^shift < d <= 2^(shift + 1): mul fits 32 bits
  f.mul = (uint32_t)((((uint64_t)1 << (32 + f.shift)) / d) + 1);
  return f;
}
struct OuterTables {
  const OuterSeg* segs;          // device
  const OuterChunk* chunks;      // device
  const DenseOwner* dense_owner; // device
  const int32_t* unit_begin;     // device [L * F/8 + 1]
  const OuterOwner* unit_owner;  // device, owners inline
  int32_t d, F;
  FastDiv div_d, div_F;
};
// sweeps chunks [chunk_lo, chunk_lo + n_chunks)
void launch_outer(const OuterTables& t, int kind, float* theta, float* buf, bf16* w16, float lr, float mu,
                  int chunk_lo, int n_chunks, cudaStream_t st);
