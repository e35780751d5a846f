// Step scheduler: enqueues the kernels of one local step (the inner loop body of Algorithm 1) and of the
// outer synchronisation (lines 12-15) on the context's stream.  No host synchronisation
// happens inside a local step.
#include <algorithm>
#include <cmath>
#include <cstring>
#include "ppu_ctx.cuh"

int ppu_fail(int code, const char* fmt, ...);
#define CUDA_OK(call)                                                                    \
  do {                                                                                   \
    cudaError_t e_ = (call);                                                             \
    if (e_ != cudaSuccess)                                                               \
      return ppu_fail(PPU_ECUDA, "%s failed: %s", #call, cudaGetErrorString(e_));        \
  } while (0)

int ppu_check_flags(ppu_ctx* c) {
  int h[PPU_FLAG_COUNT];
  CUDA_OK(cudaMemcpy(h, c->flags, sizeof(h), cudaMemcpyDeviceToHost));
  if (h[PPU_FLAG_TOKEN] || h[PPU_FLAG_TIMEOUT]) {
    CUDA_OK(cudaMemset(c->flags, 0, sizeof(h)));
    if (h[PPU_FLAG_TIMEOUT]) return ppu_fail(PPU_ETIMEOUT, "a bounded wait inside a kernel expired");
    return ppu_fail(PPU_ETOKEN, "token id outside [0, vocab) was clamped");
  }
  return PPU_OK;
}

// Puts replica k's subset (or, for k = -1, the global values) into the bf16 working copy.
int ppu_make_resident(ppu_ctx* c, int k) {
  if (c->resident == k) return PPU_OK;
  const int d = c->cfg.d_model, F = c->cfg.d_ff;
  if (c->resident >= 0) {
    ReplicaState& r = c->reps[c->resident];
    EvScope ev(c, PPU_CLS_OTHER, 6.0 * (double)r.n_sub);
    launch_slices_to_w16(r.d_segs, (int)r.segs.size(), nullptr, c->theta, c->w16, 0, d, F, r.n_ffn,
                         c->stream);
    launch_dense_move(r.d_dense, (int)r.dense.size(), nullptr, c->theta, c->w16, 2, r.n_ffn, r.n_dense, c->stream);
    c->launches += (r.segs.empty() ? 0 : 1) + (r.dense.empty() ? 0 : 1);
  }
  if (k >= 0) {
    ReplicaState& r = c->reps[k];
    EvScope ev(c, PPU_CLS_OTHER, 6.0 * (double)r.n_sub);
    launch_slices_to_w16(r.d_segs, (int)r.segs.size(), r.master, nullptr, c->w16, 1, d, F, r.n_ffn,
                         c->stream);
    launch_dense_move(r.d_dense, (int)r.dense.size(), r.master, nullptr, c->w16, 1, r.n_ffn, r.n_dense, c->stream);
    c->launches += (r.segs.empty() ? 0 : 1) + (r.dense.empty() ? 0 : 1);
  }
  c->resident = k;
  return PPU_OK;
}

constexpr size_t EV_POOL_PAIRS = 16384;

EvScope::EvScope(ppu_ctx* ctx, int cls, double work) : c(ctx) {
  if (!c->profiling) return;
  if (c->ev_recs.size() >= EV_POOL_PAIRS) { c->ev_dropped++; return; }
  slot = (int)c->ev_recs.size();
  if (c->ev_pool.size() < 2 * (size_t)(slot + 1)) {
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { slot = -1; return; }
    c->ev_pool.push_back(a); c->ev_pool.push_back(b);
  }
  c->ev_recs.push_back({cls, work});
  cudaEventRecord(c->ev_pool[2 * slot], c->stream);
}
EvScope::~EvScope() { if (slot >= 0) cudaEventRecord(c->ev_pool[2 * slot + 1], c->stream); }

namespace {

struct Sched {
  ppu_ctx* c;
  int B, S, T, d, F, V, h, dh, L;
  int rc = 0;

  explicit Sched(ppu_ctx* ctx, int B_, int S_) : c(ctx), B(B_), S(S_) {
    T = B * S; d = c->cfg.d_model; F = c->cfg.d_ff; V = c->cfg.vocab; h = c->cfg.n_head;
    dh = d / h; L = c->cfg.n_layer;
  }
  const bf16* W(int l, int64_t rel) const { return c->w16 + c->e_size + (int64_t)l * c->layer_size + rel; }
  int64_t canon(int l, int64_t rel) const { return c->e_size + (int64_t)l * c->layer_size + rel; }
  // fp32 LayerNorm gain / shift as the replica sees it: its own value where it trains them
  const float* lnp(const ReplicaState* rep, int64_t off) const {
    if (rep && rep->rest) {
      const int64_t po = rep->packed_of(off);
      if (po >= 0) return rep->master + po;
    }
    return c->theta + off;
  }
  // where the gradient of the dense run starting at canonical offset `off` goes
  float* gdense(const ReplicaState& r, int64_t off) const {
    return c->grad + c->max_ffn * c->wgrad_splits + (r.packed_of(off) - r.n_ffn);
  }

  void gemm(const bf16* A, int64_t lda, int ak, const bf16* Bm, int64_t ldb, int bk, int M, int N,
            int K, int epi, void* C, int64_t ldc, void* C2, const void* aux, int64_t ldaux,
            double* flop_counter, int splits = 1, int64_t split_stride = 0, int rope_cols = 0,
            void* C3 = nullptr, int64_t ldc3 = 0, int c3_lo = 0, int c3_hi = 0) {
    if (rc || M <= 0 || N <= 0) return;
    GemmArgs g;
    g.A = A; g.lda = lda; g.a_kmajor = ak; g.B = Bm; g.ldb = ldb; g.b_kmajor = bk;
    g.M = M; g.N = N; g.K = K; g.epilogue = epi; g.C = C; g.ldc = ldc; g.C2 = C2; g.aux = aux;
    g.ldaux = ldaux; g.flags = c->flags; g.splits = splits; g.split_stride = split_stride;
    g.rope_S = S; g.rope_dh = dh; g.rope_cols = rope_cols;
    g.C3 = C3; g.ldc3 = ldc3; g.c3_lo = c3_lo; g.c3_hi = c3_hi;
    EvScope ev(c, PPU_CLS_GEMM, 2.0 * M * N * (double)K);
    rc = c->gemm_backend == 1 ? launch_gemm_simt(g, c->stream) : launch_gemm_tc(g, c->stream);
    c->launches++;
    if (flop_counter) *flop_counter += 2.0 * M * N * (double)K;
  }
  // weight gradient dW[M,N] = X^T Y over the tokens: X [T, >=M] and Y [T, >=N] token-major, fp32 out
  void wgrad(const bf16* X, int64_t ldx, const bf16* Y, int64_t ldy, int M, int N, float* out, int64_t ldo) {
    gemm(X, ldx, 0, Y, ldy, 0, M, N, T, EPI_STORE_F32, out, ldo, nullptr, nullptr, 0, &c->flops_wgrad);
  }
  void ln_fwd(const float* x, const float* g, const float* b, bf16* y, float2* st) {
    EvScope ev(c, PPU_CLS_LN, 6.0 * T * (double)d);
    launch_ln_fwd(x, g, b, y, st, T, d, c->cfg.ln_eps, c->stream);
    c->launches++;
  }
  void ln_bwd(const bf16* dy, const float* x, const float2* st, const float* gamma, const float* gin) {
    EvScope ev(c, PPU_CLS_LN, (gin ? 16.0 : 12.0) * T * (double)d);
    launch_ln_bwd(dy, x, st, gamma, gin, c->g, c->g16, T, d, c->stream);
    c->launches++;
  }
  void ln_param_grad(const ReplicaState& r, const bf16* dy, const float* x, const float2* st,
                     int64_t off_g, int64_t off_b) {
    EvScope ev(c, PPU_CLS_LN, 6.0 * T * (double)d);
    launch_ln_param_grad(dy, x, st, gdense(r, off_g), gdense(r, off_b), c->ln_partial, T, d, c->stream);
    c->launches += 2;
  }
  // split-K partial buffers the subset weight-gradient products of this step write
  int partials() const { const int kb = (T + 63) / 64; return c->wgrad_splits < kb ? c->wgrad_splits : kb; }
  // 0: tcgen05 kernels (d_h 64 or 128), 1: SIMT
  int attn_kind() const { return (c->attn_backend == 0 && attn_tc_supported(S, dh)) ? 0 : 1; }

  // Forward pass over all parameters (Appendix C.1 forward equations), saving what the
  // restricted backward needs: nothing of the layers below the replica's lowest trained layer.
  void forward(const int32_t* tok, const ReplicaState* rep, bool keep) {
    cudaStream_t st = c->stream;
    c->saved_bytes = 0;
    const int lowest = (keep && rep && rep->lowest >= 0) ? rep->lowest : L;   // evaluation keeps nothing
    {
      EvScope ev(c, PPU_CLS_OTHER, 6.0 * T * (double)d);
      launch_embed(tok, c->w16, c->acts[0].x, T, d, V, c->flags, st); c->launches++;
    }
    for (int l = 0; l < L && !rc; ++l) {
      LayerActs& a = c->acts[l];
      float* x_next = (l + 1 < L) ? c->acts[l + 1].x : c->x_last;
      ln_fwd(a.x, lnp(rep, canon(l, c->rel_ln1g)), lnp(rep, canon(l, c->rel_ln1b)), c->a16, a.st1);
      if (c->gemm_backend == 0) {   // rotary positions applied in the projection's epilogue
        gemm(c->a16, d, 1, W(l, c->rel_wq), d, 1, T, 3 * d, d, EPI_ROPE_BF16, a.qkv, 3 * d, nullptr,
             c->rope_cs, 0, &c->flops_fwd, 1, 0, 2 * d);
      } else {
        gemm(c->a16, d, 1, W(l, c->rel_wq), d, 1, T, 3 * d, d, EPI_STORE_BF16, a.qkv, 3 * d, nullptr,
             nullptr, 0, &c->flops_fwd);
        launch_rope(a.qkv, c->rope_cs, B, S, h, dh, 0, st); c->launches++;
      }
      {
        const double fl = 4.0 * B * h * dh * 0.5 * S * (double)(S + 1);
        EvScope ev(c, PPU_CLS_ATTN, fl);
        if (attn_kind() == 0) rc |= launch_attn_fwd_tc(a.qkv, a.U, a.lse, B, S, h, dh, c->flags, st);
        else rc |= launch_attn_fwd_simt(a.qkv, a.U, a.lse, B, S, h, dh, st);
        c->launches++;
        c->flops_fwd += fl;
      }
      gemm(a.U, d, 1, W(l, c->rel_wo), d, 1, T, d, d, EPI_RESID_F32, a.x1, d, nullptr, a.x, d,
           &c->flops_fwd);
      ln_fwd(a.x1, lnp(rep, canon(l, c->rel_ln2g)), lnp(rep, canon(l, c->rel_ln2b)), a.b, a.st2);
      // gelu(Hd) goes to a buffer shared by all layers; only the replica's own columns are kept,
      // and the pre-activation only where the backward pass will come
      const bool kept = l >= lowest;
      const int lo = rep ? rep->lo[l] : 0, hi = rep ? rep->hi[l] : 0;
      gemm(a.b, d, 1, W(l, c->rel_win), d, 1, T, F, d, EPI_GELU_DUAL, kept ? a.Hd : nullptr, F, c->A_tmp,
           nullptr, 0, &c->flops_fwd, 1, 0, 0, (kept && hi > lo) ? a.As : nullptr, hi - lo, lo, hi);
      gemm(c->A_tmp, F, 1, W(l, c->rel_wout), F, 1, T, d, F, EPI_RESID_F32, x_next, d, nullptr, a.x1, d,
           &c->flops_fwd);
      if (kept)   // x, x1, both statistics, qkv, U, lse, b, Hd and the trained columns of gelu(Hd)
        c->saved_bytes += (int64_t)T * (4 * d + 4 * d + 16 + 6 * d + 2 * d + 4 * h + 2 * d + 2 * (int64_t)F + 2 * (hi - lo));
    }
    ln_fwd(c->x_last, lnp(rep, c->off_lnfg), lnp(rep, c->off_lnfb), c->f16, c->stf);
    gemm(c->f16, d, 1, c->w16, d, 1, T, V, d, EPI_STORE_BF16, c->logits, V, nullptr, nullptr, 0,
         &c->flops_fwd);
  }

  void loss(const int32_t* tok, int write_grad, float* out) {
    cudaStream_t st = c->stream;
    {
      EvScope ev(c, PPU_CLS_XENT, (write_grad ? 4.0 : 2.0) * T * (double)V);
      launch_xent(c->logits, tok, c->row_loss, B, S, V, write_grad, st); c->launches++;
    }
    launch_loss_reduce(c->row_loss, T, 1.f / (float)((int64_t)B * (S - 1)), out, st); c->launches++;
  }

  // Restricted backward (Appendix C.1): input gradients through every FFN slice and every head,
  // weight gradients only for what the replica trains - its hidden-unit range per layer, the
  // query / key / value rows of its heads, and (paper's MLP-only and MLP + head slicing) the
  // parameters that are never sliced.  When only FFN slices are trained the pass stops at the
  // lowest trained layer, where only that slice's part is computed.
  void backward(const ReplicaState& r, const int32_t* tok) {
    if (r.lowest < 0) return;
    cudaStream_t st = c->stream;
    const bool deep = r.deep();
    const int kind = attn_kind();
    // output head: dE (tied embedding) = dlogits^T f when the embedding is trained
    if (r.rest) wgrad(c->logits, V, c->f16, d, V, d, gdense(r, 0), d);
    gemm(c->logits, V, 1, c->w16, d, 0, T, d, V, EPI_STORE_BF16, c->t16, d, nullptr, nullptr, 0,
         &c->flops_dgrad);
    if (r.rest) ln_param_grad(r, c->t16, c->x_last, c->stf, c->off_lnfg, c->off_lnfb);
    ln_bwd(c->t16, c->x_last, c->stf, lnp(&r, c->off_lnfg), nullptr);
    int seg = (int)r.segs.size() - 1;
    for (int l = L - 1; l >= r.lowest && !rc; --l) {
      LayerActs& a = c->acts[l];
      const bool trained = seg >= 0 && r.seg_layer[seg] == l;
      const SliceSeg* s = trained ? &r.segs[seg] : nullptr;
      const int w = trained ? s->hi - s->lo : 0;
      const bool cut = !deep && l == r.lowest;
      if (cut) {
        // only this replica's slice: dA_n = G V_n, through the activation, then both products
        gemm(c->g16, d, 1, W(l, c->rel_wout) + s->lo, F, 0, T, w, d, EPI_DGELU, c->dHd + s->lo, F,
             nullptr, a.Hd + s->lo, F, &c->flops_dgrad);
      } else {
        gemm(c->g16, d, 1, W(l, c->rel_wout), F, 0, T, F, d, EPI_DGELU, c->dHd, F, nullptr, a.Hd, F,
             &c->flops_dgrad);
      }
      if (trained) {
        // dW_in[lo:hi,:] = dHd[:,lo:hi]^T b      dW_out[:,lo:hi] = g^T A[:,lo:hi]
        gemm(c->dHd + s->lo, F, 0, a.b, d, 0, w, d, T, EPI_STORE_F32, c->grad + s->packed_off, d,
             nullptr, nullptr, 0, &c->flops_wgrad, partials(), c->max_ffn);
        gemm(c->g16, d, 0, a.As, w, 0, d, w, T, EPI_STORE_F32,
             c->grad + s->packed_off + (int64_t)w * d, w, nullptr, nullptr, 0, &c->flops_wgrad,
             partials(), c->max_ffn);
        --seg;
      }
      if (cut) break;
      gemm(c->dHd, F, 1, W(l, c->rel_win), d, 0, T, d, F, EPI_STORE_BF16, c->t16, d, nullptr,
           nullptr, 0, &c->flops_dgrad);
      if (r.rest) ln_param_grad(r, c->t16, a.x1, a.st2, canon(l, c->rel_ln2g), canon(l, c->rel_ln2b));
      ln_bwd(c->t16, a.x1, a.st2, lnp(&r, canon(l, c->rel_ln2g)), c->g);
      // dW_o = g1^T U
      if (r.rest) wgrad(c->g16, d, a.U, d, d, d, gdense(r, canon(l, c->rel_wo)), d);
      // dU = g1 W_O^T; where the tile shape allows, its epilogue also forms delta = rowsum(dU * U)
      // per (token, head) for the attention backward
      bool delta_fused = false;
      if (kind == 0 && c->gemm_backend == 0) {
        GemmArgs q;
        q.A = c->g16; q.lda = d; q.a_kmajor = 1; q.B = W(l, c->rel_wo); q.ldb = d; q.b_kmajor = 0;
        q.M = T; q.N = d; q.K = d; q.epilogue = EPI_DELTA_BF16; q.C = c->t16; q.ldc = d; q.C2 = nullptr;
        q.aux = a.U; q.ldaux = d; q.flags = c->flags; q.C3 = c->attn_scratch; q.rope_S = S; q.rope_dh = dh;
        delta_fused = gemm_tc_fuses_delta(q);
      }
      if (delta_fused)
        gemm(c->g16, d, 1, W(l, c->rel_wo), d, 0, T, d, d, EPI_DELTA_BF16, c->t16, d, nullptr, a.U, d,
             &c->flops_dgrad, 1, 0, 0, c->attn_scratch);
      else
        gemm(c->g16, d, 1, W(l, c->rel_wo), d, 0, T, d, d, EPI_STORE_BF16, c->t16, d, nullptr, nullptr,
             0, &c->flops_dgrad);
      {
        const double fl = 10.0 * B * h * dh * 0.5 * S * (double)(S + 1);
        EvScope ev(c, PPU_CLS_ATTN, fl);
        if (kind == 0)   // rotates dq, dk back on the way out (the output drain overlaps the next item's products)
          rc |= launch_attn_bwd_tc(a.qkv, a.U, a.lse, c->t16, c->dqkv, c->attn_scratch, B, S, h, dh, c->flags, st,
                                   c->rope_cs, delta_fused);
        else
          rc |= launch_attn_bwd_simt(a.qkv, a.U, a.lse, c->t16, c->dqkv, c->attn_scratch, B, S, h, dh, st);
        c->launches += (kind == 1 ? 2 : 3) - (delta_fused ? 1 : 0);
        c->flops_dgrad += fl;
        if (kind != 0) { launch_rope(c->dqkv, c->rope_cs, B, S, h, dh, 1, st); c->launches++; }
      }
      if (r.h_hi > r.h_lo) {
        // dW_{q,k,v}[rows of the trained heads] = dqkv[:, those columns]^T a, with a = LN1(x) formed
        // again from the saved block input (it is not kept by the forward pass)
        ln_fwd(a.x, lnp(&r, canon(l, c->rel_ln1g)), lnp(&r, canon(l, c->rel_ln1b)), c->a16, a.st1);
        const int rows = (r.h_hi - r.h_lo) * dh, r0 = r.h_lo * dh;
        if (rows == d) {    // every head: W_q, W_k, W_v are adjacent, one product
          wgrad(c->dqkv, 3 * d, c->a16, d, 3 * d, d, gdense(r, canon(l, c->rel_wq)), d);
        } else {
          for (int q = 0; q < 3; ++q)
            wgrad(c->dqkv + q * d + r0, 3 * d, c->a16, d, rows, d,
                  gdense(r, canon(l, c->rel_wq) + (int64_t)q * d * d + (int64_t)r0 * d), d);
        }
      }
      if (l == 0 && !r.rest) break;      // nothing below needs the input gradient
      gemm(c->dqkv, 3 * d, 1, W(l, c->rel_wq), d, 0, T, d, 3 * d, EPI_STORE_BF16, c->t16, d, nullptr,
           nullptr, 0, &c->flops_dgrad);
      if (r.rest) ln_param_grad(r, c->t16, a.x, a.st1, canon(l, c->rel_ln1g), canon(l, c->rel_ln1b));
      ln_bwd(c->t16, a.x, a.st1, lnp(&r, canon(l, c->rel_ln1g)), c->g);
    }
    if (r.rest && !rc) {   // input embedding: the rows the batch used, added to the head's part
      EvScope ev(c, PPU_CLS_OTHER, 12.0 * T * (double)d);
      launch_embed_grad(tok, c->g, gdense(r, 0), T, d, V, st);
      c->launches++;
    }
  }
};

int check_step_args(ppu_ctx* c, int replica, const void* tokens, int batch, int seq) {
  if (!c) return ppu_fail(PPU_EINVAL, "ctx is null");
  if (replica < 0 || replica >= c->K) return ppu_fail(PPU_EINVAL, "replica %d out of range", replica);
  if (!tokens) return ppu_fail(PPU_EINVAL, "tokens is null");
  if (batch < 1 || batch > c->cfg.max_batch || seq < 2 || seq > c->cfg.max_seq)
    return ppu_fail(PPU_EINVAL, "batch/seq outside [1,%d] x [2,%d]", c->cfg.max_batch, c->cfg.max_seq);
  if ((int64_t)batch * seq > (int64_t)c->cfg.max_batch * c->cfg.max_seq)
    return ppu_fail(PPU_EINVAL, "batch*seq too large");
  return PPU_OK;
}

}  // namespace

extern "C" int ppu_local_step(ppu_ctx* c, int replica, const int32_t* tokens, int batch, int seq) {
  int rc = check_step_args(c, replica, tokens, batch, seq);
  if (rc) return rc;
  ReplicaState& r = c->reps[replica];
  const int64_t launches0 = c->launches;
  c->flops_fwd = c->flops_dgrad = c->flops_wgrad = 0;
  ppu_make_resident(c, replica);
  Sched s(c, batch, seq);
  s.forward(tokens, &r, true);
  s.loss(tokens, 1, c->loss + replica);
  s.backward(r, tokens);
  if (s.rc) return ppu_fail(PPU_ECUDA, "kernel launch failed in local step (%d)", s.rc);
  r.step += 1;
  if (r.n_sub > 0) {
    AdamHyper hp;
    hp.lr = c->adam_lr; hp.beta1 = c->cfg.adam_beta1; hp.beta2 = c->cfg.adam_beta2;
    hp.eps = c->cfg.adam_eps; hp.wd = c->cfg.adam_wd;
    hp.bc1 = (float)(1.0 - std::pow((double)hp.beta1, (double)r.step));
    hp.bc2 = (float)(1.0 - std::pow((double)hp.beta2, (double)r.step));
    c->last_partials = s.partials();
    EvScope ev(c, PPU_CLS_ADAMW, 30.0 * (double)r.n_sub + 4.0 * (c->last_partials - 1) * (double)r.n_ffn);
    launch_adamw(r.d_segs, (int)r.segs.size(), r.master, r.m, r.v, c->grad, c->last_partials, c->max_ffn, c->w16,
                 c->cfg.d_model, c->cfg.d_ff, r.n_ffn, hp, c->stream);
    launch_adamw_dense(r.d_dense, (int)r.dense.size(), r.master, r.m, r.v, c->grad + c->max_ffn * c->wgrad_splits,
                       r.n_ffn, c->w16, r.n_ffn, r.n_dense, hp, c->stream);
    c->launches += (r.segs.empty() ? 0 : 1) + (r.dense.empty() ? 0 : 1);
  }
  r.stepped = true;
  c->last_stepped = replica;
  c->launches_last_step = c->launches - launches0;
  CUDA_OK(cudaGetLastError());
  return PPU_OK;
}

extern "C" int ppu_local_step_host(ppu_ctx* c, int replica, const int32_t* tokens_host, int batch,
                                   int seq, double* loss_out) {
  int rc = check_step_args(c, replica, tokens_host, batch, seq);
  if (rc) return rc;
  if (!loss_out) return ppu_fail(PPU_EINVAL, "loss_out is null");
  CUDA_OK(cudaMemcpyAsync(c->tok_stage, tokens_host, sizeof(int32_t) * batch * seq,
                          cudaMemcpyHostToDevice, c->stream));
  rc = ppu_local_step(c, replica, c->tok_stage, batch, seq);
  if (rc) return rc;
  return ppu_loss(c, replica, loss_out);
}

extern "C" int ppu_loss(ppu_ctx* c, int replica, double* loss_out) {
  if (!c) return ppu_fail(PPU_EINVAL, "ctx is null");
  if (replica < 0 || replica >= c->K) return ppu_fail(PPU_EINVAL, "replica %d out of range", replica);
  if (!loss_out) return ppu_fail(PPU_EINVAL, "loss_out is null");
  if (!c->reps[replica].stepped) return ppu_fail(PPU_ESTATE, "replica %d has not run a local step", replica);
  float v = 0.f;
  CUDA_OK(cudaMemcpyAsync(&v, c->loss + replica, 4, cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  *loss_out = (double)v;
  return ppu_check_flags(c);
}

extern "C" int ppu_eval_loss(ppu_ctx* c, int replica, const int32_t* tokens, int batch, int seq,
                             double* loss_out) {
  int rc = check_step_args(c, replica < 0 ? 0 : replica, tokens, batch, seq);
  if (rc) return rc;
  if (replica < -1) return ppu_fail(PPU_EINVAL, "replica out of range");
  if (!loss_out) return ppu_fail(PPU_EINVAL, "loss_out is null");
  ppu_make_resident(c, replica);
  Sched s(c, batch, seq);
  s.forward(tokens, replica >= 0 ? &c->reps[replica] : nullptr, false);
  s.loss(tokens, 0, c->loss + c->K);
  if (s.rc) return ppu_fail(PPU_ECUDA, "kernel launch failed in evaluation (%d)", s.rc);
  float v = 0.f;
  CUDA_OK(cudaMemcpyAsync(&v, c->loss + c->K, 4, cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  CUDA_OK(cudaGetLastError());
  *loss_out = (double)v;
  return ppu_check_flags(c);
}

namespace {
// Builds the outer-sync tables for a list of replicas: the segments of the canonical vector with
// their owners, the chunk list the kernel walks, and the per-hidden-unit owner lists of the FFN
// matrices.  Segments never straddle a layer (or the embedding / final-norm) boundary, so a
// streaming-sync group is a contiguous range of chunks.
int build_outer_tables(ppu_ctx* c, const std::vector<int32_t>& list) {
  const int L = c->cfg.n_layer, F = c->cfg.d_ff, d = c->cfg.d_model;
  const int64_t fd = (int64_t)F * d;
  std::vector<OuterSeg> segs;
  std::vector<DenseOwner> downers;
  // dense runs of the listed replicas, as (start, end, master, shift) events
  struct Run { int64_t lo, hi; float* master; int64_t shift; };
  std::vector<Run> runs;
  for (int k : list) {
    const ReplicaState& r = c->reps[k];
    for (const auto& s : r.dense) runs.push_back({s.canon_off, s.canon_off + s.len, r.master, s.packed_off - s.canon_off});
    // a replica's rows [lo, hi) of a W_in are one contiguous run of the canonical vector and of
    // its packed array alike, so W_in is swept like the runs outside the FFNs
    for (const auto& s : r.segs) {
      const int64_t lo = s.win_off + (int64_t)s.lo * d, hi = s.win_off + (int64_t)s.hi * d;
      runs.push_back({lo, hi, r.master, s.packed_off - lo});
    }
  }
  // cuts [lo, hi) of the canonical vector at every run boundary and lists each piece's owners;
  // neighbouring pieces with the same owners and shifts are joined
  auto add_dense = [&](int64_t lo, int64_t hi, int layer) {
    std::vector<int64_t> cuts = {lo, hi};
    for (const auto& r : runs) {
      if (r.lo > lo && r.lo < hi) cuts.push_back(r.lo);
      if (r.hi > lo && r.hi < hi) cuts.push_back(r.hi);
    }
    std::sort(cuts.begin(), cuts.end());
    cuts.erase(std::unique(cuts.begin(), cuts.end()), cuts.end());
    std::vector<DenseOwner> prev; bool have_prev = false;
    for (size_t i = 0; i + 1 < cuts.size(); ++i) {
      std::vector<DenseOwner> own;
      for (const auto& r : runs)
        if (r.lo <= cuts[i] && r.hi >= cuts[i + 1]) own.push_back({r.master, r.shift});
      const bool same = have_prev && own.size() == prev.size() &&
                        std::equal(own.begin(), own.end(), prev.begin(), [](const DenseOwner& a, const DenseOwner& b) {
                          return a.master == b.master && a.shift == b.shift; });
      if (same) { segs.back().len += cuts[i + 1] - cuts[i]; continue; }
      OuterSeg sg; sg.start = cuts[i]; sg.len = cuts[i + 1] - cuts[i]; sg.base = 0; sg.kind = 0; sg.layer = layer;
      sg.ob = (int32_t)downers.size();
      downers.insert(downers.end(), own.begin(), own.end());
      sg.oe = (int32_t)downers.size();
      segs.push_back(sg);
      prev = own; have_prev = true;
    }
  };
  std::vector<int> layer_seg_begin(L + 2, 0);
  add_dense(0, c->e_size, -1);
  for (int l = 0; l < L; ++l) {
    layer_seg_begin[l] = (int)segs.size();
    const int64_t base = c->e_size + (int64_t)l * c->layer_size;
    add_dense(base, base + c->rel_wout, l);           // attention, LayerNorm and W_in
    OuterSeg sg; sg.layer = l; sg.ob = sg.oe = 0; sg.len = fd;
    sg.start = sg.base = base + c->rel_wout; sg.kind = 2; segs.push_back(sg);
  }
  layer_seg_begin[L] = (int)segs.size();
  add_dense(c->off_lnfg, c->P, -1);
  layer_seg_begin[L + 1] = (int)segs.size();
  // chunk lists, one per segment kind (each kind has its own kernel), all in canonical order; for
  // every kind the index where each layer's chunks begin ([L]: the final norm, [L + 1]: the end)
  std::vector<OuterChunk> chunks;
  for (int kind = 0; kind < 3; ++kind) {
    c->kind_chunk_base[kind] = (int)chunks.size();
    c->layer_chunk_begin[kind].assign(L + 2, 0);
    int l_next = 0;
    for (size_t i = 0; i < segs.size(); ++i) {
      while (l_next <= L + 1 && (int)i >= layer_seg_begin[l_next])
        c->layer_chunk_begin[kind][l_next++] = (int)chunks.size() - c->kind_chunk_base[kind];
      if (segs[i].kind != kind) continue;
      for (int64_t off = 0; off < segs[i].len; off += OUTER_CHUNK) chunks.push_back({(int32_t)i, 0, off});
    }
    while (l_next <= L + 1) c->layer_chunk_begin[kind][l_next++] = (int)chunks.size() - c->kind_chunk_base[kind];
  }
  c->n_chunks = (int)chunks.size();
  // owners of every group of 8 hidden units, in the order the replicas were listed
  std::vector<std::vector<OuterOwner>> per_group((size_t)L * (F / 8));
  for (int k : list) {
    const ReplicaState& r = c->reps[k];
    for (size_t i = 0; i < r.segs.size(); ++i) {
      const SliceSeg& s = r.segs[i];
      OuterOwner o;
      o.master = r.master; o.in_off = s.packed_off;
      o.out_off = s.packed_off + (int64_t)(s.hi - s.lo) * d; o.lo = s.lo; o.hi = s.hi;
      const int l = r.seg_layer[i];
      for (int u8 = s.lo / 8; u8 < s.hi / 8; ++u8) per_group[(size_t)l * (F / 8) + u8].push_back(o);
    }
  }
  std::vector<int32_t> begin(per_group.size() + 1, 0);
  std::vector<OuterOwner> flat;
  for (size_t gi = 0; gi < per_group.size(); ++gi) {
    begin[gi] = (int32_t)flat.size();
    flat.insert(flat.end(), per_group[gi].begin(), per_group[gi].end());
  }
  begin[per_group.size()] = (int32_t)flat.size();
  if (segs.size() > c->cap_oseg || chunks.size() > c->cap_ochunk || downers.size() > c->cap_downer ||
      flat.size() > c->cap_uowner)
    return ppu_fail(PPU_ESTATE, "outer-sync tables larger than the arena reserved for them");
  // the previous sync's kernel may still be reading the tables
  CUDA_OK(cudaStreamSynchronize(c->stream));
  CUDA_OK(cudaMemcpy(c->d_oseg, segs.data(), segs.size() * sizeof(OuterSeg), cudaMemcpyHostToDevice));
  CUDA_OK(cudaMemcpy(c->d_ochunk, chunks.data(), chunks.size() * sizeof(OuterChunk), cudaMemcpyHostToDevice));
  if (!downers.empty())
    CUDA_OK(cudaMemcpy(c->d_downer, downers.data(), downers.size() * sizeof(DenseOwner), cudaMemcpyHostToDevice));
  CUDA_OK(cudaMemcpy(c->d_unit_begin, begin.data(), begin.size() * 4, cudaMemcpyHostToDevice));
  if (!flat.empty())
    CUDA_OK(cudaMemcpy(c->d_unit_owner, flat.data(), flat.size() * sizeof(OuterOwner), cudaMemcpyHostToDevice));
  c->h_oseg = segs;
  c->cached_sync_list = list;
  return PPU_OK;
}

// Outer step over the listed replicas on one group of positions (group < 0: every position).
int outer_sync_impl(ppu_ctx* c, const int32_t* replicas, int n, int group, int n_groups) {
  if (!c) return ppu_fail(PPU_EINVAL, "ctx is null");
  if (n < 0 || (n > 0 && !replicas)) return ppu_fail(PPU_EINVAL, "bad replica list");
  const int L = c->cfg.n_layer, F = c->cfg.d_ff, d = c->cfg.d_model;
  if (group >= 0 && (n_groups < 1 || L % n_groups != 0 || group > n_groups))
    return ppu_fail(PPU_EINVAL, "group %d of %d does not divide %d layers", group, n_groups, L);
  std::vector<int32_t> list(replicas, replicas + n);
  {
    std::vector<int32_t> sorted = list;
    std::sort(sorted.begin(), sorted.end());
    for (int i = 0; i < n; ++i) {
      if (sorted[i] < 0 || sorted[i] >= c->K) return ppu_fail(PPU_EINVAL, "replica %d out of range", sorted[i]);
      if (i && sorted[i] == sorted[i - 1]) return ppu_fail(PPU_EINVAL, "replica %d listed twice", sorted[i]);
    }
  }
  const int64_t launches0 = c->launches;
  if (list != c->cached_sync_list || c->n_chunks == 0) {
    const int rc = build_outer_tables(c, list);
    if (rc) return rc;
  }
  // layers [l0, l1) and, for the last group, the embeddings and the final LayerNorm
  const bool all = group < 0, tail = all || group == n_groups;
  const int per = all ? L : L / n_groups;
  const int l0 = all ? 0 : (tail ? L : group * per), l1 = all ? L : (tail ? L : l0 + per);
  // positions swept and (owner, owned position) pairs inside the swept range
  const int64_t lo_pos = c->e_size + (int64_t)l0 * c->layer_size, hi_pos = c->e_size + (int64_t)l1 * c->layer_size;
  auto inside = [&](int64_t pos) { return (pos >= lo_pos && pos < hi_pos) || (tail && (pos < c->e_size || pos >= c->off_lnfg)); };
  double owned = 0;
  for (int k : list) {
    const ReplicaState& r = c->reps[k];
    for (size_t i = 0; i < r.segs.size(); ++i)
      if (r.seg_layer[i] >= l0 && r.seg_layer[i] < l1) owned += 2.0 * (double)(r.segs[i].hi - r.segs[i].lo) * d;
    for (const auto& s : r.dense) if (inside(s.canon_off)) owned += (double)s.len;
  }
  // a group step rewrites the working copy only on its own positions: everywhere else it must
  // already hold the global values, not the resident replica's
  if (!all) ppu_make_resident(c, -1);
  OuterTables t;
  t.segs = c->d_oseg; t.chunks = c->d_ochunk; t.dense_owner = c->d_downer;
  t.unit_begin = c->d_unit_begin; t.unit_owner = c->d_unit_owner; t.d = d; t.F = F;
  t.div_d = make_fast_div((uint32_t)d); t.div_F = make_fast_div((uint32_t)F);
  double swept = 0;
  if (all) swept = (double)c->P;
  else if (tail) swept = (double)c->e_size + (double)(c->P - c->off_lnfg);
  else swept = (double)(l1 - l0) * (double)c->layer_size;
  c->outer_bytes = 18.0 * swept + 8.0 * owned;
  {
    EvScope ev(c, PPU_CLS_OUTER, c->outer_bytes);     // brackets all launches of this sync
    if (all) {
      // E's chunks precede layer 0 in the kind-0 list: index 0 is the start of E
      for (int kind = 0; kind < 3; ++kind) {
        const int n = (kind < 2 ? c->kind_chunk_base[kind + 1] : c->n_chunks) - c->kind_chunk_base[kind];
        if (n <= 0) continue;
        launch_outer(t, kind, c->theta, c->buf, c->w16, c->cfg.outer_lr, c->cfg.outer_momentum,
                     c->kind_chunk_base[kind], n, c->stream);
        c->launches++;
      }
    } else if (tail) {
      // embeddings (the kind-0 chunks before layer 0) and the final LayerNorm
      launch_outer(t, 0, c->theta, c->buf, c->w16, c->cfg.outer_lr, c->cfg.outer_momentum,
                   c->kind_chunk_base[0], c->layer_chunk_begin[0][0], c->stream);
      launch_outer(t, 0, c->theta, c->buf, c->w16, c->cfg.outer_lr, c->cfg.outer_momentum,
                   c->kind_chunk_base[0] + c->layer_chunk_begin[0][L],
                   c->layer_chunk_begin[0][L + 1] - c->layer_chunk_begin[0][L], c->stream);
      c->launches += 2;
    } else {
      for (int kind = 0; kind < 3; ++kind) {
        const int lo = c->layer_chunk_begin[kind][l0], hi = c->layer_chunk_begin[kind][l1];
        if (hi <= lo) continue;
        launch_outer(t, kind, c->theta, c->buf, c->w16, c->cfg.outer_lr, c->cfg.outer_momentum,
                     c->kind_chunk_base[kind] + lo, hi - lo, c->stream);
        c->launches++;
      }
    }
  }
  c->resident = -1;   // the working copy now holds the global parameters everywhere
  c->launches_last_sync = c->launches - launches0;
  CUDA_OK(cudaGetLastError());
  return PPU_OK;
}
}  // namespace

extern "C" int ppu_outer_sync(ppu_ctx* c, const int32_t* replicas, int n) {
  return outer_sync_impl(c, replicas, n, -1, 0);
}

extern "C" int ppu_outer_sync_group(ppu_ctx* c, const int32_t* replicas, int n, int group, int n_groups) {
  if (group < 0) return ppu_fail(PPU_EINVAL, "group %d is negative", group);
  return outer_sync_impl(c, replicas, n, group, n_groups);
}

extern "C" int ppu_profile_enable(ppu_ctx* c, int enable) {
  if (!c) return ppu_fail(PPU_EINVAL, "ctx is null");
  c->profiling = enable != 0;
  return PPU_OK;
}

extern "C" int ppu_profile_read(ppu_ctx* c, ppu_profile_t* out) {
  if (!c || !out) return ppu_fail(PPU_EINVAL, "null argument");
  CUDA_OK(cudaStreamSynchronize(c->stream));
  memset(out, 0, sizeof(*out));
  for (size_t i = 0; i < c->ev_recs.size(); ++i) {
    float ms = 0.f;
    CUDA_OK(cudaEventElapsedTime(&ms, c->ev_pool[2 * i], c->ev_pool[2 * i + 1]));
    const int cls = c->ev_recs[i].cls;
    out->ms[cls] += ms; out->work[cls] += c->ev_recs[i].work; out->launches[cls]++;
  }
  out->dropped = c->ev_dropped;
  c->ev_recs.clear();
  c->ev_dropped = 0;
  return PPU_OK;
}
