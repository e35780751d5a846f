// C ABI of the ppu library: context set-up, arena layout and the accessors.  The step
// scheduler (forward, restricted backward, AdamW, outer sync) lives in ppu_step.cu.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <algorithm>
#include "ppu_ctx.cuh"

static thread_local char g_err[512] = "";

int ppu_fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}
#define CUDA_OK(call)                                                                    \
  do {                                                                                   \
    cudaError_t e_ = (call);                                                             \
    if (e_ != cudaSuccess)                                                               \
      return ppu_fail(PPU_ECUDA, "%s failed: %s", #call, cudaGetErrorString(e_));        \
  } while (0)

extern "C" const char* ppu_last_error(void) { return g_err; }

// ---------------------------------------------------------------------------------------
// validation and subset tables
// ---------------------------------------------------------------------------------------
static int validate_cfg(const ppu_model_cfg* c) {
  if (!c) return ppu_fail(PPU_EINVAL, "cfg is null");
  if (c->n_layer < 1 || c->d_model < 8 || c->n_head < 1 || c->d_ff < 8 || c->vocab < 8 ||
      c->max_batch < 1 || c->max_seq < 2)
    return ppu_fail(PPU_ESHAPE, "non-positive model dimension");
  if (c->d_model % c->n_head) return ppu_fail(PPU_ESHAPE, "d_model %% n_head != 0");
  const int dh = c->d_model / c->n_head;
  if (dh != 16 && dh != 32 && dh != 64 && dh != 128)
    return ppu_fail(PPU_ESHAPE, "d_head must be 16, 32, 64 or 128 (got %d)", dh);
  if (c->d_model % 8 || c->d_ff % 8 || c->vocab % 8)
    return ppu_fail(PPU_ESHAPE, "d_model, d_ff and vocab must be multiples of 8");
  if (c->d_model > 4096) return ppu_fail(PPU_ESHAPE, "d_model > 4096 not supported");
  if (c->vocab > 65536) return ppu_fail(PPU_ESHAPE, "vocab > 65536 not supported");
  if ((int64_t)c->max_batch * c->max_seq > (1 << 20))
    return ppu_fail(PPU_ESHAPE, "max_batch * max_seq too large");
  if (!(c->ln_eps > 0.f) || !(c->rope_base > 1.f)) return ppu_fail(PPU_EINVAL, "bad ln_eps/rope_base");
  if (!(c->adam_beta1 >= 0.f && c->adam_beta1 < 1.f && c->adam_beta2 >= 0.f && c->adam_beta2 < 1.f))
    return ppu_fail(PPU_EINVAL, "AdamW betas must lie in [0,1)");
  return PPU_OK;
}

static int build_ranges(const ppu_model_cfg* c, const ppu_subset_spec* s,
                        std::vector<ReplicaState>& reps) {
  if (!s) return ppu_fail(PPU_EINVAL, "subset spec is null");
  const int K = s->n_replicas, L = c->n_layer, F = c->d_ff;
  if (K < 1 || K > 4096) return ppu_fail(PPU_ESUBSET, "n_replicas out of range");
  reps.assign(K, ReplicaState());
  for (int k = 0; k < K; ++k) {
    reps[k].lo.assign(L, 0);
    reps[k].hi.assign(L, 0);
  }
  if (s->mode == PPU_SUBSET_FFN_SLICE) {
    const int N = s->n_slices;
    if (N < 1 || K % N) return ppu_fail(PPU_ESUBSET, "n_replicas must be a multiple of n_slices");
    if (F % N || (F / N) % 8) return ppu_fail(PPU_ESUBSET, "d_ff / n_slices must be a multiple of 8");
    const int w = F / N;
    for (int k = 0; k < K; ++k)
      for (int l = 0; l < L; ++l) { reps[k].lo[l] = (k % N) * w; reps[k].hi[l] = (k % N + 1) * w; }
  } else if (s->mode == PPU_SUBSET_FFN_LAYERS) {
    const int st = s->layer_stride;
    if (st < 1 || st > L) return ppu_fail(PPU_ESUBSET, "layer_stride out of range");
    for (int k = 0; k < K; ++k)
      for (int l = 0; l < L; ++l)
        if (l % st == k % st) { reps[k].lo[l] = 0; reps[k].hi[l] = F; }
  } else if (s->mode == PPU_SUBSET_EXPLICIT) {
    if (!s->ranges) return ppu_fail(PPU_ESUBSET, "explicit mode needs ranges");
    for (int k = 0; k < K; ++k)
      for (int l = 0; l < L; ++l) {
        const int lo = s->ranges[((int64_t)k * L + l) * 2], hi = s->ranges[((int64_t)k * L + l) * 2 + 1];
        if (lo < 0 || hi < lo || hi > F || lo % 8 || hi % 8)
          return ppu_fail(PPU_ESUBSET, "replica %d layer %d: bad range [%d,%d)", k, l, lo, hi);
        reps[k].lo[l] = lo;
        reps[k].hi[l] = hi;
      }
  } else {
    return ppu_fail(PPU_ESUBSET, "unknown subset mode %d", s->mode);
  }
  // heads whose query / key / value rows are trained, and the never-sliced rest
  const int h = c->n_head;
  if (s->train_non_mlp != 0 && s->train_non_mlp != 1)
    return ppu_fail(PPU_ESUBSET, "train_non_mlp must be 0 or 1");
  if (s->n_head_slices < 0 || (s->n_head_slices > 0 && (h % s->n_head_slices || K % s->n_head_slices)))
    return ppu_fail(PPU_ESUBSET, "n_head and n_replicas must be multiples of n_head_slices");
  for (int k = 0; k < K; ++k) {
    ReplicaState& r = reps[k];
    r.rest = s->train_non_mlp == 1;
    if (s->head_ranges) {
      r.h_lo = s->head_ranges[2 * k]; r.h_hi = s->head_ranges[2 * k + 1];
      if (r.h_lo < 0 || r.h_hi < r.h_lo || r.h_hi > h)
        return ppu_fail(PPU_ESUBSET, "replica %d: bad head range [%d,%d)", k, r.h_lo, r.h_hi);
    } else if (s->n_head_slices > 0) {
      const int per = h / s->n_head_slices;
      r.h_lo = (k % s->n_head_slices) * per; r.h_hi = r.h_lo + per;
    } else if (r.rest) {
      r.h_lo = 0; r.h_hi = h;
    }
  }
  return PPU_OK;
}

static void build_geometry(ppu_ctx* c) {
  const int64_t d = c->cfg.d_model, F = c->cfg.d_ff, V = c->cfg.vocab;
  const int L = c->cfg.n_layer;
  c->e_size = V * d;
  int64_t r = 0;
  c->rel_ln1g = r; r += d;
  c->rel_ln1b = r; r += d;
  c->rel_wq = r; r += 3 * d * d;
  c->rel_wo = r; r += d * d;
  c->rel_ln2g = r; r += d;
  c->rel_ln2b = r; r += d;
  c->rel_win = r; r += F * d;
  c->rel_wout = r; r += d * F;
  c->layer_size = r;
  c->off_lnfg = c->e_size + L * c->layer_size;
  c->off_lnfb = c->off_lnfg + d;
  c->P = c->off_lnfb + d;
  auto add = [&](const std::string& n, int64_t off, int nd, int64_t s0, int64_t s1) {
    TensorRec t; t.name = n; t.offset = off; t.ndim = nd; t.shape[0] = s0; t.shape[1] = s1;
    c->tensors.push_back(t);
  };
  c->tensors.clear();
  add("E", 0, 2, V, d);
  for (int l = 0; l < L; ++l) {
    const int64_t b = c->e_size + l * c->layer_size;
    const std::string p = "l" + std::to_string(l) + ".";
    add(p + "ln1_g", b + c->rel_ln1g, 1, d, 1);
    add(p + "ln1_b", b + c->rel_ln1b, 1, d, 1);
    add(p + "W_q", b + c->rel_wq, 2, d, d);
    add(p + "W_k", b + c->rel_wq + d * d, 2, d, d);
    add(p + "W_v", b + c->rel_wq + 2 * d * d, 2, d, d);
    add(p + "W_o", b + c->rel_wo, 2, d, d);
    add(p + "ln2_g", b + c->rel_ln2g, 1, d, 1);
    add(p + "ln2_b", b + c->rel_ln2b, 1, d, 1);
    add(p + "W_in", b + c->rel_win, 2, F, d);
    add(p + "W_out", b + c->rel_wout, 2, d, F);
  }
  add("lnf_g", c->off_lnfg, 1, d, 1);
  add("lnf_b", c->off_lnfb, 1, d, 1);
  // packed subset tables: FFN blocks first, then the dense runs in canonical order
  const int dh = (int)(d / c->cfg.n_head);
  c->max_ffn = c->max_dense = 0;
  c->min_lowest = L;
  c->any_rest = false;
  for (auto& r2 : c->reps) {
    r2.segs.clear(); r2.seg_layer.clear(); r2.dense.clear();
    r2.n_ffn = r2.n_dense = r2.n_sub = 0; r2.lowest = -1;
    for (int l = 0; l < L; ++l) {
      if (r2.hi[l] <= r2.lo[l]) continue;
      if (r2.lowest < 0) r2.lowest = l;
      SliceSeg s;
      const int64_t b = c->e_size + l * c->layer_size;
      s.win_off = b + c->rel_win; s.wout_off = b + c->rel_wout;
      s.packed_off = r2.n_ffn; s.lo = r2.lo[l]; s.hi = r2.hi[l];
      r2.segs.push_back(s); r2.seg_layer.push_back(l);
      r2.n_ffn += 2 * (int64_t)(s.hi - s.lo) * d;
    }
    int64_t at = r2.n_ffn;
    auto run = [&](int64_t off, int64_t len, int decay) {
      if (len <= 0) return;
      DenseSeg s; s.canon_off = off; s.len = len; s.packed_off = at; s.decay = decay; s.pad = 0;
      r2.dense.push_back(s);
      at += len;
    };
    const int64_t r0 = (int64_t)r2.h_lo * dh * d, rn = (int64_t)(r2.h_hi - r2.h_lo) * dh * d;
    if (r2.rest) run(0, c->e_size, 1);
    for (int l = 0; l < L && r2.deep(); ++l) {
      const int64_t b = c->e_size + l * c->layer_size;
      if (r2.rest) { run(b + c->rel_ln1g, d, 0); run(b + c->rel_ln1b, d, 0); }
      for (int q = 0; q < 3; ++q) run(b + c->rel_wq + q * d * d + r0, rn, 1);
      if (r2.rest) { run(b + c->rel_wo, d * d, 1); run(b + c->rel_ln2g, d, 0); run(b + c->rel_ln2b, d, 0); }
    }
    if (r2.rest) { run(c->off_lnfg, d, 0); run(c->off_lnfb, d, 0); }
    r2.n_dense = at - r2.n_ffn;
    r2.n_sub = at;
    if (r2.deep()) r2.lowest = 0;
    if (r2.n_ffn > c->max_ffn) c->max_ffn = r2.n_ffn;
    if (r2.n_dense > c->max_dense) c->max_dense = r2.n_dense;
    if (r2.lowest >= 0 && r2.lowest < c->min_lowest) c->min_lowest = r2.lowest;
    c->any_rest = c->any_rest || r2.rest;
  }
  c->max_ffn = (c->max_ffn + 63) & ~(int64_t)63;
  c->wmax.assign(L, 0);
  for (auto& r2 : c->reps)
    for (int l = 0; l < L; ++l) c->wmax[l] = std::max(c->wmax[l], (int)(r2.hi[l] - r2.lo[l]));
  // The subset products have few output tiles when slices are narrow: cut their reduction over
  // tokens so that about one wave of CTAs works on them.  One factor for the whole context
  // (148 SMs assumed: the factor only balances work, any value gives the same sums in order).
  int64_t min_tiles = 1 << 30;
  for (auto& r2 : c->reps)
    for (auto& s : r2.segs) {
      const int64_t t = (int64_t)((s.hi - s.lo + 127) / 128) * ((d + 127) / 128);
      if (t < min_tiles) min_tiles = t;
    }
  c->wgrad_splits = 1;
  while (min_tiles * c->wgrad_splits * 2 <= 148 && c->wgrad_splits < 8) c->wgrad_splits *= 2;
  // Slices wide enough for the SM-pair kernel (16 tiles of 256 x 256 or more) are cut so that
  // the 74 pairs are filled once: 32 tiles (a 1024-wide slice at d = 2048) run as two slices.
  int64_t min_pair_tiles = 1 << 30;
  for (auto& r2 : c->reps)
    for (auto& s : r2.segs) {
      const int64_t t = (int64_t)((s.hi - s.lo + 255) / 256) * ((d + 255) / 256);
      if (t < min_pair_tiles) min_pair_tiles = t;
    }
  if (min_pair_tiles >= 16 && min_pair_tiles < (1 << 30)) {
    c->wgrad_splits = (int)(74 / min_pair_tiles);
    if (c->wgrad_splits < 1) c->wgrad_splits = 1;
    if (c->wgrad_splits > 8) c->wgrad_splits = 8;
  }
}

// Carves the arena.  With base == nullptr only the sizes are computed.
static size_t carve(ppu_ctx* c, uint8_t* base) {
  size_t off = 0;
  // every sub-buffer is followed by a guard block that no kernel may touch (ppu_check_guards)
  c->guards.clear();
  auto take = [&](size_t bytes) -> uint8_t* {
    uint8_t* p = base ? base + off : nullptr;
    off += (bytes + 255) & ~(size_t)255;
    c->guards.push_back(off);
    off += PPU_GUARD_BYTES;
    return p;
  };
  const int64_t d = c->cfg.d_model, F = c->cfg.d_ff, V = c->cfg.vocab;
  const int L = c->cfg.n_layer, h = c->cfg.n_head;
  const int64_t T = (int64_t)c->cfg.max_batch * c->cfg.max_seq;
  c->theta = (float*)take(c->P * 4);
  c->buf = (float*)take(c->P * 4);
  c->w16 = (bf16*)take(c->P * 2);
  size_t unit_entries = 0;
  for (auto& r : c->reps) {
    r.master = (float*)take(r.n_sub * 4);
    r.m = (float*)take(r.n_sub * 4);
    r.v = (float*)take(r.n_sub * 4);
    r.d_segs = (SliceSeg*)take(sizeof(SliceSeg) * (r.segs.size() + 1));
    r.d_dense = (DenseSeg*)take(sizeof(DenseSeg) * (r.dense.size() + 1));
    for (auto& s : r.segs) unit_entries += (size_t)(s.hi - s.lo) / 8;
  }
  c->grad = (float*)take((c->max_ffn * c->wgrad_splits + c->max_dense) * 4);
  c->loss = (float*)take(sizeof(float) * (c->K + 1));
  c->flags = (int*)take(sizeof(int) * PPU_FLAG_COUNT);
  c->rope_cs = (float2*)take(sizeof(float2) * c->cfg.max_seq * (d / h / 2));
  c->tok_stage = (int32_t*)take(sizeof(int32_t) * T);
  // outer-sync tables: a layer's dense block splits at most at every head boundary of W_q/k/v and
  // at both ends of every replica's W_in rows
  c->cap_oseg = 8 + (size_t)L * (16 + 6 * (size_t)(h + 1) + 2 * (size_t)c->K + 2);
  c->cap_ochunk = (size_t)(c->P / OUTER_CHUNK) + c->cap_oseg + 8;
  c->cap_downer = c->cap_oseg * (size_t)c->K + 1;
  c->cap_uowner = unit_entries + 1;
  c->d_oseg = (OuterSeg*)take(sizeof(OuterSeg) * c->cap_oseg);
  c->d_ochunk = (OuterChunk*)take(sizeof(OuterChunk) * c->cap_ochunk);
  c->d_downer = (DenseOwner*)take(sizeof(DenseOwner) * c->cap_downer);
  c->d_unit_begin = (int32_t*)take(sizeof(int32_t) * ((size_t)L * (F / 8) + 1));
  c->d_unit_owner = (OuterOwner*)take(sizeof(OuterOwner) * c->cap_uowner);
  c->state_bytes = off;
  // Activations kept for the backward pass, per layer.  Layers below the lowest layer that any
  // replica's backward pass reaches run forward only: they share one set of buffers (two for
  // the residual stream, which alternates) and keep no pre-activation at all.
  c->acts.assign(L, LayerActs());
  const int first_kept = c->min_lowest < L ? c->min_lowest : L;
  LayerActs shared = LayerActs();
  float* shared_x[2] = {nullptr, nullptr};
  auto layer_set = [&](LayerActs& a) {
    a.x1 = (float*)take(T * d * 4);
    a.st1 = (float2*)take(T * 8);
    a.st2 = (float2*)take(T * 8);
    a.qkv = (bf16*)take(T * 3 * d * 2);
    a.U = (bf16*)take(T * d * 2);
    a.lse = (float*)take(T * h * 4);
    a.b = (bf16*)take(T * d * 2);
  };
  if (first_kept > 0) {
    layer_set(shared);
    shared_x[0] = (float*)take(T * d * 4);
    shared_x[1] = (float*)take(T * d * 4);
  }
  for (int l = 0; l < L; ++l) {
    LayerActs& a = c->acts[l];
    if (l < first_kept) {
      a = shared;
      a.x = shared_x[l & 1];
      a.Hd = nullptr;
      a.As = nullptr;
      continue;
    }
    a.x = (float*)take(T * d * 4);
    layer_set(a);
    a.Hd = (bf16*)take(T * F * 2);
    a.As = (bf16*)take(T * (int64_t)c->wmax[l] * 2);
  }
  c->x_last = (float*)take(T * d * 4);
  c->stf = (float2*)take(T * 8);
  c->a16 = (bf16*)take(T * d * 2);
  c->A_tmp = (bf16*)take(T * F * 2);
  c->f16 = (bf16*)take(T * d * 2);
  c->logits = (bf16*)take(T * V * 2);
  c->g = (float*)take(T * d * 4);
  c->g16 = (bf16*)take(T * d * 2);
  c->dHd = (bf16*)take(T * F * 2);
  c->t16 = (bf16*)take(T * d * 2);
  c->dqkv = (bf16*)take(T * 3 * d * 2);
  c->attn_scratch = (float*)take(T * h * 4);
  c->row_loss = (float*)take(T * 4);
  c->ln_partial = c->any_rest ? (float*)take((size_t)2 * ln_param_partial_blocks(T) * d * 4) : nullptr;
  c->act_bytes = off - c->state_bytes;
  return off;
}

static int init_ctx(ppu_ctx* c, const ppu_model_cfg* cfg, const ppu_subset_spec* spec) {
  int rc = validate_cfg(cfg);
  if (rc) return rc;
  c->cfg = *cfg;
  rc = build_ranges(cfg, spec, c->reps);
  if (rc) return rc;
  c->K = spec->n_replicas;
  c->adam_lr = cfg->adam_lr;
  build_geometry(c);
  return PPU_OK;
}

// every replica's packed values <- the global parameters (Algorithm 1, the replica reset)
static void ppu_restart_replicas(ppu_ctx* c) {
  for (auto& r : c->reps) {
    launch_slices_gather(r.d_segs, (int)r.segs.size(), c->theta, r.master, c->cfg.d_model,
                         c->cfg.d_ff, r.n_ffn, c->stream);
    launch_dense_move(r.d_dense, (int)r.dense.size(), r.master, c->theta, nullptr, 0, r.n_ffn, r.n_dense,
                      c->stream);
  }
}

extern "C" int ppu_query_bytes(const ppu_model_cfg* cfg, const ppu_subset_spec* spec, size_t* bytes) {
  if (!bytes) return ppu_fail(PPU_EINVAL, "bytes is null");
  ppu_ctx tmp;
  int rc = init_ctx(&tmp, cfg, spec);
  if (rc) return rc;
  *bytes = carve(&tmp, nullptr);
  return PPU_OK;
}

extern "C" int ppu_create(const ppu_model_cfg* cfg, const ppu_subset_spec* spec, void* arena,
                          size_t arena_bytes, void* cuda_stream, ppu_ctx** out) {
  if (!out) return ppu_fail(PPU_EINVAL, "out is null");
  *out = nullptr;
  if (!arena) return ppu_fail(PPU_EINVAL, "arena is null");
  if (reinterpret_cast<uintptr_t>(arena) & 255) return ppu_fail(PPU_EINVAL, "arena not 256-byte aligned");
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1)
    return ppu_fail(PPU_ECUDA, "no CUDA device: this library has no CPU path");
  ppu_ctx* c = new ppu_ctx();
  int rc = init_ctx(c, cfg, spec);
  if (rc) { delete c; return rc; }
  const size_t need = carve(c, (uint8_t*)arena);
  if (arena_bytes < need) {
    delete c;
    return ppu_fail(PPU_ENOMEM, "arena has %zu bytes, %zu needed", arena_bytes, need);
  }
  c->arena = (uint8_t*)arena;
  c->arena_bytes = need;
  c->stream = (cudaStream_t)cuda_stream;
  if (gemm_tc_init() != 0) {
    delete c;
    return ppu_fail(PPU_ECUDA, "cuTensorMapEncodeTiled not available from the driver");
  }
  cudaStream_t st = c->stream;
#define CREATE_OK(call)                                                                \
  do {                                                                                 \
    cudaError_t e_ = (call);                                                           \
    if (e_ != cudaSuccess) {                                                           \
      delete c;                                                                        \
      return ppu_fail(PPU_ECUDA, "%s failed: %s", #call, cudaGetErrorString(e_));      \
    }                                                                                  \
  } while (0)
  CREATE_OK(cudaMemsetAsync(c->arena, 0, c->state_bytes, st));
  for (size_t g : c->guards) CREATE_OK(cudaMemsetAsync(c->arena + g, PPU_GUARD_BYTE, PPU_GUARD_BYTES, st));
  // LayerNorm gains start at one
  {
    std::vector<float> ones(c->cfg.d_model, 1.f);
    for (const auto& t : c->tensors)
      if (t.name.size() > 2 && t.name.compare(t.name.size() - 2, 2, "_g") == 0)
        CREATE_OK(cudaMemcpyAsync(c->theta + t.offset, ones.data(), ones.size() * 4,
                                  cudaMemcpyHostToDevice, st));
    CREATE_OK(cudaStreamSynchronize(st));
  }
  launch_cast_bf16(c->theta, c->w16, c->P, st);
  // rotary table in double precision on the host
  {
    const int dh = c->cfg.d_model / c->cfg.n_head, hp = dh / 2;
    std::vector<float2> cs((size_t)c->cfg.max_seq * hp);
    for (int s = 0; s < c->cfg.max_seq; ++s)
      for (int i = 0; i < hp; ++i) {
        const double ang = (double)s * std::pow((double)c->cfg.rope_base, -2.0 * i / dh);
        cs[(size_t)s * hp + i] = make_float2((float)std::cos(ang), (float)std::sin(ang));
      }
    CREATE_OK(cudaMemcpyAsync(c->rope_cs, cs.data(), cs.size() * sizeof(float2),
                              cudaMemcpyHostToDevice, st));
    for (auto& r : c->reps) {
      if (!r.segs.empty())
        CREATE_OK(cudaMemcpyAsync(r.d_segs, r.segs.data(), r.segs.size() * sizeof(SliceSeg),
                                  cudaMemcpyHostToDevice, st));
      if (!r.dense.empty())
        CREATE_OK(cudaMemcpyAsync(r.d_dense, r.dense.data(), r.dense.size() * sizeof(DenseSeg),
                                  cudaMemcpyHostToDevice, st));
    }
    CREATE_OK(cudaStreamSynchronize(st));
  }
  ppu_restart_replicas(c);
  CREATE_OK(cudaStreamSynchronize(st));
  CREATE_OK(cudaGetLastError());
#undef CREATE_OK
  *out = c;
  return PPU_OK;
}

extern "C" int ppu_destroy(ppu_ctx* ctx) {
  if (!ctx) return PPU_OK;
  cudaStreamSynchronize(ctx->stream);
  for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
  delete ctx;
  return PPU_OK;
}

// ---------------------------------------------------------------------------------------
// accessors
// ---------------------------------------------------------------------------------------
int ppu_check_flags(ppu_ctx* c);                    // ppu_step.cu
int ppu_make_resident(ppu_ctx* c, int replica);     // ppu_step.cu

#define NEED_CTX(c) do { if (!(c)) return ppu_fail(PPU_EINVAL, "ctx is null"); } while (0)
#define NEED_REPLICA(c, k)                                                               \
  do { if ((k) < 0 || (k) >= (c)->K) return ppu_fail(PPU_EINVAL, "replica %d out of range", (k)); } while (0)

extern "C" int ppu_param_count(const ppu_ctx* ctx, int64_t* n) {
  NEED_CTX(ctx);
  if (!n) return ppu_fail(PPU_EINVAL, "n is null");
  *n = ctx->P;
  return PPU_OK;
}
extern "C" int ppu_tensor_count(const ppu_ctx* ctx, int32_t* n) {
  NEED_CTX(ctx);
  if (!n) return ppu_fail(PPU_EINVAL, "n is null");
  *n = (int32_t)ctx->tensors.size();
  return PPU_OK;
}
extern "C" int ppu_tensor_info(const ppu_ctx* ctx, int32_t index, char* name, int32_t name_cap,
                               int64_t* offset, int32_t* ndim, int64_t* shape) {
  NEED_CTX(ctx);
  if (index < 0 || index >= (int32_t)ctx->tensors.size()) return ppu_fail(PPU_EINVAL, "tensor index out of range");
  const TensorRec& t = ctx->tensors[index];
  if (name && name_cap > 0) { strncpy(name, t.name.c_str(), name_cap - 1); name[name_cap - 1] = 0; }
  if (offset) *offset = t.offset;
  if (ndim) *ndim = t.ndim;
  if (shape) { shape[0] = t.shape[0]; shape[1] = t.shape[1]; }
  return PPU_OK;
}

// Moves between a canonical host vector and a replica's packed host array (the order of
// ppu_subset_index).  to_packed: packed <- theta on the trained positions; else the reverse.
static void host_pack(const ppu_ctx* c, const ReplicaState& r, float* theta, float* packed, bool to_packed) {
  const int64_t d = c->cfg.d_model, F = c->cfg.d_ff;
  auto mv = [&](float* canon, float* pk, size_t n) {
    if (to_packed) memcpy(pk, canon, n * 4); else memcpy(canon, pk, n * 4);
  };
  for (const auto& s : r.segs) {
    const int w = s.hi - s.lo;
    float* p = packed + s.packed_off;
    mv(theta + s.win_off + (int64_t)s.lo * d, p, (size_t)w * d);
    p += (int64_t)w * d;
    for (int64_t row = 0; row < d; ++row) mv(theta + s.wout_off + row * F + s.lo, p + row * w, (size_t)w);
  }
  for (const auto& s : r.dense) mv(theta + s.canon_off, packed + s.packed_off, (size_t)s.len);
}

extern "C" int ppu_set_params(ppu_ctx* c, int replica, const float* theta, int64_t n) {
  NEED_CTX(c);
  if (!theta || n != c->P) return ppu_fail(PPU_EINVAL, "theta null or wrong length");
  if (replica < -1 || replica >= c->K) return ppu_fail(PPU_EINVAL, "replica out of range");
  if (replica >= 0) {
    ReplicaState& r = c->reps[replica];
    if (r.n_sub == 0) return PPU_OK;
    std::vector<float> packed(r.n_sub);
    host_pack(c, r, const_cast<float*>(theta), packed.data(), true);
    CUDA_OK(cudaStreamSynchronize(c->stream));
    CUDA_OK(cudaMemcpy(r.master, packed.data(), r.n_sub * 4, cudaMemcpyHostToDevice));
    if (c->resident == replica) {       // lay the new values over the working copy again
      c->resident = -2;                 // neither the global values nor any replica's
      ppu_make_resident(c, replica);
    }
    return PPU_OK;
  }
  CUDA_OK(cudaMemcpyAsync(c->theta, theta, n * 4, cudaMemcpyHostToDevice, c->stream));
  launch_cast_bf16(c->theta, c->w16, c->P, c->stream);
  ppu_restart_replicas(c);
  c->resident = -1;
  CUDA_OK(cudaStreamSynchronize(c->stream));
  CUDA_OK(cudaGetLastError());
  return PPU_OK;
}

extern "C" int ppu_get_params(ppu_ctx* c, int replica, float* theta, int64_t n) {
  NEED_CTX(c);
  if (!theta || n != c->P) return ppu_fail(PPU_EINVAL, "theta null or wrong length");
  if (replica < -1 || replica >= c->K) return ppu_fail(PPU_EINVAL, "replica out of range");
  CUDA_OK(cudaMemcpyAsync(theta, c->theta, n * 4, cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  if (replica < 0) return PPU_OK;
  // the replica's packed subset is laid over the global vector on the host
  ReplicaState& r = c->reps[replica];
  if (r.n_sub == 0) return PPU_OK;
  std::vector<float> packed(r.n_sub);
  CUDA_OK(cudaMemcpy(packed.data(), r.master, r.n_sub * 4, cudaMemcpyDeviceToHost));
  host_pack(c, r, theta, packed.data(), false);
  return PPU_OK;
}

extern "C" int ppu_get_working_bf16(ppu_ctx* c, uint16_t* w, int64_t n) {
  NEED_CTX(c);
  if (!w || n != c->P) return ppu_fail(PPU_EINVAL, "w null or wrong length");
  CUDA_OK(cudaMemcpyAsync(w, c->w16, n * 2, cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  return PPU_OK;
}
extern "C" int ppu_get_outer_momentum(ppu_ctx* c, float* buf, int64_t n) {
  NEED_CTX(c);
  if (!buf || n != c->P) return ppu_fail(PPU_EINVAL, "buf null or wrong length");
  CUDA_OK(cudaMemcpyAsync(buf, c->buf, n * 4, cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  return PPU_OK;
}
extern "C" int ppu_set_outer_momentum(ppu_ctx* c, const float* buf, int64_t n) {
  NEED_CTX(c);
  if (!buf || n != c->P) return ppu_fail(PPU_EINVAL, "buf null or wrong length");
  CUDA_OK(cudaMemcpyAsync(c->buf, buf, n * 4, cudaMemcpyHostToDevice, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  return PPU_OK;
}

extern "C" int ppu_subset_count(const ppu_ctx* c, int replica, int64_t* n) {
  NEED_CTX(c);
  NEED_REPLICA(c, replica);
  if (!n) return ppu_fail(PPU_EINVAL, "n is null");
  *n = c->reps[replica].n_sub;
  return PPU_OK;
}
extern "C" int ppu_subset_index(const ppu_ctx* c, int replica, int64_t* index, int64_t n) {
  NEED_CTX(c);
  NEED_REPLICA(c, replica);
  const ReplicaState& r = c->reps[replica];
  if (!index || n != r.n_sub) return ppu_fail(PPU_EINVAL, "index null or wrong length");
  const int64_t d = c->cfg.d_model, F = c->cfg.d_ff;
  int64_t j = 0;
  for (const auto& s : r.segs) {
    const int w = s.hi - s.lo;
    for (int64_t i = 0; i < (int64_t)w * d; ++i) index[j++] = s.win_off + (int64_t)s.lo * d + i;
    for (int64_t row = 0; row < d; ++row)
      for (int col = 0; col < w; ++col) index[j++] = s.wout_off + row * F + s.lo + col;
  }
  for (const auto& s : r.dense)
    for (int64_t i = 0; i < s.len; ++i) index[j++] = s.canon_off + i;
  return PPU_OK;
}
extern "C" int ppu_get_subset_grads(ppu_ctx* c, int replica, float* grads, int64_t n) {
  NEED_CTX(c);
  NEED_REPLICA(c, replica);
  if (c->last_stepped != replica) return ppu_fail(PPU_ESTATE, "gradients belong to replica %d", c->last_stepped);
  const ReplicaState& r = c->reps[replica];
  if (!grads || n != r.n_sub) return ppu_fail(PPU_EINVAL, "grads null or wrong length");
  CUDA_OK(cudaStreamSynchronize(c->stream));
  if (r.n_ffn) CUDA_OK(cudaMemcpy(grads, c->grad, r.n_ffn * 4, cudaMemcpyDeviceToHost));
  if (c->last_partials > 1 && r.n_ffn) {   // add the split-K partials in the order the optimizer kernel uses
    std::vector<float> part(r.n_ffn);
    for (int q = 1; q < c->last_partials; ++q) {
      CUDA_OK(cudaMemcpy(part.data(), c->grad + (int64_t)q * c->max_ffn, r.n_ffn * 4, cudaMemcpyDeviceToHost));
      for (int64_t i = 0; i < r.n_ffn; ++i) grads[i] += part[i];
    }
  }
  if (r.n_dense)
    CUDA_OK(cudaMemcpy(grads + r.n_ffn, c->grad + c->max_ffn * c->wgrad_splits, r.n_dense * 4,
                       cudaMemcpyDeviceToHost));
  return PPU_OK;
}
extern "C" int ppu_get_subset_state(ppu_ctx* c, int replica, float* m, float* v, int32_t* step,
                                    int64_t n) {
  NEED_CTX(c);
  NEED_REPLICA(c, replica);
  ReplicaState& r = c->reps[replica];
  if ((m || v) && n != r.n_sub) return ppu_fail(PPU_EINVAL, "wrong length");
  if (m) CUDA_OK(cudaMemcpyAsync(m, r.m, n * 4, cudaMemcpyDeviceToHost, c->stream));
  if (v) CUDA_OK(cudaMemcpyAsync(v, r.v, n * 4, cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  if (step) *step = r.step;
  return PPU_OK;
}
extern "C" int ppu_set_subset_state(ppu_ctx* c, int replica, const float* m, const float* v,
                                    int32_t step, int64_t n) {
  NEED_CTX(c);
  NEED_REPLICA(c, replica);
  ReplicaState& r = c->reps[replica];
  if ((m || v) && n != r.n_sub) return ppu_fail(PPU_EINVAL, "wrong length");
  if (step < 0) return ppu_fail(PPU_EINVAL, "negative step count");
  CUDA_OK(cudaStreamSynchronize(c->stream));
  if (m && n) CUDA_OK(cudaMemcpy(r.m, m, n * 4, cudaMemcpyHostToDevice));
  if (v && n) CUDA_OK(cudaMemcpy(r.v, v, n * 4, cudaMemcpyHostToDevice));
  r.step = step;
  return PPU_OK;
}
extern "C" int ppu_replica_values(ppu_ctx* c, int replica, void** dev_ptr, int64_t* n) {
  NEED_CTX(c);
  NEED_REPLICA(c, replica);
  if (!dev_ptr || !n) return ppu_fail(PPU_EINVAL, "null out pointer");
  *dev_ptr = c->reps[replica].master;
  *n = c->reps[replica].n_sub;
  return PPU_OK;
}
extern "C" int ppu_set_backends(ppu_ctx* c, int gemm, int attention) {
  NEED_CTX(c);
  if (gemm < 0 || gemm > 1 || attention < 0 || attention > 1)
    return ppu_fail(PPU_EINVAL, "backends are 0 (tcgen05) or 1 (SIMT check kernels)");
  c->gemm_backend = gemm;
  c->attn_backend = attention;
  return PPU_OK;
}
extern "C" int ppu_check_guards(ppu_ctx* c, int64_t* n_bad) {
  NEED_CTX(c);
  if (!n_bad) return ppu_fail(PPU_EINVAL, "n_bad is null");
  CUDA_OK(cudaStreamSynchronize(c->stream));
  // the guards are gathered with one strided copy each into a host array, then compared
  std::vector<uint8_t> host(c->guards.size() * PPU_GUARD_BYTES);
  for (size_t i = 0; i < c->guards.size(); ++i)
    CUDA_OK(cudaMemcpyAsync(host.data() + i * PPU_GUARD_BYTES, c->arena + c->guards[i], PPU_GUARD_BYTES,
                            cudaMemcpyDeviceToHost, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));
  int64_t bad = 0; size_t first = 0;
  for (size_t i = 0; i < c->guards.size(); ++i)
    for (int b = 0; b < PPU_GUARD_BYTES; ++b)
      if (host[i * PPU_GUARD_BYTES + b] != PPU_GUARD_BYTE) { if (!bad) first = i; ++bad; break; }
  *n_bad = bad;
  if (bad) return ppu_fail(PPU_ESTATE, "%lld guard blocks overwritten (first: the one after sub-buffer %zu of the arena)",
                           (long long)bad, first);
  return PPU_OK;
}
extern "C" int ppu_set_adam_lr(ppu_ctx* c, float lr) {
  NEED_CTX(c);
  c->adam_lr = lr;
  return PPU_OK;
}
extern "C" int ppu_sync(ppu_ctx* c) {
  NEED_CTX(c);
  CUDA_OK(cudaStreamSynchronize(c->stream));
  CUDA_OK(cudaGetLastError());
  return ppu_check_flags(c);
}
extern "C" int ppu_stats(ppu_ctx* c, ppu_stats_t* out) {
  NEED_CTX(c);
  if (!out) return ppu_fail(PPU_EINVAL, "out is null");
  out->param_count = c->P;
  out->arena_bytes = (int64_t)c->arena_bytes;
  out->state_bytes = (int64_t)c->state_bytes;
  out->activation_bytes = (int64_t)c->act_bytes;
  out->launches_last_step = c->launches_last_step;
  out->launches_last_sync = c->launches_last_sync;
  out->flops_fwd = c->flops_fwd;
  out->flops_dgrad = c->flops_dgrad;
  out->flops_wgrad = c->flops_wgrad;
  out->outer_bytes = c->outer_bytes;
  out->saved_bytes_last_step = c->saved_bytes;
  return PPU_OK;
}

// ---------------------------------------------------------------------------------------
// single-operator entry points
// ---------------------------------------------------------------------------------------
extern "C" int ppu_gemm(const void* A, int64_t lda, int a_kmajor, const void* B, int64_t ldb,
                        int b_kmajor, void* C, int64_t ldc, int out_f32, int M, int N, int K,
                        int backend, void* cuda_stream) {
  if (!A || !B || !C) return ppu_fail(PPU_EINVAL, "null operand");
  if (M < 0 || N < 0 || K < 0) return ppu_fail(PPU_EINVAL, "negative size");
  GemmArgs g;
  g.A = (const bf16*)A; g.lda = lda; g.a_kmajor = a_kmajor;
  g.B = (const bf16*)B; g.ldb = ldb; g.b_kmajor = b_kmajor;
  g.M = M; g.N = N; g.K = K;
  g.epilogue = out_f32 ? EPI_STORE_F32 : EPI_STORE_BF16;
  g.C = C; g.ldc = ldc; g.C2 = nullptr; g.aux = nullptr; g.ldaux = 0; g.flags = nullptr;
  if (backend < 0 || backend > 5) return ppu_fail(PPU_EINVAL, "unknown gemm backend %d", backend);
  g.tile_shape = backend == 2 ? 1 : backend == 3 ? 2 : backend == 4 ? 3 : backend == 5 ? 4 : 0;
  const int rc = backend == 1 ? launch_gemm_simt(g, (cudaStream_t)cuda_stream)
                              : launch_gemm_tc(g, (cudaStream_t)cuda_stream);
  if (rc) return ppu_fail(rc == -4 ? PPU_ESHAPE : PPU_ECUDA, "gemm launch failed (%d)", rc);
  CUDA_OK(cudaGetLastError());
  return PPU_OK;
}

extern "C" int ppu_attention_fwd(const void* qkv, void* U, float* lse, int batch, int seq,
                                 int n_head, int d_head, int backend, void* cuda_stream) {
  if (!qkv || !U || !lse) return ppu_fail(PPU_EINVAL, "null operand");
  if (backend < 0 || backend > 1) return ppu_fail(PPU_EINVAL, "unknown attention backend %d", backend);
  int rc;
  if (backend == 0) {
    if (!attn_tc_supported(seq, d_head)) return ppu_fail(PPU_ESHAPE, "shape not covered by the tensor-core attention");
    rc = launch_attn_fwd_tc((const bf16*)qkv, (bf16*)U, lse, batch, seq, n_head, d_head, nullptr, (cudaStream_t)cuda_stream);
  } else {
    rc = launch_attn_fwd_simt((const bf16*)qkv, (bf16*)U, lse, batch, seq, n_head, d_head, (cudaStream_t)cuda_stream);
  }
  if (rc) return ppu_fail(PPU_ESHAPE, "attention forward launch failed (%d)", rc);
  CUDA_OK(cudaGetLastError());
  return PPU_OK;
}
extern "C" int ppu_attention_bwd(const void* qkv, const void* U, const float* lse, const void* dU,
                                 void* dqkv, float* scratch, int batch, int seq, int n_head,
                                 int d_head, int backend, void* cuda_stream) {
  if (!qkv || !U || !lse || !dU || !dqkv || !scratch) return ppu_fail(PPU_EINVAL, "null operand");
  if (backend < 0 || backend > 1) return ppu_fail(PPU_EINVAL, "unknown attention backend %d", backend);
  int rc;
  if (backend == 0) {
    if (!attn_tc_supported(seq, d_head)) return ppu_fail(PPU_ESHAPE, "shape not covered by the tensor-core attention");
    rc = launch_attn_bwd_tc((const bf16*)qkv, (const bf16*)U, lse, (const bf16*)dU, (bf16*)dqkv, scratch, batch, seq, n_head, d_head, nullptr, (cudaStream_t)cuda_stream);
  } else {
    rc = launch_attn_bwd_simt((const bf16*)qkv, (const bf16*)U, lse, (const bf16*)dU, (bf16*)dqkv, scratch, batch, seq, n_head, d_head, (cudaStream_t)cuda_stream);
  }
  if (rc) return ppu_fail(PPU_ESHAPE, "attention backward launch failed (%d)", rc);
  CUDA_OK(cudaGetLastError());
  return PPU_OK;
}
