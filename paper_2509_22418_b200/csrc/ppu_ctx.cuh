// Host-side context of the ppu library: validated configuration, per-replica subset tables
// and the carve-up of the caller's device arena.
#pragma once
#include <string>
#include <vector>
#include "../../include/ppu.h"
#include "common.cuh"

// guard block after every sub-buffer of the arena
constexpr int PPU_GUARD_BYTES = 256;
constexpr int PPU_GUARD_BYTE = 0xA5;

struct TensorRec { std::string name; int64_t offset; int ndim; int64_t shape[2]; };

struct ReplicaState {
  std::vector<int32_t> lo, hi;     // per layer trained hidden-unit range (lo == hi: none)
  std::vector<SliceSeg> segs;      // one per trained layer, ascending layer
  std::vector<int> seg_layer;      // layer of segs[i]
  int h_lo = 0, h_hi = 0;          // heads whose W_q / W_k / W_v rows are trained (h_lo == h_hi: none)
  bool rest = false;               // trains E, W_o and every LayerNorm too
  std::vector<DenseSeg> dense;     // trained runs outside the FFNs, in canonical order
  int64_t n_ffn = 0;               // packed elements of the FFN blocks (they come first)
  int64_t n_dense = 0;             // packed elements of the dense runs
  int64_t n_sub = 0;               // |I_k^train| = n_ffn + n_dense
  int lowest = -1;                 // lowest layer the backward pass reaches (-1: trains nothing)
  int step = 0;                    // AdamW step count
  bool stepped = false;
  float *master = nullptr, *m = nullptr, *v = nullptr;  // device, packed
  SliceSeg* d_segs = nullptr;      // device copy of segs
  DenseSeg* d_dense = nullptr;     // device copy of dense
  bool deep() const { return rest || h_hi > h_lo; }
  // packed offset of the dense run that starts at canonical offset `off` (-1: not trained)
  int64_t packed_of(int64_t off) const {
    for (const auto& s : dense) if (s.canon_off == off) return s.packed_off;
    return -1;
  }
};

struct LayerActs {
  float* x;        // block input (LayerNorm-1 input), fp32 [T,d]
  float* x1;       // after the attention residual (LayerNorm-2 input), fp32 [T,d]
  float2 *st1, *st2;
  bf16* qkv;       // rotated q,k and v, [T,3d]
  bf16* U;         // attention output before W_o, [T,d]
  float* lse;      // [B,h,S]
  bf16* b;         // LayerNorm-2 output (input of W_in), [T,d]
  bf16* Hd;        // FFN pre-activation, [T,F] (null for layers no replica's backward reaches)
  bf16* As;        // gelu(Hd) restricted to the widest trained slice of this layer, packed [T,w]
};

struct ppu_ctx {
  ppu_model_cfg cfg;
  int K = 0;
  cudaStream_t stream = nullptr;
  int gemm_backend = 0;   // 0 tcgen05, 1 SIMT
  int attn_backend = 0;   // 0 tensor-core tiles when the shape allows, 1 SIMT
  // canonical geometry
  int64_t P = 0, e_size = 0, layer_size = 0;
  int64_t rel_ln1g, rel_ln1b, rel_wq, rel_wo, rel_ln2g, rel_ln2b, rel_win, rel_wout;
  int64_t off_lnfg, off_lnfb;
  std::vector<TensorRec> tensors;
  std::vector<ReplicaState> reps;
  int64_t max_ffn = 0;    // largest n_ffn over the replicas, padded: stride of the split-K partials
  int64_t max_dense = 0;  // largest n_dense
  int min_lowest = 0;     // lowest layer any replica's backward pass reaches
  bool any_rest = false;
  int wgrad_splits = 1;   // split-K factor of the subset weight-gradient products
  int last_partials = 1;  // partial gradient buffers written by the most recent step
  int resident = -1;      // replica whose subset is overlaid on the bf16 working copy
  int last_stepped = -1;
  float adam_lr;
  // arena
  uint8_t* arena = nullptr;
  size_t arena_bytes = 0, state_bytes = 0, act_bytes = 0;
  std::vector<size_t> guards;   // arena offsets of the guard blocks
  float *theta = nullptr, *buf = nullptr;
  bf16* w16 = nullptr;
  float* grad = nullptr;        // [wgrad_splits][max_ffn] partials of the FFN blocks, then [max_dense]
  std::vector<LayerActs> acts;
  float* x_last = nullptr;      // input of the final LayerNorm
  float2* stf = nullptr;
  bf16 *a16 = nullptr, *f16 = nullptr, *logits = nullptr;
  bf16* A_tmp = nullptr;        // gelu(Hd) of the layer in flight, [T,F] (only its trained slice is kept)
  std::vector<int> wmax;        // per layer: widest trained range over the replicas
  float* g = nullptr;
  bf16 *g16 = nullptr, *dHd = nullptr, *t16 = nullptr, *dqkv = nullptr;
  float *attn_scratch = nullptr, *row_loss = nullptr, *loss = nullptr;
  float* ln_partial = nullptr;  // scratch of the LayerNorm gain / shift gradients
  int* flags = nullptr;
  float2* rope_cs = nullptr;
  int32_t* tok_stage = nullptr;
  // outer-sync tables (device) and their host mirror
  OuterSeg* d_oseg = nullptr; OuterChunk* d_ochunk = nullptr; DenseOwner* d_downer = nullptr;
  int32_t* d_unit_begin = nullptr; OuterOwner* d_unit_owner = nullptr;
  size_t cap_oseg = 0, cap_ochunk = 0, cap_downer = 0, cap_uowner = 0;
  std::vector<OuterSeg> h_oseg;
  // per segment kind: where its chunk list starts in the device array, and inside that list the
  // index where layer l's chunks begin ([L]: final norm, [L + 1]: end; E's chunks precede layer 0)
  int kind_chunk_base[3] = {0, 0, 0};
  std::vector<int> layer_chunk_begin[3];
  int n_chunks = 0;
  std::vector<int32_t> cached_sync_list;
  // per-class event timing
  bool profiling = false;
  std::vector<cudaEvent_t> ev_pool;           // pairs: [2i] start, [2i+1] stop
  struct EvRec { int cls; double work; };
  std::vector<EvRec> ev_recs;
  int64_t ev_dropped = 0;
  // stats
  int64_t launches = 0, launches_last_step = 0, launches_last_sync = 0;
  double flops_fwd = 0, flops_dgrad = 0, flops_wgrad = 0, outer_bytes = 0;
  int64_t saved_bytes = 0;
};

// Brackets one launch with events when profiling is on (ppu_step.cu).
struct EvScope {
  ppu_ctx* c; int slot = -1;
  EvScope(ppu_ctx* ctx, int cls, double work);
  ~EvScope();
};
