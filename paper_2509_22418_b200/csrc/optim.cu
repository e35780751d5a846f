// Optimizer-side kernels: AdamW over a replica's packed subset (Algorithm 1, the inner update), moves
// between the packed subset arrays and the canonical vectors, and the outer synchronisation
// sweep (Algorithm 1, the outer step).  All are HBM-bound: float4 accesses, grids sized from the
// SM count of the current device.
#include "common.cuh"

namespace {

// Canonical index of packed element j (multiple of 4) of a trained FFN block.
__device__ __forceinline__ int64_t canon_index(const SliceSeg& s, int64_t j, int d, int F) {
  const int w = s.hi - s.lo;
  const int64_t n_in = (int64_t)w * d;
  if (j < n_in) return s.win_off + (int64_t)s.lo * d + j;
  const int64_t j2 = j - n_in;
  const int64_t r = j2 / w;
  const int c = (int)(j2 - r * w);
  return s.wout_off + r * F + s.lo + c;
}

__device__ __forceinline__ void store_bf16x4(bf16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}

// One AdamW step (bias-corrected, decoupled decay on the value before the step) on four elements.
__device__ __forceinline__ void adamw4(float4& p, float4& mm, float4& vv, const float4& g,
                                       const AdamHyper& hp, float wd) {
  float* pp = &p.x; float* pm = &mm.x; float* pv = &vv.x; const float* pg = &g.x;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float gi = pg[e];
    const float mi = hp.beta1 * pm[e] + (1.f - hp.beta1) * gi;
    const float vi = hp.beta2 * pv[e] + (1.f - hp.beta2) * gi * gi;
    const float mhat = mi / hp.bc1;
    const float vhat = vi / hp.bc2;
    pp[e] = pp[e] - hp.lr * (mhat / (sqrtf(vhat) + hp.eps) + wd * pp[e]);
    pm[e] = mi;
    pv[e] = vi;
  }
}

__global__ void __launch_bounds__(256)
adamw_kernel(const SliceSeg* __restrict__ segs, float* __restrict__ master, float* __restrict__ m,
             float* __restrict__ v, const float* __restrict__ grad, int n_partials,
             int64_t grad_stride, bf16* __restrict__ w16, int d, int F, AdamHyper hp) {
  const SliceSeg s = segs[blockIdx.y];
  const int64_t n = 2 * (int64_t)(s.hi - s.lo) * d;
  for (int64_t j = 4 * (blockIdx.x * (int64_t)blockDim.x + threadIdx.x); j < n;
       j += 4 * (int64_t)gridDim.x * blockDim.x) {
    const int64_t pj = s.packed_off + j;
    float4 g = *reinterpret_cast<const float4*>(grad + pj);
    for (int q = 1; q < n_partials; ++q) {
      float4 h = *reinterpret_cast<const float4*>(grad + q * grad_stride + pj);
      g.x += h.x; g.y += h.y; g.z += h.z; g.w += h.w;
    }
    float4 p = *reinterpret_cast<float4*>(master + pj);
    float4 mm = *reinterpret_cast<float4*>(m + pj);
    float4 vv = *reinterpret_cast<float4*>(v + pj);
    adamw4(p, mm, vv, g, hp, hp.wd);
    *reinterpret_cast<float4*>(master + pj) = p;
    *reinterpret_cast<float4*>(m + pj) = mm;
    *reinterpret_cast<float4*>(v + pj) = vv;
    store_bf16x4(w16 + canon_index(s, j, d, F), p);
  }
}

// The dense runs of a replica are contiguous in its packed arrays (positions [base, base + n)) but
// of very different lengths (a LayerNorm vector, the embedding), so the kernels that walk them
// cut the packed range into equal chunks instead of giving every run the same number of blocks:
// a block finds the run its chunk starts in by bisection and steps to the next run where a
// float4 lies past the current one's end.  f(run, offset inside the run, packed position).
constexpr int64_t DENSE_CHUNK = 16384;
template <class F>
__device__ __forceinline__ void dense_walk(const DenseSeg* __restrict__ segs, int n_seg, int64_t base,
                                           int64_t n, F f) {
  for (int64_t p0 = base + blockIdx.x * DENSE_CHUNK; p0 < base + n; p0 += (int64_t)gridDim.x * DENSE_CHUNK) {
    const int64_t p1 = p0 + DENSE_CHUNK < base + n ? p0 + DENSE_CHUNK : base + n;
    int lo = 0, hi = n_seg - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (segs[mid].packed_off <= p0) lo = mid; else hi = mid - 1;
    }
    int si = lo;
    DenseSeg s = segs[si];
    for (int64_t p = p0 + 4 * threadIdx.x; p < p1; p += 4 * blockDim.x) {
      while (p >= s.packed_off + s.len) s = segs[++si];
      f(s, p - s.packed_off, p);
    }
  }
}

__global__ void __launch_bounds__(256)
adamw_dense_kernel(const DenseSeg* __restrict__ segs, int n_seg, int64_t base, int64_t n,
                   float* __restrict__ master, float* __restrict__ m, float* __restrict__ v,
                   const float* __restrict__ grad, int64_t grad_shift, bf16* __restrict__ w16, AdamHyper hp) {
  dense_walk(segs, n_seg, base, n, [&](const DenseSeg& s, int64_t j, int64_t pj) {
    const float4 g = *reinterpret_cast<const float4*>(grad + (pj - grad_shift));
    float4 p = *reinterpret_cast<float4*>(master + pj);
    float4 mm = *reinterpret_cast<float4*>(m + pj);
    float4 vv = *reinterpret_cast<float4*>(v + pj);
    adamw4(p, mm, vv, g, hp, s.decay ? hp.wd : 0.f);
    *reinterpret_cast<float4*>(master + pj) = p;
    *reinterpret_cast<float4*>(m + pj) = mm;
    *reinterpret_cast<float4*>(v + pj) = vv;
    store_bf16x4(w16 + s.canon_off + j, p);
  });
}

// mode 0: packed = theta[subset]; 1: w16[subset] = bf16(packed); 2: w16[subset] = bf16(theta);
// 3: dense[subset] = packed
__global__ void __launch_bounds__(256)
slice_move_kernel(const SliceSeg* __restrict__ segs, float* packed, float* dense, bf16* w16, int d,
                  int F, int mode) {
  const SliceSeg s = segs[blockIdx.y];
  const int64_t n = 2 * (int64_t)(s.hi - s.lo) * d;
  for (int64_t j = 4 * (blockIdx.x * (int64_t)blockDim.x + threadIdx.x); j < n;
       j += 4 * (int64_t)gridDim.x * blockDim.x) {
    const int64_t ci = canon_index(s, j, d, F);
    const int64_t pj = s.packed_off + j;
    if (mode == 0) {
      *reinterpret_cast<float4*>(packed + pj) = *reinterpret_cast<const float4*>(dense + ci);
    } else if (mode == 1) {
      store_bf16x4(w16 + ci, *reinterpret_cast<const float4*>(packed + pj));
    } else if (mode == 2) {
      store_bf16x4(w16 + ci, *reinterpret_cast<const float4*>(dense + ci));
    } else {
      *reinterpret_cast<float4*>(dense + ci) = *reinterpret_cast<const float4*>(packed + pj);
    }
  }
}

__global__ void __launch_bounds__(256)
dense_move_kernel(const DenseSeg* __restrict__ segs, int n_seg, int64_t base, int64_t n, float* packed,
                  const float* theta, bf16* w16, int mode) {
  dense_walk(segs, n_seg, base, n, [&](const DenseSeg& s, int64_t j, int64_t pj) {
    const int64_t ci = s.canon_off + j;
    if (mode == 0) *reinterpret_cast<float4*>(packed + pj) = *reinterpret_cast<const float4*>(theta + ci);
    else if (mode == 1) store_bf16x4(w16 + ci, *reinterpret_cast<const float4*>(packed + pj));
    else store_bf16x4(w16 + ci, *reinterpret_cast<const float4*>(theta + ci));
  });
}

// ---------------------------------------------------------------------------------------------
// Outer sweep (Algorithm 1, the outer step): Delta = sum over owners (theta_k - theta) / m, 0 where
// m = 0; g = -Delta; buf = mu buf + g; theta -= lr (g + mu buf); the bf16 copy is refreshed and
// every owner restarts from the new value.
//
// A persistent grid walks a list of chunks (OUTER_CHUNK elements of one segment each), so the
// decoding of "which tensor, which owners" is uniform per block and chunk, and segments of any
// length share the machine evenly.  Per chunk a thread handles OUTER_U float4 at a time, all
// loads of theta and buf issued before the owner lookups.
// ---------------------------------------------------------------------------------------------
constexpr int OUTER_U = 4;
constexpr int OUTER_THREADS = 256;

__device__ __forceinline__ void outer_update(float4& th, float4& bu, const float4& total, int count,
                                             float lr, float mu) {
  // (a division by m = 1 or by the stand-in for m = 0 changes nothing and is skipped: the sweep
  // runs at the power-capped SM clock and is sensitive to its instruction count)
  float* pt = &th.x; float* pb = &bu.x; const float* pd = &total.x;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float g = count > 1 ? -(pd[e] / (float)count) : -pd[e];
    const float b = mu * pb[e] + g;
    pt[e] = pt[e] - lr * (g + mu * b);
    pb[e] = b;
  }
}

// n / divisor for n < 2^31 with the divisor's precomputed multiplier and shift
__device__ __forceinline__ uint32_t fast_div(uint32_t n, FastDiv f) {
  return (uint32_t)(((uint64_t)n * f.mul) >> 32) >> f.shift;
}

template <int KIND>
__device__ __forceinline__ void outer_chunk(const OuterTables& t, const OuterSeg& sg, int64_t off,
                                            float* __restrict__ theta, float* __restrict__ buf,
                                            bf16* __restrict__ w16, float lr, float mu) {
  const int64_t left = sg.len - off;
  const uint32_t n4 = (uint32_t)((left < OUTER_CHUNK ? left : OUTER_CHUNK) / 4);
  float* th_p = theta + sg.start + off;
  float* bu_p = buf + sg.start + off;
  bf16* w_p = w16 + sg.start + off;
  // element index of the chunk's first float inside its matrix (kind 2)
  const uint32_t rel0 = KIND ? (uint32_t)(sg.start + off - sg.base) : 0u;
  // kind 0: the common owner counts are none and one; the single owner's record is read once
  const int n_own = KIND == 0 ? sg.oe - sg.ob : 0;
  DenseOwner own0{nullptr, 0};
  if (KIND == 0 && n_own == 1) own0 = t.dense_owner[sg.ob];
  const int32_t* ub = KIND ? t.unit_begin + (int64_t)sg.layer * (t.F / 8) : nullptr;
  for (uint32_t e0 = threadIdx.x; e0 < n4; e0 += OUTER_U * OUTER_THREADS) {
    float4 th[OUTER_U], bu[OUTER_U];
#pragma unroll
    for (int k = 0; k < OUTER_U; ++k) {
      const uint32_t e = e0 + k * OUTER_THREADS;
      if (e < n4) {
        th[k] = __ldcs(reinterpret_cast<const float4*>(th_p) + e);
        bu[k] = __ldcs(reinterpret_cast<const float4*>(bu_p) + e);
      }
    }
#pragma unroll
    for (int k = 0; k < OUTER_U; ++k) {
      const uint32_t e = e0 + k * OUTER_THREADS;
      if (e >= n4) break;
      float4 total = make_float4(0.f, 0.f, 0.f, 0.f);
      int count = 0;
      const float4 old = th[k];
      if (KIND == 0) {
        const int64_t ci = sg.start + off + 4 * (int64_t)e;
        if (n_own == 1) {
          const float4 v = __ldcs(reinterpret_cast<const float4*>(own0.master + ci + own0.shift));
          total.x = v.x - old.x; total.y = v.y - old.y; total.z = v.z - old.z; total.w = v.w - old.w;
          count = 1;
        } else {
          for (int o = sg.ob; o < sg.oe; ++o) {
            const DenseOwner ow = t.dense_owner[o];
            const float4 v = __ldcs(reinterpret_cast<const float4*>(ow.master + ci + ow.shift));
            total.x += v.x - old.x; total.y += v.y - old.y; total.z += v.z - old.z; total.w += v.w - old.w;
            ++count;
          }
        }
        outer_update(th[k], bu[k], total, count, lr, mu);
        __stcs(reinterpret_cast<float4*>(th_p) + e, th[k]);
        __stcs(reinterpret_cast<float4*>(bu_p) + e, bu[k]);
        store_bf16x4(w_p + 4 * (int64_t)e, th[k]);
        // the owners restart from the new parameters
        if (n_own == 1) {
          *reinterpret_cast<float4*>(own0.master + ci + own0.shift) = th[k];
        } else {
          for (int o = sg.ob; o < sg.oe; ++o) {
            const DenseOwner ow = t.dense_owner[o];
            *reinterpret_cast<float4*>(ow.master + ci + ow.shift) = th[k];
          }
        }
      } else {
        const uint32_t rel = rel0 + 4u * e;
        const uint32_t inner = fast_div(rel, t.div_F), unit = rel - inner * (uint32_t)t.F;
        const int ob = ub[unit >> 3], oe = ub[(unit >> 3) + 1];
        for (int o = ob; o < oe; ++o) {
          const OuterOwner ow = t.unit_owner[o];
          const float* p = ow.master + ow.out_off + (int64_t)inner * (ow.hi - ow.lo) + ((int)unit - ow.lo);
          const float4 v = __ldcs(reinterpret_cast<const float4*>(p));
          total.x += v.x - old.x; total.y += v.y - old.y; total.z += v.z - old.z; total.w += v.w - old.w;
          ++count;
        }
        outer_update(th[k], bu[k], total, count, lr, mu);
        __stcs(reinterpret_cast<float4*>(th_p) + e, th[k]);
        __stcs(reinterpret_cast<float4*>(bu_p) + e, bu[k]);
        store_bf16x4(w_p + 4 * (int64_t)e, th[k]);
        for (int o = ob; o < oe; ++o) {
          const OuterOwner ow = t.unit_owner[o];
          float* p = ow.master + ow.out_off + (int64_t)inner * (ow.hi - ow.lo) + ((int)unit - ow.lo);
          *reinterpret_cast<float4*>(p) = th[k];
        }
      }
    }
  }
}

// One kernel per segment kind (no kind branches inside, three resident blocks per SM); each walks
// its own chunk list.
template <int KIND>
__global__ void __launch_bounds__(OUTER_THREADS, 3)
outer_kernel(OuterTables t, const OuterChunk* __restrict__ chunks, float* __restrict__ theta,
             float* __restrict__ buf, bf16* __restrict__ w16, float lr, float mu, int n_chunks) {
  for (int c = blockIdx.x; c < n_chunks; c += gridDim.x) {
    const OuterChunk ch = chunks[c];
    const OuterSeg sg = t.segs[ch.seg];
    outer_chunk<KIND>(t, sg, ch.off, theta, buf, w16, lr, mu);
  }
}

// blocks for `work_items` threads' worth of work, at most cap_per_sm per SM
inline unsigned grid_for(int64_t work_items, int threads, int cap_per_sm) {
  int64_t b = (work_items + threads - 1) / threads;
  const int64_t cap = (int64_t)ppu_sm_count() * cap_per_sm;
  if (b > cap) b = cap;
  if (b < 1) b = 1;
  return (unsigned)b;
}

// grid (x, n_seg) with about 16 blocks per SM in total
inline dim3 seg_grid(int64_t n_total, int n_seg) {
  const int64_t per_seg = (n_total / n_seg + 3) / 4;
  dim3 grid(grid_for(per_seg, 256, 8), n_seg);
  while ((int64_t)grid.x * grid.y > (int64_t)ppu_sm_count() * 16 && grid.x > 1) grid.x = (grid.x + 1) / 2;
  return grid;
}

}  // namespace

void launch_adamw(const SliceSeg* segs, int n_seg, float* master, float* m, float* v,
                  const float* grad, int n_partials, int64_t grad_stride, bf16* w16, int d, int F,
                  int64_t n_total, AdamHyper hp, cudaStream_t st) {
  if (n_seg == 0) return;
  adamw_kernel<<<seg_grid(n_total, n_seg), 256, 0, st>>>(segs, master, m, v, grad, n_partials,
                                                         grad_stride, w16, d, F, hp);
}

static unsigned dense_grid(int64_t n) {
  const int64_t chunks = (n + DENSE_CHUNK - 1) / DENSE_CHUNK, cap = (int64_t)ppu_sm_count() * 8;
  return (unsigned)(chunks < cap ? chunks : cap);
}

void launch_adamw_dense(const DenseSeg* segs, int n_seg, float* master, float* m, float* v,
                        const float* grad, int64_t grad_shift, bf16* w16, int64_t packed_base,
                        int64_t n_total, AdamHyper hp, cudaStream_t st) {
  if (n_seg == 0 || n_total <= 0) return;
  adamw_dense_kernel<<<dense_grid(n_total), 256, 0, st>>>(segs, n_seg, packed_base, n_total, master, m, v,
                                                          grad, grad_shift, w16, hp);
}

static void slice_move(const SliceSeg* segs, int n_seg, float* packed, float* dense, bf16* w16,
                       int d, int F, int64_t n_total, int mode, cudaStream_t st) {
  if (n_seg == 0) return;
  slice_move_kernel<<<seg_grid(n_total, n_seg), 256, 0, st>>>(segs, packed, dense, w16, d, F, mode);
}

void launch_slices_gather(const SliceSeg* segs, int n_seg, const float* theta, float* packed,
                          int d, int F, int64_t n_total, cudaStream_t st) {
  slice_move(segs, n_seg, packed, const_cast<float*>(theta), nullptr, d, F, n_total, 0, st);
}
void launch_slices_to_w16(const SliceSeg* segs, int n_seg, const float* packed, const float* theta,
                          bf16* w16, int from_packed, int d, int F, int64_t n_total,
                          cudaStream_t st) {
  slice_move(segs, n_seg, const_cast<float*>(packed), const_cast<float*>(theta), w16, d, F,
             n_total, from_packed ? 1 : 2, st);
}

void launch_dense_move(const DenseSeg* segs, int n_seg, float* packed, const float* theta, bf16* w16,
                       int mode, int64_t packed_base, int64_t n_total, cudaStream_t st) {
  if (n_seg == 0 || n_total <= 0) return;
  dense_move_kernel<<<dense_grid(n_total), 256, 0, st>>>(segs, n_seg, packed_base, n_total, packed, theta,
                                                         w16, mode);
}

void launch_outer(const OuterTables& t, int kind, float* theta, float* buf, bf16* w16, float lr, float mu,
                  int chunk_lo, int n_chunks, cudaStream_t st) {
  if (n_chunks <= 0) return;
  // three resident blocks per SM; a chunk gives every thread 16 float4 per array
  int grid = ppu_sm_count() * 3;
  if (grid > n_chunks) grid = n_chunks;
  const OuterChunk* ch = t.chunks + chunk_lo;
  if (kind == 0) outer_kernel<0><<<grid, OUTER_THREADS, 0, st>>>(t, ch, theta, buf, w16, lr, mu, n_chunks);
  else if (kind == 2) outer_kernel<2><<<grid, OUTER_THREADS, 0, st>>>(t, ch, theta, buf, w16, lr, mu, n_chunks);
}
