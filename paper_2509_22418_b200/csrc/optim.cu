// Optimizer-side kernels: AdamW over a replica's packed subset (Algorithm 1 line 10), moves
// between the packed subset arrays and the canonical vectors, and the outer synchronisation
// sweep (Algorithm 1 lines 12-15).  All are HBM-bound: float4 accesses, grid sized from the
// SM count.
#include "common.cuh"

namespace {

// Canonical index of packed element j (multiple of 4) of a trained block.
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
    float* pg = &g.x; float* pp = &p.x; float* pm = &mm.x; float* pv = &vv.x;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float gi = pg[e];
      const float mi = hp.beta1 * pm[e] + (1.f - hp.beta1) * gi;
      const float vi = hp.beta2 * pv[e] + (1.f - hp.beta2) * gi * gi;
      const float mhat = mi / hp.bc1;
      const float vhat = vi / hp.bc2;
      pp[e] = pp[e] - hp.lr * (mhat / (sqrtf(vhat) + hp.eps) + hp.wd * pp[e]);
      pm[e] = mi;
      pv[e] = vi;
    }
    *reinterpret_cast<float4*>(master + pj) = p;
    *reinterpret_cast<float4*>(m + pj) = mm;
    *reinterpret_cast<float4*>(v + pj) = vv;
    store_bf16x4(w16 + canon_index(s, j, d, F), p);
  }
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

// Outer sweep over the whole canonical vector, one float4 per thread-iteration.
__global__ void __launch_bounds__(256)
outer_kernel(OuterTables t, float* __restrict__ theta, float* __restrict__ buf,
             bf16* __restrict__ w16, float lr, float mu) {
  const int64_t n4 = t.P / 4;
  const int64_t win_end = t.win_rel + (int64_t)t.F * t.d;
  const int64_t wout_end = t.wout_rel + (int64_t)t.F * t.d;
  for (int64_t i4 = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i4 < n4;
       i4 += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = 4 * i4;
    float4 th = *reinterpret_cast<const float4*>(theta + i);
    float4 bu = *reinterpret_cast<const float4*>(buf + i);
    float4 total = make_float4(0.f, 0.f, 0.f, 0.f);
    int count = 0;
    float* slot[8];  // owners' packed positions to restart (at most 8 kept inline)
    int ob = 0, oe = 0;
    int64_t rel = i - t.e_size;
    int layer = -1, unit = 0, which = 0;
    int64_t inner = 0;  // W_in: column; W_out: row
    if (rel >= 0) {
      const int64_t l = rel / t.layer_size;
      if (l < t.L) {
        const int64_t r = rel - l * t.layer_size;
        if (r >= t.win_rel && r < win_end) {
          const int64_t q = r - t.win_rel;
          unit = (int)(q / t.d); inner = q - (int64_t)unit * t.d; which = 1; layer = (int)l;
        } else if (r >= t.wout_rel && r < wout_end) {
          const int64_t q = r - t.wout_rel;
          inner = q / t.F; unit = (int)(q - inner * t.F); which = 2; layer = (int)l;
        }
      }
    }
    if (which) {
      const int64_t grp = (int64_t)layer * (t.F / 8) + unit / 8;
      ob = t.unit_begin[grp];
      oe = t.unit_begin[grp + 1];
    }
    for (int o = ob; o < oe; ++o) {
      const OuterOwner ow = t.owners[t.unit_owner[o]];
      float* p = which == 1
                     ? ow.master + ow.in_off + (int64_t)(unit - ow.lo) * t.d + inner
                     : ow.master + ow.out_off + inner * (ow.hi - ow.lo) + (unit - ow.lo);
      const float4 e = *reinterpret_cast<const float4*>(p);
      total.x += e.x - th.x; total.y += e.y - th.y; total.z += e.z - th.z; total.w += e.w - th.w;
      if (count < 8) slot[count] = p;
      ++count;
    }
    float4 nt;
    {
      const float inv_m = count > 0 ? (float)count : 1.f;
      float* pt = &th.x; float* pb = &bu.x; float* pd = &total.x; float* pn = &nt.x;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float g = -(pd[e] / inv_m);
        const float b = mu * pb[e] + g;
        pn[e] = pt[e] - lr * (g + mu * b);
        pb[e] = b;
      }
    }
    *reinterpret_cast<float4*>(theta + i) = nt;
    *reinterpret_cast<float4*>(buf + i) = bu;
    store_bf16x4(w16 + i, nt);
    for (int c = 0; c < count && c < 8; ++c) *reinterpret_cast<float4*>(slot[c]) = nt;
    if (count > 8) {  // rare: more than 8 replicas share this position
      int c = 0;
      for (int o = ob; o < oe; ++o, ++c) {
        if (c < 8) continue;
        const OuterOwner ow = t.owners[t.unit_owner[o]];
        float* p = which == 1
                       ? ow.master + ow.in_off + (int64_t)(unit - ow.lo) * t.d + inner
                       : ow.master + ow.out_off + inner * (ow.hi - ow.lo) + (unit - ow.lo);
        *reinterpret_cast<float4*>(p) = nt;
      }
    }
  }
}

inline unsigned grid_for(int64_t work_items, int threads, int cap_per_sm) {
  int64_t b = (work_items + threads - 1) / threads;
  const int64_t cap = 148LL * cap_per_sm;
  if (b > cap) b = cap;
  if (b < 1) b = 1;
  return (unsigned)b;
}

}  // namespace

void launch_adamw(const SliceSeg* segs, int n_seg, float* master, float* m, float* v,
                  const float* grad, int n_partials, int64_t grad_stride, bf16* w16, int d, int F,
                  int64_t n_total, AdamHyper hp, cudaStream_t st) {
  if (n_seg == 0) return;
  const int64_t per_seg = (n_total / n_seg + 3) / 4;
  dim3 grid(grid_for(per_seg, 256, 8), n_seg);
  // keep the total near a few waves of the 148 SMs
  while ((int64_t)grid.x * grid.y > 148LL * 16 && grid.x > 1) grid.x = (grid.x + 1) / 2;
  adamw_kernel<<<grid, 256, 0, st>>>(segs, master, m, v, grad, n_partials, grad_stride, w16, d, F,
                                     hp);
}

static void slice_move(const SliceSeg* segs, int n_seg, float* packed, float* dense, bf16* w16,
                       int d, int F, int64_t n_total, int mode, cudaStream_t st) {
  if (n_seg == 0) return;
  const int64_t per_seg = (n_total / n_seg + 3) / 4;
  dim3 grid(grid_for(per_seg, 256, 8), n_seg);
  while ((int64_t)grid.x * grid.y > 148LL * 16 && grid.x > 1) grid.x = (grid.x + 1) / 2;
  slice_move_kernel<<<grid, 256, 0, st>>>(segs, packed, dense, w16, d, F, mode);
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
void launch_slices_scatter_f32(const SliceSeg* segs, int n_seg, const float* packed, float* dense,
                               int d, int F, int64_t n_total, cudaStream_t st) {
  slice_move(segs, n_seg, const_cast<float*>(packed), dense, nullptr, d, F, n_total, 3, st);
}

void launch_outer(const OuterTables& t, float* theta, float* buf, bf16* w16, float lr, float mu,
                  cudaStream_t st) {
  outer_kernel<<<grid_for(t.P / 4, 256, 8), 256, 0, st>>>(t, theta, buf, w16, lr, mu);
}
