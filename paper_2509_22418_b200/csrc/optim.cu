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

// Outer sweep (Algorithm 1 lines 12-15).  blockIdx.y selects a segment of the canonical
// vector - a quarter of E, a layer's non-FFN block, its W_in, its W_out, or the final
// LayerNorm - so that the position decoding is block-uniform; within a segment every thread
// keeps four independent float4 streams in flight.
constexpr int OUTER_U = 4;

__device__ __forceinline__ void outer_update(float4& th, float4& bu, const float4& total, int count,
                                             float lr, float mu) {
  const float m = count > 0 ? (float)count : 1.f;
  float* pt = &th.x; float* pb = &bu.x; const float* pd = &total.x;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float g = -(pd[e] / m);
    const float b = mu * pb[e] + g;
    pt[e] = pt[e] - lr * (g + mu * b);
    pb[e] = b;
  }
}

__global__ void __launch_bounds__(256)
outer_kernel(OuterTables t, float* __restrict__ theta, float* __restrict__ buf,
             bf16* __restrict__ w16, float lr, float mu, int seg_lo) {
  // ---- segment decoding (uniform per block) ----
  const int seg = seg_lo + blockIdx.y;
  int64_t start; int64_t len; int kind = 0, layer = 0;
  const int64_t fd = (int64_t)t.F * t.d;
  if (seg < 4) {
    const int64_t q = ((t.e_size / 4 + 3) / 4) * 4;          // quarter of E, whole float4s
    start = seg * q;
    len = seg < 3 ? q : t.e_size - 3 * q;
    if (len < 0) len = 0;
    if (start > t.e_size) { start = t.e_size; len = 0; }
  } else if (seg == 4 + 3 * t.L) {
    start = t.e_size + (int64_t)t.L * t.layer_size;
    len = t.P - start;
  } else {
    layer = (seg - 4) / 3;
    const int w = (seg - 4) - 3 * layer;
    const int64_t base = t.e_size + (int64_t)layer * t.layer_size;
    if (w == 0) { start = base; len = t.win_rel; }
    else if (w == 1) { start = base + t.win_rel; len = fd; kind = 1; }
    else { start = base + t.wout_rel; len = fd; kind = 2; }
  }
  const uint32_t n4 = (uint32_t)(len / 4);
  const uint32_t stride = gridDim.x * blockDim.x;
  float* th_p = theta + start;
  float* bu_p = buf + start;
  bf16* w_p = w16 + start;
  const int32_t* ub = t.unit_begin + (int64_t)layer * (t.F / 8);

  for (uint32_t e0 = blockIdx.x * blockDim.x + threadIdx.x; e0 < n4; e0 += OUTER_U * stride) {
    float4 th[OUTER_U], bu[OUTER_U];
#pragma unroll
    for (int k = 0; k < OUTER_U; ++k) {
      const uint32_t e = e0 + k * stride;
      if (e < n4) {
        th[k] = reinterpret_cast<const float4*>(th_p)[e];
        bu[k] = reinterpret_cast<const float4*>(bu_p)[e];
      }
    }
#pragma unroll
    for (int k = 0; k < OUTER_U; ++k) {
      const uint32_t e = e0 + k * stride;
      if (e >= n4) break;
      float4 total = make_float4(0.f, 0.f, 0.f, 0.f);
      int count = 0, ob = 0, oe = 0;
      uint32_t unit = 0, inner = 0;
      if (kind == 1) { unit = (4u * e) / (uint32_t)t.d; inner = 4u * e - unit * (uint32_t)t.d; }
      else if (kind == 2) { inner = (4u * e) / (uint32_t)t.F; unit = 4u * e - inner * (uint32_t)t.F; }
      if (kind) { ob = ub[unit >> 3]; oe = ub[(unit >> 3) + 1]; }
      const float4 old = th[k];
      for (int o = ob; o < oe; ++o) {
        const OuterOwner ow = t.owners[t.unit_owner[o]];
        const float* p = kind == 1
                             ? ow.master + ow.in_off + (int64_t)((int)unit - ow.lo) * t.d + inner
                             : ow.master + ow.out_off + (int64_t)inner * (ow.hi - ow.lo) + ((int)unit - ow.lo);
        const float4 v = *reinterpret_cast<const float4*>(p);
        total.x += v.x - old.x; total.y += v.y - old.y; total.z += v.z - old.z; total.w += v.w - old.w;
        ++count;
      }
      outer_update(th[k], bu[k], total, count, lr, mu);
      reinterpret_cast<float4*>(th_p)[e] = th[k];
      reinterpret_cast<float4*>(bu_p)[e] = bu[k];
      store_bf16x4(w_p + 4 * (int64_t)e, th[k]);
      for (int o = ob; o < oe; ++o) {       // the owners restart from the new parameters
        const OuterOwner ow = t.owners[t.unit_owner[o]];
        float* p = kind == 1
                       ? ow.master + ow.in_off + (int64_t)((int)unit - ow.lo) * t.d + inner
                       : ow.master + ow.out_off + (int64_t)inner * (ow.hi - ow.lo) + ((int)unit - ow.lo);
        *reinterpret_cast<float4*>(p) = th[k];
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
                  int seg_lo, int seg_count, cudaStream_t st) {
  if (seg_count <= 0) return;
  // 4 segments for E, 3 per layer, 1 for the final LayerNorm
  // enough blocks for about four waves of three resident blocks per SM, never fewer than 32 per
  // segment (a streaming-sync group has few segments)
  int gx = (4 * 3 * 148 + seg_count - 1) / seg_count;
  gx = gx < 32 ? 32 : (gx > 256 ? 256 : gx);
  dim3 grid(gx, seg_count);
  outer_kernel<<<grid, 256, 0, st>>>(t, theta, buf, w16, lr, mu, seg_lo);
}
