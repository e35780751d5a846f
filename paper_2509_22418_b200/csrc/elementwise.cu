// Bandwidth-bound kernels of the local step: embedding gather, LayerNorm forward and
// input-gradient backward, rotary positions, fused cross-entropy, loss reduction.
// All accesses are 16-byte vectors on rows that are multiples of 8 elements.
#include "common.cuh"

namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Block-wide sum with a fixed combination order (deterministic).
template <int NW>
__device__ __forceinline__ float block_sum(float v, float* red) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int i = 0; i < NW; ++i) t += red[i];
  return t;
}
template <int NW>
__device__ __forceinline__ float block_max(float v, float* red) {
  v = warp_max(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float t = red[0];
#pragma unroll
  for (int i = 1; i < NW; ++i) t = fmaxf(t, red[i]);
  return t;
}

__device__ __forceinline__ void unpack8(const uint4& u, float* f) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 t = __bfloat1622float2(p[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}
__device__ __forceinline__ uint4 pack8(const float* f) {
  uint4 u;
  __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  return u;
}

// ---- embedding gather: x[t,:] = E[tok[t],:] (bf16 working copy -> fp32 stream) ----
__global__ void embed_kernel(const int32_t* __restrict__ tok, const bf16* __restrict__ E,
                             float* __restrict__ x, int T, int d, int V, int* flags) {
  const int t = blockIdx.x;
  int id = tok[t];
  if (id < 0 || id >= V) {
    if (threadIdx.x == 0) atomicExch(flags + PPU_FLAG_TOKEN, 1);
    id = id < 0 ? 0 : V - 1;
  }
  const uint4* src = reinterpret_cast<const uint4*>(E + (int64_t)id * d);
  float4* dst = reinterpret_cast<float4*>(x + (int64_t)t * d);
  for (int i = threadIdx.x; i < d / 8; i += blockDim.x) {
    float f[8];
    unpack8(src[i], f);
    dst[2 * i] = make_float4(f[0], f[1], f[2], f[3]);
    dst[2 * i + 1] = make_float4(f[4], f[5], f[6], f[7]);
  }
}

// ---- LayerNorm forward: one block per row, row staged in shared memory ----
constexpr int LN_THREADS = 256;
__global__ void __launch_bounds__(LN_THREADS)
ln_fwd_kernel(const float* __restrict__ x, const float* __restrict__ g, const float* __restrict__ b,
              bf16* __restrict__ y, float2* __restrict__ stats, int d, float eps) {
  extern __shared__ float row[];
  __shared__ float red[LN_THREADS / 32];
  const int64_t t = blockIdx.x;
  const float4* src = reinterpret_cast<const float4*>(x + t * d);
  float s = 0.f;
  for (int i = threadIdx.x; i < d / 4; i += LN_THREADS) {
    float4 v = src[i];
    reinterpret_cast<float4*>(row)[i] = v;
    s += (v.x + v.y) + (v.z + v.w);
  }
  const float mean = block_sum<LN_THREADS / 32>(s, red) / d;
  float q = 0.f;
  for (int i = threadIdx.x; i < d / 4; i += LN_THREADS) {
    float4 v = reinterpret_cast<float4*>(row)[i];
    float a = v.x - mean, bb = v.y - mean, c = v.z - mean, e = v.w - mean;
    q += (a * a + bb * bb) + (c * c + e * e);
  }
  const float var = block_sum<LN_THREADS / 32>(q, red) / d;
  const float rstd = rsqrtf(var + eps);
  if (threadIdx.x == 0) stats[t] = make_float2(mean, rstd);
  uint4* dst = reinterpret_cast<uint4*>(y + t * d);
  for (int i = threadIdx.x; i < d / 8; i += LN_THREADS) {
    float f[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int c = 8 * i + j;
      f[j] = (row[c] - mean) * rstd * g[c] + b[c];
    }
    dst[i] = pack8(f);
  }
}

// ---- LayerNorm backward, input gradient only (gamma/beta are frozen) ----
// gout = gin + rstd * (dy*gamma - mean(dy*gamma) - xhat * mean(dy*gamma*xhat))
__global__ void __launch_bounds__(LN_THREADS)
ln_bwd_kernel(const bf16* __restrict__ dy, const float* __restrict__ x,
              const float2* __restrict__ stats, const float* __restrict__ gamma,
              const float* gin, float* gout, bf16* __restrict__ gout16, int d) {
  extern __shared__ float sm[];
  float* dyg = sm;
  float* xh = sm + d;
  __shared__ float red[LN_THREADS / 32];
  const int64_t t = blockIdx.x;
  const float2 st = stats[t];
  const uint4* dsrc = reinterpret_cast<const uint4*>(dy + t * d);
  const float4* xsrc = reinterpret_cast<const float4*>(x + t * d);
  float s1 = 0.f, s2 = 0.f;
  for (int i = threadIdx.x; i < d / 8; i += LN_THREADS) {
    float f[8];
    unpack8(dsrc[i], f);
    float4 xa = xsrc[2 * i], xb = xsrc[2 * i + 1];
    float xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int c = 8 * i + j;
      const float a = f[j] * gamma[c];
      const float h = (xv[j] - st.x) * st.y;
      dyg[c] = a;
      xh[c] = h;
      s1 += a;
      s2 += a * h;
    }
  }
  const float m1 = block_sum<LN_THREADS / 32>(s1, red) / d;
  const float m2 = block_sum<LN_THREADS / 32>(s2, red) / d;
  const float4* gsrc = gin ? reinterpret_cast<const float4*>(gin + t * d) : nullptr;
  float4* gdst = reinterpret_cast<float4*>(gout + t * d);
  uint4* g16 = reinterpret_cast<uint4*>(gout16 + t * d);
  for (int i = threadIdx.x; i < d / 8; i += LN_THREADS) {
    float f[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int c = 8 * i + j;
      f[j] = st.y * (dyg[c] - m1 - xh[c] * m2);
    }
    if (gsrc) {
      float4 a = gsrc[2 * i], bq = gsrc[2 * i + 1];
      f[0] += a.x; f[1] += a.y; f[2] += a.z; f[3] += a.w;
      f[4] += bq.x; f[5] += bq.y; f[6] += bq.z; f[7] += bq.w;
    }
    gdst[2 * i] = make_float4(f[0], f[1], f[2], f[3]);
    gdst[2 * i + 1] = make_float4(f[4], f[5], f[6], f[7]);
    g16[i] = pack8(f);
  }
}

// ---- warp-per-row LayerNorm (d a multiple of 256): the row lives in registers, lane l owns
// the 8-element chunks l, l+32, ...; no shared memory, no block barrier ----
template <int NV>
__global__ void __launch_bounds__(128)
ln_fwd_warp_kernel(const float* __restrict__ x, const float* __restrict__ g,
                   const float* __restrict__ b, bf16* __restrict__ y, float2* __restrict__ stats,
                   int T, float eps) {
  constexpr int d = NV * 256;
  const int64_t t = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (t >= T) return;
  const float4* src = reinterpret_cast<const float4*>(x + t * d);
  float v[NV][8];
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = lane + 32 * i;
    const float4 a = src[2 * c], bq = src[2 * c + 1];
    v[i][0] = a.x; v[i][1] = a.y; v[i][2] = a.z; v[i][3] = a.w;
    v[i][4] = bq.x; v[i][5] = bq.y; v[i][6] = bq.z; v[i][7] = bq.w;
#pragma unroll
    for (int j = 0; j < 8; ++j) s += v[i][j];
  }
  // gain and bias are fetched before the reductions, so that their latency overlaps them
  float4 gq[NV][2], bq2[NV][2];
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = lane + 32 * i;
    gq[i][0] = reinterpret_cast<const float4*>(g)[2 * c]; gq[i][1] = reinterpret_cast<const float4*>(g)[2 * c + 1];
    bq2[i][0] = reinterpret_cast<const float4*>(b)[2 * c]; bq2[i][1] = reinterpret_cast<const float4*>(b)[2 * c + 1];
  }
  const float mean = warp_sum(s) * (1.f / d);
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) { const float e = v[i][j] - mean; q += e * e; }
  const float rstd = rsqrtf(warp_sum(q) * (1.f / d) + eps);
  if (lane == 0) stats[t] = make_float2(mean, rstd);
  uint4* dst = reinterpret_cast<uint4*>(y + t * d);
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = lane + 32 * i;
    const float gg[8] = {gq[i][0].x, gq[i][0].y, gq[i][0].z, gq[i][0].w, gq[i][1].x, gq[i][1].y, gq[i][1].z, gq[i][1].w};
    const float bb[8] = {bq2[i][0].x, bq2[i][0].y, bq2[i][0].z, bq2[i][0].w, bq2[i][1].x, bq2[i][1].y, bq2[i][1].z, bq2[i][1].w};
    float f[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) f[j] = (v[i][j] - mean) * rstd * gg[j] + bb[j];
    dst[c] = pack8(f);
  }
}

template <int NV>
__global__ void __launch_bounds__(128)
ln_bwd_warp_kernel(const bf16* __restrict__ dy, const float* __restrict__ x,
                   const float2* __restrict__ stats, const float* __restrict__ gamma,
                   const float* gin, float* gout, bf16* __restrict__ gout16, int T) {
  constexpr int d = NV * 256;
  const int64_t t = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (t >= T) return;
  const float2 st = stats[t];
  const uint4* dsrc = reinterpret_cast<const uint4*>(dy + t * d);
  const float4* xsrc = reinterpret_cast<const float4*>(x + t * d);
  float a[NV][8], hh[NV][8];
  float s1 = 0.f, s2 = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = lane + 32 * i;
    float f[8];
    unpack8(dsrc[c], f);
    const float4 xa = xsrc[2 * c], xb = xsrc[2 * c + 1];
    const float4 g0 = reinterpret_cast<const float4*>(gamma)[2 * c], g1 = reinterpret_cast<const float4*>(gamma)[2 * c + 1];
    const float xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
    const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      a[i][j] = f[j] * gg[j];
      hh[i][j] = (xv[j] - st.x) * st.y;
      s1 += a[i][j];
      s2 += a[i][j] * hh[i][j];
    }
  }
  // the incoming gradient is fetched before the reductions, so that its latency overlaps them
  const float4* gsrc = gin ? reinterpret_cast<const float4*>(gin + t * d) : nullptr;
  float4 pin[NV][2];
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = lane + 32 * i;
    if (gsrc) { pin[i][0] = gsrc[2 * c]; pin[i][1] = gsrc[2 * c + 1]; }
    else { pin[i][0] = pin[i][1] = make_float4(0.f, 0.f, 0.f, 0.f); }
  }
  const float m1 = warp_sum(s1) * (1.f / d), m2 = warp_sum(s2) * (1.f / d);
  float4* gdst = reinterpret_cast<float4*>(gout + t * d);
  uint4* g16 = reinterpret_cast<uint4*>(gout16 + t * d);
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = lane + 32 * i;
    float f[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) f[j] = st.y * (a[i][j] - m1 - hh[i][j] * m2);
    f[0] += pin[i][0].x; f[1] += pin[i][0].y; f[2] += pin[i][0].z; f[3] += pin[i][0].w;
    f[4] += pin[i][1].x; f[5] += pin[i][1].y; f[6] += pin[i][1].z; f[7] += pin[i][1].w;
    gdst[2 * c] = make_float4(f[0], f[1], f[2], f[3]);
    gdst[2 * c + 1] = make_float4(f[4], f[5], f[6], f[7]);
    g16[c] = pack8(f);
  }
}

// ---- rotary positions on the q and k parts of qkv[T,3d], in place ----
// cs: [S, dh/2] (cos, sin) pairs computed on the host in double precision.
__global__ void rope_kernel(bf16* __restrict__ qkv, const float2* __restrict__ cs, int S, int d,
                            int dh, int64_t n_vec, int inverse) {
  // one thread per 8 consecutive elements (4 pairs) of q or k
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= n_vec) return;
  const int per_row = 2 * d / 8;
  const int64_t t = i / per_row;
  const int c = (int)(i % per_row) * 8;       // column in [0, 2d)
  const int pos = (int)(t % S);
  const int pair0 = (c % dh) / 2;
  uint4* p = reinterpret_cast<uint4*>(qkv + t * (int64_t)(3 * d) + c);
  float f[8];
  unpack8(*p, f);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    float2 w = cs[(int64_t)pos * (dh / 2) + pair0 + j];
    if (inverse) w.y = -w.y;
    const float a = f[2 * j], b = f[2 * j + 1];
    f[2 * j] = a * w.x - b * w.y;
    f[2 * j + 1] = a * w.y + b * w.x;
  }
  *p = pack8(f);
}

// ---- fused cross-entropy: a persistent block per SM walks token rows, row held in registers ----
// Reads the logits once; writes dlogits = (softmax - onehot) / count in place.  The next row's
// loads are issued before the current row's reductions and exponentials, so that they (and the
// current row's stores) overlap the arithmetic instead of following it.
constexpr int XE_THREADS = 1024;
template <int NCH>
__global__ void __launch_bounds__(XE_THREADS, 1)
xent_kernel(bf16* __restrict__ logits, const int32_t* __restrict__ tok,
            float* __restrict__ row_loss, int T, int S, int V, float inv_count, int write_grad) {
  __shared__ float red[XE_THREADS / 32];
  const int nvec = V / 8;
  uint4 nxt[NCH];
  auto load_row = [&](int64_t row) {
    const uint4* rp = reinterpret_cast<const uint4*>(logits + row * V);
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int i = threadIdx.x + c * XE_THREADS;
      if (i < nvec) nxt[c] = rp[i];
    }
  };
  int64_t t = blockIdx.x;
  if (t < T) load_row(t);
  for (; t < T; t += gridDim.x) {
    const int s = (int)(t % S);
    uint4* rowp = reinterpret_cast<uint4*>(logits + t * V);
    float v[NCH][8];
    float mx = -INFINITY;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int i = threadIdx.x + c * XE_THREADS;
      if (i < nvec) {
        unpack8(nxt[c], v[c]);
#pragma unroll
        for (int j = 0; j < 8; ++j) mx = fmaxf(mx, v[c][j]);
      }
    }
    if (t + gridDim.x < T) load_row(t + gridDim.x);
    if (s == S - 1) {  // no next token: no loss, zero gradient (block-uniform)
      if (write_grad)
        for (int i = threadIdx.x; i < nvec; i += XE_THREADS) rowp[i] = make_uint4(0, 0, 0, 0);
      if (threadIdx.x == 0) row_loss[t] = 0.f;
      continue;
    }
    int target = tok[t + 1];
    target = target < 0 ? 0 : (target >= V ? V - 1 : target);
    // the thread that holds the target logit takes it from its registers
    const int oc = (target >> 3) / XE_THREADS, oj = target & 7;
    const bool owner = (target >> 3) % XE_THREADS == (int)threadIdx.x;
    float zt = 0.f;
    if (owner) {
#pragma unroll
      for (int c = 0; c < NCH; ++c)
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (c == oc && j == oj) zt = v[c][j];
    }
    mx = block_max<XE_THREADS / 32>(mx, red);
    float sum = 0.f;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int i = threadIdx.x + c * XE_THREADS;
      if (i < nvec) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          v[c][j] = __expf(v[c][j] - mx);
          sum += v[c][j];
        }
      }
    }
    sum = block_sum<XE_THREADS / 32>(sum, red);
    const float inv = 1.f / sum;
    if (owner) row_loss[t] = logf(sum) + mx - zt;
    if (!write_grad) continue;
    const float scale = inv * inv_count;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int i = threadIdx.x + c * XE_THREADS;
      if (i < nvec) {
        float f[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) f[j] = v[c][j] * scale;
        if (owner && c == oc) {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (j == oj) f[j] = (v[c][j] * inv - 1.f) * inv_count;
        }
        rowp[i] = pack8(f);
      }
    }
  }
}

__global__ void __launch_bounds__(1024)
loss_reduce_kernel(const float* __restrict__ row_loss, int T, float inv_count, float* out) {
  __shared__ float red[32];
  float s = 0.f;
  for (int i = threadIdx.x; i < T; i += 1024) s += row_loss[i];
  s = block_sum<32>(s, red);
  if (threadIdx.x == 0) *out = s * inv_count;
}

__global__ void cast_bf16_kernel(const float* __restrict__ src, bf16* __restrict__ dst, int64_t n8) {
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n8;
       i += (int64_t)gridDim.x * blockDim.x) {
    float4 a = reinterpret_cast<const float4*>(src)[2 * i];
    float4 b = reinterpret_cast<const float4*>(src)[2 * i + 1];
    float f[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    reinterpret_cast<uint4*>(dst)[i] = pack8(f);
  }
}

// ---- gradient of the embedding rows a batch touches -----------------------------------------
// dE[id, :] += sum over the positions t with tok[t] == id, in ascending t, of g[t, :].  One warp
// per position: the warp of an id's first occurrence gathers all of them (ids are compared after
// the same clamping the forward gather applies), every other warp leaves at once - so each row
// of dE has one writer and a fixed summation order.
__global__ void __launch_bounds__(256)
embed_grad_kernel(const int32_t* __restrict__ tok, const float* __restrict__ g, float* __restrict__ dE,
                  int T, int d, int V) {
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (t >= T) return;
  auto clampv = [V](int id) { return id < 0 ? 0 : (id >= V ? V - 1 : id); };
  const int id = clampv(tok[t]);
  bool seen = false;
  for (int j = lane; j < t && !seen; j += 32) seen = clampv(tok[j]) == id;
  if (__any_sync(0xffffffffu, seen)) return;
  float* row = dE + (int64_t)id * d;
  for (int c0 = 0; c0 < d; c0 += 512) {          // 512 columns at a time: four float4 per lane
    float4 acc[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c = c0 + 4 * (lane + 32 * i);
      acc[i] = c < d ? *reinterpret_cast<const float4*>(row + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int j0 = t & ~31; j0 < T; j0 += 32) {
      const int j = j0 + lane;
      const bool hit = j >= t && j < T && clampv(tok[j]) == id;
      unsigned mask = __ballot_sync(0xffffffffu, hit);
      while (mask) {
        const int src = j0 + __ffs(mask) - 1;
        mask &= mask - 1;
        const float* gr = g + (int64_t)src * d;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = c0 + 4 * (lane + 32 * i);
          if (c < d) {
            const float4 v = *reinterpret_cast<const float4*>(gr + c);
            acc[i].x += v.x; acc[i].y += v.y; acc[i].z += v.z; acc[i].w += v.w;
          }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c = c0 + 4 * (lane + 32 * i);
      if (c < d) *reinterpret_cast<float4*>(row + c) = acc[i];
    }
  }
}

constexpr int LNP_ROWS = 16;
// ---- LayerNorm gain / shift gradients: column sums over the tokens, two stages -------------
// stage 1: block b sums rows [16 b, 16 b + 16) for every column -> partial[b][0][c] (dy * xhat),
// partial[b][1][c] (dy); stage 2: a block takes 32 columns, each of its 32 warps adds a 32nd of
// the partials in order of b, and the 32 sums are added in order - a fixed order throughout.
__global__ void __launch_bounds__(256)
ln_param_partial_kernel(const bf16* __restrict__ dy, const float* __restrict__ x,
                        const float2* __restrict__ stats, float* __restrict__ partial, int T, int d) {
  const int r0 = blockIdx.x * LNP_ROWS;
  const int r1 = r0 + LNP_ROWS < T ? r0 + LNP_ROWS : T;
  float* pg = partial + (int64_t)blockIdx.x * 2 * d;
  float* pb = pg + d;
  for (int c = 8 * threadIdx.x; c < d; c += 8 * 256) {
    float sg[8] = {}, sb[8] = {};
#pragma unroll 4
    for (int t = r0; t < r1; ++t) {
      const float2 st = stats[t];
      float f[8];
      unpack8(*reinterpret_cast<const uint4*>(dy + (int64_t)t * d + c), f);
      const float4 xa = *reinterpret_cast<const float4*>(x + (int64_t)t * d + c);
      const float4 xb = *reinterpret_cast<const float4*>(x + (int64_t)t * d + c + 4);
      const float xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        sg[j] += f[j] * ((xv[j] - st.x) * st.y);
        sb[j] += f[j];
      }
    }
    *reinterpret_cast<float4*>(pg + c) = make_float4(sg[0], sg[1], sg[2], sg[3]);
    *reinterpret_cast<float4*>(pg + c + 4) = make_float4(sg[4], sg[5], sg[6], sg[7]);
    *reinterpret_cast<float4*>(pb + c) = make_float4(sb[0], sb[1], sb[2], sb[3]);
    *reinterpret_cast<float4*>(pb + c + 4) = make_float4(sb[4], sb[5], sb[6], sb[7]);
  }
}
__global__ void __launch_bounds__(1024)
ln_param_final_kernel(const float* __restrict__ partial, float* __restrict__ dgamma,
                      float* __restrict__ dbeta, int n_blocks, int d) {
  __shared__ float sh[2][32][32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + lane;
  const int per = (n_blocks + 31) / 32;
  const int b0 = w * per, b1 = b0 + per < n_blocks ? b0 + per : n_blocks;
  float sg = 0.f, sb = 0.f;
  if (c < d) {
#pragma unroll 8
    for (int b = b0; b < b1; ++b) {
      sg += partial[(int64_t)b * 2 * d + c];
      sb += partial[(int64_t)b * 2 * d + d + c];
    }
  }
  sh[0][w][lane] = sg; sh[1][w][lane] = sb;
  __syncthreads();
  if (w == 0 && c < d) {
    float tg = 0.f, tb = 0.f;
#pragma unroll
    for (int q = 0; q < 32; ++q) { tg += sh[0][q][lane]; tb += sh[1][q][lane]; }
    dgamma[c] = tg;
    dbeta[c] = tb;
  }
}

}  // namespace

int ppu_current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= PPU_MAX_DEVICES) dev = 0;
  return dev;
}

int ppu_sm_count() {
  static int n_sm[PPU_MAX_DEVICES] = {};
  const int dev = ppu_current_device();
  if (n_sm[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 1;
    n_sm[dev] = n;
  }
  return n_sm[dev];
}

void launch_embed_grad(const int32_t* tok, const float* g, float* dE, int T, int d, int V,
                       cudaStream_t st) {
  embed_grad_kernel<<<(unsigned)((T + 7) / 8), 256, 0, st>>>(tok, g, dE, T, d, V);
}

int ln_param_partial_blocks(int T) { return (T + LNP_ROWS - 1) / LNP_ROWS; }

void launch_ln_param_grad(const bf16* dy, const float* x, const float2* stats, float* dgamma,
                          float* dbeta, float* partial, int T, int d, cudaStream_t st) {
  const int nb = ln_param_partial_blocks(T);
  ln_param_partial_kernel<<<nb, 256, 0, st>>>(dy, x, stats, partial, T, d);
  ln_param_final_kernel<<<(d + 31) / 32, 1024, 0, st>>>(partial, dgamma, dbeta, nb, d);
}

void launch_embed(const int32_t* tok, const bf16* E16, float* x, int T, int d, int V, int* flags,
                  cudaStream_t st) {
  embed_kernel<<<T, 128, 0, st>>>(tok, E16, x, T, d, V, flags);
}

void launch_ln_fwd(const float* x, const float* g, const float* b, bf16* y, float2* stats, int T,
                   int d, float eps, cudaStream_t st) {
  const unsigned wb = (unsigned)((T + 3) / 4);
  switch (d % 256 == 0 ? d / 256 : 0) {
#define LNF(NV) case NV: ln_fwd_warp_kernel<NV><<<wb, 128, 0, st>>>(x, g, b, y, stats, T, eps); return;
    LNF(1) LNF(2) LNF(3) LNF(4) LNF(6) LNF(8) LNF(12) LNF(16)
#undef LNF
    default: break;
  }
  ln_fwd_kernel<<<T, LN_THREADS, d * sizeof(float), st>>>(x, g, b, y, stats, d, eps);
}

void launch_ln_bwd(const bf16* dy, const float* x, const float2* stats, const float* gamma,
                   const float* gin, float* gout, bf16* gout16, int T, int d, cudaStream_t st) {
  const unsigned wb = (unsigned)((T + 3) / 4);
  switch (d % 256 == 0 ? d / 256 : 0) {
#define LNB(NV) case NV: ln_bwd_warp_kernel<NV><<<wb, 128, 0, st>>>(dy, x, stats, gamma, gin, gout, gout16, T); return;
    LNB(1) LNB(2) LNB(3) LNB(4) LNB(6) LNB(8) LNB(12) LNB(16)
#undef LNB
    default: break;
  }
  ln_bwd_kernel<<<T, LN_THREADS, 2 * d * sizeof(float), st>>>(dy, x, stats, gamma, gin, gout,
                                                              gout16, d);
}

void launch_rope(bf16* qkv, const float2* cs, int B, int S, int h, int dh, int inverse,
                 cudaStream_t st) {
  const int d = h * dh;
  const int64_t n_vec = (int64_t)B * S * (2 * d / 8);
  const int threads = 256;
  rope_kernel<<<(unsigned)((n_vec + threads - 1) / threads), threads, 0, st>>>(
      qkv, cs, S, d, dh, n_vec, inverse);
}

void launch_xent(bf16* logits, const int32_t* tok, float* row_loss, int B, int S, int V,
                 int write_grad, cudaStream_t st) {
  const int T = B * S;
  const float inv_count = 1.f / (float)((int64_t)B * (S - 1));
  const int nch = (V / 8 + XE_THREADS - 1) / XE_THREADS;
  const int grid = T < ppu_sm_count() ? T : ppu_sm_count();
  if (nch <= 1)
    xent_kernel<1><<<grid, XE_THREADS, 0, st>>>(logits, tok, row_loss, T, S, V, inv_count, write_grad);
  else if (nch <= 2)
    xent_kernel<2><<<grid, XE_THREADS, 0, st>>>(logits, tok, row_loss, T, S, V, inv_count, write_grad);
  else if (nch <= 4)
    xent_kernel<4><<<grid, XE_THREADS, 0, st>>>(logits, tok, row_loss, T, S, V, inv_count, write_grad);
  else
    xent_kernel<8><<<grid, XE_THREADS, 0, st>>>(logits, tok, row_loss, T, S, V, inv_count, write_grad);
}

void launch_loss_reduce(const float* row_loss, int T, float inv_count, float* out, cudaStream_t st) {
  loss_reduce_kernel<<<1, 1024, 0, st>>>(row_loss, T, inv_count, out);
}

void launch_cast_bf16(const float* src, bf16* dst, int64_t n, cudaStream_t st) {
  const int64_t n8 = n / 8;
  const int threads = 256;
  int64_t blocks = (n8 + threads - 1) / threads;
  if (blocks > (int64_t)ppu_sm_count() * 16) blocks = (int64_t)ppu_sm_count() * 16;
  if (blocks < 1) blocks = 1;
  cast_bf16_kernel<<<(unsigned)blocks, threads, 0, st>>>(src, dst, n8);
}
