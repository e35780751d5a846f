// Plain SIMT causal attention (one thread per query or key row, online softmax).  Serves the
// head sizes the tensor-core kernels do not cover and as an in-library cross-check.
// Appendix C.1: S = q k^T / sqrt(d_h), A = softmax_row(S) under the causal mask, U = A v, and
// the backward dV = A^T dU, dA = dU v^T, dS = A * (dA - rowsum(dA * A)), dq = dS k, dk = dS^T q.
#include "common.cuh"

namespace {

constexpr int ROWS = 128;  // rows per block
constexpr int KT = 16;     // rows of the other operand staged per iteration

template <int DH>
__global__ void __launch_bounds__(ROWS)
attn_fwd_simt_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ U, float* __restrict__ lse,
                     int S, int h) {
  __shared__ float Ks[KT][DH];
  __shared__ float Vs[KT][DH];
  const int d = h * DH;
  const int head = blockIdx.y, b = blockIdx.z;
  const int s0 = blockIdx.x * ROWS;
  const int s = s0 + threadIdx.x;
  const bool live = s < S;
  const float scale = rsqrtf((float)DH);
  const bf16* base = qkv + (int64_t)b * S * 3 * d + head * DH;
  float q[DH], acc[DH];
#pragma unroll
  for (int e = 0; e < DH; ++e) {
    q[e] = live ? __bfloat162float(base[(int64_t)s * 3 * d + e]) * scale : 0.f;
    acc[e] = 0.f;
  }
  float mx = -INFINITY, l = 0.f;
  const int t_end = min(S, s0 + ROWS);
  for (int t0 = 0; t0 < t_end; t0 += KT) {
    __syncthreads();
    for (int i = threadIdx.x; i < KT * DH; i += ROWS) {
      const int tt = i / DH, e = i % DH;
      const int t = t0 + tt;
      Ks[tt][e] = t < S ? __bfloat162float(base[(int64_t)t * 3 * d + d + e]) : 0.f;
      Vs[tt][e] = t < S ? __bfloat162float(base[(int64_t)t * 3 * d + 2 * d + e]) : 0.f;
    }
    __syncthreads();
    if (!live) continue;
    for (int tt = 0; tt < KT; ++tt) {
      const int t = t0 + tt;
      if (t > s) break;
      float sc = 0.f;
#pragma unroll
      for (int e = 0; e < DH; ++e) sc += q[e] * Ks[tt][e];
      const float nm = fmaxf(mx, sc);
      const float corr = __expf(mx - nm);
      const float p = __expf(sc - nm);
      l = l * corr + p;
#pragma unroll
      for (int e = 0; e < DH; ++e) acc[e] = acc[e] * corr + p * Vs[tt][e];
      mx = nm;
    }
  }
  if (!live) return;
  const float inv = 1.f / l;
  bf16* out = U + ((int64_t)b * S + s) * d + head * DH;
#pragma unroll
  for (int e = 0; e < DH; ++e) out[e] = __float2bfloat16_rn(acc[e] * inv);
  lse[((int64_t)b * h + head) * S + s] = mx + logf(l);
}

// dq and delta = rowsum(dU * U) per query row
template <int DH>
__global__ void __launch_bounds__(ROWS)
attn_bwd_dq_simt_kernel(const bf16* __restrict__ qkv, const bf16* __restrict__ U,
                        const float* __restrict__ lse, const bf16* __restrict__ dU,
                        bf16* __restrict__ dqkv, float* __restrict__ delta, int S, int h) {
  __shared__ float Ks[KT][DH];
  __shared__ float Vs[KT][DH];
  const int d = h * DH;
  const int head = blockIdx.y, b = blockIdx.z;
  const int s0 = blockIdx.x * ROWS;
  const int s = s0 + threadIdx.x;
  const bool live = s < S;
  const float scale = rsqrtf((float)DH);
  const bf16* base = qkv + (int64_t)b * S * 3 * d + head * DH;
  float q[DH], go[DH], dq[DH];
  float dl = 0.f, ls = 0.f;
  if (live) {
    const bf16* up = U + ((int64_t)b * S + s) * d + head * DH;
    const bf16* gp = dU + ((int64_t)b * S + s) * d + head * DH;
#pragma unroll
    for (int e = 0; e < DH; ++e) {
      q[e] = __bfloat162float(base[(int64_t)s * 3 * d + e]) * scale;
      go[e] = __bfloat162float(gp[e]);
      dl += go[e] * __bfloat162float(up[e]);
      dq[e] = 0.f;
    }
    ls = lse[((int64_t)b * h + head) * S + s];
    delta[((int64_t)b * h + head) * S + s] = dl;
  }
  const int t_end = min(S, s0 + ROWS);
  for (int t0 = 0; t0 < t_end; t0 += KT) {
    __syncthreads();
    for (int i = threadIdx.x; i < KT * DH; i += ROWS) {
      const int tt = i / DH, e = i % DH;
      const int t = t0 + tt;
      Ks[tt][e] = t < S ? __bfloat162float(base[(int64_t)t * 3 * d + d + e]) : 0.f;
      Vs[tt][e] = t < S ? __bfloat162float(base[(int64_t)t * 3 * d + 2 * d + e]) : 0.f;
    }
    __syncthreads();
    if (!live) continue;
    for (int tt = 0; tt < KT; ++tt) {
      const int t = t0 + tt;
      if (t > s) break;
      float sc = 0.f, dp = 0.f;
#pragma unroll
      for (int e = 0; e < DH; ++e) { sc += q[e] * Ks[tt][e]; dp += go[e] * Vs[tt][e]; }
      const float p = __expf(sc - ls);
      const float ds = p * (dp - dl) * scale;
#pragma unroll
      for (int e = 0; e < DH; ++e) dq[e] += ds * Ks[tt][e];
    }
  }
  if (!live) return;
  bf16* out = dqkv + ((int64_t)b * S + s) * 3 * d + head * DH;
#pragma unroll
  for (int e = 0; e < DH; ++e) out[e] = __float2bfloat16_rn(dq[e]);
}

// dk and dv per key row
template <int DH>
__global__ void __launch_bounds__(ROWS)
attn_bwd_dkv_simt_kernel(const bf16* __restrict__ qkv, const float* __restrict__ lse,
                         const bf16* __restrict__ dU, bf16* __restrict__ dqkv,
                         const float* __restrict__ delta, int S, int h) {
  __shared__ float Qs[KT][DH];
  __shared__ float Gs[KT][DH];
  __shared__ float Ls[KT], Ds[KT];
  const int d = h * DH;
  const int head = blockIdx.y, b = blockIdx.z;
  const int t0 = blockIdx.x * ROWS;
  const int t = t0 + threadIdx.x;
  const bool live = t < S;
  const float scale = rsqrtf((float)DH);
  const bf16* base = qkv + (int64_t)b * S * 3 * d + head * DH;
  float k[DH], v[DH], dk[DH], dv[DH];
#pragma unroll
  for (int e = 0; e < DH; ++e) {
    k[e] = live ? __bfloat162float(base[(int64_t)t * 3 * d + d + e]) : 0.f;
    v[e] = live ? __bfloat162float(base[(int64_t)t * 3 * d + 2 * d + e]) : 0.f;
    dk[e] = 0.f;
    dv[e] = 0.f;
  }
  for (int s0 = t0; s0 < S; s0 += KT) {
    __syncthreads();
    for (int i = threadIdx.x; i < KT * DH; i += ROWS) {
      const int ss = i / DH, e = i % DH;
      const int s = s0 + ss;
      Qs[ss][e] = s < S ? __bfloat162float(base[(int64_t)s * 3 * d + e]) * scale : 0.f;
      Gs[ss][e] = s < S ? __bfloat162float(dU[((int64_t)b * S + s) * d + head * DH + e]) : 0.f;
    }
    if (threadIdx.x < KT) {
      const int s = s0 + threadIdx.x;
      Ls[threadIdx.x] = s < S ? lse[((int64_t)b * h + head) * S + s] : 0.f;
      Ds[threadIdx.x] = s < S ? delta[((int64_t)b * h + head) * S + s] : 0.f;
    }
    __syncthreads();
    if (!live) continue;
    for (int ss = 0; ss < KT; ++ss) {
      const int s = s0 + ss;
      if (s >= S) break;
      if (s < t) continue;
      float sc = 0.f, dp = 0.f;
#pragma unroll
      for (int e = 0; e < DH; ++e) { sc += Qs[ss][e] * k[e]; dp += Gs[ss][e] * v[e]; }
      const float p = __expf(sc - Ls[ss]);
      const float ds = p * (dp - Ds[ss]);   // Qs already carries the 1/sqrt(d_h)
#pragma unroll
      for (int e = 0; e < DH; ++e) { dv[e] += p * Gs[ss][e]; dk[e] += ds * Qs[ss][e]; }
    }
  }
  if (!live) return;
  bf16* out = dqkv + ((int64_t)b * S + t) * 3 * d + head * DH;
#pragma unroll
  for (int e = 0; e < DH; ++e) {
    out[d + e] = __float2bfloat16_rn(dk[e]);
    out[2 * d + e] = __float2bfloat16_rn(dv[e]);
  }
}

}  // namespace

#define DISPATCH_DH(dh, CALL)                 \
  switch (dh) {                               \
    case 16: { constexpr int DH = 16; CALL; } break;   \
    case 32: { constexpr int DH = 32; CALL; } break;   \
    case 64: { constexpr int DH = 64; CALL; } break;   \
    case 128: { constexpr int DH = 128; CALL; } break; \
    default: return -1;                       \
  }

int launch_attn_fwd_simt(const bf16* qkv, bf16* U, float* lse, int B, int S, int h, int dh,
                         cudaStream_t st) {
  dim3 grid((S + ROWS - 1) / ROWS, h, B);
  DISPATCH_DH(dh, (attn_fwd_simt_kernel<DH><<<grid, ROWS, 0, st>>>(qkv, U, lse, S, h)));
  return 0;
}

int launch_attn_bwd_simt(const bf16* qkv, const bf16* U, const float* lse, const bf16* dU,
                         bf16* dqkv, float* scratch, int B, int S, int h, int dh, cudaStream_t st) {
  dim3 grid((S + ROWS - 1) / ROWS, h, B);
  DISPATCH_DH(dh, (attn_bwd_dq_simt_kernel<DH><<<grid, ROWS, 0, st>>>(qkv, U, lse, dU, dqkv,
                                                                      scratch, S, h)));
  DISPATCH_DH(dh, (attn_bwd_dkv_simt_kernel<DH><<<grid, ROWS, 0, st>>>(qkv, lse, dU, dqkv, scratch,
                                                                       S, h)));
  return 0;
}
