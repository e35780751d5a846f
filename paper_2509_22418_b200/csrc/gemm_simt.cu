// Plain SIMT GEMM with the same operand conventions and epilogues as the tcgen05 kernel.
// It exists as an in-library cross-check (selected explicitly) and is not tuned.
#include "common.cuh"

namespace {

__device__ __forceinline__ float gelu_f(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  return 0.5f * x * (1.f + tanhf(u));
}
__device__ __forceinline__ float gelu_grad_f(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  const float t = tanhf(u);
  const float du = 0.7978845608028654f * (1.f + 3.f * 0.044715f * x * x);
  return 0.5f * (1.f + t) + 0.5f * x * (1.f - t * t) * du;
}

constexpr int TS = 64, TK = 16;

__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs g) {
  __shared__ float As[TK][TS + 1];
  __shared__ float Bs[TK][TS + 1];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const int m0 = blockIdx.y * TS, n0 = blockIdx.x * TS;
  const int64_t sam = g.a_kmajor ? g.lda : 1, sak = g.a_kmajor ? 1 : g.lda;
  const int64_t sbn = g.b_kmajor ? g.ldb : 1, sbk = g.b_kmajor ? 1 : g.ldb;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < g.K; k0 += TK) {
    for (int i = threadIdx.x; i < TS * TK; i += 256) {
      int mm, kk;
      if (g.a_kmajor) { kk = i % TK; mm = i / TK; } else { mm = i % TS; kk = i / TS; }
      const int m = m0 + mm, ka = k0 + kk;
      As[kk][mm] = (m < g.M && ka < g.K) ? __bfloat162float(g.A[m * sam + ka * sak]) : 0.f;
      int nn;
      if (g.b_kmajor) { kk = i % TK; nn = i / TK; } else { nn = i % TS; kk = i / TS; }
      const int n = n0 + nn, kb = k0 + kk;
      Bs[kk][nn] = (n < g.N && kb < g.K) ? __bfloat162float(g.B[n * sbn + kb * sbk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] += a[i] * b[j];
    }
    __syncthreads();
  }
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= g.M) continue;
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= g.N) continue;
      const float a = acc[i][j];
      const int64_t ci = (int64_t)m * g.ldc + n;
      switch (g.epilogue) {
        case EPI_STORE_BF16: ((bf16*)g.C)[ci] = __float2bfloat16_rn(a); break;
        case EPI_STORE_F32: ((float*)g.C)[ci] = a; break;
        case EPI_GELU_DUAL:
          if (g.C) ((bf16*)g.C)[ci] = __float2bfloat16_rn(a);
          ((bf16*)g.C2)[ci] = __float2bfloat16_rn(gelu_f(a));
          if (g.C3 && n >= g.c3_lo && n < g.c3_hi)
            ((bf16*)g.C3)[(int64_t)m * g.ldc3 + (n - g.c3_lo)] = __float2bfloat16_rn(gelu_f(a));
          break;
        case EPI_RESID_F32:
          ((float*)g.C)[ci] = ((const float*)g.aux)[(int64_t)m * g.ldaux + n] + a;
          break;
        case EPI_DGELU: {
          const float h = __bfloat162float(((const bf16*)g.aux)[(int64_t)m * g.ldaux + n]);
          ((bf16*)g.C)[ci] = __float2bfloat16_rn(a * gelu_grad_f(h));
        } break;
      }
    }
  }
}

}  // namespace

int launch_gemm_simt(const GemmArgs& g, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0) return 0;
  dim3 grid((g.N + TS - 1) / TS, (g.M + TS - 1) / TS);
  const int k_blocks = (g.K + 63) / 64;      // same reduction ranges as the tcgen05 kernel
  const int splits = g.splits < 1 ? 1 : (g.splits > k_blocks ? k_blocks : g.splits);
  for (int sp = 0; sp < splits; ++sp) {
    const int k0 = (int)((long long)sp * k_blocks / splits) * 64;
    int k1 = (int)((long long)(sp + 1) * k_blocks / splits) * 64;
    if (k1 > g.K) k1 = g.K;
    GemmArgs s = g;
    s.K = k1 - k0;
    s.A = g.A + (g.a_kmajor ? (int64_t)k0 : (int64_t)k0 * g.lda);
    s.B = g.B + (g.b_kmajor ? (int64_t)k0 : (int64_t)k0 * g.ldb);
    if (g.epilogue == EPI_STORE_F32) s.C = (float*)g.C + (int64_t)sp * g.split_stride;
    else s.C = (bf16*)g.C + (int64_t)sp * g.split_stride;
    gemm_simt_kernel<<<grid, 256, 0, st>>>(s);
  }
  return 0;
}
