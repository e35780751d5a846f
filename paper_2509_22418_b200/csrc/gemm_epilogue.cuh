// Pieces shared by the tcgen05 GEMM kernels: launch parameters, the fused-epilogue arithmetic and
// the routine that drains one accumulator tile from tensor memory to global memory.
#pragma once
#include "tc_common.cuh"

namespace gemm_tc_detail {
using namespace tc;

constexpr int BM = 128;
constexpr int BK = 64;            // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int EPI_WARPS = 8;      // two per TMEM lane quarter, each draining half the columns
constexpr int GEMM_THREADS = 64 + 32 * EPI_WARPS;  // warp 0: TMA, warp 1: MMA + TMEM owner, then epilogue

// hardware tanh (relative error about 2^-11, below the bf16 rounding of the stored result)
__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float gelu_dev(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  const float t = tanh_fast(u);
  return 0.5f * x * (1.f + t);
}
__device__ __forceinline__ float gelu_grad_dev(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  const float t = tanh_fast(u);
  const float du = 0.7978845608028654f * (1.f + 3.f * 0.044715f * x * x);
  return 0.5f * (1.f + t) + 0.5f * x * (1.f - t * t) * du;
}
__device__ __forceinline__ uint4 pack8_bf16(const float* f) {
  uint4 u;
  __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  return u;
}

// 32-byte global accesses (one full sector per lane and instruction)
__device__ __forceinline__ void st_v8(void* p, const uint32_t* v) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v[0]), "r"(v[1]),
               "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}
__device__ __forceinline__ void ld_v8(uint32_t* v, const void* p) {
  asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
                 "=r"(v[7])
               : "l"(p));
}
__device__ __forceinline__ uint32_t pack2_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

// rotary positions on `pairs` adjacent pairs of f starting at column n0 of a [.., heads x dh] row
__device__ __forceinline__ void rope_pairs(float* f, int pairs, const float2* cs_row, int n0, int dh) {
#pragma unroll
  for (int q = 0; q < 16; ++q) {
    if (q >= pairs) break;
    const float2 w = __ldg(cs_row + ((n0 + 2 * q) % dh) / 2);
    const float a = f[2 * q], b = f[2 * q + 1];
    f[2 * q] = a * w.x - b * w.y;
    f[2 * q + 1] = a * w.y + b * w.x;
  }
}

struct TcParams {
  int M, N, K;
  int epilogue;
  void* C; long long ldc;
  void* C2;
  const void* aux; long long ldaux;
  int* flags;
  int tiles_m, tiles_n;
  int tail_from;   // SM-pair kernel: tiles from this index on are worked as two 128-column halves
  int n_fastest;   // SM-pair kernel: consecutive tile indices walk along N (else along M)
  int splits; long long split_stride;
  int wide;   // every output / auxiliary row start is 32-byte aligned: use 32-byte accesses
  int rope_S, rope_dh, rope_cols;
  void* C3; long long ldc3; int c3_lo, c3_hi;
};

// host side (gemm_tc.cu / gemm_tc_pair.cu)
bool encode_map(CUtensorMap* map, const bf16* base, long long ld, bool kmajor, int rows, int K, int box_rows);
TcParams make_params(const GemmArgs& g);
int launch_gemm_tc_pair(const GemmArgs& g, const TcParams& p, int bn, cudaStream_t st);   // bn: 256 or 128

// Drains rows [m0 + 32 quarter, +32) x columns [n0 + half BN/2, + BN/2) of the accumulator at
// TMEM column t_acc through registers into global memory, applying the epilogue p.epilogue.
// One row per lane; `sp` is the split-K slice (offsets the output by sp * split_stride).
// (drain_cols: the same for an explicit range [c_begin, c_end) of the tile's columns, both
// multiples of 32)
__device__ __forceinline__ void drain_cols(const TcParams& p, int m0, int n0, int sp, uint32_t t_acc,
                                           int quarter, int c_begin, int c_end, int lane) {
  const int m = m0 + quarter * 32 + lane;
  const bool row_ok = m < p.M;
  const uint32_t t_row = t_acc + ((uint32_t)(quarter * 32) << 16);
  float head_dot = 0.f;   // EPI_DELTA_BF16: running sum over the current head's columns
#pragma unroll 1
  for (int c0 = c_begin; c0 < c_end; c0 += 32) {
    const int nb = n0 + c0;
    if (nb >= p.N) break;                  // warp-uniform
    uint32_t r[32];
    tmem_ld32(t_row + c0, r);              // asynchronous until tmem_ld_wait
    const long long ci = (long long)m * p.ldc + nb + (long long)sp * p.split_stride;
    const bool full = nb + 32 <= p.N;
    if (p.wide && full) {
      // whole 32-column chunk with 32-byte accesses
      if (p.epilogue == EPI_RESID_F32) {
        uint32_t x[32];
        const float* rs = (const float*)p.aux + (long long)m * p.ldaux + nb;
        if (row_ok) {
#pragma unroll
          for (int j = 0; j < 4; ++j) ld_v8(x + 8 * j, rs + 8 * j);
        }
        tmem_ld_wait();
        if (row_ok) {
#pragma unroll
          for (int j = 0; j < 32; ++j) x[j] = __float_as_uint(__uint_as_float(x[j]) + __uint_as_float(r[j]));
#pragma unroll
          for (int j = 0; j < 4; ++j) st_v8((float*)p.C + ci + 8 * j, x + 8 * j);
        }
      } else if (p.epilogue == EPI_DGELU) {
        uint32_t hv[16];
        const bf16* hs = (const bf16*)p.aux + (long long)m * p.ldaux + nb;
        if (row_ok) { ld_v8(hv, hs); ld_v8(hv + 8, hs + 16); }
        tmem_ld_wait();
        if (row_ok) {
          uint32_t o[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float2 h2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&hv[j]));
            o[j] = pack2_bf16(__uint_as_float(r[2 * j]) * gelu_grad_dev(h2.x),
                              __uint_as_float(r[2 * j + 1]) * gelu_grad_dev(h2.y));
          }
          st_v8((bf16*)p.C + ci, o);
          st_v8((bf16*)p.C + ci + 16, o + 8);
        }
      } else if (p.epilogue == EPI_STORE_F32) {
        tmem_ld_wait();
        if (row_ok) {
#pragma unroll
          for (int j = 0; j < 4; ++j) st_v8((float*)p.C + ci + 8 * j, r + 8 * j);
        }
      } else {
        uint32_t uv[16];
        if (p.epilogue == EPI_DELTA_BF16 && row_ok) {
          const bf16* us = (const bf16*)p.aux + (long long)m * p.ldaux + nb;
          ld_v8(uv, us); ld_v8(uv + 8, us + 16);
        }
        tmem_ld_wait();
        if (row_ok) {
          if (p.epilogue == EPI_ROPE_BF16 && nb < p.rope_cols) {
            const float2* cs_row = (const float2*)p.aux + (long long)(m % p.rope_S) * (p.rope_dh / 2);
            if (p.rope_dh % 32 == 0) {
              // the chunk lies inside one head: its 16 (cos, sin) pairs are 128 contiguous bytes
              uint32_t w[32];
              const float2* src = cs_row + (nb % p.rope_dh) / 2;
#pragma unroll
              for (int j = 0; j < 4; ++j) ld_v8(w + 8 * j, src + 4 * j);
#pragma unroll
              for (int q = 0; q < 16; ++q) {
                const float cw = __uint_as_float(w[2 * q]), sw = __uint_as_float(w[2 * q + 1]);
                const float a = __uint_as_float(r[2 * q]), b = __uint_as_float(r[2 * q + 1]);
                r[2 * q] = __float_as_uint(a * cw - b * sw);
                r[2 * q + 1] = __float_as_uint(a * sw + b * cw);
              }
            } else {
              rope_pairs(reinterpret_cast<float*>(r), 16, cs_row, nb, p.rope_dh);
            }
          }
          uint32_t o[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) o[j] = pack2_bf16(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
          if (p.C) {       // (the pre-activation store of EPI_GELU_DUAL is optional)
            st_v8((bf16*)p.C + ci, o);
            st_v8((bf16*)p.C + ci + 16, o + 8);
          }
          if (p.epilogue == EPI_DELTA_BF16) {
            // the product uses the stored (rounded) values, as the attention kernels will
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float2 gv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&o[j]));
              const float2 u2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&uv[j]));
              head_dot = fmaf(gv.x, u2.x, fmaf(gv.y, u2.y, head_dot));
            }
            if ((nb + 32) % p.rope_dh == 0) {
              const int heads = p.N / p.rope_dh;
              ((float*)p.C3)[((long long)(m / p.rope_S) * heads + nb / p.rope_dh) * p.rope_S + m % p.rope_S] = head_dot;
              head_dot = 0.f;
            }
          }
          if (p.epilogue == EPI_GELU_DUAL) {
#pragma unroll
            for (int j = 0; j < 16; ++j)
              o[j] = pack2_bf16(gelu_dev(__uint_as_float(r[2 * j])), gelu_dev(__uint_as_float(r[2 * j + 1])));
            st_v8((bf16*)p.C2 + ci, o);
            st_v8((bf16*)p.C2 + ci + 16, o + 8);
            if (p.C3 && nb < p.c3_hi && nb + 32 > p.c3_lo) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int col = nb + 8 * j;
                if (col >= p.c3_lo && col + 8 <= p.c3_hi)
                  *reinterpret_cast<uint4*>((bf16*)p.C3 + (long long)m * p.ldc3 + (col - p.c3_lo)) =
                      make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
              }
            }
          }
        }
      }
      continue;
    }
    if (p.epilogue == EPI_RESID_F32) {
      float4 x[8];
      const float4* rs = reinterpret_cast<const float4*>((const float*)p.aux + (long long)m * p.ldaux + nb);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        x[j] = (row_ok && (full || nb + 4 * j < p.N)) ? rs[j] : make_float4(0.f, 0.f, 0.f, 0.f);
      tmem_ld_wait();
      if (row_ok) {
        float4* o = reinterpret_cast<float4*>((float*)p.C + ci);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (full || nb + 4 * j < p.N)
            o[j] = make_float4(x[j].x + __uint_as_float(r[4 * j]), x[j].y + __uint_as_float(r[4 * j + 1]),
                               x[j].z + __uint_as_float(r[4 * j + 2]), x[j].w + __uint_as_float(r[4 * j + 3]));
      }
    } else if (p.epilogue == EPI_DGELU) {
      uint4 hv[4];
      const uint4* hs = reinterpret_cast<const uint4*>((const bf16*)p.aux + (long long)m * p.ldaux + nb);
#pragma unroll
      for (int j = 0; j < 4; ++j)
        hv[j] = (row_ok && (full || nb + 8 * j < p.N)) ? hs[j] : make_uint4(0, 0, 0, 0);
      tmem_ld_wait();
      if (row_ok) {
        uint4* o = reinterpret_cast<uint4*>((bf16*)p.C + ci);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (!(full || nb + 8 * j < p.N)) break;
          const __nv_bfloat162* hp = reinterpret_cast<const __nv_bfloat162*>(&hv[j]);
          float a[8];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float2 h2 = __bfloat1622float2(hp[q]);
            a[2 * q] = __uint_as_float(r[8 * j + 2 * q]) * gelu_grad_dev(h2.x);
            a[2 * q + 1] = __uint_as_float(r[8 * j + 2 * q + 1]) * gelu_grad_dev(h2.y);
          }
          o[j] = pack8_bf16(a);
        }
      }
    } else {
      tmem_ld_wait();
      if (row_ok) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (!(full || nb + 8 * j < p.N)) break;
          float f[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) f[q] = __uint_as_float(r[8 * j + q]);
          if (p.epilogue == EPI_ROPE_BF16 && nb + 8 * j < p.rope_cols)
            rope_pairs(f, 4, (const float2*)p.aux + (long long)(m % p.rope_S) * (p.rope_dh / 2), nb + 8 * j,
                       p.rope_dh);
          if (p.epilogue == EPI_STORE_F32) {
            float4* o = reinterpret_cast<float4*>((float*)p.C + ci + 8 * j);
            o[0] = make_float4(f[0], f[1], f[2], f[3]);
            o[1] = make_float4(f[4], f[5], f[6], f[7]);
          } else {
            if (p.C) *reinterpret_cast<uint4*>((bf16*)p.C + ci + 8 * j) = pack8_bf16(f);
            if (p.epilogue == EPI_GELU_DUAL) {
#pragma unroll
              for (int q = 0; q < 8; ++q) f[q] = gelu_dev(f[q]);
              const uint4 gv = pack8_bf16(f);
              *reinterpret_cast<uint4*>((bf16*)p.C2 + ci + 8 * j) = gv;
              const int col = nb + 8 * j;
              if (p.C3 && col >= p.c3_lo && col + 8 <= p.c3_hi)
                *reinterpret_cast<uint4*>((bf16*)p.C3 + (long long)m * p.ldc3 + (col - p.c3_lo)) = gv;
            }
          }
        }
      }
    }
  }
}

template <int BN>
__device__ __forceinline__ void drain_tile(const TcParams& p, int m0, int n0, int sp, uint32_t t_acc,
                                           int quarter, int half, int lane) {
  drain_cols(p, m0, n0, sp, t_acc, quarter, half * (BN / 2), (half + 1) * (BN / 2), lane);
}

}  // namespace gemm_tc_detail
