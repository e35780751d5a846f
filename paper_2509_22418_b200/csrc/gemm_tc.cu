// tcgen05 GEMM for sm_100a: C[M,N] = A . B^T with bf16 operands and fp32 accumulation in
// tensor memory.  One persistent CTA per SM walks 128 x BN output tiles; a producer thread
// streams 64-deep operand slabs into a shared-memory ring with TMA (128-byte swizzle), one
// thread issues tcgen05.mma (M=128, N=BN, K=16) into one of two TMEM accumulators, and four
// epilogue warps drain the other accumulator through registers into global memory, so the
// epilogue of tile i overlaps the main loop of tile i+1.  Both operands may be K-major
// (row-major [rows, K]) or MN-major (stored [K, rows]) - forward products are K/K, input
// gradients K/MN, subset weight gradients MN/MN (the reduction runs over tokens).
//
// Every mbarrier wait is bounded: on expiry the CTA raises a shared abort flag and a device
// error word, all roles leave their loops, tensor memory is released and the kernel returns.
#include "tc_common.cuh"

namespace tc {
static EncodeTiledFn g_encode = nullptr;
EncodeTiledFn get_encoder() { return g_encode; }
}  // namespace tc

namespace {
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
  int splits; long long split_stride;
  int wide;   // every output / auxiliary row start is 32-byte aligned: use 32-byte accesses
  int rope_S, rope_dh, rope_cols;
  void* C3; long long ldc3; int c3_lo, c3_hi;
};

template <int BN> struct Cfg {
  static constexpr int STAGES = BN == 256 ? 4 : 6;
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int SMEM = STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
  static constexpr int TMEM_COLS = 2 * BN;
};

template <int BN, bool A_K, bool B_K>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
               const TcParams p) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::STAGES * C::STAGE_BYTES);
  // bars[0..ST): full, [ST..2ST): empty, [2ST..2ST+2): tmem_full, [2ST+2..2ST+4): tmem_empty
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * C::STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (C::STAGES + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * C::STAGES + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * C::STAGES + 2 + a); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), (uint32_t)C::TMEM_COLS);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int tiles_mn = p.tiles_m * p.tiles_n;
  const int num_tiles = tiles_mn * p.splits;
  const int k_blocks = (p.K + BK - 1) / BK;

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer ----------------
      int s = 0; uint32_t ph = 0;
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
        const int sp = tile / tiles_mn, t2 = tile - sp * tiles_mn;
        const int m0 = (t2 % p.tiles_m) * BM, n0 = (t2 / p.tiles_m) * BN;
        const int kb0 = (int)((long long)sp * k_blocks / p.splits);
        const int kb1 = (int)((long long)(sp + 1) * k_blocks / p.splits);
        bool ok = true;
        for (int kb = kb0; kb < kb1 && ok; ++kb) {
          ok = mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.flags);
          if (!ok) break;
          const uint32_t a_dst = smem_u32(smem + s * C::STAGE_BYTES);
          const uint32_t b_dst = a_dst + C::A_BYTES;
          mbar_expect_tx(full_bar(s), C::STAGE_BYTES);
          if (A_K) {
            tma_load_2d(a_dst, &mapA, full_bar(s), kb * BK, m0);
          } else {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i)
              tma_load_2d(a_dst + i * 8192, &mapA, full_bar(s), m0 + 64 * i, kb * BK);
          }
          if (B_K) {
            tma_load_2d(b_dst, &mapB, full_bar(s), kb * BK, n0);
          } else {
#pragma unroll
            for (int i = 0; i < BN / 64; ++i)
              tma_load_2d(b_dst + i * 8192, &mapB, full_bar(s), n0 + 64 * i, kb * BK);
          }
          if (++s == C::STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      // instruction descriptor: D fp32, A/B bf16, majors, N >> 3, M >> 4
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_K ? 0u : 1u) << 15) |
                             ((B_K ? 0u : 1u) << 16) | ((uint32_t)(BN >> 3) << 17) |
                             ((uint32_t)(BM >> 4) << 24);
      int s = 0; uint32_t ph = 0;
      int acc = 0; uint32_t acc_ph = 0;
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
        const int sp = tile / tiles_mn;
        const int kb0 = (int)((long long)sp * k_blocks / p.splits);
        const int kb1 = (int)((long long)(sp + 1) * k_blocks / p.splits);
        if (!mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag, p.flags)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        bool ok = true;
        for (int kb = kb0; kb < kb1; ++kb) {
          ok = mbar_wait(full_bar(s), ph, abort_flag, p.flags);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + s * C::STAGE_BYTES);
          const uint32_t b_addr = a_addr + C::A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t adesc = A_K ? make_desc(a_addr + k * 32, 16, 1024)
                                       : make_desc(a_addr + k * 2048, 8192, 1024);
            const uint64_t bdesc = B_K ? make_desc(b_addr + k * 32, 16, 1024)
                                       : make_desc(b_addr + k * 2048, 8192, 1024);
            umma_bf16(d_tmem, adesc, bdesc, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          }
          umma_commit(empty_bar(s));           // slot is free once these MMAs have read it
          if (++s == C::STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        umma_commit(tfull_bar(acc));           // accumulator complete
        if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue warps ----------------
    const int quarter = warp & 3;              // TMEM lanes [32 q, 32 q + 32) belong to this warp
    const int half = (warp - 2) >> 2;          // which half of the tile's columns
    int acc = 0; uint32_t acc_ph = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      const int sp = tile / tiles_mn, t2 = tile - sp * tiles_mn;
      const int m0 = (t2 % p.tiles_m) * BM, n0 = (t2 / p.tiles_m) * BN;
      if (!mbar_wait(tfull_bar(acc), acc_ph, abort_flag, p.flags)) break;
      tc_fence_after();
      const int m = m0 + quarter * 32 + lane;
      const bool row_ok = m < p.M;
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
#pragma unroll 1
      for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
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
              st_v8((bf16*)p.C + ci, o);
              st_v8((bf16*)p.C + ci + 16, o + 8);
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
                *reinterpret_cast<uint4*>((bf16*)p.C + ci + 8 * j) = pack8_bf16(f);
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
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
    }
  }

  // ---------------- common exit ----------------
  if (*abort_flag) {
    // give copies and MMAs already in flight time to land before memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(2000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)C::TMEM_COLS);
  }
}

bool encode_map(CUtensorMap* map, const bf16* base, long long ld, bool kmajor, int rows, int K,
                int box_rows) {
  // kmajor: memory is [rows, K] (inner = K).  else: memory is [K, rows] (inner = rows).
  cuuint64_t gdim[2];
  cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2];
  cuuint32_t estr[2] = {1, 1};
  if (kmajor) {
    gdim[0] = (cuuint64_t)K; gdim[1] = (cuuint64_t)rows;
    box[0] = BK; box[1] = (cuuint32_t)box_rows;
  } else {
    gdim[0] = (cuuint64_t)rows; gdim[1] = (cuuint64_t)K;
    box[0] = 64; box[1] = BK;
  }
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)base, gdim, gstride, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int BN, bool A_K, bool B_K>
int launch_t(const GemmArgs& g, cudaStream_t st) {
  using C = Cfg<BN>;
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(gemm_tc_kernel<BN, A_K, B_K>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM) != cudaSuccess)
      return -1;
    attr_done = true;
  }
  CUtensorMap mapA, mapB;
  if (!encode_map(&mapA, g.A, g.lda, A_K, g.M, g.K, BM)) return -2;
  if (!encode_map(&mapB, g.B, g.ldb, B_K, g.N, g.K, BN)) return -2;
  TcParams p;
  p.M = g.M; p.N = g.N; p.K = g.K; p.epilogue = g.epilogue;
  p.C = g.C; p.ldc = g.ldc; p.C2 = g.C2; p.aux = g.aux; p.ldaux = g.ldaux; p.flags = g.flags;
  p.tiles_m = (g.M + BM - 1) / BM;
  p.tiles_n = (g.N + BN - 1) / BN;
  const int k_blocks = (g.K + BK - 1) / BK;
  p.splits = g.splits < 1 ? 1 : (g.splits > k_blocks ? k_blocks : g.splits);
  p.split_stride = g.split_stride;
  p.C3 = g.C3; p.ldc3 = g.ldc3; p.c3_lo = g.c3_lo; p.c3_hi = g.c3_hi;
  p.rope_S = g.rope_S > 0 ? g.rope_S : 1; p.rope_dh = g.rope_dh > 0 ? g.rope_dh : 2; p.rope_cols = g.rope_cols;
  {
    const bool f32 = g.epilogue == EPI_STORE_F32 || g.epilogue == EPI_RESID_F32;
    const long long out_unit = f32 ? 8 : 16;   // elements per 32 bytes
    bool w = (reinterpret_cast<uintptr_t>(g.C) % 32 == 0) && (g.ldc % out_unit == 0) &&
             (g.split_stride % out_unit == 0);
    if (g.epilogue == EPI_GELU_DUAL) w = w && (reinterpret_cast<uintptr_t>(g.C2) % 32 == 0);
    if (g.epilogue == EPI_RESID_F32) w = w && (reinterpret_cast<uintptr_t>(g.aux) % 32 == 0) && (g.ldaux % 8 == 0);
    if (g.epilogue == EPI_DGELU) w = w && (reinterpret_cast<uintptr_t>(g.aux) % 32 == 0) && (g.ldaux % 16 == 0);
    p.wide = w ? 1 : 0;
  }
  const int tiles = p.tiles_m * p.tiles_n * p.splits;
  static int n_sm = 0;
  if (n_sm == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (n_sm <= 0) n_sm = 148;
  }
  const int grid = tiles < n_sm ? tiles : n_sm;
  gemm_tc_kernel<BN, A_K, B_K><<<grid, GEMM_THREADS, C::SMEM, st>>>(mapA, mapB, p);
  return cudaGetLastError() == cudaSuccess ? 0 : -3;
}

template <int BN>
int launch_bn(const GemmArgs& g, cudaStream_t st) {
  if (g.a_kmajor && g.b_kmajor) return launch_t<BN, true, true>(g, st);
  if (g.a_kmajor && !g.b_kmajor) return launch_t<BN, true, false>(g, st);
  if (!g.a_kmajor && g.b_kmajor) return launch_t<BN, false, true>(g, st);
  return launch_t<BN, false, false>(g, st);
}

}  // namespace

int gemm_tc_init() {
  if (tc::g_encode) return 0;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess || !fn)
    return -1;
  tc::g_encode = (tc::EncodeTiledFn)fn;
  return 0;
}

int launch_gemm_tc(const GemmArgs& g, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return 0;
  if (gemm_tc_init() != 0) return -1;
  if ((g.lda % 8) || (g.ldb % 8) || (g.ldc % 8) || (g.N % 8) ||
      (reinterpret_cast<uintptr_t>(g.A) & 15) || (reinterpret_cast<uintptr_t>(g.B) & 15) ||
      (reinterpret_cast<uintptr_t>(g.C) & 15))
    return -4;
  // Wide tiles when the grid still fills the machine; narrow ones for small outputs.
  const long long tiles256 = (long long)((g.M + BM - 1) / BM) * ((g.N + 255) / 256) * (g.splits > 1 ? g.splits : 1);
  if (g.N > 128 && tiles256 >= 148) return launch_bn<256>(g, st);
  return launch_bn<128>(g, st);
}
