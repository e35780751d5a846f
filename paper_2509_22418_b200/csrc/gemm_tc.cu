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
#include <cuda.h>
#include "common.cuh"

namespace {

constexpr int BM = 128;
constexpr int BK = 64;            // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int EPI_WARPS = 8;      // two per TMEM lane quarter, each draining half the columns
constexpr int GEMM_THREADS = 64 + 32 * EPI_WARPS;  // warp 0: TMA, warp 1: MMA + TMEM owner, then epilogue
constexpr uint32_t WAIT_LIMIT = 1u << 20;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the CTA is aborting or the wait expired.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* flags) {
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  if (flags) atomicExch(flags + PPU_FLAG_TIMEOUT, 1);
  return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   bar)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
        "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor (128-byte swizzle, descriptor version 1).  Offsets in bytes.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;   // version
  d |= (uint64_t)2 << 61;   // SWIZZLE_128B
  return d;
}

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

struct TcParams {
  int M, N, K;
  int epilogue;
  void* C; long long ldc;
  void* C2;
  const void* aux; long long ldaux;
  int* flags;
  int tiles_m, tiles_n;
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
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_slot)),
                 "r"((uint32_t)C::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int num_tiles = p.tiles_m * p.tiles_n;
  const int k_blocks = (p.K + BK - 1) / BK;

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer ----------------
      int s = 0; uint32_t ph = 0;
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
        const int m0 = (tile % p.tiles_m) * BM, n0 = (tile / p.tiles_m) * BN;
        bool ok = true;
        for (int kb = 0; kb < k_blocks && ok; ++kb) {
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
        if (!mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag, p.flags)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        bool ok = true;
        for (int kb = 0; kb < k_blocks; ++kb) {
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
            umma_bf16(d_tmem, adesc, bdesc, idesc, (kb > 0 || k > 0) ? 1u : 0u);
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
      const int m0 = (tile % p.tiles_m) * BM, n0 = (tile / p.tiles_m) * BN;
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
        const long long ci = (long long)m * p.ldc + nb;
        const bool full = nb + 32 <= p.N;
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
              if (p.epilogue == EPI_STORE_F32) {
                float4* o = reinterpret_cast<float4*>((float*)p.C + ci + 8 * j);
                o[0] = make_float4(f[0], f[1], f[2], f[3]);
                o[1] = make_float4(f[4], f[5], f[6], f[7]);
              } else {
                *reinterpret_cast<uint4*>((bf16*)p.C + ci + 8 * j) = pack8_bf16(f);
                if (p.epilogue == EPI_GELU_DUAL) {
#pragma unroll
                  for (int q = 0; q < 8; ++q) f[q] = gelu_dev(f[q]);
                  *reinterpret_cast<uint4*>((bf16*)p.C2 + ci + 8 * j) = pack8_bf16(f);
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
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"((uint32_t)C::TMEM_COLS)
                 : "memory");
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
  const int tiles = p.tiles_m * p.tiles_n;
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
  if (g_encode) return 0;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess || !fn)
    return -1;
  g_encode = (EncodeTiledFn)fn;
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
  const long long tiles256 = (long long)((g.M + BM - 1) / BM) * ((g.N + 255) / 256);
  if (g.N > 128 && tiles256 >= 148) return launch_bn<256>(g, st);
  return launch_bn<128>(g, st);
}
