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
#include <mutex>
#include <unordered_map>
#include "gemm_epilogue.cuh"

namespace tc {
static EncodeTiledFn g_encode = nullptr;
EncodeTiledFn get_encoder() { return g_encode; }
}  // namespace tc

namespace {
using namespace tc;
using namespace gemm_tc_detail;

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
      drain_tile<BN>(p, m0, n0, sp, tmem_base + (uint32_t)(acc * BN), quarter, half, lane);
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

}  // namespace

namespace gemm_tc_detail {
// Tensor maps are cached per (address, leading dimension, order, extents, box): a training step
// issues the same few hundred products every time, and encoding is a driver call.
namespace mapcache {
struct MapKey {
  const void* base; long long ld; int kmajor, rows, K, box_rows;
  bool operator==(const MapKey& o) const {
    return base == o.base && ld == o.ld && kmajor == o.kmajor && rows == o.rows && K == o.K && box_rows == o.box_rows;
  }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    size_t h = std::hash<const void*>()(k.base);
    auto mix = [&h](size_t v) { h ^= v + 0x9e3779b97f4a7c15ull + (h << 6) + (h >> 2); };
    mix((size_t)k.ld); mix((size_t)k.kmajor); mix((size_t)k.rows); mix((size_t)k.K); mix((size_t)k.box_rows);
    return h;
  }
};
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_maps;
std::mutex g_maps_lock;
constexpr size_t MAP_CACHE_LIMIT = 1 << 16;
}  // namespace mapcache
using namespace mapcache;

bool encode_map(CUtensorMap* map, const bf16* base, long long ld, bool kmajor, int rows, int K,
                int box_rows) {
  const MapKey key{base, ld, kmajor ? 1 : 0, rows, K, box_rows};
  {
    std::lock_guard<std::mutex> lk(g_maps_lock);
    auto it = g_maps.find(key);
    if (it != g_maps.end()) { *map = it->second; return true; }
  }
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
  CUresult r = tc::g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)base, gdim, gstride, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  std::lock_guard<std::mutex> lk(g_maps_lock);
  if (g_maps.size() >= MAP_CACHE_LIMIT) g_maps.clear();
  g_maps.emplace(key, *map);
  return true;
}

// launch parameters common to every tile shape (tile counts and split-K are set by the launcher)
TcParams make_params(const GemmArgs& g) {
  TcParams p;
  p.M = g.M; p.N = g.N; p.K = g.K; p.epilogue = g.epilogue;
  p.C = g.C; p.ldc = g.ldc; p.C2 = g.C2; p.aux = g.aux; p.ldaux = g.ldaux; p.flags = g.flags;
  p.tiles_m = p.tiles_n = 0; p.tail_from = 1 << 30; p.n_fastest = 0; p.splits = 1; p.split_stride = 0;
  p.C3 = g.C3; p.ldc3 = g.ldc3; p.c3_lo = g.c3_lo; p.c3_hi = g.c3_hi;
  p.rope_S = g.rope_S > 0 ? g.rope_S : 1; p.rope_dh = g.rope_dh > 0 ? g.rope_dh : 2; p.rope_cols = g.rope_cols;
  const bool f32 = g.epilogue == EPI_STORE_F32 || g.epilogue == EPI_RESID_F32;
  const long long out_unit = f32 ? 8 : 16;   // elements per 32 bytes
  bool w = (reinterpret_cast<uintptr_t>(g.C) % 32 == 0) && (g.ldc % out_unit == 0) &&
           (g.split_stride % out_unit == 0);
  if (g.epilogue == EPI_GELU_DUAL) w = w && (reinterpret_cast<uintptr_t>(g.C2) % 32 == 0);
  if (g.epilogue == EPI_RESID_F32) w = w && (reinterpret_cast<uintptr_t>(g.aux) % 32 == 0) && (g.ldaux % 8 == 0);
  if (g.epilogue == EPI_DGELU) w = w && (reinterpret_cast<uintptr_t>(g.aux) % 32 == 0) && (g.ldaux % 16 == 0);
  if (g.epilogue == EPI_DELTA_BF16) w = w && (reinterpret_cast<uintptr_t>(g.aux) % 32 == 0) && (g.ldaux % 16 == 0);
  p.wide = w ? 1 : 0;
  return p;
}
}  // namespace gemm_tc_detail

namespace {
template <int BN, bool A_K, bool B_K>
int launch_t(const GemmArgs& g, cudaStream_t st) {
  using C = Cfg<BN>;
  static PerDeviceFlag attr;
  if (!ppu_set_smem_once(attr, gemm_tc_kernel<BN, A_K, B_K>, C::SMEM)) return -1;
  CUtensorMap mapA, mapB;
  if (!encode_map(&mapA, g.A, g.lda, A_K, g.M, g.K, BM)) return -2;
  if (!encode_map(&mapB, g.B, g.ldb, B_K, g.N, g.K, BN)) return -2;
  TcParams p = make_params(g);
  p.tiles_m = (g.M + BM - 1) / BM;
  p.tiles_n = (g.N + BN - 1) / BN;
  const int k_blocks = (g.K + BK - 1) / BK;
  p.splits = g.splits < 1 ? 1 : (g.splits > k_blocks ? k_blocks : g.splits);
  p.split_stride = g.split_stride;
  const int tiles = p.tiles_m * p.tiles_n * p.splits;
  const int n_sm = ppu_sm_count();
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

namespace {
// the SM-pair kernel on 256 x 256 tiles is chosen for this product: from 16 tiles up it is at
// least as fast as one CTA per 128 x 128 tile even though it then leaves SM pairs idle
// (2048 x 2048 x 8192, 64 tiles: 0.053 ms against 0.092; 512 x 2048 x 8192, 16 tiles: equal)
bool picks_pair256(const GemmArgs& g) {
  const long long tiles_pair = (long long)((g.M + 255) / 256) * ((g.N + 255) / 256);
  // (a split product needs as many 128-k blocks as slices, or the pair kernel would write fewer
  // partial outputs than the caller adds up)
  const bool split_ok = g.splits <= 1 || g.splits <= (g.K + 127) / 128;
  return split_ok && (g.tile_shape == 2 || g.tile_shape == 4 ||
                      (g.tile_shape == 0 && g.M > 128 && g.N > 128 && tiles_pair >= 16));
}
}  // namespace

bool gemm_tc_fuses_delta(const GemmArgs& g) {
  // a thread drains 128 consecutive columns of its row in 32-column chunks with 32-byte accesses:
  // heads must be whole multiples of a chunk and must not straddle the 128-column boundary
  GemmArgs probe = g;
  probe.epilogue = EPI_DELTA_BF16;
  const int dh = g.rope_dh;
  return picks_pair256(g) && (dh == 32 || dh == 64 || dh == 128) && g.N % dh == 0 && g.N % 32 == 0 &&
         g.rope_S > 0 && g.M % g.rope_S == 0 && g.aux && g.C3 && gemm_tc_detail::make_params(probe).wide;
}

int launch_gemm_tc(const GemmArgs& g, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return 0;
  if (gemm_tc_init() != 0) return -1;
  if (g.epilogue == EPI_DELTA_BF16 && !gemm_tc_fuses_delta(g)) return -4;
  if ((g.lda % 8) || (g.ldb % 8) || (g.ldc % 8) || (g.N % 8) ||
      (reinterpret_cast<uintptr_t>(g.A) & 15) || (reinterpret_cast<uintptr_t>(g.B) & 15) ||
      (reinterpret_cast<uintptr_t>(g.C) & 15))
    return -4;
  // Wide tiles when the grid still fills the machine; narrow ones for small outputs.
  // SM pairs on 256 x 256 tiles from 16 tiles up when the product is not split.
  // (256 x 128 pair tiles throughout would fill the last wave of the N = 2048 products better -
  // 512 tiles instead of 256 on the 74 pairs of a B200 - but the narrower product measured 25 %
  // slower, so only a half-empty last wave is worked that way, inside the 256-wide kernel;
  // tile_shape 3 keeps the narrow kernel testable, 4 is the 256-wide kernel without narrow units.)
  if (g.splits > 1 && (g.tile_shape == 3 || g.epilogue != EPI_STORE_F32)) return -4;
  if (g.tile_shape == 3) return launch_gemm_tc_pair(g, make_params(g), 128, st);
  if (picks_pair256(g)) return launch_gemm_tc_pair(g, make_params(g), 256, st);
  const long long tiles256 = (long long)((g.M + BM - 1) / BM) * ((g.N + 255) / 256) * (g.splits > 1 ? g.splits : 1);
  if (g.N > 128 && tiles256 >= ppu_sm_count()) return launch_bn<256>(g, st);
  return launch_bn<128>(g, st);
}
