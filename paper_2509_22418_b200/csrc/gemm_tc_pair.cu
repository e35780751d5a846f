// tcgen05 GEMM on SM pairs (cta_group::2): C[M,N] = A . B^T, bf16 operands, fp32 accumulation.
//
// A cluster of two CTAs (the two SMs of one TPC) owns a 256 x 256 output tile.  CTA r of the
// pair loads rows [128 r, 128 r + 128) of the A tile and of the B tile; one thread of the
// leader CTA (rank 0) issues tcgen05.mma.cta_group::2 with M = 256, N = 256, K = 16, for which
// each SM reads its own A half and shares its B half with its peer, and each SM's tensor memory
// receives its 128 rows of the 256-column accumulator.  Per SM and MMA that is 8 KB of operands
// read from shared memory for 128 x 256 x 16 multiply-adds, against 12 KB for a single-CTA
// 128 x 256 tile: the operand path, not the tensor pipe, limits the single-CTA kernel.
//
// Protocol.  Stage barriers live at the same shared-memory offsets in both CTAs.
//   full[s]    only the leader's is used: its producer posts the expected bytes of BOTH CTAs'
//              loads, and both CTAs' TMA loads complete on it (.cta_group::2 form of the copy).
//   empty[s]   one per CTA, signalled in both by the MMA thread's multicast commit.
//   tfull[a]   one per CTA (multicast commit): accumulator a is complete.
//   tempty[a]  the leader's counts the epilogue warps of both CTAs (the peer's arrive remotely).
// Every wait is bounded; on expiry the CTA raises its abort flag and an error word and all roles
// fall through to the common exit, where both CTAs meet at a cluster barrier (reached
// unconditionally by every thread) before tensor memory is released.
#include "gemm_epilogue.cuh"

namespace {
using namespace tc;
using namespace gemm_tc_detail;

// The pair's tile is 256 rows x BN columns, BN = 256 or 128.  The narrow tile is for outputs whose
// 256-wide tiling leaves the last wave of SM pairs half empty (N = 2048 with 8192 rows: 256 tiles
// on the 74 SM pairs of a B200: three full waves and 34 tiles).  The 256-wide kernel can work the
// tiles from index p.tail_from on as two 128-column halves each, so that the 34 leftover tiles
// become 68 units on 74 pairs: the narrow product runs at about 0.7 of the wide one's rate, so
// the last wave takes 0.7 of a tile's time instead of a whole one.
// A stage holds PAIR_KH slabs of 64 k: the issuing thread stalls while the tensor pipe is busy, so
// a barrier wait per 64 k (four instructions) is not hidden behind the products; one per 128 k is.
constexpr int PAIR_KH = 2;
constexpr int SLAB_BYTES = 128 * BK * 2;     // 128 rows x 64 k of one operand
template <int BN> struct PairCfg {
  static constexpr int STAGES = BN == 256 ? 3 : 4;
  static constexpr int A_HALF = PAIR_KH * SLAB_BYTES;            // this CTA's 128 rows of A
  static constexpr int B_SLAB = (BN / 2) * BK * 2;               // this CTA's BN/2 rows of B, 64 k
  static constexpr int B_HALF = PAIR_KH * B_SLAB;
  static constexpr int STAGE_BYTES = A_HALF + B_HALF;
  static constexpr int SMEM = STAGES * STAGE_BYTES + 1024 + 256;
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load of a CTA pair: the bytes land in this CTA's shared memory, the completion is
// counted on the barrier at cluster address `bar` (the leader's)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
  const uint32_t z = 0;
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(z)
      : "memory");
}
// arrives, once the pair's earlier MMAs have completed, on the barrier at this offset in both CTAs
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
      "h"(mask)
      : "memory");
}

// one unit of work of a pair: rows [m0, m0 + 256) x columns [n0, n0 + bn)
// (kb0, kb1: the unit's range of 128-k blocks; sp: its split-K slice)
struct PairUnit { int m0, n0, bn, sp, kb0, kb1; };
template <int PAIR_BN>
__device__ __forceinline__ PairUnit pair_unit(const TcParams& p, int u, int num_tiles, int k_blocks) {
  PairUnit w;
  int tile = u, half = 0;
  w.bn = PAIR_BN; w.sp = 0; w.kb0 = 0; w.kb1 = k_blocks;
  if (p.splits > 1) {          // split-K products have whole tiles only
    w.sp = u / num_tiles; tile = u - w.sp * num_tiles;
    w.kb0 = (int)((long long)w.sp * k_blocks / p.splits);
    w.kb1 = (int)((long long)(w.sp + 1) * k_blocks / p.splits);
  }
  if (PAIR_BN == 256 && u >= p.tail_from) {
    const int v = u - p.tail_from;
    tile = p.tail_from + (v >> 1); half = v & 1; w.bn = 128;
  }
  // consecutive tiles (which the pairs work on at the same time) walk along the smaller operand:
  // the rows of A they share then stay in L2 while B is swept, or the other way round
  const int row = p.n_fastest ? tile / p.tiles_n : tile % p.tiles_m;
  const int col = p.n_fastest ? tile % p.tiles_n : tile / p.tiles_m;
  w.m0 = row * 256;
  w.n0 = col * PAIR_BN + half * 128;
  return w;
}

// mapB2: B with a box of 64 rows (the narrow units of a K-major B); otherwise a copy of mapB
template <int PAIR_BN, bool A_K, bool B_K>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                    const __grid_constant__ CUtensorMap mapB2, const TcParams p) {
  using PC = PairCfg<PAIR_BN>;
  constexpr int ST = PC::STAGES, PAIR_STAGE_BYTES = PC::STAGE_BYTES, HALF_BYTES = PC::A_HALF, B_SLAB = PC::B_SLAB;
  extern __shared__ uint8_t smem_raw[];
  // the dynamic window starts at the same offset in both CTAs, so aligned offsets match too
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + ST * PAIR_STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * ST + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const bool leader = rank == 0;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (ST + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * ST + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * ST + 2 + a); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < ST; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int n_pairs = gridDim.x >> 1, pair = blockIdx.x >> 1;
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int k_blocks = (p.K + PAIR_KH * BK - 1) / (PAIR_KH * BK);
  const int num_units = p.splits > 1 ? num_tiles * p.splits
                                     : num_tiles + (PAIR_BN == 256 && num_tiles > p.tail_from ? num_tiles - p.tail_from : 0);

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer (both CTAs) ----------------
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      for (int u = pair; u < num_units && ok; u += n_pairs) {
        const PairUnit w = pair_unit<PAIR_BN>(p, u, num_tiles, k_blocks);
        const int m0 = w.m0 + (int)rank * 128;
        const int n0 = w.n0 + (int)rank * (w.bn / 2);
        const bool narrow = w.bn != PAIR_BN;
        const int b_slab = narrow ? B_SLAB / 2 : B_SLAB;          // this CTA's bn/2 rows of B, 64 k
        const CUtensorMap* mB = narrow ? &mapB2 : &mapB;
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          ok = mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.flags);
          if (!ok) break;
          const uint32_t a_dst = smem_u32(smem + s * PAIR_STAGE_BYTES);
          const uint32_t b_dst = a_dst + HALF_BYTES;
          const uint32_t fb = map_to_rank(full_bar(s), 0);
          if (leader) mbar_expect_tx(full_bar(s), 2 * (HALF_BYTES + PAIR_KH * b_slab));
          // (k past the end of the reduction reads zeros)
#pragma unroll
          for (int kh = 0; kh < PAIR_KH; ++kh) {
            const int k0 = (kb * PAIR_KH + kh) * BK;
            if (A_K) {
              tma_load_2d_pair(a_dst + kh * SLAB_BYTES, &mapA, fb, k0, m0);
            } else {
              tma_load_2d_pair(a_dst + kh * SLAB_BYTES, &mapA, fb, m0, k0);
              tma_load_2d_pair(a_dst + kh * SLAB_BYTES + 8192, &mapA, fb, m0 + 64, k0);
            }
            if (B_K) {
              tma_load_2d_pair(b_dst + kh * b_slab, mB, fb, k0, n0);
            } else {
#pragma unroll
              for (int i = 0; i < PAIR_BN / 128; ++i)
                if (i < w.bn / 128) tma_load_2d_pair(b_dst + kh * b_slab + i * 8192, &mapB, fb, n0 + 64 * i, k0);
            }
          }
          if (++s == ST) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      // ---------------- MMA issuer (leader CTA only) ----------------
      const uint32_t idesc0 = (1u << 4) | (1u << 7) | (1u << 10) | ((A_K ? 0u : 1u) << 15) |
                              ((B_K ? 0u : 1u) << 16) | ((uint32_t)(256 >> 4) << 24);
      int s = 0; uint32_t ph = 0;
      int acc = 0; uint32_t acc_ph = 0;
      for (int u = pair; u < num_units; u += n_pairs) {
        const PairUnit w = pair_unit<PAIR_BN>(p, u, num_tiles, k_blocks);
        const uint32_t idesc = idesc0 | ((uint32_t)(w.bn >> 3) << 17);
        const uint32_t b_slab = w.bn != PAIR_BN ? B_SLAB / 2 : B_SLAB;
        if (!mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag, p.flags)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * PAIR_BN);
        bool ok = true;
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          ok = mbar_wait(full_bar(s), ph, abort_flag, p.flags);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + s * PAIR_STAGE_BYTES);
          const uint32_t b_addr = a_addr + HALF_BYTES;
#pragma unroll
          for (int k = 0; k < PAIR_KH * (BK / UMMA_K); ++k) {
            const uint32_t kh = (uint32_t)(k / (BK / UMMA_K)), kk = (uint32_t)(k % (BK / UMMA_K));
            const uint32_t slab = kh * SLAB_BYTES, slab_b = kh * b_slab;
            const uint64_t adesc = A_K ? make_desc(a_addr + slab + kk * 32, 16, 1024) : make_desc(a_addr + slab + kk * 2048, 8192, 1024);
            const uint64_t bdesc = B_K ? make_desc(b_addr + slab_b + kk * 32, 16, 1024) : make_desc(b_addr + slab_b + kk * 2048, 8192, 1024);
            umma_bf16_pair(d_tmem, adesc, bdesc, idesc, (kb > w.kb0 || k > 0) ? 1u : 0u);
          }
          umma_commit_pair(empty_bar(s));        // both CTAs' slots are free once these MMAs have read them
          if (++s == ST) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(tfull_bar(acc));        // both halves of the accumulator are complete
        if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
      }
    }
  } else {
    // ---------------- epilogue warps (both CTAs, 128 rows each) ----------------
    const int quarter = warp & 3;
    const int half = (warp - 2) >> 2;
    int acc = 0; uint32_t acc_ph = 0;
    for (int u = pair; u < num_units; u += n_pairs) {
      const PairUnit w = pair_unit<PAIR_BN>(p, u, num_tiles, k_blocks);
      const int m0 = w.m0 + (int)rank * 128;
      if (!mbar_wait(tfull_bar(acc), acc_ph, abort_flag, p.flags)) break;
      tc_fence_after();
      drain_cols(p, m0, w.n0, w.sp, tmem_base + (uint32_t)(acc * PAIR_BN), quarter, half * (w.bn / 2),
                 (half + 1) * (w.bn / 2), lane);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_rank(tempty_bar(acc), 0));
      if (++acc == 2) { acc = 0; acc_ph ^= 1u; }
    }
  }

  // ---------------- common exit ----------------
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(2000);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // neither CTA leaves (or frees tensor memory) while its peer may still signal it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

template <int PAIR_BN, bool A_K, bool B_K>
int launch_pair_t(const GemmArgs& g, const TcParams& p0, cudaStream_t st) {
  static PerDeviceFlag attr;
  if (!ppu_set_smem_once(attr, gemm_tc_pair_kernel<PAIR_BN, A_K, B_K>, PairCfg<PAIR_BN>::SMEM)) return -1;
  CUtensorMap mapA, mapB, mapB2;
  if (!encode_map(&mapA, g.A, g.lda, A_K, g.M, g.K, 128)) return -2;
  if (!encode_map(&mapB, g.B, g.ldb, B_K, g.N, g.K, PAIR_BN / 2)) return -2;
  TcParams p = p0;
  p.tiles_m = (g.M + 255) / 256;
  p.tiles_n = (g.N + PAIR_BN - 1) / PAIR_BN;
  // split-K (fp32 partial outputs sp * split_stride apart, summed by the consumer): each unit of
  // work is a whole tile over a slice of the 128-k blocks
  const int k_blocks = (g.K + PAIR_KH * BK - 1) / (PAIR_KH * BK);
  p.splits = g.splits < 1 ? 1 : (g.splits > k_blocks ? k_blocks : g.splits);
  p.split_stride = g.split_stride;
  // tiles that run at the same time share operand rows through L2: walk along the shorter side
  // of the output, so that a wave of pairs covers few rows of the larger operand and all of the
  // smaller one (8192 x 2048 x 8192: 1341 -> 1452 TFLOP/s; the 134 MB A operand no longer
  // passes through L2 once per wave)
  p.n_fastest = g.M > g.N ? 1 : 0;
  const int tiles = p.tiles_m * p.tiles_n * p.splits;
  const int n_sm = ppu_sm_count();
  // as many pairs as give every pair the same number of tiles: 256 tiles on 74 pairs take four
  // waves whether 74 or 64 pairs work on them, and on a power-capped part the idle SMs' share of
  // the budget raises the clock of the busy ones
  const int max_pairs = n_sm / 2;
  const int waves = (tiles + max_pairs - 1) / max_pairs;
  int pairs = tiles < max_pairs ? tiles : (tiles + waves - 1) / waves;
  // a last wave that fills at most half of the pairs is worked as 128-column halves by all of
  // them (not with the row-sum epilogue, whose running sum spans a thread's 128 columns)
  const int rem = tiles % max_pairs;
  p.tail_from = 1 << 30;
  if (PAIR_BN == 256 && p.splits == 1 && g.tile_shape != 4 && g.epilogue != EPI_DELTA_BF16 && tiles > max_pairs && rem > 0 &&
      2 * rem <= max_pairs) {
    p.tail_from = tiles - rem;
    pairs = max_pairs;
  }
  mapB2 = mapB;
  if (B_K && p.tail_from < tiles && !encode_map(&mapB2, g.B, g.ldb, true, g.N, g.K, 64)) return -2;
  gemm_tc_pair_kernel<PAIR_BN, A_K, B_K><<<2 * pairs, GEMM_THREADS, PairCfg<PAIR_BN>::SMEM, st>>>(mapA, mapB, mapB2, p);
  return cudaGetLastError() == cudaSuccess ? 0 : -3;
}

}  // namespace

namespace {
template <int PAIR_BN>
int launch_pair_bn(const GemmArgs& g, const TcParams& p, cudaStream_t st) {
  if (g.a_kmajor && g.b_kmajor) return launch_pair_t<PAIR_BN, true, true>(g, p, st);
  if (g.a_kmajor && !g.b_kmajor) return launch_pair_t<PAIR_BN, true, false>(g, p, st);
  if (!g.a_kmajor && g.b_kmajor) return launch_pair_t<PAIR_BN, false, true>(g, p, st);
  return launch_pair_t<PAIR_BN, false, false>(g, p, st);
}
}  // namespace

namespace gemm_tc_detail {
int launch_gemm_tc_pair(const GemmArgs& g, const TcParams& p, int bn, cudaStream_t st) {
  return bn == 128 ? launch_pair_bn<128>(g, p, st) : launch_pair_bn<256>(g, p, st);
}
}  // namespace gemm_tc_detail
