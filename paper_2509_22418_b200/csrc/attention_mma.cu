// Fused causal attention on tensor cores (bf16 mma.sync m16n8k16, fp32 accumulation) with an
// online softmax, for head sizes 64 and 128.  Scores never reach global memory.
//   forward : U = softmax_row(q k^T / sqrt(d_h) + causal) v, lse = log-sum-exp of the scaled scores
//   backward: delta = rowsum(dU * U); one kernel owns query blocks and forms dq, a second owns key
//             blocks and forms dk, dv.  Both recompute the probabilities from q, k and lse, so no
//             floating-point atomics are needed and results are bitwise reproducible.
// Tiles are 64 rows x d_h, staged with cp.async into XOR-swizzled shared memory and read with
// ldmatrix.  (Appendix C.1, MHA equations; softmax backward dS = A * (dA - rowsum(dA * A)).)
#include "common.cuh"

namespace {

constexpr int BT = 64;          // rows per tile (queries and keys)
constexpr int NTHREADS = 128;   // 4 warps x 16 rows
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes)
               : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t* r, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

// byte offset of 16-byte chunk `ch` of row `r` in a swizzled [rows][DH] bf16 tile
template <int DH> __device__ __forceinline__ uint32_t sw(int r, int ch) {
  return (uint32_t)(r * DH * 2 + ((ch ^ (r & 7)) << 4));
}

// 64 x DH tile of rows [row0, row0+64) of a [S, ld] matrix; rows >= S are zero-filled
template <int DH>
__device__ __forceinline__ void load_tile(uint32_t tile, const bf16* g, int64_t ld, int row0, int S) {
  constexpr int CH = DH / 8;
  for (int c = threadIdx.x; c < BT * CH; c += NTHREADS) {
    const int r = c / CH, ch = c % CH;
    const int row = row0 + r;
    const bool ok = row < S;
    cp_async16(tile + sw<DH>(r, ch), g + (int64_t)(ok ? row : 0) * ld + ch * 8, ok ? 16 : 0);
  }
}
__device__ __forceinline__ void load_vec64(uint32_t dst, const float* g, int row0, int S) {
  // 64 floats = 16 chunks of 16 bytes; rows >= S zero-filled (S need not be a multiple of 4)
  if (threadIdx.x < 64) {
    const int row = row0 + threadIdx.x;
    const bool ok = row < S;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst + 4 * threadIdx.x),
                 "l"(g + (ok ? row : 0)), "r"(ok ? 4 : 0) : "memory");
  }
}

// A fragment (16 rows x 16 k) of a swizzled tile at (row_base, k0)
template <int DH>
__device__ __forceinline__ void frag_a(uint32_t* a, uint32_t tile, int row_base, int k0) {
  const int l = threadIdx.x & 31;
  ldsm_x4(a, tile + sw<DH>(row_base + (l & 7) + ((l >> 3) & 1) * 8, (k0 >> 3) + (l >> 4)));
}
// B fragments for two n-tiles (rows n0..n0+15 of the tile are the n index, k contiguous):
// b[0],b[1] -> n-tile n0 ; b[2],b[3] -> n-tile n0+8
template <int DH>
__device__ __forceinline__ void frag_b(uint32_t* b, uint32_t tile, int n0, int k0) {
  const int l = threadIdx.x & 31;
  ldsm_x4(b, tile + sw<DH>(n0 + (l & 7) + (l >> 4) * 8, (k0 >> 3) + ((l >> 3) & 1)));
}
// B fragments where tile rows are the k index and columns the n index (transposed load):
// b[0],b[1] -> n-tile n0 ; b[2],b[3] -> n-tile n0+8
template <int DH>
__device__ __forceinline__ void frag_bt(uint32_t* b, uint32_t tile, int k0, int n0) {
  const int l = threadIdx.x & 31;
  ldsm_x4_t(b, tile + sw<DH>(k0 + (l & 7) + ((l >> 3) & 1) * 8, (n0 >> 3) + (l >> 4)));
}

// acc[8][4] (16 x 64) = X[rows row_base..+16, :] . Y^T with X, Y swizzled [64][DH] tiles
template <int DH>
__device__ __forceinline__ void mm_xyT(float (*acc)[4], uint32_t X, int row_base, uint32_t Y) {
#pragma unroll
  for (int k0 = 0; k0 < DH; k0 += 16) {
    uint32_t a[4];
    frag_a<DH>(a, X, row_base, k0);
#pragma unroll
    for (int n0 = 0; n0 < BT; n0 += 16) {
      uint32_t b[4];
      frag_b<DH>(b, Y, n0, k0);
      mma16816(acc[n0 / 8], a, b[0], b[1]);
      mma16816(acc[n0 / 8 + 1], a, b[2], b[3]);
    }
  }
}
// out[DH/8][4] (16 x DH) += P (16 x 64, as bf16 A fragments pa[4][4]) . Z with Z a swizzled [64][DH] tile
template <int DH>
__device__ __forceinline__ void mm_pz(float (*out)[4], const uint32_t (*pa)[4], uint32_t Z) {
#pragma unroll
  for (int k0 = 0; k0 < BT; k0 += 16) {
#pragma unroll
    for (int n0 = 0; n0 < DH; n0 += 16) {
      uint32_t b[4];
      frag_bt<DH>(b, Z, k0, n0);
      mma16816(out[n0 / 8], pa[k0 / 16], b[0], b[1]);
      mma16816(out[n0 / 8 + 1], pa[k0 / 16], b[2], b[3]);
    }
  }
}
__device__ __forceinline__ void to_a_frags(uint32_t (*pa)[4], const float (*s)[4]) {
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    pa[j][0] = pack_bf16(s[2 * j][0], s[2 * j][1]);
    pa[j][1] = pack_bf16(s[2 * j][2], s[2 * j][3]);
    pa[j][2] = pack_bf16(s[2 * j + 1][0], s[2 * j + 1][1]);
    pa[j][3] = pack_bf16(s[2 * j + 1][2], s[2 * j + 1][3]);
  }
}

// ------------------------------------------------------------------ forward
template <int DH>
__global__ void __launch_bounds__(NTHREADS)
attn_fwd_mma_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ U, float* __restrict__ lse,
                    int S, int h) {
  extern __shared__ __align__(128) uint8_t sm[];
  constexpr int TILE = BT * DH * 2;
  const uint32_t Qs = smem_u32(sm), Ks = Qs + TILE, Vs = Ks + 2 * TILE;
  const int d = h * DH;
  const int qb = gridDim.x - 1 - blockIdx.x;   // long rows first
  const int head = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int64_t ld = 3 * d;
  const bf16* base = qkv + (int64_t)b * S * ld + head * DH;
  const float c = rsqrtf((float)DH) * LOG2E;

  load_tile<DH>(Qs, base, ld, qb * BT, S);
  load_tile<DH>(Ks, base + d, ld, 0, S);
  load_tile<DH>(Vs, base + 2 * d, ld, 0, S);
  cp_commit();

  float o[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};
  const int row0 = qb * BT + warp * 16 + g;    // this thread's rows: row0 and row0 + 8

  for (int kb = 0; kb <= qb; ++kb) {
    const int cur = kb & 1;
    if (kb < qb) {
      load_tile<DH>(Ks + (cur ^ 1) * TILE, base + d, ld, (kb + 1) * BT, S);
      load_tile<DH>(Vs + (cur ^ 1) * TILE, base + 2 * d, ld, (kb + 1) * BT, S);
      cp_commit();
      cp_wait<1>();
    } else {
      cp_wait<0>();
    }
    __syncthreads();
    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
    mm_xyT<DH>(s, Qs, warp * 16, Ks + cur * TILE);
    // scale into the log2 domain, mask, row maxima
    float mx[2] = {mrow[0], mrow[1]};
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int col = kb * BT + i * 8 + 2 * t + (e & 1);
        const int row = row0 + (e >> 1) * 8;
        float v = s[i][e] * c;
        if (col > row || col >= S) v = -INFINITY;
        s[i][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
    }
    float corr[2], sum[2] = {0.f, 0.f};
#pragma unroll
    for (int r = 0; r < 2; ++r) corr[r] = ex2(mrow[r] - mx[r]);
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float p = ex2(s[i][e] - mx[e >> 1]);
        s[i][e] = p;
        sum[e >> 1] += p;
      }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      lrow[r] = lrow[r] * corr[r] + sum[r];   // per-thread partial; combined across the quad at the end
      mrow[r] = mx[r];
    }
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      o[i][0] *= corr[0]; o[i][1] *= corr[0]; o[i][2] *= corr[1]; o[i][3] *= corr[1];
    }
    uint32_t pa[4][4];
    to_a_frags(pa, s);
    mm_pz<DH>(o, pa, Vs + cur * TILE);
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int row = row0 + r * 8;
    if (row >= S) continue;
    const float inv = 1.f / lrow[r];
    bf16* out = U + ((int64_t)b * S + row) * d + head * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i)
      *reinterpret_cast<uint32_t*>(out + i * 8 + 2 * t) = pack_bf16(o[i][2 * r] * inv, o[i][2 * r + 1] * inv);
    if (t == 0) lse[((int64_t)b * h + head) * S + row] = (mrow[r] + log2f(lrow[r])) * (1.f / LOG2E);
  }
}

// ------------------------------------------------------------------ backward: delta
__global__ void attn_delta_kernel(const bf16* __restrict__ U, const bf16* __restrict__ dU,
                                  float* __restrict__ delta, int S, int h, int dh, int64_t rows) {
  // one warp per (token, head)
  const int64_t w = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= rows * h) return;
  const int64_t tok = w / h;
  const int head = (int)(w % h);
  const bf16* u = U + tok * (int64_t)h * dh + head * dh;
  const bf16* g = dU + tok * (int64_t)h * dh + head * dh;
  float s = 0.f;
  for (int e = lane * 2; e < dh; e += 64) {
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(u + e));
    const float2 bq = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(g + e));
    s += a.x * bq.x + a.y * bq.y;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) {
    const int64_t bb = tok / S;
    const int sidx = (int)(tok % S);
    delta[(bb * h + head) * S + sidx] = s;
  }
}

// ------------------------------------------------------------------ backward: dq (owns a query block)
template <int DH>
__global__ void __launch_bounds__(NTHREADS)
attn_bwd_dq_mma_kernel(const bf16* __restrict__ qkv, const float* __restrict__ lse,
                       const bf16* __restrict__ dU, const float* __restrict__ delta,
                       bf16* __restrict__ dqkv, int S, int h) {
  extern __shared__ __align__(128) uint8_t sm[];
  constexpr int TILE = BT * DH * 2;
  const uint32_t Qs = smem_u32(sm), Gs = Qs + TILE, Ks = Gs + TILE, Vs = Ks + 2 * TILE;
  const int d = h * DH;
  const int qb = gridDim.x - 1 - blockIdx.x;
  const int head = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int64_t ld = 3 * d;
  const bf16* base = qkv + (int64_t)b * S * ld + head * DH;
  const float scale = rsqrtf((float)DH), c = scale * LOG2E;

  load_tile<DH>(Qs, base, ld, qb * BT, S);
  load_tile<DH>(Gs, dU + (int64_t)b * S * d + head * DH, d, qb * BT, S);
  load_tile<DH>(Ks, base + d, ld, 0, S);
  load_tile<DH>(Vs, base + 2 * d, ld, 0, S);
  cp_commit();

  const int row0 = qb * BT + warp * 16 + g;
  float l2[2], dl[2];
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int row = row0 + r * 8;
    const int64_t si = ((int64_t)b * h + head) * S + (row < S ? row : S - 1);
    l2[r] = lse[si] * LOG2E;
    dl[r] = delta[si];
  }
  float dq[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) { dq[i][0] = dq[i][1] = dq[i][2] = dq[i][3] = 0.f; }

  for (int kb = 0; kb <= qb; ++kb) {
    const int cur = kb & 1;
    if (kb < qb) {
      load_tile<DH>(Ks + (cur ^ 1) * TILE, base + d, ld, (kb + 1) * BT, S);
      load_tile<DH>(Vs + (cur ^ 1) * TILE, base + 2 * d, ld, (kb + 1) * BT, S);
      cp_commit();
      cp_wait<1>();
    } else {
      cp_wait<0>();
    }
    __syncthreads();
    float s[8][4], dp[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
      dp[i][0] = dp[i][1] = dp[i][2] = dp[i][3] = 0.f;
    }
    mm_xyT<DH>(s, Qs, warp * 16, Ks + cur * TILE);
    mm_xyT<DH>(dp, Gs, warp * 16, Vs + cur * TILE);
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int col = kb * BT + i * 8 + 2 * t + (e & 1);
        const int row = row0 + (e >> 1) * 8;
        const float p = (col > row || col >= S) ? 0.f : ex2(s[i][e] * c - l2[e >> 1]);
        s[i][e] = p * (dp[i][e] - dl[e >> 1]);
      }
    uint32_t pa[4][4];
    to_a_frags(pa, s);
    mm_pz<DH>(dq, pa, Ks + cur * TILE);
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int row = row0 + r * 8;
    if (row >= S) continue;
    bf16* out = dqkv + ((int64_t)b * S + row) * ld + head * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i)
      *reinterpret_cast<uint32_t*>(out + i * 8 + 2 * t) =
          pack_bf16(dq[i][2 * r] * scale, dq[i][2 * r + 1] * scale);
  }
}

// ------------------------------------------------------------------ backward: dk, dv (owns a key block)
template <int DH>
__global__ void __launch_bounds__(NTHREADS)
attn_bwd_dkv_mma_kernel(const bf16* __restrict__ qkv, const float* __restrict__ lse,
                        const bf16* __restrict__ dU, const float* __restrict__ delta,
                        bf16* __restrict__ dqkv, int S, int h) {
  extern __shared__ __align__(128) uint8_t sm[];
  constexpr int TILE = BT * DH * 2;
  const uint32_t Ks = smem_u32(sm), Vs = Ks + TILE, Qs = Vs + TILE, Gs = Qs + 2 * TILE;
  const uint32_t Ls = Gs + 2 * TILE, Ds = Ls + 2 * BT * 4;
  const float* Lsp = reinterpret_cast<const float*>(sm + 6 * TILE);
  const float* Dsp = Lsp + 2 * BT;
  const int d = h * DH;
  const int kb = blockIdx.x;                    // early key blocks have the most work and start first
  const int head = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int64_t ld = 3 * d;
  const bf16* base = qkv + (int64_t)b * S * ld + head * DH;
  const bf16* gbase = dU + (int64_t)b * S * d + head * DH;
  const float* lbase = lse + ((int64_t)b * h + head) * S;
  const float* dbase = delta + ((int64_t)b * h + head) * S;
  const float scale = rsqrtf((float)DH), c = scale * LOG2E;
  const int nqb = (S + BT - 1) / BT;

  load_tile<DH>(Ks, base + d, ld, kb * BT, S);
  load_tile<DH>(Vs, base + 2 * d, ld, kb * BT, S);
  load_tile<DH>(Qs, base, ld, kb * BT, S);
  load_tile<DH>(Gs, gbase, d, kb * BT, S);
  load_vec64(Ls, lbase, kb * BT, S);
  load_vec64(Ds, dbase, kb * BT, S);
  cp_commit();

  const int key0 = kb * BT + warp * 16 + g;     // this thread's keys: key0 and key0 + 8
  float dk[DH / 8][4], dv[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) {
    dk[i][0] = dk[i][1] = dk[i][2] = dk[i][3] = 0.f;
    dv[i][0] = dv[i][1] = dv[i][2] = dv[i][3] = 0.f;
  }
  for (int qb = kb; qb < nqb; ++qb) {
    const int cur = (qb - kb) & 1;
    if (qb + 1 < nqb) {
      load_tile<DH>(Qs + (cur ^ 1) * TILE, base, ld, (qb + 1) * BT, S);
      load_tile<DH>(Gs + (cur ^ 1) * TILE, gbase, d, (qb + 1) * BT, S);
      load_vec64(Ls + (cur ^ 1) * BT * 4, lbase, (qb + 1) * BT, S);
      load_vec64(Ds + (cur ^ 1) * BT * 4, dbase, (qb + 1) * BT, S);
      cp_commit();
      cp_wait<1>();
    } else {
      cp_wait<0>();
    }
    __syncthreads();
    float s[8][4], dp[8][4];   // transposed: rows = keys, columns = queries
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
      dp[i][0] = dp[i][1] = dp[i][2] = dp[i][3] = 0.f;
    }
    mm_xyT<DH>(s, Ks, warp * 16, Qs + cur * TILE);
    mm_xyT<DH>(dp, Vs, warp * 16, Gs + cur * TILE);
    float ds[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int qi = i * 8 + 2 * t + (e & 1);
        const int q = qb * BT + qi;
        const int key = key0 + (e >> 1) * 8;
        const float p = (key > q || q >= S) ? 0.f : ex2(s[i][e] * c - Lsp[cur * BT + qi] * LOG2E);
        s[i][e] = p;
        ds[i][e] = p * (dp[i][e] - Dsp[cur * BT + qi]);
      }
    uint32_t pa[4][4];
    to_a_frags(pa, s);
    mm_pz<DH>(dv, pa, Gs + cur * TILE);
    to_a_frags(pa, ds);
    mm_pz<DH>(dk, pa, Qs + cur * TILE);
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int key = key0 + r * 8;
    if (key >= S) continue;
    bf16* out = dqkv + ((int64_t)b * S + key) * ld + head * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      *reinterpret_cast<uint32_t*>(out + d + i * 8 + 2 * t) =
          pack_bf16(dk[i][2 * r] * scale, dk[i][2 * r + 1] * scale);
      *reinterpret_cast<uint32_t*>(out + 2 * d + i * 8 + 2 * t) =
          pack_bf16(dv[i][2 * r], dv[i][2 * r + 1]);
    }
  }
}

template <typename K>
bool set_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

}  // namespace

void launch_attn_delta(const bf16* U, const bf16* dU, float* delta, int B, int S, int h, int dh,
                       cudaStream_t st) {
  const int64_t rows = (int64_t)B * S;
  const int64_t warps = rows * h;
  attn_delta_kernel<<<(unsigned)((warps * 32 + 255) / 256), 256, 0, st>>>(U, dU, delta, S, h, dh, rows);
}

bool attn_mma_supported(int S, int dh) { return (dh == 64 || dh == 128) && S >= 1; }

int launch_attn_fwd_mma(const bf16* qkv, bf16* U, float* lse, int B, int S, int h, int dh,
                        cudaStream_t st) {
  dim3 grid((S + BT - 1) / BT, h, B);
  if (dh == 64) {
    constexpr int SM = 5 * BT * 64 * 2;
    static bool ok = set_smem(attn_fwd_mma_kernel<64>, SM);
    if (!ok) return -2;
    attn_fwd_mma_kernel<64><<<grid, NTHREADS, SM, st>>>(qkv, U, lse, S, h);
  } else if (dh == 128) {
    constexpr int SM = 5 * BT * 128 * 2;
    static bool ok = set_smem(attn_fwd_mma_kernel<128>, SM);
    if (!ok) return -2;
    attn_fwd_mma_kernel<128><<<grid, NTHREADS, SM, st>>>(qkv, U, lse, S, h);
  } else {
    return -1;
  }
  return 0;
}

int launch_attn_bwd_mma(const bf16* qkv, const bf16* U, const float* lse, const bf16* dU,
                        bf16* dqkv, float* scratch, int B, int S, int h, int dh, cudaStream_t st) {
  launch_attn_delta(U, dU, scratch, B, S, h, dh, st);
  dim3 grid((S + BT - 1) / BT, h, B);
  if (dh == 64) {
    constexpr int SM = 6 * BT * 64 * 2 + 4 * BT * 4;
    static bool ok = set_smem(attn_bwd_dq_mma_kernel<64>, SM) && set_smem(attn_bwd_dkv_mma_kernel<64>, SM);
    if (!ok) return -2;
    attn_bwd_dq_mma_kernel<64><<<grid, NTHREADS, SM, st>>>(qkv, lse, dU, scratch, dqkv, S, h);
    attn_bwd_dkv_mma_kernel<64><<<grid, NTHREADS, SM, st>>>(qkv, lse, dU, scratch, dqkv, S, h);
  } else if (dh == 128) {
    constexpr int SM = 6 * BT * 128 * 2 + 4 * BT * 4;
    static bool ok = set_smem(attn_bwd_dq_mma_kernel<128>, SM) && set_smem(attn_bwd_dkv_mma_kernel<128>, SM);
    if (!ok) return -2;
    attn_bwd_dq_mma_kernel<128><<<grid, NTHREADS, SM, st>>>(qkv, lse, dU, scratch, dqkv, S, h);
    attn_bwd_dkv_mma_kernel<128><<<grid, NTHREADS, SM, st>>>(qkv, lse, dU, scratch, dqkv, S, h);
  } else {
    return -1;
  }
  return 0;
}
