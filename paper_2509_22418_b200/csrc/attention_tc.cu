// Fused causal attention on the 5th-generation tensor cores (tcgen05.mma, accumulators in
// tensor memory, operands brought in by TMA), head sizes 64 and 128.
//
//   forward   128 queries per work item; per 128-key block S = Q K^T lands in TMEM, two groups of
//             128 softmax threads (one query row each, half of the block's key columns per
//             group, so row maxima and sums need no shuffles) turn it into bf16 probabilities
//             written back to TMEM over the scores, and P V (A operand from TMEM) accumulates in
//             TMEM, one accumulator per group, with lazy online-softmax rescaling; the two
//             partial softmaxes are merged at the end.
//   dq        128 queries per work item, 128-key slabs; S = Q K^T and dP = dU V^T in TMEM, the
//             threads form dS = P (dP - delta) and write it back to TMEM as bf16, from where it is
//             the A operand of dQ += dS K, which accumulates in TMEM over all slabs (no rescaling
//             is needed in the backward).
//   dk, dv    128 keys per work item, 128-query slabs; the transposed products S^T = K Q^T,
//             dP^T = V dU^T; P^T and dS^T overwrite them in TMEM as bf16 and feed dV += P^T dU and
//             dK += dS^T Q, which accumulate in TMEM.
// All three kernels are persistent: one CTA per SM walks a balanced list of (sequence, head,
// query or key block) items, so set-up, the first loads and the output drain of an item overlap
// with the products of its neighbours.
// The two backward kernels recompute P from q, k and the saved log-sum-exp; nothing is
// accumulated with atomics, so results are bitwise reproducible.  (Appendix C.1, MHA.)
//
// Warp roles: warp 0 issues TMA, warp 1 issues MMAs and owns the TMEM allocation, warps 2-5 and
// 6-9 are two groups of 128 row threads; every kernel has a second MMA-issuing
// thread in warp 10 (a thread that issues tcgen05.mma stalls while the tensor pipe is busy, so
// one thread alone would serialise its barrier waits with the products).  Every mbarrier wait is
// bounded; on expiry the CTA raises an abort flag, all roles fall through to the common exit,
// TMEM is released and an error word is set.
#include "tc_common.cuh"

namespace {
using namespace tc;

// backward kernels: warp 0 TMA, warp 1 first MMA-issuing thread, warps 2-5 and 6-9 two row groups (half
// the slab columns each), warp 10 second MMA-issuing thread
constexpr int DQ_THREADS = 352;
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}
// 32 consecutive head columns starting at c0, scaled by f and (optionally) rotated back by the
// position's angle, packed to bf16 and stored
__device__ __forceinline__ void drain32(bf16* out, const uint32_t* r, float f, const float2* cs_row, int c0) {
  float v[32];
#pragma unroll
  for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(r[e]) * f;
  if (cs_row) {
    // the chunk's 16 (cos, sin) pairs are 128 contiguous, 128-byte aligned bytes of the table
    const float4* w4 = reinterpret_cast<const float4*>(cs_row + c0 / 2);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float4 w = __ldg(w4 + q);
      const float a0 = v[4 * q], b0 = v[4 * q + 1], a1 = v[4 * q + 2], b1 = v[4 * q + 3];
      v[4 * q] = a0 * w.x + b0 * w.y;
      v[4 * q + 1] = b0 * w.x - a0 * w.y;
      v[4 * q + 2] = a1 * w.z + b1 * w.w;
      v[4 * q + 3] = b1 * w.z - a1 * w.w;
    }
  }
#pragma unroll
  for (int e = 0; e < 32; e += 8) {
    uint4 u;
    u.x = pack2(v[e], v[e + 1]); u.y = pack2(v[e + 2], v[e + 3]);
    u.z = pack2(v[e + 4], v[e + 5]); u.w = pack2(v[e + 6], v[e + 7]);
    *reinterpret_cast<uint4*>(out + e) = u;
  }
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// 16-byte chunk `idx` (8 bf16) of row `row` in a K-major operand made of [rows x 64] swizzled
// half-tiles that are `half_bytes` apart
__device__ __forceinline__ uint32_t op_chunk(uint32_t base, uint32_t half_bytes, int row, int idx) {
  return base + (uint32_t)(idx >> 3) * half_bytes + (uint32_t)row * 128u + (uint32_t)(((idx & 7) ^ (row & 7)) << 4);
}
// 32 fp32 values -> 32 bf16 -> four 16-byte chunks starting at chunk index idx0
__device__ __forceinline__ void store_row32(uint32_t base, uint32_t half_bytes, int row, int idx0, const float* v) {
#pragma unroll
  for (int q = 0; q < 4; ++q)
    st_shared_v4(op_chunk(base, half_bytes, row, idx0 + q), pack2(v[8 * q], v[8 * q + 1]),
                 pack2(v[8 * q + 2], v[8 * q + 3]), pack2(v[8 * q + 4], v[8 * q + 5]),
                 pack2(v[8 * q + 6], v[8 * q + 7]));
}

// One arrival per warp: 128 single-thread arrivals on one mbarrier serialise in shared memory
// and cost more than the arithmetic between them.  __syncwarp orders the lanes' earlier
// accesses before lane 0's releasing arrive.
__device__ __forceinline__ void warp_arrive(uint32_t bar) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}

struct AttnParams {
  const float* lse; const float* delta;
  bf16* U; float* lse_out; bf16* dqkv;
  int S, h, B; int* flags;
  const float2* inv_rope;   // (cos, sin) table [S][d_h/2]: rotate dq, dk by -angle on the way out (or null)
};

// A [ROWS x DH] K-major operand tile: DH/64 half-tiles of ROWS*128 bytes.  K-step ks (16 columns).
template <int ROWS>
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t tile, int ks) {
  return make_desc(tile + (uint32_t)(ks >> 2) * (ROWS * 128u) + (uint32_t)(ks & 3) * 32u, 16, 1024);
}
// The same tile read as an MN-major B operand (rows are the reduction index): step ks = 16 rows.
template <int ROWS>
__device__ __forceinline__ uint64_t mnmajor_desc(uint32_t tile, int ks) {
  return make_desc(tile + (uint32_t)ks * 2048u, ROWS * 128u, 1024);
}
// Lean MMA issue: the issuing thread is the critical resource here (each K=16 step of a
// 64-column product is only 32 tensor cycles), so descriptors are kept as a precomputed low word
// plus compile-time step offsets, and the constant high word (SBO 1024 B, version 1, 128-byte
// swizzle) is shared.
constexpr uint32_t DESC_HI = 64u | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t klo(uint32_t tile) { return ((tile >> 4) & 0x3FFFu) | (1u << 16); }
template <int ROWS>
__device__ __forceinline__ uint32_t mlo(uint32_t tile) { return ((tile >> 4) & 0x3FFFu) | ((uint32_t)(ROWS * 8) << 16); }
template <int ROWS> __host__ __device__ constexpr uint32_t kstep(int ks) { return (uint32_t)((ks >> 2) * ROWS * 8 + (ks & 3) * 2); }
__host__ __device__ constexpr uint32_t mstep(int ks) { return (uint32_t)(ks * 128); }
__device__ __forceinline__ void umma_lo(uint32_t tmem_d, uint32_t alo, uint32_t blo, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n.reg .pred p;\n.reg .b64 da, db;\nsetp.ne.b32 p, %4, 0;\n"
      "mov.b64 da, {%1, %5};\nmov.b64 db, {%2, %5};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n}" ::"r"(tmem_d),
      "r"(alo), "r"(blo), "r"(idesc), "r"(acc), "r"(DESC_HI)
      : "memory");
}
__device__ __forceinline__ uint8_t* align1k(uint8_t* p) {
  return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~(uintptr_t)1023);
}

// ------------------------------------------------------------------ forward
// A work item is 128 queries, walked in 128-key blocks.  S = Q K^T of block j+1 is issued into the second TMEM
// buffer while the row threads work on block j.  Two groups of 128 row threads share a block by
// key columns: group g owns columns [64g, 64g+64) of every block, keeps its own softmax
// reference and row sum, writes its bf16 probabilities back into tensor memory over the first
// half of the scores they came from, and its half of P V (A operand straight from tensor memory,
// two K=64 products per block) accumulates in its own accumulator O_g.  At the end the two
// partial softmaxes are merged exactly: with m = max(m_A, m_B),
// O = (2^(m_A-m) O_A + 2^(m_B-m) O_B) / (2^(m_A-m) l_A + 2^(m_B-m) l_B).
// A reference is only raised when a row's block maximum exceeds it by more than 2^8 (stored
// probabilities then stay below 256); raising it rescales that group's rows of O_g in TMEM.
// Two threads issue the products (one S, one P V): an issuing thread stalls while the tensor
// pipe is busy, so with a single one every barrier wait would serialise with the products.
constexpr float RESCALE_LOG2 = 8.f;
constexpr int FWD_THREADS = 352;   // warp 0 TMA, warp 1 S products, warps 2-5 group A, warps 6-9 group B, warp 10 P V products

// A operand from tensor memory (bf16 pairs, one row per lane), B from shared memory
__device__ __forceinline__ void umma_ts_lo(uint32_t tmem_d, uint32_t tmem_a, uint32_t blo, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n.reg .pred p;\n.reg .b64 db;\nsetp.ne.b32 p, %4, 0;\n"
      "mov.b64 db, {%2, %5};\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n}" ::"r"(tmem_d),
      "r"(tmem_a), "r"(blo), "r"(idesc), "r"(acc), "r"(DESC_HI)
      : "memory");
}

// Work items (128 queries of one head of one sequence) are ordered heavy first - the last query
// block of every (sequence, head), then the one before, ... - and dealt to the resident CTAs in
// boustrophedon order, so every CTA gets a near-equal number of key blocks.  A CTA walks its items
// without leaving: barriers, tensor memory and the K/V rings carry over, and the next item's Q
// and first K/V tiles arrive while the current item's last blocks and its output drain.
struct WorkItem { int qb, head, b; };
__device__ __forceinline__ bool work_item(int k, int n_batch, int h, int nq, WorkItem& w) {
  const int G = gridDim.x, cta = blockIdx.x;
  const int t = k * G + ((k & 1) ? (G - 1 - cta) : cta);
  const int hb = h * n_batch;
  if (t >= nq * hb) return false;
  w.qb = nq - 1 - t / hb;
  const int rem = t % hb;
  w.head = rem % h; w.b = rem / h;
  return true;
}

constexpr int FWD_ALIGN_SLACK = 768;   // the full 1 KB would put the 128-wide head over the 227 KB limit
template <int DH>
__global__ void __launch_bounds__(FWD_THREADS, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap mapQKV, const AttnParams p) {
  constexpr int NH = DH / 64, QT = 128 * DH * 2, NS = 3;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align1k(smem_raw);
  const uint32_t Qs = smem_u32(smem), Ks = Qs + QT, Vs = Ks + NS * QT;
  float2* exch = reinterpret_cast<float2*>(smem + (1 + 2 * NS) * QT);   // (reference, sum) of each row and group
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (1 + 2 * NS) * QT + 2 * 128 * 8);
  // P_FULL is indexed [group * 2 + buffer], PV_DONE by group
  enum { Q_FULL = 0, Q_EMPTY, K_FULL, K_EMPTY = K_FULL + NS, V_FULL = K_EMPTY + NS, V_EMPTY = V_FULL + NS,
         S_FULL = V_EMPTY + NS, S_EMPTY = S_FULL + 2, P_FULL = S_EMPTY + 2, PV_DONE = P_FULL + 4,
         ALL_DONE = PV_DONE + 2, MERGE, O_EMPTY, NBAR };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NBAR);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto B = [&](int i) { return bar0 + 8u * i; };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int d = p.h * DH, S = p.S, nq = (S + 127) / 128;
  // the launch provides FWD_ALIGN_SLACK bytes for the 1 KB alignment of the tiles
  if (smem - smem_raw > FWD_ALIGN_SLACK) {
    if (threadIdx.x == 0 && p.flags) atomicExch(p.flags + PPU_FLAG_TIMEOUT, 1);
    return;
  }

  if (threadIdx.x == 0) {
    for (int i = 0; i < NBAR; ++i) mbar_init(B(i), 1);
    for (int i = 0; i < 4; ++i) mbar_init(B(P_FULL + i), 4);
    mbar_init(B(MERGE), 8);
    mbar_init(B(O_EMPTY), 8);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tS = tmem, tO = tmem + 256;   // S buffer s at tS + 128 s; O_g at tO + g * DH
  // c counts the key blocks this CTA has gone through (every role keeps its own copy): it selects
  // ring stages, score buffers and barrier phases across items

  if (warp == 0) {
    if (lane == 0) {
      WorkItem w; uint32_t c = 0; bool ok = true;
      for (int k = 0; ok && work_item(k, p.B, p.h, nq, w); ++k) {
        // the Q tile is free once the previous item's last S product is done
        if (k > 0 && !mbar_wait(B(Q_EMPTY), (uint32_t)(k - 1) & 1u, abort_flag, p.flags)) break;
        mbar_expect_tx(B(Q_FULL), QT);
        for (int hf = 0; hf < NH; ++hf)
          tma_load_3d(Qs + hf * 16384, &mapQKV, B(Q_FULL), w.head * DH + hf * 64, w.qb * 128, w.b);
        for (int j = 0; j <= w.qb; ++j, ++c) {
          const int st = c % NS; const uint32_t ph = (c / NS) & 1;
          if (!mbar_wait(B(K_EMPTY + st), ph ^ 1u, abort_flag, p.flags)) { ok = false; break; }
          mbar_expect_tx(B(K_FULL + st), QT);
          for (int hf = 0; hf < NH; ++hf)
            tma_load_3d(Ks + st * QT + hf * 16384, &mapQKV, B(K_FULL + st), d + w.head * DH + hf * 64, j * 128, w.b);
          if (!mbar_wait(B(V_EMPTY + st), ph ^ 1u, abort_flag, p.flags)) { ok = false; break; }
          mbar_expect_tx(B(V_FULL + st), QT);
          for (int hf = 0; hf < NH; ++hf)
            tma_load_3d(Vs + st * QT + hf * 16384, &mapQKV, B(V_FULL + st), 2 * d + w.head * DH + hf * 64, j * 128, w.b);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc(128, 128, false, false);
      const uint32_t q_lo = klo(Qs);
      WorkItem w; uint32_t c = 0; bool ok = true;
      for (int k = 0; ok && work_item(k, p.B, p.h, nq, w); ++k) {
        if (!mbar_wait(B(Q_FULL), (uint32_t)k & 1u, abort_flag, p.flags)) break;
        for (int j = 0; j <= w.qb; ++j, ++c) {
          const int st = c % NS, sb = c & 1;
          if (!mbar_wait(B(K_FULL + st), (c / NS) & 1, abort_flag, p.flags)) { ok = false; break; }
          // buffer sb still holds the probabilities of two blocks ago until their P V products are done
          if (!mbar_wait(B(S_EMPTY + sb), ((c >> 1) & 1) ^ 1u, abort_flag, p.flags)) { ok = false; break; }
          tc_fence_after();
          const uint32_t k_lo = klo(Ks + st * QT);
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks)
            umma_lo(tS + sb * 128, q_lo + kstep<128>(ks), k_lo + kstep<128>(ks), idesc_s, ks > 0);
          umma_commit(B(S_FULL + sb));
          umma_commit(B(K_EMPTY + st));
        }
        if (ok) umma_commit(B(Q_EMPTY));
      }
    }
  } else if (warp == 10) {
    if (lane == 0) {
      constexpr uint32_t idesc_o = make_idesc(128, DH, false, true);
      WorkItem w; uint32_t c = 0; bool ok = true;
      for (int k = 0; ok && work_item(k, p.B, p.h, nq, w); ++k) {
        // the accumulators are free once the row threads have drained the previous item's output
        if (k > 0 && !mbar_wait(B(O_EMPTY), (uint32_t)(k - 1) & 1u, abort_flag, p.flags)) break;
        for (int j = 0; j <= w.qb && ok; ++j, ++c) {
          const int st = c % NS, sb = c & 1; const uint32_t ph = (c >> 1) & 1;
          const uint32_t v_lo = mlo<128>(Vs + st * QT);
          if (!mbar_wait(B(V_FULL + st), (c / NS) & 1, abort_flag, p.flags)) { ok = false; break; }
#pragma unroll
          for (int g = 0; g < 2; ++g) {
            if (!mbar_wait(B(P_FULL + g * 2 + sb), ph, abort_flag, p.flags)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              umma_ts_lo(tO + g * DH, tS + sb * 128 + 64 * g + 8 * ks, v_lo + mstep(4 * g + ks), idesc_o,
                         (j > 0 || ks > 0));
            umma_commit(B(PV_DONE + g));
          }
          if (!ok) break;
          umma_commit(B(S_EMPTY + sb));
          umma_commit(B(V_EMPTY + st));
        }
        if (ok) umma_commit(B(ALL_DONE));
      }
    }
  } else {
    const int g = (warp - 2) >> 2;                // column group
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may access
    const int row = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const uint32_t tOg = tO + g * DH + lane_off;
    const float c = rsqrtf((float)DH) * LOG2E;
    WorkItem w; uint32_t cb = 0; bool ok = true;
    for (int k = 0; ok && work_item(k, p.B, p.h, nq, w); ++k) {
      const int qb = w.qb, grow = qb * 128 + row;
      float m_ref = -INFINITY, l = 0.f;
      for (int j = 0; j <= qb && ok; ++j, ++cb) {
        const int sb = cb & 1; const uint32_t ph = (cb >> 1) & 1;
        const uint32_t tSg = tS + lane_off + sb * 128 + g * 64;
        if (!mbar_wait(B(S_FULL + sb), ph, abort_flag, p.flags)) { ok = false; break; }
        tc_fence_after();
        uint32_t r[64];
        tmem_ld32(tSg, r);
        tmem_ld32(tSg + 32, r + 32);
        tmem_ld_wait();
        const int col0 = j * 128 + g * 64;
        const bool diag = (j == qb) || ((j + 1) * 128 > S);
        // eight independent partial maxima / sums: a single warp per scheduler cannot hide the
        // latency of one long dependent chain
        float mx8[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) mx8[q] = -INFINITY;
        if (!diag) {
#pragma unroll
          for (int e = 0; e < 64; ++e) mx8[e & 7] = fmaxf(mx8[e & 7], __uint_as_float(r[e]));
        } else {
#pragma unroll
          for (int e = 0; e < 64; ++e) {
            const int col = col0 + e;
            if (col <= grow && col < S) mx8[e & 7] = fmaxf(mx8[e & 7], __uint_as_float(r[e]));
          }
        }
        const float mx = fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])),
                               fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
        const float m_blk = mx * c;
        const bool need = m_blk > m_ref + RESCALE_LOG2;
        if (__any_sync(0xffffffffu, need)) {
          const float new_ref = need ? m_blk : m_ref;
          const float factor = need ? ex2(m_ref - new_ref) : 1.f;
          if (j > 0) {
            // O_g must be complete up to the previous block before its rows are rescaled in place
            if (!mbar_wait(B(PV_DONE + g), (cb - 1) & 1u, abort_flag, p.flags)) { ok = false; break; }
            tc_fence_after();
#pragma unroll 1
            for (int cc = 0; cc < DH / 32; ++cc) {
              uint32_t o[32];
              tmem_ld32(tOg + cc * 32, o);
              tmem_ld_wait();
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * factor);
              tmem_st32(tOg + cc * 32, o);
            }
          }
          l *= factor;
          m_ref = new_ref;
        }
        float sum8[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) sum8[q] = 0.f;
        // a group whose columns are all masked so far still has m_ref = -inf; the selects below
        // discard whatever the exponential made of that
        if (!diag) {
#pragma unroll
          for (int e = 0; e < 64; e += 2) {
            const float p0 = ex2(fmaf(__uint_as_float(r[e]), c, -m_ref));
            const float p1 = ex2(fmaf(__uint_as_float(r[e + 1]), c, -m_ref));
            sum8[e & 7] += p0; sum8[(e + 1) & 7] += p1;
            r[e >> 1] = pack2(p0, p1);
          }
        } else {
#pragma unroll
          for (int e = 0; e < 64; e += 2) {
            const int col = col0 + e;
            float p0 = ex2(fmaf(__uint_as_float(r[e]), c, -m_ref));
            float p1 = ex2(fmaf(__uint_as_float(r[e + 1]), c, -m_ref));
            if (col > grow || col >= S) p0 = 0.f;
            if (col + 1 > grow || col + 1 >= S) p1 = 0.f;
            sum8[e & 7] += p0; sum8[(e + 1) & 7] += p1;
            r[e >> 1] = pack2(p0, p1);
          }
        }
        l += ((sum8[0] + sum8[1]) + (sum8[2] + sum8[3])) + ((sum8[4] + sum8[5]) + (sum8[6] + sum8[7]));
        // the probabilities replace the first half of this thread's own scores
        tmem_st32(tSg, r);
        tmem_st_wait();
        tc_fence_before();
        warp_arrive(B(P_FULL + g * 2 + sb));
      }
      if (!ok) break;
      // the item's last P V product is done: merge the two partial softmaxes and write the output
      const uint32_t kp = (uint32_t)k & 1u;
      if (!mbar_wait(B(ALL_DONE), kp, abort_flag, p.flags)) { ok = false; break; }
      tc_fence_after();
      exch[g * 128 + row] = make_float2(m_ref, l);
      warp_arrive(B(MERGE));
      if (!mbar_wait(B(MERGE), kp, abort_flag, p.flags)) { ok = false; break; }
      {
        const float2 other = exch[(g ^ 1) * 128 + row];
        const float m = fmaxf(m_ref, other.x);
        // group A always has a finite reference (key 0 is visible to every query), so m is finite
        const float w_own = ex2(m_ref - m), w_oth = ex2(other.x - m);
        const float l_tot = w_own * l + w_oth * other.y;
        const float inv = 1.f / l_tot;
        const float fa = (g == 0 ? w_own : w_oth) * inv, fb = (g == 0 ? w_oth : w_own) * inv;
        bf16* out = p.U + ((int64_t)w.b * S + grow) * d + w.head * DH;
        // each group writes half of the head's columns
#pragma unroll 1
        for (int cc = g * (DH / 64); cc < (g + 1) * (DH / 64); ++cc) {
          uint32_t oa[32], ob[32];
          tmem_ld32(tO + lane_off + cc * 32, oa);
          tmem_ld32(tO + DH + lane_off + cc * 32, ob);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e)
            oa[e] = __float_as_uint(__uint_as_float(oa[e]) * fa + __uint_as_float(ob[e]) * fb);
          if (grow < S) drain32(out + cc * 32, oa, 1.f, nullptr, 0);
        }
        if (g == 0 && grow < S)
          p.lse_out[((int64_t)w.b * p.h + w.head) * S + grow] = (m + log2f(l_tot)) * (1.f / LOG2E);
      }
      // both accumulators have been read: the next item's P V products may overwrite them (this
      // arrival also orders this thread's reads of the exchange buffer before the next item's writes)
      tc_fence_before();
      warp_arrive(B(O_EMPTY));
    }
  }
  if (*abort_flag) for (int i = 0; i < 64; ++i) __nanosleep(2000);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

// ------------------------------------------------------------------ backward: dq
// A work item owns 128 queries (Q and dU tiles resident) and streams 128-key slabs of K and V through
// a two-deep TMA ring.  S = Q K^T and dP = dU V^T of a slab land in tensor memory; the 256 row
// threads (one query row each, half of the slab's key columns per group) pull them into
// registers, which frees the two accumulators for the next slab, form dS = P (dP - delta) and
// write it as bf16 into one of two tensor-memory buffers, from where it is the A operand of
// dQ += dS K.  The MMA-issuing thread is the scarce resource of this kernel (its waits, commits
// and instruction issue are latency-bound), hence few, wide instructions: 24 per 128 keys.
template <int DH>
__global__ void __launch_bounds__(DQ_THREADS, 1)
attn_dq_tc_kernel(const __grid_constant__ CUtensorMap mapQKV, const __grid_constant__ CUtensorMap mapG,
                  const AttnParams p) {
  constexpr int NH = DH / 64, QT = 128 * DH * 2, NK = 3, NV = 2;   // K lives until its slab's dQ product, V only until dP
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align1k(smem_raw);
  const uint32_t Qs = smem_u32(smem), Gs = Qs + QT, Kr = Gs + QT, Vr = Kr + NK * QT;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (2 + NK + NV) * QT);
  enum { Q_FULL = 0, QG_EMPTY, K_FULL, V_FULL = K_FULL + NK, K_EMPTY = V_FULL + NV, V_EMPTY = K_EMPTY + NK,
         SDP_FULL = V_EMPTY + NV, SDP_EMPTY, DS_FULL, DS_EMPTY = DS_FULL + 2, DQ_FULL = DS_EMPTY + 2, TQ_EMPTY, NBAR };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NBAR);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto B = [&](int i) { return bar0 + 8u * i; };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int d = p.h * DH, S = p.S, nq = (S + 127) / 128;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NBAR; ++i) mbar_init(B(i), 1);
    mbar_init(B(SDP_EMPTY), 8); mbar_init(B(DS_FULL), 8); mbar_init(B(DS_FULL + 1), 8); mbar_init(B(TQ_EMPTY), 8);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tS = tmem, tP = tmem + 128, tD = tmem + 256, tQ = tmem + 384;   // dS buffer b at tD + 64 b
  // c counts the key slabs this CTA has gone through (every role keeps its own copy)

  if (warp == 0) {
    if (lane == 0) {
      WorkItem w; uint32_t c = 0; bool ok = true;
      for (int k = 0; ok && work_item(k, p.B, p.h, nq, w); ++k) {
        // the Q and dU tiles are free once the previous item's last S / dP products are done
        if (k > 0 && !mbar_wait(B(QG_EMPTY), (uint32_t)(k - 1) & 1u, abort_flag, p.flags)) break;
        mbar_expect_tx(B(Q_FULL), 2 * QT);
        for (int hf = 0; hf < NH; ++hf) {
          tma_load_3d(Qs + hf * 16384, &mapQKV, B(Q_FULL), w.head * DH + hf * 64, w.qb * 128, w.b);
          tma_load_3d(Gs + hf * 16384, &mapG, B(Q_FULL), w.head * DH + hf * 64, w.qb * 128, w.b);
        }
        for (int it = 0; it <= w.qb; ++it, ++c) {
          const int sk = c % NK, sv = c % NV;
          if (!mbar_wait(B(K_EMPTY + sk), ((c / NK) & 1) ^ 1u, abort_flag, p.flags)) { ok = false; break; }
          mbar_expect_tx(B(K_FULL + sk), QT);
          for (int hf = 0; hf < NH; ++hf)
            tma_load_3d(Kr + sk * QT + hf * 16384, &mapQKV, B(K_FULL + sk), d + w.head * DH + hf * 64, it * 128, w.b);
          if (!mbar_wait(B(V_EMPTY + sv), ((c / NV) & 1) ^ 1u, abort_flag, p.flags)) { ok = false; break; }
          mbar_expect_tx(B(V_FULL + sv), QT);
          for (int hf = 0; hf < NH; ++hf)
            tma_load_3d(Vr + sv * QT + hf * 16384, &mapQKV, B(V_FULL + sv), 2 * d + w.head * DH + hf * 64, it * 128, w.b);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc(128, 128, false, false);
      const uint32_t q_lo = klo(Qs), g_lo = klo(Gs);
      WorkItem w; uint32_t c = 0; bool ok = true;
      for (int k = 0; ok && work_item(k, p.B, p.h, nq, w); ++k) {
        if (!mbar_wait(B(Q_FULL), (uint32_t)k & 1u, abort_flag, p.flags)) break;
        for (int it = 0; it <= w.qb; ++it, ++c) {
          const int sk = c % NK, sv = c % NV;
          if (!mbar_wait(B(K_FULL + sk), (c / NK) & 1, abort_flag, p.flags)) { ok = false; break; }
          if (!mbar_wait(B(V_FULL + sv), (c / NV) & 1, abort_flag, p.flags)) { ok = false; break; }
          if (c > 0 && !mbar_wait(B(SDP_EMPTY), (c - 1) & 1u, abort_flag, p.flags)) { ok = false; break; }
          tc_fence_after();
          const uint32_t k_lo = klo(Kr + sk * QT), v_lo = klo(Vr + sv * QT);
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks)
            umma_lo(tS, q_lo + kstep<128>(ks), k_lo + kstep<128>(ks), idesc_s, ks > 0);
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks)
            umma_lo(tP, g_lo + kstep<128>(ks), v_lo + kstep<128>(ks), idesc_s, ks > 0);
          umma_commit(B(SDP_FULL));
          umma_commit(B(V_EMPTY + sv));
        }
        if (ok) umma_commit(B(QG_EMPTY));
      }
    }
  } else if (warp == 10) {
    // second issuing thread: its waits overlap the first thread's instructions and vice versa
    // (an issuing thread stalls while the tensor pipe is busy, so one thread alone would
    // serialise every wait with the products)
    if (lane == 0) {
      constexpr uint32_t idesc_q = make_idesc(128, DH, false, true);
      WorkItem w; uint32_t c = 0; bool ok = true;
      for (int k = 0; ok && work_item(k, p.B, p.h, nq, w); ++k) {
        // the accumulator is free once the row threads have drained the previous item's dQ
        if (k > 0 && !mbar_wait(B(TQ_EMPTY), (uint32_t)(k - 1) & 1u, abort_flag, p.flags)) break;
        for (int it = 0; it <= w.qb; ++it, ++c) {
          const int sk = c % NK, db = c & 1;
          if (!mbar_wait(B(K_FULL + sk), (c / NK) & 1, abort_flag, p.flags)) { ok = false; break; }
          if (!mbar_wait(B(DS_FULL + db), (c >> 1) & 1, abort_flag, p.flags)) { ok = false; break; }
          tc_fence_after();
          const uint32_t kmn_lo = mlo<128>(Kr + sk * QT);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            umma_ts_lo(tQ, tD + 64 * db + 8 * ks, kmn_lo + mstep(ks), idesc_q, (it > 0 || ks > 0));
          umma_commit(B(DS_EMPTY + db));
          umma_commit(B(K_EMPTY + sk));
        }
        if (ok) umma_commit(B(DQ_FULL));
      }
    }
  } else {
    const int grp = (warp - 2) >> 2;               // column half of every slab this thread handles
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const float scale = rsqrtf((float)DH), c = scale * LOG2E;
    WorkItem w; uint32_t cs = 0; bool ok = true;
    for (int k = 0; ok && work_item(k, p.B, p.h, nq, w); ++k) {
      const int qb = w.qb, grow = qb * 128 + row;
      const int64_t si = ((int64_t)w.b * p.h + w.head) * S + (grow < S ? grow : S - 1);
      const float l2 = p.lse[si] * LOG2E, dl = p.delta[si];
      for (int it = 0; it <= qb && ok; ++it, ++cs) {
        const int db = cs & 1;
        if (!mbar_wait(B(SDP_FULL), cs & 1u, abort_flag, p.flags)) { ok = false; break; }
        tc_fence_after();
        uint32_t rs[64], rd[64];
        tmem_ld32(tS + lane_off + 64 * grp, rs);
        tmem_ld32(tS + lane_off + 64 * grp + 32, rs + 32);
        tmem_ld32(tP + lane_off + 64 * grp, rd);
        tmem_ld32(tP + lane_off + 64 * grp + 32, rd + 32);
        tmem_ld_wait();
        tc_fence_before();
        warp_arrive(B(SDP_EMPTY));               // the accumulators are in registers: free them early
        const bool diag = (it == qb) || ((it + 1) * 128 > S);
        const int col0 = it * 128 + 64 * grp;
        if (!diag) {
#pragma unroll
          for (int e = 0; e < 64; e += 2) {
            const float p0 = ex2(fmaf(__uint_as_float(rs[e]), c, -l2));
            const float p1 = ex2(fmaf(__uint_as_float(rs[e + 1]), c, -l2));
            rs[e >> 1] = pack2(p0 * (__uint_as_float(rd[e]) - dl), p1 * (__uint_as_float(rd[e + 1]) - dl));
          }
        } else {
#pragma unroll
          for (int e = 0; e < 64; e += 2) {
            const int col = col0 + e;
            float p0 = ex2(fmaf(__uint_as_float(rs[e]), c, -l2));
            float p1 = ex2(fmaf(__uint_as_float(rs[e + 1]), c, -l2));
            if (col > grow || col >= S) p0 = 0.f;
            if (col + 1 > grow || col + 1 >= S) p1 = 0.f;
            rs[e >> 1] = pack2(p0 * (__uint_as_float(rd[e]) - dl), p1 * (__uint_as_float(rd[e + 1]) - dl));
          }
        }
        if (!mbar_wait(B(DS_EMPTY + db), ((cs >> 1) & 1) ^ 1u, abort_flag, p.flags)) { ok = false; break; }
        tc_fence_after();
        tmem_st32(tD + 64 * db + lane_off + 32 * grp, rs);
        tmem_st_wait();
        tc_fence_before();
        warp_arrive(B(DS_FULL + db));
      }
      if (!ok) break;
      if (!mbar_wait(B(DQ_FULL), (uint32_t)k & 1u, abort_flag, p.flags)) { ok = false; break; }
      tc_fence_after();
      bf16* out = p.dqkv + ((int64_t)w.b * S + grow) * (3 * d) + w.head * DH;
#pragma unroll 1
      for (int cc = grp; cc < DH / 32; cc += 2) {       // the two groups drain alternate column chunks
        uint32_t r[32];
        tmem_ld32(tQ + lane_off + cc * 32, r);
        tmem_ld_wait();
        if (grow < S)
          drain32(out + cc * 32, r, scale, p.inv_rope ? p.inv_rope + (int64_t)grow * (DH / 2) : nullptr, cc * 32);
      }
      tc_fence_before();
      warp_arrive(B(TQ_EMPTY));                 // the next item's dQ products may overwrite the accumulator
    }
  }
  if (*abort_flag) for (int i = 0; i < 64; ++i) __nanosleep(2000);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

// ------------------------------------------------------------------ backward: dk, dv
// A work item owns 128 keys (K and V tiles resident) and streams 128-query slabs of Q and dU through
// a two-deep TMA ring.  The transposed products S^T = K Q^T and dP^T = V dU^T of a slab land in
// tensor memory; the 256 row threads (one key each, half of the slab's queries per group) turn
// S^T into bf16 P^T and then dP^T into bf16 dS^T, each written back over the first half of the
// thread's own accumulator columns, and dV += P^T dU, dK += dS^T Q take those as A operands
// straight from tensor memory.  The tensor-memory budget (two 128-column accumulators for dV and
// dK plus the two score buffers) leaves no room to double-buffer the scores, and with one score
// buffer S^T -> P^T -> dV -> next S^T is a serial chain that leaves the tensor pipe idle while
// the row threads work.  So the chain is split by query half: S^T and dV are issued per half
// (64-column / 64-deep products) with their own barriers, S^T of slab i+1's half h may start
// as soon as dV of slab i's half h has consumed that half's P^T, and the two row groups drift
// half a period apart - one group's exponentials run under the other's products.  One thread
// issues S^T and dP^T, a second one dV and dK; dP^T of slab i+1 may start as soon as dK of
// slab i is done.
// Work items of the dk/dv kernel: 128 keys of one head of one sequence, heavy (first key block)
// first; qb of the item is its key block.
__device__ __forceinline__ bool work_item_kv(int k, int n_batch, int h, int nq, WorkItem& w) {
  const int G = gridDim.x, cta = blockIdx.x;
  const int t = k * G + ((k & 1) ? (G - 1 - cta) : cta);
  const int hb = h * n_batch;
  if (t >= nq * hb) return false;
  w.qb = t / hb;
  const int rem = t % hb;
  w.head = rem % h; w.b = rem / h;
  return true;
}

template <int DH>
__global__ void __launch_bounds__(DQ_THREADS, 1)
attn_dkv_tc_kernel(const __grid_constant__ CUtensorMap mapQKV, const __grid_constant__ CUtensorMap mapG,
                   const AttnParams p) {
  constexpr int NH = DH / 64, QT = 128 * DH * 2, NS = 2;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align1k(smem_raw);
  const uint32_t Ks = smem_u32(smem), Vs = Ks + QT, Rs = Vs + QT;   // ring: Q then dU per stage
  // per-query statistics of a slab, staged one slab ahead: [slab % 3][lse * log2e | delta][128]
  float* row_stat = reinterpret_cast<float*>(smem + (2 + 2 * NS) * QT);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (2 + 2 * NS) * QT + 3 * 2 * 128 * 4);
  // S_FULL, P_FULL and TS_EMPTY exist per query half of the slab (= per row group)
  enum { KV_FULL = 0, KV_EMPTY, QG_FULL, QG_EMPTY = QG_FULL + NS, S_FULL = QG_EMPTY + NS, DP_FULL = S_FULL + 2,
         P_FULL, DS_FULL = P_FULL + 2, TS_EMPTY, TP_EMPTY = TS_EMPTY + 2, OUT_FULL, ACC_EMPTY, NBAR };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NBAR);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto B = [&](int i) { return bar0 + 8u * i; };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int d = p.h * DH, S = p.S, nq = (S + 127) / 128;
  // Row thread (grp, row) stages one statistic of one of its own group's 64 queries of query block
  // qblk: threads 0-63 the log-sum-exp, threads 64-127 delta.  A group reads only what its own
  // threads staged, so its hand-over needs no one but itself.
  auto fetch_stat = [&](const WorkItem& w, int qblk, int grp, int row) -> float {
    const int q = qblk * 128 + 64 * grp + (row & 63);
    const int64_t i = ((int64_t)w.b * p.h + w.head) * S + (q < S ? q : S - 1);
    return row < 64 ? __ldg(p.lse + i) * LOG2E : __ldg(p.delta + i);
  };
  // where that value goes inside a staging slot laid out [lse | delta][128 queries]
  auto stat_slot = [](int grp, int row) { return (row >> 6) * 128 + 64 * grp + (row & 63); };

  if (threadIdx.x == 0) {
    for (int i = 0; i < NBAR; ++i) mbar_init(B(i), 1);
    mbar_init(B(P_FULL), 4); mbar_init(B(P_FULL + 1), 4); mbar_init(B(DS_FULL), 8); mbar_init(B(ACC_EMPTY), 8);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
  if (warp >= 2 && warp < 10) {
    WorkItem w0;
    if (work_item_kv(0, p.B, p.h, nq, w0)) {
      const int g0 = (warp - 2) >> 2, r0 = (warp & 3) * 32 + lane;
      row_stat[stat_slot(g0, r0)] = fetch_stat(w0, w0.qb, g0, r0);
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tS = tmem, tP = tmem + 128, tV = tmem + 256, tK = tmem + 384;   // P^T overlays S^T, dS^T overlays dP^T
  // c counts the query slabs this CTA has gone through (every role keeps its own copy)

  if (warp == 0) {
    if (lane == 0) {
      WorkItem w; uint32_t c = 0; bool ok = true;
      for (int k = 0; ok && work_item_kv(k, p.B, p.h, nq, w); ++k) {
        const int kb = w.qb;
        // the K and V tiles are free once the previous item's last S^T / dP^T products are done
        if (k > 0 && !mbar_wait(B(KV_EMPTY), (uint32_t)(k - 1) & 1u, abort_flag, p.flags)) break;
        mbar_expect_tx(B(KV_FULL), 2 * QT);
        for (int hf = 0; hf < NH; ++hf) {
          tma_load_3d(Ks + hf * 16384, &mapQKV, B(KV_FULL), d + w.head * DH + hf * 64, kb * 128, w.b);
          tma_load_3d(Vs + hf * 16384, &mapQKV, B(KV_FULL), 2 * d + w.head * DH + hf * 64, kb * 128, w.b);
        }
        for (int it = 0; it < nq - kb; ++it, ++c) {
          const int st = c % NS; const uint32_t ph = (c / NS) & 1;
          if (!mbar_wait(B(QG_EMPTY + st), ph ^ 1u, abort_flag, p.flags)) { ok = false; break; }
          mbar_expect_tx(B(QG_FULL + st), 2 * QT);
          for (int hf = 0; hf < NH; ++hf) {
            tma_load_3d(Rs + st * 2 * QT + hf * 16384, &mapQKV, B(QG_FULL + st), w.head * DH + hf * 64, (kb + it) * 128, w.b);
            tma_load_3d(Rs + st * 2 * QT + QT + hf * 16384, &mapG, B(QG_FULL + st), w.head * DH + hf * 64, (kb + it) * 128, w.b);
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc(128, 128, false, false), idesc_h = make_idesc(128, 64, false, false);
      const uint32_t k_lo = klo(Ks), v_lo = klo(Vs);
      WorkItem w; uint32_t c = 0; bool ok = true;
      for (int k = 0; ok && work_item_kv(k, p.B, p.h, nq, w); ++k) {
        if (!mbar_wait(B(KV_FULL), (uint32_t)k & 1u, abort_flag, p.flags)) break;
        for (int it = 0; it < nq - w.qb; ++it, ++c) {
          const int st = c % NS; const uint32_t prev = (c - 1) & 1u;
          const uint32_t Qst = Rs + st * 2 * QT, Gst = Qst + QT;
          if (!mbar_wait(B(QG_FULL + st), (c / NS) & 1, abort_flag, p.flags)) { ok = false; break; }
          const uint32_t q_lo = klo(Qst), g_lo = klo(Gst);
          // S^T is formed per query half (64-column products), each half as soon as dV has consumed
          // that half's P^T of the previous slab: the two row groups then work out of phase, and
          // one group's exponentials overlap the other's products
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            if (c > 0 && !mbar_wait(B(TS_EMPTY + hh), prev, abort_flag, p.flags)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks)
              umma_lo(tS + 64 * hh, k_lo + kstep<128>(ks), q_lo + 512u * hh + kstep<128>(ks), idesc_h, ks > 0);
            umma_commit(B(S_FULL + hh));
          }
          if (!ok) break;
          // dP^T overwrites dS^T of the previous slab: wait until dK has consumed it
          if (c > 0 && !mbar_wait(B(TP_EMPTY), prev, abort_flag, p.flags)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks)
            umma_lo(tP, v_lo + kstep<128>(ks), g_lo + kstep<128>(ks), idesc_s, ks > 0);
          umma_commit(B(DP_FULL));
        }
        if (ok) umma_commit(B(KV_EMPTY));
      }
    }
  } else if (warp == 10) {
    if (lane == 0) {
      constexpr uint32_t idesc_o = make_idesc(128, DH, false, true);
      WorkItem w; uint32_t c = 0; bool ok = true;
      for (int k = 0; ok && work_item_kv(k, p.B, p.h, nq, w); ++k) {
        // the accumulators are free once the row threads have drained the previous item's dV, dK
        if (k > 0 && !mbar_wait(B(ACC_EMPTY), (uint32_t)(k - 1) & 1u, abort_flag, p.flags)) break;
        for (int it = 0; it < nq - w.qb; ++it, ++c) {
          const int st = c % NS; const uint32_t ph = c & 1u;
          const uint32_t Qst = Rs + st * 2 * QT, Gst = Qst + QT;
          if (!mbar_wait(B(QG_FULL + st), (c / NS) & 1, abort_flag, p.flags)) { ok = false; break; }
          const uint32_t gmn_lo = mlo<128>(Gst), qmn_lo = mlo<128>(Qst);
          // group g's 64 queries sit in the first 32 columns of its own half of the accumulator
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            if (!mbar_wait(B(P_FULL + hh), ph, abort_flag, p.flags)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int ks = 4 * hh; ks < 4 * hh + 4; ++ks)
              umma_ts_lo(tV, tS + hh * 64 + (ks & 3) * 8, gmn_lo + mstep(ks), idesc_o, (it > 0 || ks > 0));
            umma_commit(B(TS_EMPTY + hh));
          }
          if (!ok) break;
          if (!mbar_wait(B(DS_FULL), ph, abort_flag, p.flags)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            umma_ts_lo(tK, tP + (ks >> 2) * 64 + (ks & 3) * 8, qmn_lo + mstep(ks), idesc_o, (it > 0 || ks > 0));
          umma_commit(B(TP_EMPTY));
          umma_commit(B(QG_EMPTY + st));
        }
        if (ok) umma_commit(B(OUT_FULL));
      }
    }
  } else {
    const int grp = (warp - 2) >> 2;               // query half of every slab this thread handles
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const float scale = rsqrtf((float)DH), c = scale * LOG2E;
    WorkItem w, wn; uint32_t cs = 0; bool ok = true;
    bool have = work_item_kv(0, p.B, p.h, nq, w);
    for (int k = 0; ok && have; ++k) {
      const int kb = w.qb, n = nq - kb, key = kb * 128 + row;
      const bool have_next = work_item_kv(k + 1, p.B, p.h, nq, wn);
      for (int it = 0; it < n && ok; ++it, ++cs) {
        const uint32_t ph = cs & 1u;
        const float4* sl = reinterpret_cast<const float4*>(row_stat + ((cs % 3) * 2 + 0) * 128 + 64 * grp);
        const float4* sd = reinterpret_cast<const float4*>(row_stat + ((cs % 3) * 2 + 1) * 128 + 64 * grp);
        const int q0 = (kb + it) * 128 + 64 * grp;
        const bool diag = (it == 0) || ((kb + it + 1) * 128 > S);
        // the next slab's statistic (of this item or of the next one) is fetched now so that its
        // latency hides behind this slab's work
        const bool more = it + 1 < n || have_next;
        const float next_stat = it + 1 < n ? fetch_stat(w, kb + it + 1, grp, row)
                                           : (have_next ? fetch_stat(wn, wn.qb, grp, row) : 0.f);
        // ---- P^T from S^T
        if (!mbar_wait(B(S_FULL + grp), ph, abort_flag, p.flags)) { ok = false; break; }
        tc_fence_after();
        uint32_t rs[64], pk[32];
        tmem_ld32(tS + lane_off + 64 * grp, rs);
        tmem_ld32(tS + lane_off + 64 * grp + 32, rs + 32);
        tmem_ld_wait();
#pragma unroll
        for (int e4 = 0; e4 < 16; ++e4) {
          const float4 l4 = sl[e4];
          const float lv[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int e = 4 * e4 + u;
            float x = ex2(fmaf(__uint_as_float(rs[e]), c, -lv[u]));
            if (diag && (key > q0 + e || q0 + e >= S)) x = 0.f;
            rs[e] = __float_as_uint(x);
          }
          pk[2 * e4] = pack2(__uint_as_float(rs[4 * e4]), __uint_as_float(rs[4 * e4 + 1]));
          pk[2 * e4 + 1] = pack2(__uint_as_float(rs[4 * e4 + 2]), __uint_as_float(rs[4 * e4 + 3]));
        }
        tmem_st32(tS + lane_off + 64 * grp, pk);
        tmem_st_wait();
        tc_fence_before();
        // next slab's statistics: written before this arrival, they are visible to every thread of
        // the group that later sees its half of the next slab's S^T (issued only after this half's dV)
        if (more) row_stat[((cs + 1) % 3) * 256 + stat_slot(grp, row)] = next_stat;
        warp_arrive(B(P_FULL + grp));
        // ---- dS^T from dP^T
        if (!mbar_wait(B(DP_FULL), ph, abort_flag, p.flags)) { ok = false; break; }
        tc_fence_after();
        {
          uint32_t rd[64];
          tmem_ld32(tP + lane_off + 64 * grp, rd);
          tmem_ld32(tP + lane_off + 64 * grp + 32, rd + 32);
          tmem_ld_wait();
#pragma unroll
          for (int e4 = 0; e4 < 16; ++e4) {
            const float4 d4 = sd[e4];
            const float dv[4] = {d4.x, d4.y, d4.z, d4.w};
            float de[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
              de[u] = __uint_as_float(rs[4 * e4 + u]) * (__uint_as_float(rd[4 * e4 + u]) - dv[u]);
            pk[2 * e4] = pack2(de[0], de[1]);
            pk[2 * e4 + 1] = pack2(de[2], de[3]);
          }
        }
        tmem_st32(tP + lane_off + 64 * grp, pk);
        tmem_st_wait();
        tc_fence_before();
        warp_arrive(B(DS_FULL));
      }
      if (!ok) break;
      if (!mbar_wait(B(OUT_FULL), (uint32_t)k & 1u, abort_flag, p.flags)) { ok = false; break; }
      tc_fence_after();
      bf16* out = p.dqkv + ((int64_t)w.b * S + key) * (3 * d) + w.head * DH;
#pragma unroll 1
      for (int cc = grp; cc < 2 * DH / 32; cc += 2) {
        const bool is_k = cc >= DH / 32;
        const int c0 = (is_k ? cc - DH / 32 : cc) * 32;
        uint32_t r[32];
        tmem_ld32((is_k ? tK : tV) + lane_off + c0, r);
        tmem_ld_wait();
        if (key < S)
          drain32(out + (is_k ? d : 2 * d) + c0, r, is_k ? scale : 1.f,
                  (is_k && p.inv_rope) ? p.inv_rope + (int64_t)key * (DH / 2) : nullptr, c0);
      }
      tc_fence_before();
      warp_arrive(B(ACC_EMPTY));                // the next item's products may overwrite dV, dK
      w = wn; have = have_next;
    }
  }
  if (*abort_flag) for (int i = 0; i < 64; ++i) __nanosleep(2000);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

// 3-D tensor map over a [B, S, cols] bf16 array (row stride ld elements), boxes of 64 columns
bool encode3d(CUtensorMap* map, const bf16* base, int cols, int S, int B, int64_t ld, int box_rows) {
  EncodeTiledFn enc = get_encoder();
  if (!enc) return false;
  cuuint64_t gdim[3] = {(cuuint64_t)cols, (cuuint64_t)S, (cuuint64_t)B};
  cuuint64_t gstride[2] = {(cuuint64_t)ld * 2, (cuuint64_t)S * ld * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, (void*)base, gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() { return ppu_sm_count(); }

// delta[b, head, s] = sum over the head's columns of dU * U: one warp per (token, head)
__global__ void attn_delta_kernel(const bf16* __restrict__ U, const bf16* __restrict__ dU,
                                  float* __restrict__ delta, int S, int h, int dh, int64_t rows) {
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
  if (lane == 0) delta[((tok / S) * h + head) * S + (int)(tok % S)] = s;
}

constexpr int EXTRA = 1024 + 256;   // alignment slack + barriers

template <int DH>
int fwd_t(const bf16* qkv, bf16* U, float* lse, int B, int S, int h, int* flags, cudaStream_t st) {
  constexpr int SM = 7 * 128 * DH * 2 + 2 * 128 * 8 + 256 + FWD_ALIGN_SLACK;
  static PerDeviceFlag attr;
  if (!ppu_set_smem_once(attr, attn_fwd_tc_kernel<DH>, SM)) return -2;
  CUtensorMap m;
  if (!encode3d(&m, qkv, 3 * h * DH, S, B, 3 * (int64_t)h * DH, 128)) return -3;
  AttnParams p{}; p.U = U; p.lse_out = lse; p.S = S; p.h = h; p.B = B; p.flags = flags;
  const int items = ((S + 127) / 128) * h * B;
  attn_fwd_tc_kernel<DH><<<items < sm_count() ? items : sm_count(), FWD_THREADS, SM, st>>>(m, p);
  return 0;
}

template <int DH>
int bwd_t(const bf16* qkv, const float* lse, const bf16* dU, bf16* dqkv, const float* delta, int B,
          int S, int h, int* flags, cudaStream_t st, const float2* inv_rope) {
  constexpr int SM_DQ = 7 * 128 * DH * 2 + EXTRA;
  constexpr int SM_KV = 6 * 128 * DH * 2 + 3 * 2 * 128 * 4 + EXTRA;
  static PerDeviceFlag attr_dq, attr_kv;
  if (!ppu_set_smem_once(attr_dq, attn_dq_tc_kernel<DH>, SM_DQ) || !ppu_set_smem_once(attr_kv, attn_dkv_tc_kernel<DH>, SM_KV)) return -2;
  const int d = h * DH;
  CUtensorMap mQKV, mG;
  if (!encode3d(&mQKV, qkv, 3 * d, S, B, 3 * (int64_t)d, 128) || !encode3d(&mG, dU, d, S, B, d, 128))
    return -3;
  AttnParams p{}; p.lse = lse; p.delta = delta; p.dqkv = dqkv; p.S = S; p.h = h; p.B = B; p.flags = flags;
  p.inv_rope = inv_rope;
  const int items = ((S + 127) / 128) * h * B, ctas = items < sm_count() ? items : sm_count();
  attn_dq_tc_kernel<DH><<<ctas, DQ_THREADS, SM_DQ, st>>>(mQKV, mG, p);
  attn_dkv_tc_kernel<DH><<<ctas, DQ_THREADS, SM_KV, st>>>(mQKV, mG, p);
  return 0;
}

}  // namespace

bool attn_tc_supported(int S, int dh) { return (dh == 64 || dh == 128) && S >= 1; }

void launch_attn_delta(const bf16* U, const bf16* dU, float* delta, int B, int S, int h, int dh,
                       cudaStream_t st) {
  const int64_t rows = (int64_t)B * S;
  const int64_t warps = rows * h;
  attn_delta_kernel<<<(unsigned)((warps * 32 + 255) / 256), 256, 0, st>>>(U, dU, delta, S, h, dh, rows);
}

int launch_attn_fwd_tc(const bf16* qkv, bf16* U, float* lse, int B, int S, int h, int dh, int* flags,
                       cudaStream_t st) {
  if (gemm_tc_init() != 0) return -1;
  if (dh == 64) return fwd_t<64>(qkv, U, lse, B, S, h, flags, st);
  if (dh == 128) return fwd_t<128>(qkv, U, lse, B, S, h, flags, st);
  return -1;
}

int launch_attn_bwd_tc(const bf16* qkv, const bf16* U, const float* lse, const bf16* dU, bf16* dqkv,
                       float* scratch, int B, int S, int h, int dh, int* flags, cudaStream_t st,
                       const float2* inv_rope_cs, bool delta_done) {
  if (gemm_tc_init() != 0) return -1;
  if (!delta_done) launch_attn_delta(U, dU, scratch, B, S, h, dh, st);
  if (dh == 64) return bwd_t<64>(qkv, lse, dU, dqkv, scratch, B, S, h, flags, st, inv_rope_cs);
  if (dh == 128) return bwd_t<128>(qkv, lse, dU, dqkv, scratch, B, S, h, flags, st, inv_rope_cs);
  return -1;
}
