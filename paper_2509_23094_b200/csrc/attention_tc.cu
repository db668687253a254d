// Selected-query bidirectional attention on the 5th-generation tensor cores (head_dim 128).
//
//   attn_fwd_tc    O = softmax(Q K^T / sqrt(Dh)) V and the log-sum-exp per (row, head).  One CTA per
//                  (256 selected rows, head, sequence); keys stream in tiles of 128 through TMA.
//                  S = Q K^T is a tcgen05.mma into TMEM; softmax warps (one row per thread) read it
//                  with tcgen05.ld, write the bf16 probabilities back over the same TMEM columns and the
//                  PV product takes them from there as its A operand (V is the MN-major B operand straight
//                  from the TMA tile) and accumulates O in TMEM.
//   attn_abar_tc   Abar[r][j] = 1/Hq sum_h exp(s_h[r][j] - lse_h[r]) (Section 4.2): one CTA per
//                  (128 rows x 128 keys) loops over the heads, S by tcgen05.mma, the sum over heads in
//                  registers in a fixed order (deterministic).
//
// Warp roles in both: warp 0 TMA producer, warp 1 MMA issuer + TMEM owner, warps 2.. softmax/epilogue.
// No cluster, no multicast.  Every mbarrier wait is bounded (see gemm_tc.cu for the protocol).
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace d2c {
namespace {

constexpr int AQ = 128, AKEYS = 128, ADH = 128;
constexpr int HALF_BYTES = 128 * 64 * 2;          // one 128-row x 64-column swizzled box: 16 KB
constexpr int TILE_BYTES = 2 * HALF_BYTES;        // 128 x 128 bf16
constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;

__device__ int g_attn_status[4];

// D (TMEM) (+)= A (TMEM) x B (shared memory): the probabilities stay in TMEM
__device__ __forceinline__ void umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
               ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
               ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                 "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// MN-major bf16 operand: 64 contiguous N elements per 128-byte row, 8 K-rows per 1024-byte group
// (stride offset), the next 64 N elements 16 KB further (leading offset).
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(HALF_BYTES >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// bf16 x bf16 -> fp32, M = 128, N = 128; bit 16 set: B is MN-major.
constexpr uint32_t kIdescKK = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescKMn = kIdescKK | (1u << 16);

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

struct AttnTcParams { AttnArgs a; int* status; int sm_count; int head_groups; };

// ------------------------------------------------------------------------------------------------
// Forward kernel.  One CTA owns up to 256 selected rows of one (sequence, head): two query tiles of
// 128 rows that share every K/V tile brought in by TMA.  Each query tile has its own softmax warp
// group (4 warps, one row per thread) and its own TMEM columns: 128 for the scores S (overwritten in
// place by the bf16 probabilities P) and 128 for the output accumulator O, which stays in TMEM across
// the key tiles.  The running maximum is only raised when it grows by more than 2^8 (P stays exactly
// representable in bf16's exponent range); the rare raise rescales O in TMEM between two PV products.
constexpr int FWD_THREADS = 320;
constexpr float kRescaleStep = 8.f;

// Packed pairs of fp32 for Blackwell's two-wide FMA-pipe instructions: one issue slot for two elements.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
               "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
               ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                 "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
                 "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
                 "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]) : "memory");
}

__global__ void __launch_bounds__(FWD_THREADS, 1)
attn_fwd_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
            const __grid_constant__ CUtensorMap tmV, const AttnTcParams p) {
  pdl_prologue();
  const AttnArgs& a = p.a;
  const int b = blockIdx.z, h = blockIdx.y, g = h / (a.hq / a.hkv);
  // With few selected rows every 128-row tile gets a CTA of its own (more SMs busy); otherwise a CTA
  // takes two tiles, which halves the K/V traffic per row and keeps both softmax warp groups busy.
  const int nb = a.row_off[b + 1] - a.row_off[b];
  const bool pairs = ((nb + AQ - 1) / AQ) * a.hq * a.batch > p.sm_count;
  const int r0 = a.row_off[b] + blockIdx.x * (pairs ? 2 * AQ : AQ);
  const int nrows = min(pairs ? 2 * AQ : AQ, a.row_off[b + 1] - r0);
  if (nrows <= 0) return;                                          // uniform: nothing allocated yet
  const int nq = nrows > AQ ? 2 : 1;                                // live query tiles
  const int L = a.seq_len, T = (L + AKEYS - 1) / AKEYS;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int* status = p.status ? p.status : g_attn_status;

  extern __shared__ unsigned char smem_raw[];
  const uint32_t sbase = ((uint32_t)__cvta_generic_to_shared(smem_raw) + 1023u) & ~1023u;
  auto sQ = [&](int q) { return sbase + q * TILE_BYTES; };
  auto sK = [&](int s) { return sbase + (2 + 2 * s) * TILE_BYTES; };
  auto sV = [&](int s) { return sbase + (3 + 2 * s) * TILE_BYTES; };
  // barriers: 0 q_full | 1,2 k_full | 3,4 v_full | 5,6 kv_empty | 7,8 s_full[q] | 9,10 p_full[q] | 11,12 o_full[q]
  __shared__ __align__(8) uint64_t bars[13];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
  auto B = [&](int i) { return bar0 + 8u * i; };
  if (threadIdx.x == 0) {
    for (int i = 0; i < 9; ++i) mbar_init(B(i), 1);
    mbar_init(B(9), 4); mbar_init(B(10), 4);
    mbar_init(B(11), 1); mbar_init(B(12), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) { tmem_alloc((uint32_t)__cvta_generic_to_shared(&tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = tmem_slot;                                    // tile q: S/P at q*256, O at q*256 + 128
  volatile int* abortp = &abort_flag;
  const int kv_row0 = b * a.cache_seq;

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(B(0), nq * TILE_BYTES);
      for (int q = 0; q < nq; ++q) {
        tma_load_2d(sQ(q), &tmQ, h * ADH, r0 + q * AQ, B(0));
        tma_load_2d(sQ(q) + HALF_BYTES, &tmQ, h * ADH + 64, r0 + q * AQ, B(0));
      }
      int issued = 0;
      for (int j = 0; j < T; ++j) {
        const int s = j & 1, u = j >> 1;
        if (!mbar_wait(B(5 + s), (u & 1) ^ 1, abortp, status, 11)) break;
        mbar_expect_tx(B(1 + s), TILE_BYTES);
        tma_load_2d(sK(s), &tmK, g * ADH, kv_row0 + j * AKEYS, B(1 + s));
        tma_load_2d(sK(s) + HALF_BYTES, &tmK, g * ADH + 64, kv_row0 + j * AKEYS, B(1 + s));
        mbar_expect_tx(B(3 + s), TILE_BYTES);
        tma_load_2d(sV(s), &tmV, g * ADH, kv_row0 + j * AKEYS, B(3 + s));
        tma_load_2d(sV(s) + HALF_BYTES, &tmV, g * ADH + 64, kv_row0 + j * AKEYS, B(3 + s));
        issued = j + 1;
      }
      if (*abortp) {
        const long long t0 = clock64();
        while (!mbar_try_wait(B(0), 0) && clock64() - t0 < kWaitCycles) {}
        for (int j = max(0, issued - 2); j < issued; ++j) {
          const long long t1 = clock64();
          while (!(mbar_try_wait(B(1 + (j & 1)), (j >> 1) & 1) && mbar_try_wait(B(3 + (j & 1)), (j >> 1) & 1)) &&
                 clock64() - t1 < kWaitCycles) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      auto issue_s = [&](int q, int j) {                            // S_{q,j} = Q_q K_j^T
        const int s = j & 1;
#pragma unroll
        for (int i = 0; i < ADH / 16; ++i) {
          const uint32_t off = (i >> 2) * HALF_BYTES;
          umma_ss(tm + q * 256, smem_desc_sw128(sQ(q) + off) + 2 * (i & 3), smem_desc_sw128(sK(s) + off) + 2 * (i & 3), kIdescKK, i != 0);
        }
        umma_commit(B(7 + q));
      };
      bool ok = mbar_wait(B(0), 0, abortp, status, 12) && mbar_wait(B(1), 0, abortp, status, 13);
      if (nq == 1) {
        // One live query tile: the second tile's TMEM columns are free, so the scores of key tile j + 1 are
        // computed there while the softmax warps work on tile j (S/P buffer = j & 1, O stays in the first half).
        auto issue_s1 = [&](int j) {
          const int s = j & 1;
#pragma unroll
          for (int i = 0; i < ADH / 16; ++i) {
            const uint32_t off = (i >> 2) * HALF_BYTES;
            umma_ss(tm + s * 256, smem_desc_sw128(sQ(0) + off) + 2 * (i & 3), smem_desc_sw128(sK(s) + off) + 2 * (i & 3), kIdescKK, i != 0);
          }
          umma_commit(B(7 + s));
        };
        if (ok) {
          tc_fence_after();
          issue_s1(0);
        }
        for (int j = 0; j < T && ok; ++j) {
          const int s = j & 1, u = j >> 1;
          if (j + 1 < T) {
            if (!mbar_wait(B(1 + ((j + 1) & 1)), ((j + 1) >> 1) & 1, abortp, status, 16)) { ok = false; break; }
            tc_fence_after();
            issue_s1(j + 1);                                        // its buffer held P_{j-1}, consumed by the product issued before
          }
          if (!mbar_wait(B(9 + s), u & 1, abortp, status, 14)) { ok = false; break; }
          if (!mbar_wait(B(3 + s), u & 1, abortp, status, 15)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int i = 0; i < AKEYS / 16; ++i)
            umma_ts(tm + 128, tm + s * 256 + 8 * i, desc_mnmajor(sV(s) + i * 2048), kIdescKMn, (j | i) != 0);
          umma_commit(B(11));
          umma_commit(B(5 + s));
        }
        ok = false;                                                 // done: skip the two-tile schedule below
      } else if (ok) {
        tc_fence_after();
        for (int q = 0; q < nq; ++q) issue_s(q, 0);
      }
      for (int j = 0; j < T && ok; ++j) {
        const int s = j & 1, u = j >> 1;
        for (int q = 0; q < nq && ok; ++q) {
          if (!mbar_wait(B(9 + q), j & 1, abortp, status, 14)) { ok = false; break; }
          if (q == 0 && !mbar_wait(B(3 + s), u & 1, abortp, status, 15)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int i = 0; i < AKEYS / 16; ++i)                     // O_q += P_{q,j} (TMEM, 8 columns per 16 keys) x V_j
            umma_ts(tm + q * 256 + 128, tm + q * 256 + 8 * i, desc_mnmajor(sV(s) + i * 2048), kIdescKMn, (j | i) != 0);
          umma_commit(B(11 + q));
          if (q == nq - 1) umma_commit(B(5 + s));                   // both products of tile j issued: K/V stage free when done
          if (j + 1 < T) {
            if (q == 0 && !mbar_wait(B(1 + ((j + 1) & 1)), ((j + 1) >> 1) & 1, abortp, status, 16)) { ok = false; break; }
            tc_fence_after();
            issue_s(q, j + 1);                                      // after PV_{q,j} in program order: P_{q,j} is consumed first
          }
        }
      }
    }
    __syncwarp();
  } else {
    const int q = (warp - 2) >> 2;                                  // softmax warp group = query tile
    if (q < nq) {
      const int quarter = warp & 3, lrow = q * AQ + quarter * 32 + lane;
      const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
      const bool dbuf = nq == 1;                                    // one query tile: S/P alternate between the TMEM halves
      const uint32_t to = tm + q * 256 + 128 + lane_base;
      const float sc = kLog2e * rsqrtf((float)ADH);
      float m_used = -INFINITY, l = 0.f;
      bool ok = true;
      for (int j = 0; j < T && ok; ++j) {
        const int sp = dbuf ? (j & 1) : q;                          // S/P buffer of this tile
        const uint32_t ts = tm + sp * 256 + lane_base;
        // a wait that gave up ends the loop for the whole warp: the tcgen05.ld / st below are warp-collective
        if (!__all_sync(0xffffffffu, mbar_wait(B(7 + sp), (dbuf ? (j >> 1) : j) & 1, abortp, status, 18))) { ok = false; break; }
        tc_fence_after();
        const int key0 = j * AKEYS;
        const bool full = key0 + AKEYS <= L;
        uint32_t sv[4][32];                                         // the whole score row of this thread
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(ts + c * 32, sv[c]);
        tmem_ld_wait();
        if (!full) {                                                // last, ragged key tile: keys past L score -inf (probability 0)
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (key0 + c * 32 + i >= L) sv[c][i] = __float_as_uint(-INFINITY);
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
#pragma unroll
          for (int i = 0; i < 32; i += 2)                               // three-input maximum: two scores per instruction
            mx4[(i >> 1) & 3] = fmax3(mx4[(i >> 1) & 3], __uint_as_float(sv[c][i]), __uint_as_float(sv[c][i + 1]));
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sc;
        const bool raise = mx > m_used + kRescaleStep;              // always true on the first tile
        if (__any_sync(0xffffffffu, raise)) {
          const float alpha = raise ? exp2f(m_used - mx) : 1.f;     // first tile: exp2(-inf) = 0
          if (raise) m_used = mx;
          l *= alpha;
          if (j > 0) {                                              // O holds the sum of tiles 0..j-1: rescale it in place
            if (!__all_sync(0xffffffffu, mbar_wait(B(11 + q), (j - 1) & 1, abortp, status, 17))) { ok = false; break; }
            tc_fence_after();
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              uint32_t v[32];
              tmem_ld32(to + c * 32, v);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
              tmem_st32(to + c * 32, v);
            }
            tmem_st_wait();
          }
        }
        // scale-and-subtract and the row sums run two elements per instruction (fma / add .f32x2): 2.7 % on the
        // forward kernel at 8 x 4096 keys; the exponentials and the bf16 rounding stay one instruction per pair or element
        unsigned long long rs2[4] = {0ull, 0ull, 0ull, 0ull};     // packed pairs of partial row sums (the bits of 0.f are 0)
        const unsigned long long sc2 = pack2(sc, sc), nm2 = pack2(-m_used, -m_used);
#pragma unroll
        for (int c = 0; c < 4; ++c) {                               // probabilities, written back as bf16 over the scores
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            float x0, x1;
            unpack2(fma2(pack2(__uint_as_float(sv[c][2 * i]), __uint_as_float(sv[c][2 * i + 1])), sc2, nm2), x0, x1);
            const float p0 = exp2f(x0), p1 = exp2f(x1);
            rs2[i & 3] = add2(rs2[i & 3], pack2(p0, p1));
            pk[i] = pack_bf16(p0, p1);
          }
          tmem_st16(ts + c * 16, pk);
        }
        float rs4[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) { float lo, hi; unpack2(rs2[t], lo, hi); rs4[t] = lo + hi; }
        const float rs = (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
        l += rs;
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(B(9 + sp));
      }
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(B(11 + q), (T - 1) & 1, abortp, status, 19));
      tc_fence_after();
      if (ok) {
        const bool row_ok = lrow < nrows;
        const float inv = 1.f / l;
        bf16* dst = a.o + (size_t)(r0 + lrow) * ((size_t)a.hq * ADH) + (size_t)h * ADH;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t v[32];
          tmem_ld32(to + c * 32, v);
          tmem_ld_wait();
          if (row_ok) {
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              uint4 w;
              w.x = pack_bf16(__uint_as_float(v[8 * t + 0]) * inv, __uint_as_float(v[8 * t + 1]) * inv);
              w.y = pack_bf16(__uint_as_float(v[8 * t + 2]) * inv, __uint_as_float(v[8 * t + 3]) * inv);
              w.z = pack_bf16(__uint_as_float(v[8 * t + 4]) * inv, __uint_as_float(v[8 * t + 5]) * inv);
              w.w = pack_bf16(__uint_as_float(v[8 * t + 6]) * inv, __uint_as_float(v[8 * t + 7]) * inv);
              reinterpret_cast<uint4*>(dst)[c * 4 + t] = w;
            }
          }
        }
        if (row_ok) a.lse[(size_t)(r0 + lrow) * a.hq + h] = (m_used + log2f(l)) * kLn2;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tm, 512); }
}

// ------------------------------------------------------------------------------------------------
constexpr int ABS = 3;                             // stages of the Q ring and of the K ring in attn_abar_tc

__global__ void __launch_bounds__(FWD_THREADS, 1)
attn_abar_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const AttnTcParams p) {
  pdl_prologue();
  const AttnArgs& a = p.a;
  const int b = blockIdx.z;
  const int r0 = a.row_off[b] + blockIdx.y * AQ;
  const int nrows = min(AQ, a.row_off[b + 1] - r0);
  const int L = a.seq_len, ktiles = (L + AKEYS - 1) / AKEYS;
  const int key0 = ((int)blockIdx.x % ktiles) * AKEYS, hg = (int)blockIdx.x / ktiles;
  if (nrows <= 0) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int group = a.hq / a.hkv;
  const int nh = a.hq / p.head_groups, h_first = hg * nh;          // this CTA's heads (whole kv groups)
  int* status = p.status ? p.status : g_attn_status;

  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = ((uint32_t)__cvta_generic_to_shared(smem_raw) + 1023u) & ~1023u;
  auto sQ = [&](int s) { return base + s * TILE_BYTES; };           // ABS query stages, then ABS key stages
  auto sK = [&](int s) { return base + (ABS + s) * TILE_BYTES; };
  // barriers: q_full[ABS] | k_full[ABS] | q_empty[ABS] | k_empty[ABS] | s_full[2] | s_empty[2]
  __shared__ __align__(8) uint64_t bars[4 * ABS + 4];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
  auto QF = [&](int i) { return bar0 + 8u * i; };
  auto KF = [&](int i) { return bar0 + 8u * (ABS + i); };
  auto QE = [&](int i) { return bar0 + 8u * (2 * ABS + i); };
  auto KE = [&](int i) { return bar0 + 8u * (3 * ABS + i); };
  auto SF = [&](int i) { return bar0 + 8u * (4 * ABS + i); };
  auto SE = [&](int i) { return bar0 + 8u * (4 * ABS + 2 + i); };
  if (threadIdx.x == 0) {
    for (int i = 0; i < 4 * ABS + 2; ++i) mbar_init(bar0 + 8u * i, 1);
    mbar_init(SE(0), 8); mbar_init(SE(1), 8);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) { tmem_alloc((uint32_t)__cvta_generic_to_shared(&tmem_slot), 256); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = tmem_slot;
  volatile int* abortp = &abort_flag;
  const int kv_row = b * a.cache_seq + key0;

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int h = 0; h < nh; ++h) {                                // h: local head index, hgl: head of the model
        const int s = h % ABS, u = h / ABS, hgl = h_first + h;
        if (!mbar_wait(QE(s), (u & 1) ^ 1, abortp, status, 21)) break;
        mbar_expect_tx(QF(s), TILE_BYTES);
        tma_load_2d(sQ(s), &tmQ, hgl * ADH, r0, QF(s));
        tma_load_2d(sQ(s) + HALF_BYTES, &tmQ, hgl * ADH + 64, r0, QF(s));
        if (h % group == 0) {
          const int gi = h / group, ks = gi % ABS, ku = gi / ABS, ggl = hgl / group;
          if (!mbar_wait(KE(ks), (ku & 1) ^ 1, abortp, status, 22)) break;
          mbar_expect_tx(KF(ks), TILE_BYTES);
          tma_load_2d(sK(ks), &tmK, ggl * ADH, kv_row, KF(ks));
          tma_load_2d(sK(ks) + HALF_BYTES, &tmK, ggl * ADH + 64, kv_row, KF(ks));
        }
        issued = h + 1;
      }
      if (*abortp) {
        for (int h = max(0, issued - ABS); h < issued; ++h) {
          const long long t1 = clock64();
          while (!mbar_try_wait(QF(h % ABS), (h / ABS) & 1) && clock64() - t1 < kWaitCycles) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      for (int h = 0; h < nh; ++h) {
        const int s = h % ABS, u = h / ABS, gi = h / group, ks = gi % ABS, ku = gi / ABS, sb = h & 1;
        if (!mbar_wait(QF(s), u & 1, abortp, status, 23)) break;
        if (h % group == 0 && !mbar_wait(KF(ks), ku & 1, abortp, status, 24)) break;
        if (!mbar_wait(SE(sb), ((h >> 1) & 1) ^ 1, abortp, status, 25)) break;
        tc_fence_after();
#pragma unroll
        for (int i = 0; i < ADH / 16; ++i) {
          const uint32_t off = (i >> 2) * HALF_BYTES;
          umma_ss(tm + sb * 128, smem_desc_sw128(sQ(s) + off) + 2 * (i & 3), smem_desc_sw128(sK(ks) + off) + 2 * (i & 3), kIdescKK, i != 0);
        }
        umma_commit(QE(s));                                         // Q stage free
        if ((h + 1) % group == 0 || h + 1 == nh) umma_commit(KE(ks));        // last head of the group: K stage free
        umma_commit(SF(sb));
      }
    }
    __syncwarp();
  } else {
    // eight warps: two per TMEM lane quarter, each owning 64 of the tile's 128 key columns, so that the
    // two warps of a scheduler hide each other's TMEM-load latency
    const int quarter = warp & 3, half = (warp - 2) >> 2, lrow = quarter * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const float sc = kLog2e * rsqrtf((float)ADH);
    const bool row_ok = lrow < nrows;
    float acc[64];
#pragma unroll
    for (int i = 0; i < 64; ++i) acc[i] = 0.f;
    bool ok = true;
    for (int h = 0; h < nh && ok; ++h) {
      const int sb = h & 1;
      const float e = row_ok ? a.lse[(size_t)(r0 + lrow) * a.hq + h_first + h] * kLog2e : 0.f;
      if (!__all_sync(0xffffffffu, mbar_wait(SF(sb), (h >> 1) & 1, abortp, status, 26))) { ok = false; break; }   // whole warp or nobody: tcgen05.ld below
      tc_fence_after();
      uint32_t v[2][32];
      tmem_ld32(tm + sb * 128 + lane_base + half * 64, v[0]);
      tmem_ld32(tm + sb * 128 + lane_base + half * 64 + 32, v[1]);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(SE(sb));                           // scores are in registers: the buffer may be refilled
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int i = 0; i < 32; ++i) acc[c * 32 + i] += exp2f(fmaf(__uint_as_float(v[c][i]), sc, -e));
    }
    if (ok && row_ok) {
      const float inv = 1.f / (float)a.hq;
      const int k0 = key0 + half * 64;
      float* out = p.head_groups > 1 ? a.abar_partial + (size_t)hg * ((size_t)a.q_rows * L) : a.abar;
      float* dst = out + (size_t)(r0 + lrow) * L + k0;
      if (k0 + 64 <= L && (L & 3) == 0) {
#pragma unroll
        for (int q = 0; q < 16; ++q)
          reinterpret_cast<float4*>(dst)[q] = make_float4(acc[4 * q] * inv, acc[4 * q + 1] * inv, acc[4 * q + 2] * inv, acc[4 * q + 3] * inv);
      } else {
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (k0 + i < L) dst[i] = acc[i] * inv;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tm, 256); }
}

// Abar = sum of the head groups' partial sums, in group order (deterministic).
__global__ void __launch_bounds__(256)
abar_sum_kernel(const float* __restrict__ part, size_t group_stride, int groups, const int32_t* __restrict__ n_rows,
                int L, float* __restrict__ abar) {
  pdl_prologue();
  const size_t total4 = ((size_t)(*n_rows) * L) >> 2;               // L is a multiple of 4 on this path
  const float4* p4 = reinterpret_cast<const float4*>(part);
  const size_t gs4 = group_stride >> 2;
  for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < total4; i += (size_t)gridDim.x * 256) {
    float4 acc = p4[i];
    for (int g2 = 1; g2 < groups; ++g2) {
      const float4 t = p4[i + (size_t)g2 * gs4];
      acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
    }
    reinterpret_cast<float4*>(abar)[i] = acc;
  }
}

}  // namespace

// True if the tcgen05 kernels can take this problem (otherwise the caller uses the mma.sync ones).
bool attention_tc_supported(const AttnArgs& a) {
  return a.dh == ADH && a.q_rows >= AQ && (long long)a.batch * a.cache_seq >= AKEYS && (a.ldq & 7) == 0 &&
         (reinterpret_cast<uintptr_t>(a.q) & 15) == 0 && (reinterpret_cast<uintptr_t>(a.kc) & 15) == 0 &&
         (reinterpret_cast<uintptr_t>(a.vc) & 15) == 0;
}

int launch_attention_tc(const AttnArgs& a, cudaStream_t st, int* status) {
  const int smem_fwd = 6 * TILE_BYTES + 1024, smem_ab = 2 * ABS * TILE_BYTES + 1024;
  static PerDevice attr_set;
  if (attr_set.first()) {
    D2C_CUDA_OK(cudaFuncSetAttribute(attn_fwd_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_fwd));
    D2C_CUDA_OK(cudaFuncSetAttribute(attn_abar_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_ab));
  }
  CUtensorMap tmQ, tmK, tmV;
  const uint64_t kv_cols = (uint64_t)a.hkv * a.dh, kv_rows = (uint64_t)a.batch * a.cache_seq;
  int rc = make_bf16_map(&tmQ, a.q, (uint64_t)a.q_rows, (uint64_t)a.hq * a.dh, (uint64_t)a.ldq, 128);
  if (rc == D2C_OK) rc = make_bf16_map(&tmK, a.kc, kv_rows, kv_cols, kv_cols, 128);
  if (rc == D2C_OK) rc = make_bf16_map(&tmV, a.vc, kv_rows, kv_cols, kv_cols, 128);
  if (rc != D2C_OK) return rc;
  const int sms = sm_count_current();
  const int qtiles = ceil_div(a.max_rows_per_seq, AQ), ktiles = ceil_div(a.seq_len, AKEYS);
  // split the heads over several CTAs while the (row tile x key tile) grid leaves a quarter of the SMs idle
  int groups = 1;
  const int kv_group = a.hq / a.hkv;
  while (a.abar_partial && a.n_rows && (a.seq_len & 3) == 0 && groups < 8 && 4LL * ktiles * qtiles * a.batch * groups < 3LL * sms &&
         a.hq % (groups * 2) == 0 && (a.hq / (groups * 2)) % kv_group == 0 &&
         (size_t)(groups * 2) * a.q_rows * a.seq_len <= a.abar_partial_floats)
    groups *= 2;
  AttnTcParams p{a, status, sms, groups};
  if (a.which != 2) {
    D2C_LAUNCH((attn_fwd_tc), dim3(qtiles, a.hq, a.batch), FWD_THREADS, smem_fwd, st, tmQ, tmK, tmV, p);
  }
  if (a.abar && a.which != 1) {
    D2C_LAUNCH((attn_abar_tc), dim3(ktiles * groups, qtiles, a.batch), FWD_THREADS, smem_ab, st, tmQ, tmK, p);
    if (groups > 1)
      D2C_LAUNCH((abar_sum_kernel), 4 * sms, 256, 0, st, (const float*)a.abar_partial, (size_t)a.q_rows * a.seq_len, groups, a.n_rows,
                 a.seq_len, a.abar);
  }
  return D2C_OK;
}

}  // namespace d2c
