// tcgen05 / TMEM GEMM for sm_100a with the step's fused epilogues.
//
//   C[m][n] = sum_k A[m][k] * W[n][k]      A: [max_rows][K] bf16, W: [N][K] bf16 (both K-major)
//
// Persistent CTAs (one per SM) walk over 128 x 256 accumulator tiles (256 output columns, or 128 gate +
// 128 up columns for the SwiGLU epilogue).  Warp roles:
//   warp 0      TMA producer: cp.async.bulk.tensor loads of 128 x 64 bf16 boxes (128-byte swizzle) into a
//               ring of shared-memory stages, completion signalled on mbarriers;
//   warp 1      MMA issuer: one thread issues tcgen05.mma (M=128, N=256, K=16) from shared-memory
//               descriptors into one of two TMEM accumulators; tcgen05.commit releases each stage back
//               to the producer and finally signals the epilogue;
//   warps 2-5   epilogue: tcgen05.ld brings one accumulator row per thread into registers, the fused
//               epilogue (bias / residual / SwiGLU / soft-max statistics) runs there, rows go to HBM.
// The live row count is read from device memory: the tile list is derived from it on the device.
// Every mbarrier wait is bounded; a wait that runs out raises D2C_ETIMEOUT in the status word, the
// CTA drains its copies, frees its TMEM and returns.
#include "common.cuh"
#include "epilogue_tiles.cuh"
#include "sm100_ptx.cuh"

namespace d2c {
namespace {

constexpr int TM = 128, TK = 64;                 // tile rows, K elements per stage (one 128-byte swizzle atom)
constexpr int TC_THREADS = 192;
constexpr int A_BYTES = TM * TK * 2;             // 16 KB

__device__ int g_tc_status[4];                   // status word used when the caller passes none

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
}


struct TcParams {
  GemmArgs g;
  int* status;
};

constexpr int ST = 4;                            // ring size: 4 x (16 KB of A + 32 KB of B) = 192 KB
constexpr int KSUB = 2;                          // 64-wide k-blocks per pipeline stage (see gemm_tc2.cu on why two)
constexpr int kSkMaxParts = 8;                   // split-K parts per tile at most
constexpr int ST_MAX = 12;                       // narrow tiles use smaller stages and more of them
constexpr int ACC_COLS = 256;                    // TMEM columns of one accumulator; two are allocated
constexpr int B_BYTES = ACC_COLS * TK * 2;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;

// Persistent kernel: CTA b works on tiles b, b + gridDim.x, ...  Tiles are numbered with the row
// tile fastest, so the CTAs that run together share one weight tile (read once from HBM, then L2).
// A tile is 128 rows x 256 accumulator columns (for SwiGLU: 128 gate + 128 up columns of the same 128
// outputs).  Two accumulators live in TMEM: the epilogue warps drain one while the MMA warp fills
// the other.
template <int EPI>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA128, const __grid_constant__ CUtensorMap tmA64,
               const __grid_constant__ CUtensorMap tmA32, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmB64, const TcParams p) {
  // Everything that does not read a predecessor's results (barriers, TMEM, descriptor prefetch) runs before
  // the wait on the preceding kernel, so it overlaps that kernel's tail.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const GemmArgs& g = p.g;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int* status = p.status ? p.status : g_tc_status;

  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = ((uint32_t)__cvta_generic_to_shared(smem_raw) + 1023u) & ~1023u;
  __shared__ __align__(8) uint64_t bars[2 * ST_MAX + 4];     // full[], empty[], acc_full[2], acc_empty[2]
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (ST_MAX + s); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * ST_MAX + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * ST_MAX + 2 + b); };
  if (threadIdx.x == 0) {
    for (int s = 0; s < ST_MAX; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 4); }
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    prefetch_tensormap(&tmA128); prefetch_tensormap(&tmB); prefetch_tensormap(&tmB2);
  }
  if (warp == 1) {
    tmem_alloc((uint32_t)__cvta_generic_to_shared(&tmem_slot), 2 * ACC_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = tmem_slot;
  volatile int* abortp = &abort_flag;

  // The live row count is read, and the weight boxes of the first ring fill are requested, before the wait on the
  // preceding kernel: neither is that kernel's output (the count is the selection kernel's, which has completed
  // before any GEMM's CTA runs: every kernel between it and a GEMM waits for its own predecessor before it lets
  // its successor launch, or is a GEMM behind such a kernel).  What the predecessor may have written (A rows, the
  // residual, split-K scratch) is touched only behind each role's own griddepcontrol.wait.
  const int n = max(*g.n_rows, 0);
  const int MT = (n + TM - 1) / TM;
  const int KT = g.K / TK, G = gridDim.x;
  const bool sk_ok = g.sk_partials != nullptr && g.sk_counters != nullptr;
  // Split-K for launches with fewer tiles than SMs (few live rows: the launch streams weights and every
  // idle SM is lost bandwidth): each tile's K range is cut into S equal parts of at least four k-blocks,
  // one (tile, part) item per CTA at most, so all parts of a tile run at the same time.  Parts park their fp32
  // accumulators in scratch and meet at a counter (a bounded wait); then each part adds, in part order
  // (deterministic), the partial sums of its own share of the tile's columns and runs the epilogue on them,
  // so the reduction and the epilogue are spread over S CTAs instead of falling on one.
  auto split_of = [&](int tiles) {
    if (!sk_ok || EPI == EPI_LMSTATS || tiles <= 0 || tiles >= G) return 1;
    const int s = max(1, min(min(G / tiles, KT / 4), kSkMaxParts));
    return tiles * s <= g.sk_max_tiles ? s : 1;
  };
  // Accumulator width of this launch.  One thread issues every MMA and pays a fixed issue latency per k-block
  // whatever the tile's width, so a narrow tile moves fewer weight bytes per unit of that latency: the tile
  // stays 256 columns wide and idle SMs are filled by splitting K.  Only when K is too short to split (or the
  // epilogue has no split form) is the tile narrowed to 128 or 64 columns.  The LM head covers several waves of
  // tiles and is bound by HBM: 128-column tiles make its last, partial wave shorter.
  int bn = ACC_COLS;
  const int bn_min = (EPI == EPI_SWIGLU) ? 256 : (EPI == EPI_LMSTATS ? 128 : (EPI == EPI_QKV_ROPE ? max(64, g.q_dh) : 64));
  if (EPI == EPI_LMSTATS) {
    if (MT * ((g.N + 255) / 256) > G) bn = 128;
  }
  while (bn > bn_min) {
    const int t = MT * ((g.N + bn - 1) / bn);
    if (2 * t * split_of(t) <= G) bn >>= 1; else break;
  }
  const int OUT_COLS = (EPI == EPI_SWIGLU) ? 128 : bn;       // output columns per tile
  const int NT = (g.N + OUT_COLS - 1) / OUT_COLS;
  const int total = MT * NT;                                 // 0 when no row is live: every role loop is empty
  const int S = split_of(total);
  const int items = total * S;
  // A pipeline stage holds two 64-wide k-blocks, each an A box of at most 128 rows (sized to the live rows) and
  // the tile's weight rows; shared memory left over by small boxes becomes more stages, i.e. more bytes in
  // flight per SM when the launch streams weights.
  const int a_rows_max = n >= 128 ? 128 : (n > 64 ? 128 : (n > 32 ? 64 : 32));
  const int b_rows = (EPI == EPI_SWIGLU) ? ACC_COLS : bn;
  const int sub_bytes = ((a_rows_max + b_rows) * TK * 2 + 1023) & ~1023;
  const int ring_bytes = ST * STAGE_BYTES - (128 - a_rows_max) * TK * 2;
  // two k-blocks per stage halve the issuing thread's barrier round-trips, but a ring of only two such stages
  // leaves one stage in flight while the other is consumed: big boxes (few-row weight streaming) keep one
  // k-block per stage and so twice as many stages
  const int ksub = ring_bytes / (KSUB * sub_bytes) >= 3 ? KSUB : 1;
  const int stage_bytes = ksub * sub_bytes;
  // the MMA always reads 128 rows of A: keep that read inside the allocation when the A box is smaller
  const int nst = min(ST_MAX, ring_bytes / stage_bytes);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;                                        // stages issued so far (ring position)
      bool ok = true;
      auto load_w = [&](uint32_t sb, int kc, int n0, uint32_t bar) {      // the weight rows of one k-block
        if (bn == 64) {
          tma_load_2d(sb, &tmB64, kc, n0, bar);
        } else {
          tma_load_2d(sb, &tmB, kc, n0, bar);
          if (EPI == EPI_SWIGLU) tma_load_2d(sb + 128 * TK * 2, &tmB2, kc, n0, bar);
          else if (bn == 256) tma_load_2d(sb + 128 * TK * 2, &tmB, kc, n0 + 128, bar);
        }
      };
      auto a_box_rows = [&](int m0) { const int rows = n - m0; return rows <= 32 ? 32 : (rows <= 64 ? 64 : 128); };   // live rows of a tile: load no more than needed
      uint32_t early = 0;                                     // stages whose byte count and weight boxes are already out
      for (int item = blockIdx.x; item < items && early < (uint32_t)nst; item += G) {
        const int tile = item % total, part = item / total;
        const int k0 = part * KT / S, k1 = (part + 1) * KT / S;
        const int m0 = (tile % MT) * TM, n0 = (tile / MT) * OUT_COLS;
        const uint32_t kb_bytes = (uint32_t)a_box_rows(m0) * TK * 2 + (uint32_t)b_rows * TK * 2;
        for (int kt = k0; kt < k1 && early < (uint32_t)nst; kt += ksub, ++early) {
          const int nsub = min(ksub, k1 - kt);
          mbar_expect_tx(full_bar(early), (uint32_t)nsub * kb_bytes);
#pragma unroll
          for (int u = 0; u < KSUB; ++u)
            if (u < nsub) load_w(smem_base + early * stage_bytes + u * sub_bytes + a_rows_max * TK * 2, (kt + u) * TK, n0, full_bar(early));
        }
      }
      asm volatile("griddepcontrol.wait;" ::: "memory");
      if (g.clock_probe && blockIdx.x == 0) { g.clock_probe[0] = clock64(); g.clock_probe[1] = global_timer_ns(); }
      for (int item = blockIdx.x; item < items && ok; item += G) {
        const int tile = item % total, part = item / total;
        const int k0 = part * KT / S, k1 = (part + 1) * KT / S;
        const int m0 = (tile % MT) * TM, n0 = (tile / MT) * OUT_COLS;
        const int arows = a_box_rows(m0);
        const CUtensorMap* ma = arows == 32 ? &tmA32 : (arows == 64 ? &tmA64 : &tmA128);
        const uint32_t kb_bytes = (uint32_t)arows * TK * 2 + (uint32_t)b_rows * TK * 2;
        for (int kt = k0; kt < k1; kt += ksub, ++it) {
          const int s = it % nst;
          const int nsub = min(ksub, k1 - kt);
          const bool fresh = it >= early;                     // not one of the stages started before the wait
          if (!mbar_wait(empty_bar(s), ((it / nst) & 1) ^ 1, abortp, status, 1)) { ok = false; break; }
          if (fresh) mbar_expect_tx(full_bar(s), (uint32_t)nsub * kb_bytes);
#pragma unroll
          for (int u = 0; u < KSUB; ++u) {
            if (u < nsub) {
              const uint32_t sa = smem_base + s * stage_bytes + u * sub_bytes, sb = sa + a_rows_max * TK * 2;
              const int kc = (kt + u) * TK;
              tma_load_2d(sa, ma, kc, m0, full_bar(s));
              if (fresh) load_w(sb, kc, n0, full_bar(s));
            }
          }
        }
      }
      if (*abortp) {
        // give the copies already in flight a bounded chance to land before the CTA goes away
        for (uint32_t j = it > (uint32_t)nst ? it - nst : 0; j < it; ++j) {
          const long long t0 = clock64();
          while (!mbar_try_wait(full_bar(j % nst), (j / nst) & 1) && clock64() - t0 < kWaitCycles) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc(bn);
      uint32_t tcount = 0;
      bool ok = true;
      const uint64_t desc0 = smem_desc_sw128(smem_base);     // A operand of stage 0, k-block 0
      const uint32_t b_off = (uint32_t)(a_rows_max * TK * 2) >> 4, sub_step = (uint32_t)sub_bytes >> 4;
      int st = 0; uint32_t ph = 0;                           // ring position of the next stage
      for (int item = blockIdx.x; item < items && ok; item += G, ++tcount) {
        const int part = item / total;
        const int nk = (part + 1) * KT / S - part * KT / S;
        const uint32_t buf = tcount & 1, use = tcount >> 1;
        if (!mbar_wait(acc_empty(buf), (use & 1) ^ 1, abortp, status, 4)) { ok = false; break; }
        const uint32_t tacc = tmem_acc + buf * ACC_COLS;
        for (int j = 0; j < nk; j += ksub) {
          const int nsub = min(ksub, nk - j);
          if (!mbar_wait(full_bar(st), ph, abortp, status, 2)) { ok = false; break; }
          tc_fence_after();
          const uint64_t adesc = desc0 + (uint64_t)(st * (stage_bytes >> 4)), bdesc = adesc + b_off;
#pragma unroll
          for (int u = 0; u < KSUB; ++u) {
            if (u < nsub) {
#pragma unroll
              for (int k = 0; k < TK / 16; ++k)               // +32 bytes per K=16 slice inside the swizzle atom
                umma_ss(tacc, adesc + u * sub_step + 2 * k, bdesc + u * sub_step + 2 * k, idesc, (j | u | k) != 0);
            }
          }
          umma_commit(empty_bar(st));                         // stage reusable once these MMAs have read it
          if (++st == nst) { st = 0; ph ^= 1; }
        }
        if (ok) umma_commit(acc_full(buf));                   // accumulator complete
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;                             // TMEM lanes this warp may touch
    const int lrow = quarter * 32 + lane;
    asm volatile("griddepcontrol.wait;" ::: "memory");        // the residual, the scratch and the outputs belong to the step's chain
    uint32_t tcount = 0;
    for (int item = blockIdx.x; item < items; item += G, ++tcount) {
      const int tile = item % total, part = item / total;
      const uint32_t buf = tcount & 1, use = tcount >> 1;
      const int m0 = (tile % MT) * TM, nt = tile / MT, n0 = nt * OUT_COLS;
      const int row = m0 + lrow;
      const bool row_ok = row < n;
      const float rscale = folded_row_scale(g, row, row_ok);     // RMSNorm of the A rows folded into this GEMM (1 if none)
      // a wait that gave up ends the loop for the whole warp (the tcgen05.ld below is warp-collective) ...
      const bool got = __all_sync(0xffffffffu, mbar_wait(acc_full(buf), use & 1, abortp, status, 3));
      if (S > 1) {
        // ... and, where the four warps meet at named barriers below, for all of them together
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (*abortp) break;
      } else if (!got) {
        break;
      }
      tc_fence_after();
      const uint32_t tbase = tmem_acc + buf * ACC_COLS + ((uint32_t)(quarter * 32) << 16);
      bool reduce = false;
      if (S > 1) {
        const int acc_cols = (EPI == EPI_SWIGLU) ? ACC_COLS : bn;
        float4* mine = reinterpret_cast<float4*>(g.sk_partials + (size_t)(tile * S + part) * (TM * ACC_COLS));
#pragma unroll 1
        for (int c = 0; c < acc_cols / 32; ++c) {
          uint32_t v[32];
          tmem_ld32(tbase + c * 32, v);
          tmem_ld_wait();
          if (row_ok) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              mine[(size_t)(c * 8 + q) * TM + lrow] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                                                  __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
          }
        }
        tc_fence_before();
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (warp == 2 && lane == 0) {
          mbar_arrive(acc_empty(buf)); mbar_arrive(acc_empty(buf)); mbar_arrive(acc_empty(buf)); mbar_arrive(acc_empty(buf));
          atomicAdd(&g.sk_counters[tile], 1);
          // every other part of this tile is running on another SM: wait (bounded) until all have parked their sums
          const long long t0 = clock64();
          volatile int32_t* cnt = g.sk_counters + tile;
          while (*cnt < S) {
            if (*abortp) break;
            if (clock64() - t0 > kWaitCycles) {
              *abortp = 1;
              if (atomicCAS(status, 0, D2C_ETIMEOUT) == 0) status[1] = 5;
              break;
            }
          }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (*abortp) break;
        __threadfence();
        reduce = true;
      }
      auto load_chunk = [&](int col, uint32_t (&v)[32]) {     // 32 accumulator columns of this thread's row
        if (!reduce) {
          tmem_ld32(tbase + col, v);
          tmem_ld_wait();
          if (g.in_ssq) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * rscale);
          }
        } else {
          const float4* sp = reinterpret_cast<const float4*>(g.sk_partials + (size_t)(tile * S) * (TM * ACC_COLS)) +
                             (size_t)(col >> 2) * TM + lrow;
          float4 acc[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
          for (int c0 = 0; c0 < S; c0 += 4) {                 // parts are added in part order, four loads in flight
            float4 t[4][8];
#pragma unroll
            for (int c2 = 0; c2 < 4; ++c2)
#pragma unroll
              for (int q = 0; q < 8; ++q)
                t[c2][q] = (c0 + c2 < S && row_ok) ? __ldcg(sp + (size_t)(c0 + c2) * (TM * ACC_COLS / 4) + (size_t)q * TM) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int c2 = 0; c2 < 4; ++c2)
#pragma unroll
              for (int q = 0; q < 8; ++q) { acc[q].x += t[c2][q].x; acc[q].y += t[c2][q].y; acc[q].z += t[c2][q].z; acc[q].w += t[c2][q].w; }
          }
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            v[4 * q] = __float_as_uint(acc[q].x * rscale); v[4 * q + 1] = __float_as_uint(acc[q].y * rscale);
            v[4 * q + 2] = __float_as_uint(acc[q].z * rscale); v[4 * q + 3] = __float_as_uint(acc[q].w * rscale);
          }
        }
      };
      const EpiWarp ew{smem_base + (uint32_t)(ST * STAGE_BYTES) + (uint32_t)(quarter * kEpiStageBytes), m0 + quarter * 32, n, lane};
      // a split-K part finishes its share of the tile's epilogue passes; an unsplit tile all of them
      const int units = (EPI == EPI_STORE || EPI == EPI_RESIDUAL) ? OUT_COLS >> 5 : (EPI == EPI_SWIGLU ? OUT_COLS >> 5 : OUT_COLS >> 6);
      const int u0 = reduce ? part * units / S : 0, u1 = reduce ? (part + 1) * units / S : units;
      if (EPI == EPI_QKV_ROPE) {
        epilogue_qkv_rope(load_chunk, g, ew, n0, OUT_COLS, u0, u1);
      } else if (EPI == EPI_STORE || EPI == EPI_RESIDUAL) {
        epilogue_rows<EPI>(load_chunk, g, ew, n0, OUT_COLS, u0, u1);
      } else if (EPI == EPI_SWIGLU) {
        epilogue_swiglu(load_chunk, g, ew, n0, OUT_COLS, u0, u1);
      } else {  // EPI_LMSTATS: one thread owns a whole row of the tile, so the statistics need no exchange
#pragma unroll 1
        for (int half = 0; half < bn / 128; ++half) {         // statistics are kept per 128 columns
          float mx = -INFINITY, sum = 0.f; int arg = 0x7fffffff;
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t v[32];
            load_chunk(half * 128 + c * 32, v);
            const int col0 = n0 + half * 128 + c * 32;
            if (col0 >= g.N) continue;
            float cmx = -INFINITY; int carg = 0x7fffffff;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float f = __uint_as_float(v[j]);
              if (col0 + j < g.N && f > cmx) { cmx = f; carg = col0 + j; }   // ascending columns: first maximum wins
            }
            const float nmx = fmaxf(mx, cmx);
            float csum = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (col0 + j < g.N) csum += __expf(__uint_as_float(v[j]) - nmx);
            sum = sum * __expf(mx - nmx) + csum;                              // exp(-inf) = 0 on the first chunk
            if (cmx > mx) arg = carg;
            mx = nmx;
            if (g.logits && row_ok) {
              float* lp = g.logits + (size_t)row * g.N + col0;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j < g.N) lp[j] = __uint_as_float(v[j]);
            }
          }
          const int stile = nt * (bn / 128) + half;
          if (row_ok && stile < g.n_tiles) {
            const size_t o = (size_t)row * g.n_tiles + stile;
            g.st_max[o] = mx; g.st_sum[o] = sum; g.st_arg[o] = arg;
          }
        }
      }
      if (reduce) {
        // the part that finishes reading last puts both counters back for the next launch
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (warp == 2 && lane == 0) {
          const int old = atomicAdd(&g.sk_counters[g.sk_max_tiles + tile], 1);
          if (old == S - 1) { g.sk_counters[tile] = 0; g.sk_counters[g.sk_max_tiles + tile] = 0; }
        }
      }
      // hand the accumulator back to the MMA warp (a split-K part has done so already)
      if (!reduce) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty(buf));
      }
    }
  }
  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_acc, 2 * ACC_COLS);
  }
  if (g.clock_probe && blockIdx.x == 0 && threadIdx.x == 0) { g.clock_probe[2] = clock64(); g.clock_probe[3] = global_timer_ns(); }
}

template <int EPI>
int launch_one(const GemmArgs& g, int* status, cudaStream_t st) {
  const int smem = ST * STAGE_BYTES + 1024 + 4 * kEpiStageBytes;   // stage ring, alignment slack, epilogue staging
  static PerDevice attr_set;
  if (attr_set.first()) {
    D2C_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  }
  CUtensorMap tmA128, tmA64, tmA32, tmB, tmB2, tmB64;
  int rc = make_bf16_map(&tmA128, g.A, (uint64_t)g.max_rows, (uint64_t)g.K, (uint64_t)g.lda, 128);
  if (rc == D2C_OK) rc = make_bf16_map(&tmA64, g.A, (uint64_t)g.max_rows, (uint64_t)g.K, (uint64_t)g.lda, 64);
  if (rc == D2C_OK) rc = make_bf16_map(&tmA32, g.A, (uint64_t)g.max_rows, (uint64_t)g.K, (uint64_t)g.lda, 32);
  if (rc == D2C_OK) rc = make_bf16_map(&tmB, g.W, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.K, 128);
  if (rc == D2C_OK) rc = make_bf16_map(&tmB2, EPI == EPI_SWIGLU ? g.W2 : g.W, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.K, 128);
  if (rc == D2C_OK) rc = make_bf16_map(&tmB64, g.W, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.K, 64);
  if (rc != D2C_OK) return rc;
  TcParams p{g, status};
  const int out_cols = EPI == EPI_SWIGLU ? 128 : (EPI == EPI_LMSTATS ? 128 : (EPI == EPI_QKV_ROPE ? (g.q_dh > 64 ? g.q_dh : 64) : 64));   // narrowest tile
  const long long tiles = (long long)ceil_div(g.max_rows, TM) * ceil_div(g.N, out_cols);
  const int grid = (int)(tiles < sm_count_current() ? tiles : sm_count_current());
  D2C_LAUNCH((gemm_tc_kernel<EPI>), grid, TC_THREADS, smem, st, tmA128, tmA64, tmA32, tmB, tmB2, tmB64, p);
  return D2C_OK;
}
}  // namespace

bool gemm_tc_supported(const GemmArgs& g) {
  return !(g.max_rows < TM || g.N < 128 || g.K % TK != 0 || (g.lda & 7) || (g.N & 1) ||
           (reinterpret_cast<uintptr_t>(g.A) & 15) || (reinterpret_cast<uintptr_t>(g.W) & 15));
}

int launch_gemm_tc(const GemmArgs& g, GemmEpilogue epi, cudaStream_t st, int* status) {
  if (g.max_rows <= 0 || g.N <= 0) return D2C_OK;
  // shapes the TMA boxes cannot express fall back to the portable kernel
  if (!gemm_tc_supported(g)) {
    if (epi == EPI_QKV_ROPE) { set_global_error("gemm: the fused QKV epilogue needs the tcgen05 kernel"); return D2C_ESHAPE; }
    return launch_gemm_mma(g, epi, st);
  }
  switch (epi) {
    case EPI_STORE: return launch_one<EPI_STORE>(g, status, st);
    case EPI_RESIDUAL: return launch_one<EPI_RESIDUAL>(g, status, st);
    case EPI_SWIGLU: return launch_one<EPI_SWIGLU>(g, status, st);
    case EPI_LMSTATS: return launch_one<EPI_LMSTATS>(g, status, st);
    case EPI_QKV_ROPE: return launch_one<EPI_QKV_ROPE>(g, status, st);
  }
  return D2C_EINVAL;
}

}  // namespace d2c
