// Two-SM tcgen05 GEMM (cta_group::2) with the same fused epilogues as gemm_tc.cu.
//
// A cluster of two CTAs (two SMs) computes a 256 x 256 accumulator tile: CTA r of the pair owns rows
// [128 r, 128 r + 128) of the tile (its own TMEM holds them) and brings in only half of the weight tile,
// 128 of the 256 weight rows (for SwiGLU: CTA 0 the gate rows, CTA 1 the up rows).  One thread of the
// even CTA issues tcgen05.mma.cta_group::2 (M = 256, N = 256, K = 16): each SM's tensor core multiplies
// its own A rows by the whole B tile, whose halves it reads from both CTAs' shared memory.  Per SM and
// k-block that is 32 KB of TMA traffic instead of 48 KB, which lifts the shared-memory bound of the
// one-SM kernel.  TMA loads of both CTAs signal the even CTA's mbarrier (cta_group::2 form, no multicast
// load); stage release and accumulator hand-over reach both CTAs through multicast tcgen05.commit.
// Persistent: cluster c works on pair-tiles c, c + #clusters, ... with the row tile fastest.  Per CTA: warp 0
// loads, warp 1 issues the MMAs, warps 2-9 run the epilogue, two per TMEM lane quarter, each on half of a
// tile's columns (measured alone, the epilogue of the last tile of a launch is 3 us with one warp per quarter).
//
// Ragged waves: when the tile count does not fill whole waves of clusters, tiles are not handed out one by one.
// The clusters form groups of as many clusters as there are row tiles; the run of (column tile, pipeline stage)
// pairs is cut into equal shares, one per group, and cluster j of a group walks its group's share for row tile j
// (stream-K; the clusters of a group read the same weight k-blocks at about the same time, so the weights still
// cross from HBM once).  A cluster whose share starts inside a tile parks that tile's partial sums (fp32) in its
// own scratch slot first thing; the cluster holding the tile's first stages adds the parked parts in cluster
// order and runs the epilogue.  Nobody waits for work that has not started, and an owner works on its shared
// tile before its whole tiles, so the adding overlaps the next tile's MMAs.
//
// One thread issues every tcgen05.mma of a pair, and each step of its loop costs issue latency that does not
// shrink with the tile: about 115 clocks for the full-barrier test, 58 per MMA and 95 for the commit (measured
// with clock stamps on B200).  With one 64-wide k-block per pipeline stage that is ~560 clocks against the 512
// clocks four M256 x N256 x K16 instructions run, so the tensor pipe waited on the issuing thread.  A stage
// therefore holds two k-blocks (K = 128): eight MMAs per barrier round-trip, ~750 clocks of issue for 1024
// clocks of tensor work.
#include "common.cuh"
#include "epilogue_tiles.cuh"
#include "sm100_ptx.cuh"

namespace d2c {
namespace {

constexpr int TM = 128, TK = 64;
constexpr int EPI_WARPS = 8;                      // two per TMEM lane quarter: each takes half of a tile's columns
constexpr int TC_THREADS = 64 + 32 * EPI_WARPS;
constexpr int A_BYTES = TM * TK * 2;             // 16 KB: this CTA's rows
constexpr int BH_BYTES = 128 * TK * 2;           // 16 KB: this CTA's half of the weight tile
constexpr int SUB2 = A_BYTES + BH_BYTES;         // 32 KB per CTA and k-block
constexpr int KSUB = 2;                          // k-blocks per pipeline stage
constexpr int STAGE2 = KSUB * SUB2;              // 64 KB per CTA and stage
constexpr int ST2 = 3;
constexpr int ACC_COLS = 256;
constexpr uint32_t kPeerMask = 0xFEFFFFFFu;      // clears the CTA-rank bit of a shared::cluster address: the even CTA

__device__ int g_tc_status[4];

// ------------------------------------------------------------------------------------------- PTX
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
}
// TMA load of one CTA of a pair; completion bytes go to the even CTA's barrier.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar & kPeerMask), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma2_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are done.
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void mbar_arrive_even_cta(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar & kPeerMask) : "memory");
}

struct Tc2Params { GemmArgs g; int* status; };

// The pieces of work of one cluster, in order.  Round-robin: whole tiles (or (tile, part) items of a split-K
// launch) cl, cl + #clusters, ...  Stream-K: the end of the tile its group's share starts in, then the start of
// the tile the share ends in, then the whole tiles between.  All roles of both CTAs walk the same sequence.
struct WorkIter {
  int ncl, total, S, KT, KS;           // KS: pipeline stages per tile
  int item;                            // round-robin: tile = item % total, part = item / total
  int sk, MT, mt, phase;               // stream-K: on/off, row tiles, this cluster's row tile, next piece
  int nt_tail, s_tail0, s_tail1;       // column tile and stages of the piece the share starts with (empty if s_tail1 <= s_tail0)
  int nt_head, s_head1;                // column tile and end stage of the piece the share ends with (empty if 0)
  int nt_full, n_full;                 // whole column tiles
  __device__ void set_share(long long u0, long long u1) {
    const int nt0 = (int)(u0 / KS), s0 = (int)(u0 - (long long)nt0 * KS);
    nt_tail = nt0; s_tail0 = s_tail1 = 0;
    if (s0 > 0) { s_tail0 = s0; s_tail1 = (int)min((long long)KS, s0 + (u1 - u0)); u0 += s_tail1 - s_tail0; }
    nt_full = (int)(u0 / KS); n_full = (int)((u1 - u0) / KS);
    nt_head = nt_full + n_full; s_head1 = (int)((u1 - u0) - (long long)n_full * KS);
  }
  __device__ bool next(int& tile, int& part, int& kb0, int& kb1) {
    if (!sk) {
      if (item >= total * S) return false;
      tile = item % total; part = item / total;
      kb0 = part * KT / S; kb1 = (part + 1) * KT / S;
      item += ncl;
      return true;
    }
    part = 0;
    if (phase == 0) {
      phase = 1;
      if (s_tail1 > s_tail0) { tile = nt_tail * MT + mt; kb0 = s_tail0 * KSUB; kb1 = min(s_tail1 * KSUB, KT); return true; }
    }
    if (phase == 1) {
      phase = 2;
      if (s_head1 > 0) { tile = nt_head * MT + mt; kb0 = 0; kb1 = s_head1 * KSUB; return true; }
    }
    if (n_full > 0) { tile = nt_full * MT + mt; ++nt_full; --n_full; kb0 = 0; kb1 = KT; return true; }
    return false;
  }
};

template <int EPI>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmB64,
                const __grid_constant__ CUtensorMap tmB32, const Tc2Params p) {
  // Everything that does not read a predecessor's results (barriers, TMEM, descriptor prefetch) runs before
  // the wait on the preceding kernel, so it overlaps that kernel's tail.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const GemmArgs& g = p.g;
  const int cl = blockIdx.x >> 1, ncl = gridDim.x >> 1;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int* status = p.status ? p.status : g_tc_status;

  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = ((uint32_t)__cvta_generic_to_shared(smem_raw) + 1023u) & ~1023u;
  __shared__ __align__(8) uint64_t bars[2 * ST2 + 4];        // full[ST2], empty[ST2], acc_full[2], acc_empty[2]
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag, sk_last;
  const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (ST2 + s); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * ST2 + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * ST2 + 2 + b); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < ST2; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 2 * EPI_WARPS); }   // epilogue warps of both CTAs
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    prefetch_tensormap(&tmA); prefetch_tensormap(&tmB); prefetch_tensormap(&tmB2);
  }
  if (warp == 1) {
    tmem_alloc2((uint32_t)__cvta_generic_to_shared(&tmem_slot), 2 * ACC_COLS);
    tmem_relinquish2();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                        // both CTAs' barriers exist before anyone signals them
  tc_fence_after();
  const uint32_t tmem_acc = tmem_slot;
  volatile int* abortp = &abort_flag;

  // The live row count is read, and the weight boxes of the first ring fill are requested, before the wait on the
  // preceding kernel: neither is that kernel's output.  The count was written by the selection kernel at the start
  // of the step, and every kernel between it and a GEMM either waits for its own predecessor before it lets its
  // successor launch (the row kernels, attention) or is a GEMM behind such a kernel, so selection has completed
  // before any GEMM's CTA runs.  Everything the predecessor may have written (A rows, the residual, split-K
  // scratch) is touched only behind each role's own griddepcontrol.wait.
  const int n = *g.n_rows;
  const int MT = (max(n, 0) + 2 * TM - 1) / (2 * TM);
  const int KT = g.K / TK;
  const bool sk_ok = g.sk_partials != nullptr && g.sk_counters != nullptr;
  // Accumulator width of this launch.  With the issue latency out of the way a tile's time follows the bytes
  // each SM pulls from L2 per k-block (its 128 rows of A plus its half of the weight rows; about 90 GB/s per SM
  // measured), so a tile of half the width costs about 0.75 of a full one and a quarter-width one 0.73 (there
  // the issuing thread is the limit again).  Narrow tiles only pay when they fill the launch's waves of
  // clusters that much better; split-K (below) is preferred when few tiles are live.
  int bn = ACC_COLS;
  const int KS = (KT + KSUB - 1) / KSUB;                     // pipeline stages per tile
  // Stream-K (see the top of the file) when the evenly shared stages plus the hand-over (parking and adding a
  // partial tile, about four stages' time) undercut whole waves of tiles.  Returns the number of groups.  Only the
  // gate/up projection takes it: measured inside the step at 835 rows x d 4096 it gains 6 us of 143 there (and 6 %
  // at 488 rows), while the QKV and down projections, whose shares hold at most two whole tiles to hide the adding
  // behind, lose 3 and 8 us; the code below is written for every epilogue and was parity-tested with all of them.
  auto stream_k_groups = [&](int col_tiles) {
    if (EPI != EPI_SWIGLU || !sk_ok || MT <= 0 || 2 * MT > ncl || 2 * ncl > g.sk_max_tiles) return 0;
    const int G = ncl / MT;
    const long long stages = (long long)col_tiles * KS;
    if (stages < 4LL * G) return 0;                          // every group gets a share worth starting
    const long long shared = (stages + G - 1) / G + 4, in_waves = (long long)((MT * col_tiles + ncl - 1) / ncl) * KS;
    return shared < in_waves ? G : 0;
  };
  auto waves = [&](int out_cols) { const int t = MT * ((g.N + out_cols - 1) / out_cols); return (t + ncl - 1) / ncl; };
  const int t256 = MT * ((g.N + 255) / 256);
  // Few tiles: either K is split (below), which costs a split tile about 28 k-blocks' time for parking, meeting and
  // adding its parts, or the tiles are narrowed; with K = 4096 the narrow tiles win, with K = 12288 the split.
  const int s256 = (sk_ok && 2 * t256 <= ncl && KT >= 16 && 2 * t256 <= g.sk_max_tiles) ? max(1, min(min(ncl / max(t256, 1), KT / 8), 4)) : 1;
  if (MT > 0 && (EPI == EPI_STORE || EPI == EPI_RESIDUAL) && stream_k_groups((g.N + 255) / 256) == 0) {
    float best = s256 > 1 ? ((float)((KT + s256 - 1) / s256) + 28.f) / (float)KT : (float)waves(256);
    if ((float)waves(128) * 0.75f < best) { best = (float)waves(128) * 0.75f; bn = 128; }
    if ((float)waves(64) * 0.73f < best) { bn = 64; }
  }
  const int OUT_COLS = (EPI == EPI_SWIGLU) ? bn / 2 : bn;    // output columns per pair-tile
  const int NT = (g.N + OUT_COLS - 1) / OUT_COLS;
  const int total = MT * NT;                                 // 0 when no row is live: every role loop is empty
  // Split-K when there are fewer pair-tiles than clusters: K is cut into S equal parts, one (tile, part)
  // item per cluster; every CTA parks its 128 rows of fp32 partial sums in scratch and, per (tile, CTA
  // rank), the part that arrives last adds all parts in part order (no waiting, deterministic).
  int S = 1;
  if (sk_ok && total > 0 && total < ncl && 2 * total <= g.sk_max_tiles)
    S = max(1, min(min(ncl / total, KT / 8), 4));
  const int G = (S == 1 && bn == ACC_COLS) ? stream_k_groups(NT) : 0;
  const long long sk_stages = (long long)NT * KS;            // stream-K: group q takes stages [q, q + 1) * sk_stages / G
  WorkIter work;
  work.ncl = ncl; work.total = max(total, 1); work.S = total > 0 ? S : 0; work.KT = KT; work.KS = KS; work.item = cl;
  work.sk = G > 0; work.MT = max(MT, 1); work.mt = cl % max(MT, 1); work.phase = 0;
  const int grp = cl / max(MT, 1);
  if (G > 0) {
    if (grp < G) work.set_share((long long)grp * sk_stages / G, (long long)(grp + 1) * sk_stages / G);
    else work.set_share(0, 0);                               // clusters beyond the last whole group have no share
  }
  const int b_box_rows = bn / 2;                             // weight rows this CTA brings in per k-block

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      uint32_t it = 0;                                        // stages issued so far (ring position)
      bool ok = true;
      const uint32_t kb_bytes = 2 * (A_BYTES + (uint32_t)b_box_rows * TK * 2);   // both CTAs' boxes of one k-block
      const CUtensorMap* mb = (EPI == EPI_SWIGLU && rank == 1) ? &tmB2 : (bn == 256 ? &tmB : (bn == 128 ? &tmB64 : &tmB32));
      int tile, part, k0, k1;
      uint32_t early = 0;                                     // stages whose byte count and weight boxes are already out
      {
        WorkIter w = work;
        while (early < (uint32_t)ST2 && w.next(tile, part, k0, k1)) {
          const int n0 = (tile / MT) * OUT_COLS;
          const int brow = (EPI == EPI_SWIGLU) ? n0 : n0 + (int)rank * (bn / 2);
          for (int kt = k0; kt < k1 && early < (uint32_t)ST2; kt += KSUB, ++early) {
            const int nsub = min(KSUB, k1 - kt);
            if (leader) mbar_expect_tx(full_bar(early), (uint32_t)nsub * kb_bytes);
#pragma unroll
            for (int u = 0; u < KSUB; ++u)
              if (u < nsub) tma_load_2d_pair(smem_base + early * STAGE2 + u * SUB2 + A_BYTES, mb, (kt + u) * TK, brow, full_bar(early));
          }
        }
      }
      asm volatile("griddepcontrol.wait;" ::: "memory");
      if (g.clock_probe && blockIdx.x == 0) { g.clock_probe[0] = clock64(); g.clock_probe[1] = global_timer_ns(); }
      WorkIter w = work;
      while (ok && w.next(tile, part, k0, k1)) {
        const int m0 = (tile % MT) * 2 * TM + (int)rank * TM, n0 = (tile / MT) * OUT_COLS;
        const int brow = (EPI == EPI_SWIGLU) ? n0 : n0 + (int)rank * (bn / 2);
        for (int kt = k0; kt < k1; kt += KSUB, ++it) {
          const int s = it % ST2;
          const int nsub = min(KSUB, k1 - kt);
          const bool fresh = it >= early;                     // not one of the stages started before the wait
          if (!mbar_wait(empty_bar(s), ((it / ST2) & 1) ^ 1, abortp, status, 31)) { ok = false; break; }
          if (leader && fresh) mbar_expect_tx(full_bar(s), (uint32_t)nsub * kb_bytes);
#pragma unroll
          for (int u = 0; u < KSUB; ++u) {
            if (u < nsub) {
              const uint32_t sa = smem_base + s * STAGE2 + u * SUB2, sb = sa + A_BYTES;
              tma_load_2d_pair(sa, &tmA, (kt + u) * TK, m0, full_bar(s));
              if (fresh) tma_load_2d_pair(sb, mb, (kt + u) * TK, brow, full_bar(s));
            }
          }
        }
      }
      if (*abortp && leader) {
        for (uint32_t j = it > (uint32_t)ST2 ? it - ST2 : 0; j < it; ++j) {
          const long long t0 = clock64();
          while (!mbar_try_wait(full_bar(j % ST2), (j / ST2) & 1) && clock64() - t0 < kWaitCycles) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (even CTA only)
    if (lane == 0 && leader) {
      uint32_t tcount = 0;
      bool ok = true;
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((256u >> 4) << 24);
      const uint64_t desc0 = smem_desc_sw128(smem_base);     // A operand of stage 0, k-block 0
      int st = 0; uint32_t ph = 0;                           // ring position of the next stage
      WorkIter w = work;
      int tile, part, k0, k1;
      for (; ok && w.next(tile, part, k0, k1); ++tcount) {
        const int nk = k1 - k0;
        const uint32_t buf = tcount & 1, use = tcount >> 1;
        if (!mbar_wait(acc_empty(buf), (use & 1) ^ 1, abortp, status, 34)) { ok = false; break; }
        const uint32_t tacc = tmem_acc + buf * ACC_COLS;
        for (int j = 0; j < nk; j += KSUB) {
          const int nsub = min(KSUB, nk - j);
          if (!mbar_wait(full_bar(st), ph, abortp, status, 32)) { ok = false; break; }
          tc_fence_after();
          const uint64_t adesc = desc0 + (uint64_t)(st * (STAGE2 >> 4)), bdesc = adesc + (A_BYTES >> 4);
#pragma unroll
          for (int u = 0; u < KSUB; ++u) {
            if (u < nsub) {
#pragma unroll
              for (int k = 0; k < TK / 16; ++k)               // +32 bytes per K=16 slice inside the swizzle atom
                umma2_bf16(tacc, adesc + u * (SUB2 >> 4) + 2 * k, bdesc + u * (SUB2 >> 4) + 2 * k, idesc, (j | u | k) != 0);
            }
          }
          umma2_commit_both(empty_bar(st));                   // both CTAs may refill this stage
          if (++st == ST2) { st = 0; ph ^= 1; }
        }
        if (ok) umma2_commit_both(acc_full(buf));             // both CTAs' epilogues may read their rows
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    const int quarter = warp & 3;                             // TMEM lanes this warp may touch
    const int ehalf = (warp - 2) >> 2;                        // which half of a tile's columns it takes
    asm volatile("griddepcontrol.wait;" ::: "memory");        // the residual, the scratch and the outputs belong to the step's chain
    const int lrow = quarter * 32 + lane;
    uint32_t tcount = 0;
    WorkIter w = work;
    int tile, part, k0, k1;
    for (; w.next(tile, part, k0, k1); ++tcount) {
      const uint32_t buf = tcount & 1, use = tcount >> 1;
      const int m0 = (tile % MT) * 2 * TM + (int)rank * TM, nt = tile / MT, n0 = nt * OUT_COLS;
      const int row = m0 + lrow;
      const bool row_ok = row < n;
      const float rscale = folded_row_scale(g, row, row_ok);     // RMSNorm of the A rows folded into this GEMM (1 if none)
      const bool sk_piece = S == 1 && (k0 > 0 || k1 < KT);       // part of a tile shared between clusters (stream-K)
      // a wait that gave up ends the loop for the whole warp (the tcgen05.ld below is warp-collective) ...
      const bool got = __all_sync(0xffffffffu, mbar_wait(acc_full(buf), use & 1, abortp, status, 33));
      if (S > 1 || sk_piece) {
        // ... and, where the epilogue warps meet at named barriers below, for all of them together
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (*abortp) break;
      } else if (!got) {
        break;
      }
      tc_fence_after();
      const uint32_t tbase = tmem_acc + buf * ACC_COLS + ((uint32_t)(quarter * 32) << 16);
      bool reduce = false;
      int sk_parts = 0;                                          // parked parts this tile owner adds to its own
      const size_t slot_floats = (size_t)TM * ACC_COLS;
      const bool parks = S > 1 || (sk_piece && k0 > 0);          // this piece's sums go to scratch
      if (parks) {
        const int acc_cols = bn;
        const size_t slot = S > 1 ? (size_t)(tile * S + part) * 2 + rank : (size_t)cl * 2 + rank;
        float4* mine = reinterpret_cast<float4*>(g.sk_partials + slot * slot_floats);
#pragma unroll 1
        for (int c = ehalf * (acc_cols / 64); c < (ehalf + 1) * (acc_cols / 64); ++c) {
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
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (S == 1) {
          // stream-K: tell the tile's owner (same row tile and CTA rank in the group holding the tile's first stage)
          if (warp == 2 && lane == 0) {
            for (int w4 = 0; w4 < EPI_WARPS; ++w4) mbar_arrive_even_cta(acc_empty(buf));
            int og = grp - 1;
            while (og > 0 && (long long)og * sk_stages / G > (long long)nt * KS) --og;
            atomicAdd(&g.sk_counters[(og * MT + work.mt) * 2 + rank], 1);
          }
          continue;
        }
        if (warp == 2 && lane == 0) {
          for (int w4 = 0; w4 < EPI_WARPS; ++w4) mbar_arrive_even_cta(acc_empty(buf));
          const int old = atomicAdd(&g.sk_counters[tile * 2 + rank], 1);
          const int last = (old == S - 1) ? 1 : 0;
          if (last) g.sk_counters[tile * 2 + rank] = 0;      // every part has arrived: ready for the next launch
          sk_last = last;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        reduce = sk_last != 0;
        asm volatile("bar.sync 1, 256;" ::: "memory");      // sk_last may be rewritten only after everyone has read it
        if (!reduce) continue;
        __threadfence();
      } else if (sk_piece) {
        // stream-K tile owner: the groups after this one hold the rest of the tile's stages, up to the tile's end
        for (int g2 = grp + 1; g2 < G && (long long)g2 * sk_stages / G < (long long)(nt + 1) * KS; ++g2) ++sk_parts;
        if (warp == 2 && lane == 0) {
          volatile int32_t* cnt = g.sk_counters + cl * 2 + rank;
          const long long t0 = clock64();
          bool there = true;
          while (*cnt < sk_parts) {
            if (*abortp || clock64() - t0 > kWaitCycles) { there = false; break; }
            __nanosleep(64);
          }
          if (there) *cnt = 0;                                 // all parts are in: ready for the next launch
          else if (!*abortp) { *abortp = 1; if (atomicCAS(status, 0, D2C_ETIMEOUT) == 0) status[1] = 35; }
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (*abortp) break;
        __threadfence();
      }
      auto load_chunk = [&](int col, uint32_t (&v)[32]) {     // 32 accumulator columns of this thread's row
        if (!reduce) {
          tmem_ld32(tbase + col, v);
          tmem_ld_wait();
#pragma unroll 1
          for (int j = 0; j < sk_parts; ++j) {                  // parked parts of this row tile, in group order
            const float4* sp = reinterpret_cast<const float4*>(g.sk_partials + ((size_t)(cl + (1 + j) * MT) * 2 + rank) * slot_floats) +
                               (size_t)(col >> 2) * TM + lrow;
            float4 t[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) t[q] = row_ok ? __ldcg(sp + (size_t)q * TM) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              v[4 * q] = __float_as_uint(__uint_as_float(v[4 * q]) + t[q].x); v[4 * q + 1] = __float_as_uint(__uint_as_float(v[4 * q + 1]) + t[q].y);
              v[4 * q + 2] = __float_as_uint(__uint_as_float(v[4 * q + 2]) + t[q].z); v[4 * q + 3] = __float_as_uint(__uint_as_float(v[4 * q + 3]) + t[q].w);
            }
          }
          if (g.in_ssq) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * rscale);
          }
        } else {
          float4 t[4][8];
          const float4* sp = reinterpret_cast<const float4*>(g.sk_partials + ((size_t)(tile * S) * 2 + rank) * slot_floats) +
                             (size_t)(col >> 2) * TM + lrow;
#pragma unroll
          for (int c2 = 0; c2 < 4; ++c2)
#pragma unroll
            for (int q = 0; q < 8; ++q)
              t[c2][q] = (c2 < S && row_ok) ? __ldcg(sp + (size_t)c2 * (2 * slot_floats / 4) + (size_t)q * TM) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            float4 acc = t[0][q];
#pragma unroll
            for (int c2 = 1; c2 < 4; ++c2) { acc.x += t[c2][q].x; acc.y += t[c2][q].y; acc.z += t[c2][q].z; acc.w += t[c2][q].w; }
            v[4 * q] = __float_as_uint(acc.x * rscale); v[4 * q + 1] = __float_as_uint(acc.y * rscale);
            v[4 * q + 2] = __float_as_uint(acc.z * rscale); v[4 * q + 3] = __float_as_uint(acc.w * rscale);
          }
        }
      };
      const EpiWarp ew{smem_base + (uint32_t)(ST2 * STAGE2) + (uint32_t)((warp - 2) * kEpiStageBytes), m0 + quarter * 32, n, lane};
      if (EPI == EPI_QKV_ROPE) {
        const int units = OUT_COLS >> 6;
        epilogue_qkv_rope(load_chunk, g, ew, n0, OUT_COLS, ehalf * units / 2, (ehalf + 1) * units / 2);
      } else if (EPI == EPI_STORE || EPI == EPI_RESIDUAL) {
        const int units = OUT_COLS >> 5;
        epilogue_rows<EPI>(load_chunk, g, ew, n0, OUT_COLS, ehalf * units / 2, (ehalf + 1) * units / 2);
      } else if (EPI == EPI_SWIGLU) {
        const int units = OUT_COLS >> 5;
        epilogue_swiglu(load_chunk, g, ew, n0, OUT_COLS, ehalf * units / 2, (ehalf + 1) * units / 2);
      } else if (ehalf == 0) {  // EPI_LMSTATS: one thread owns a whole row of the tile, so the statistics need no exchange
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {         // statistics are kept per 128 columns
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
          const int stile = nt * 2 + half;
          if (row_ok && stile < g.n_tiles) {
            const size_t o = (size_t)row * g.n_tiles + stile;
            g.st_max[o] = mx; g.st_sum[o] = sum; g.st_arg[o] = arg;
          }
        }
      }
      // hand the accumulator back to the MMA thread in the even CTA (a split-K part has done so already)
      if (!reduce) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_even_cta(acc_empty(buf));
      }
    }
  }
  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                        // nobody leaves while the peer may still signal it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc2(tmem_acc, 2 * ACC_COLS);
  }
  if (g.clock_probe && blockIdx.x == 0 && threadIdx.x == 0) { g.clock_probe[2] = clock64(); g.clock_probe[3] = global_timer_ns(); }
}

template <int EPI>
int launch_one(const GemmArgs& g, int* status, cudaStream_t st) {
  const int smem = ST2 * STAGE2 + 1024 + EPI_WARPS * kEpiStageBytes;   // stage ring, alignment slack, epilogue staging
  static PerDevice attr_set;
  if (attr_set.first()) {
    D2C_CUDA_OK(cudaFuncSetAttribute(gemm_tc2_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  }
  CUtensorMap tmA, tmB, tmB2, tmB64, tmB32;
  int rc = make_bf16_map(&tmA, g.A, (uint64_t)g.max_rows, (uint64_t)g.K, (uint64_t)g.lda, 128);
  if (rc == D2C_OK) rc = make_bf16_map(&tmB, g.W, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.K, 128);
  if (rc == D2C_OK) rc = make_bf16_map(&tmB2, EPI == EPI_SWIGLU ? g.W2 : g.W, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.K, 128);
  if (rc == D2C_OK) rc = make_bf16_map(&tmB64, g.W, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.K, 64);
  if (rc == D2C_OK) rc = make_bf16_map(&tmB32, g.W, (uint64_t)g.N, (uint64_t)g.K, (uint64_t)g.K, 32);
  if (rc != D2C_OK) return rc;
  Tc2Params p{g, status};
  const int out_cols = (EPI == EPI_STORE || EPI == EPI_RESIDUAL) ? 64 : (EPI == EPI_SWIGLU ? 128 : 256);   // narrowest tile (QKV: 256)
  const long long tiles = (long long)ceil_div(g.max_rows, 2 * TM) * ceil_div(g.N, out_cols);
  const int pairs = (int)(tiles < sm_count_current() / 2 ? tiles : sm_count_current() / 2);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  D2C_CUDA_OK(cudaLaunchKernelEx(&cfg, gemm_tc2_kernel<EPI>, tmA, tmB, tmB2, tmB64, tmB32, p));
  count_launch(1);
  return D2C_OK;
}
}  // namespace

// Shapes the pair kernel takes; everything else goes to the one-SM kernel.
bool gemm_tc2_supported(const GemmArgs& g) {
  return g.max_rows >= 2 * TM && g.N >= 256 && g.K % TK == 0 && (g.lda & 7) == 0 && (g.N & 1) == 0 &&
         (reinterpret_cast<uintptr_t>(g.A) & 15) == 0 && (reinterpret_cast<uintptr_t>(g.W) & 15) == 0;
}

int launch_gemm_tc2(const GemmArgs& g, GemmEpilogue epi, cudaStream_t st, int* status) {
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
