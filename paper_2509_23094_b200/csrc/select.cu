// Two-stage token selection of d2Cache (Section 4.1-4.2) and the compaction of the selected set.
//
// One CTA per sequence.  Every sum that decides an index is an integer sum, so the result does
// not depend on the order in which threads add:
//   stage 1 (Eq. 3-4): D(i) = sum over known j of phi(|i-j|), with phi tabulated as round(phi*2^30);
//                      key = fp32(D) * conf (one multiply); the k largest keys among masked positions.
//   stage 2 (after Eq. 9): candidates sorted by score c_j (ties: lower position first); the shortest
//                      prefix whose mass sum floor(c_j*2^32) exceeds p times the total.
// Sorting is a bitonic network over 64-bit words (score bits << 32 | ~position) in shared memory.
#include <math.h>

#include "common.cuh"

namespace d2c {

static constexpr int kSelThreads = 1024;
static constexpr int kPhiMax = 512;              // phi entries kept in shared memory; a wider window reads the rest from global memory
enum : uint8_t { F_SEL = 1, F_MSTAR = 2 };

// Descending bitonic sort of n 64-bit words in shared memory by the whole block.  Pair p of a stage exchanges
// elements lo = 2p - (p & (stride - 1)) and lo + stride; for stride <= 32 the pairs of one warp touch only that
// warp's 64 elements, so only the stages that reach further need the block to synchronise.  (Keeping the words in
// registers and exchanging by warp shuffles was no faster: with 32 warps on one SM the stages are bound by
// instruction issue, not by the shared-memory round trip.)
__device__ __forceinline__ void bitonic_sort_desc(uint64_t* buf, int n) {
  bool wide_before = true;                                  // the caller's writes count as a block-wide stage
  for (int size = 2; size <= n; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      const bool wide = stride >= 64;
      if (wide || wide_before) __syncthreads(); else __syncwarp();
      wide_before = wide;
      for (int t = threadIdx.x; t < (n >> 1); t += blockDim.x) {
        const int lo = 2 * t - (t & (stride - 1));
        const int hi = lo + stride;
        const bool desc = (lo & size) == 0;
        const uint64_t x = buf[lo], y = buf[hi];
        if ((x < y) == desc) { buf[lo] = y; buf[hi] = x; }
      }
    }
  }
  __syncthreads();
}

// Exclusive block scan of one value per thread; returns the exclusive prefix, *total gets the sum.
template <typename T>
__device__ __forceinline__ T block_exclusive_scan(T v, T* warp_buf, T* total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  T inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    T up = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += up;
  }
  if (lane == 31) warp_buf[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    T w = lane < nw ? warp_buf[lane] : T(0);
    T winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      T up = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += up;
    }
    warp_buf[lane] = winc - w;                     // exclusive prefix of warp sums
    if (lane == 31) *total = winc;
  }
  __syncthreads();
  T res = warp_buf[wid] + inc - v;
  __syncthreads();
  return res;
}

// NaN, negative and infinite scores count as 0; finite ones are capped at 2^18 so that the fixed-point
// mass of 8192 positions stays inside 64 bits.
__device__ __forceinline__ float clean_score(float x) { return (x > 0.f && x < INFINITY) ? fminf(x, 262144.f) : 0.f; }

__global__ void __launch_bounds__(kSelThreads) select_kernel(SelectArgs a, int P2) {
  pdl_prologue();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint64_t* sbuf = reinterpret_cast<uint64_t*>(smem_raw);
  uint8_t* flags = reinterpret_cast<uint8_t*>(sbuf + P2);
  uint8_t* smask = flags + a.seq_len;
  __shared__ uint64_t warp_buf64[32];
  __shared__ uint64_t s_total64;
  __shared__ int warp_buf32[32];
  __shared__ int s_total32, s_cnt, s_take;
  __shared__ uint32_t s_phi[kPhiMax];                          // the non-zero head of the phi table (window +-65 at sigma 10)

  const int b = blockIdx.x, L = a.seq_len, tid = threadIdx.x;
  const uint8_t* mask = a.mask + (size_t)b * L;
  const float* conf = a.conf + (size_t)b * L;
  const float* cs = a.c + (size_t)b * L;
  const float* okey = a.override_key ? a.override_key + (size_t)b * L : nullptr;

  // stage 1 may be confined to one block of positions (semi-autoregressive decoding); whole sequence otherwise
  const int blk_lo = a.block_hi > a.block_lo ? a.block_lo : 0, blk_hi = a.block_hi > a.block_lo ? a.block_hi : L;
  for (int i = tid; i < L; i += kSelThreads) { smask[i] = mask[i] ? 1 : 0; flags[i] = 0; }
  for (int r = tid; r < min(a.phi_len, kPhiMax); r += kSelThreads) s_phi[r] = a.phi_q30[r];
  if (tid == 0) { s_cnt = 0; }
  __syncthreads();

  if (a.stage2_candidates == 0) {
    // ---- default candidate mode: masked positions (stage 1) and known positions (stage 2) are disjoint,
    //      so one sort orders both: bit 63 = masked, bits 62..32 = score bits, bits 31..0 = ~position ----
    for (int i = tid; i < P2; i += kSelThreads) {
      uint64_t comp = 0;
      if (i < L) {
        float key = 0.f;
        if (smask[i] && i >= blk_lo && i < blk_hi) {
          if (okey) {
            key = clean_score(okey[i]);
          } else {
            unsigned long long dq = 0;
            for (int r = 1; r < a.phi_len; ++r) {
              const int lo = i - r, hi = i + r;
              int known = 0;
              if (lo >= 0) known += 1 - smask[lo];
              if (hi < L) known += 1 - smask[hi];
              dq += (unsigned long long)(r < kPhiMax ? s_phi[r] : a.phi_q30[r]) * (unsigned)known;
            }
            const float D = __ull2float_rn(dq) * 9.31322574615478515625e-10f;   // * 2^-30, exact
            key = clean_score(__fmul_rn(D, conf[i]));
          }
          comp = (1ull << 63) | ((uint64_t)__float_as_uint(key) << 32) | (uint64_t)(0xFFFFFFFFu - (uint32_t)i);
        } else if (!smask[i]) {
          comp = ((uint64_t)__float_as_uint(clean_score(cs[i])) << 32) | (uint64_t)(0xFFFFFFFFu - (uint32_t)i);
        }                                                           // masked outside the block: in neither stage
        a.key[(size_t)b * L + i] = key;
      }
      sbuf[i] = comp;
    }
    bitonic_sort_desc(sbuf, P2);
    if (tid == 0) { s_cnt = 0; s_take = 0; }                      // s_take doubles as the masked count here
    __syncthreads();
    for (int t = tid; t < P2; t += kSelThreads) {
      const uint64_t x = sbuf[t], y = t + 1 < P2 ? sbuf[t + 1] : 0ull;
      if ((x >> 63) && !(y >> 63)) s_take = t + 1;
      if (x != 0 && y == 0) s_cnt = t + 1;
    }
    __syncthreads();
    const int nm = s_take, ntot = s_cnt;
    {
      const int take = min(max(a.k, 0), nm);
      for (int t = tid; t < take; t += kSelThreads) {
        const uint32_t idx = 0xFFFFFFFFu - (uint32_t)(sbuf[t] & 0xFFFFFFFFull);
        flags[idx] = F_SEL | F_MSTAR;
      }
    }
    const int per = max(1, P2 / kSelThreads);
    const int t0 = tid * per;
    unsigned long long local = 0;
    if (t0 < P2) {
      for (int e = 0; e < per; ++e) {
        const uint64_t x = sbuf[t0 + e];
        if (!(x >> 63)) local += __double2ull_rd((double)__uint_as_float((uint32_t)(x >> 32)) * 4294967296.0);
      }
    }
    const unsigned long long excl =
        block_exclusive_scan<unsigned long long>(local, (unsigned long long*)warp_buf64, (unsigned long long*)&s_total64);
    if (tid == 0) s_take = (a.p > 0.f) ? ntot : nm;                // end (exclusive) of the selected candidates
    __syncthreads();
    if (a.p > 0.f && t0 < P2) {
      const double thr = __dmul_rn((double)a.p, __ull2double_rn(s_total64));
      unsigned long long run = excl;
      for (int e = 0; e < per; ++e) {
        const int t = t0 + e;
        if (t >= ntot) break;
        if (t < nm) continue;
        run += __double2ull_rd((double)__uint_as_float((uint32_t)(sbuf[t] >> 32)) * 4294967296.0);
        if (__ull2double_rn(run) > thr) { atomicMin(&s_take, t + 1); break; }
      }
    }
    __syncthreads();
    {
      const int end = s_take;
      for (int t = nm + tid; t < end; t += kSelThreads) {
        const uint32_t idx = 0xFFFFFFFFu - (uint32_t)(sbuf[t] & 0xFFFFFFFFull);
        flags[idx] |= F_SEL;
      }
    }
    __syncthreads();
  } else {
  // ---- stage 1: keys ----
  for (int i = tid; i < P2; i += kSelThreads) {
    uint64_t comp = 0;
    if (i < L) {
      float key = 0.f;
      if (smask[i] && i >= blk_lo && i < blk_hi) {
        if (okey) {
          key = clean_score(okey[i]);
        } else {
          unsigned long long dq = 0;
          for (int r = 1; r < a.phi_len; ++r) {
            const int lo = i - r, hi = i + r;
            int known = 0;
            if (lo >= 0) known += 1 - smask[lo];
            if (hi < L) known += 1 - smask[hi];
            dq += (unsigned long long)(r < kPhiMax ? s_phi[r] : a.phi_q30[r]) * (unsigned)known;
          }
          const float D = __ull2float_rn(dq) * 9.31322574615478515625e-10f;   // * 2^-30, exact
          key = clean_score(__fmul_rn(D, conf[i]));
        }
        comp = ((uint64_t)__float_as_uint(key) << 32) | (uint64_t)(0xFFFFFFFFu - (uint32_t)i);
      }
      a.key[(size_t)b * L + i] = key;
    }
    sbuf[i] = comp;
  }
  bitonic_sort_desc(sbuf, P2);
  for (int t = tid; t < P2; t += kSelThreads)
    if (sbuf[t] != 0 && (t + 1 == P2 || sbuf[t + 1] == 0)) s_cnt = t + 1;
  __syncthreads();
  {
    const int take = min(max(a.k, 0), s_cnt);
    for (int t = tid; t < take; t += kSelThreads) {
      const uint32_t idx = 0xFFFFFFFFu - (uint32_t)(sbuf[t] & 0xFFFFFFFFull);
      flags[idx] = F_SEL | F_MSTAR;
    }
  }
  __syncthreads();

  // ---- stage 2: top-p over the candidates ----
  if (tid == 0) s_cnt = 0;
  for (int j = tid; j < P2; j += kSelThreads) {
    uint64_t comp = 0;
    if (j < L) {
      const bool cand = a.stage2_candidates == 0 ? (smask[j] == 0) : ((flags[j] & F_MSTAR) == 0);
      if (cand) comp = ((uint64_t)__float_as_uint(clean_score(cs[j])) << 32) | (uint64_t)(0xFFFFFFFFu - (uint32_t)j);
    }
    sbuf[j] = comp;
  }
  bitonic_sort_desc(sbuf, P2);
  for (int t = tid; t < P2; t += kSelThreads)
    if (sbuf[t] != 0 && (t + 1 == P2 || sbuf[t + 1] == 0)) s_cnt = t + 1;
  __syncthreads();
  {
    const int ncand = s_cnt;
    const int per = max(1, P2 / kSelThreads);
    const int t0 = tid * per;
    unsigned long long local = 0;
    if (t0 < P2) {
      for (int e = 0; e < per; ++e) {
        const float cv = __uint_as_float((uint32_t)(sbuf[t0 + e] >> 32));
        local += __double2ull_rd((double)cv * 4294967296.0);
      }
    }
    const unsigned long long excl =
        block_exclusive_scan<unsigned long long>(local, (unsigned long long*)warp_buf64,
                                                 (unsigned long long*)&s_total64);
    if (tid == 0) s_take = (a.p > 0.f) ? ncand : 0;
    __syncthreads();
    if (a.p > 0.f && t0 < P2) {
      const double thr = __dmul_rn((double)a.p, __ull2double_rn(s_total64));
      unsigned long long run = excl;
      for (int e = 0; e < per; ++e) {
        const int t = t0 + e;
        if (t >= ncand) break;
        const float cv = __uint_as_float((uint32_t)(sbuf[t] >> 32));
        run += __double2ull_rd((double)cv * 4294967296.0);
        if (__ull2double_rn(run) > thr) { atomicMin(&s_take, t + 1); break; }
      }
    }
    __syncthreads();
    const int take = s_take;
    for (int t = tid; t < take; t += kSelThreads) {
      const uint32_t idx = 0xFFFFFFFFu - (uint32_t)(sbuf[t] & 0xFFFFFFFFull);
      flags[idx] |= F_SEL;
    }
  }
  __syncthreads();

  }

  // ---- forced rows ----
  if (a.forced && a.forced_off) {
    const int f0 = a.forced_off[b], f1 = a.forced_off[b + 1];
    for (int f = f0 + tid; f < f1; f += kSelThreads) {
      const int pos = a.forced[f];
      if (pos >= 0 && pos < L) flags[pos] = flags[pos] | F_SEL;   // duplicates write the same value
    }
  }
  __syncthreads();

  // ---- ranks of the selected positions (ascending) and of the selected masked positions ----
  {
    const int per = (L + kSelThreads - 1) / kSelThreads;
    const int j0 = tid * per;
    int local = 0;                                     // low 16 bits: selected, high 16: selected & masked
    for (int e = 0; e < per; ++e) {
      const int j = j0 + e;
      if (j < L && (flags[j] & F_SEL)) local += 1 + (smask[j] ? (1 << 16) : 0);
    }
    int excl = block_exclusive_scan<int>(local, warp_buf32, &s_total32);
    for (int e = 0; e < per; ++e) {
      const int j = j0 + e;
      if (j >= L) break;
      int rs = -1, rl = -1;
      if (flags[j] & F_SEL) {
        rs = excl & 0xFFFF;
        if (smask[j]) { rl = excl >> 16; excl += 1 << 16; }
        excl += 1;
      }
      a.rank_s[(size_t)b * L + j] = rs;
      a.rank_lm[(size_t)b * L + j] = rl;
      if (a.batch == 1) {
        // one sequence: its ranks are the global row numbers, so the second kernel's work is done here
        if (rs >= 0) {
          a.sel_idx[rs] = j; a.row_seq[rs] = 0;
          if (rl >= 0) a.lm_rows[rl] = rs;
        }
        a.slot_of_pos[j] = rs;
      }
    }
    if (tid == 0) { a.n_b[b] = s_total32 & 0xFFFF; a.nm_b[b] = s_total32 >> 16; }
    if (a.batch == 1) {
      if (tid == 0) {
        a.row_off[0] = 0; a.lm_off[0] = 0; a.row_off[1] = s_total32 & 0xFFFF; a.lm_off[1] = s_total32 >> 16;
        if (a.n_host) *a.n_host = s_total32 & 0xFFFF;
      }
    }
  }
}

// Turns the per-sequence ranks into global row numbers.
__global__ void __launch_bounds__(256) select_finalize_kernel(SelectArgs a) {
  pdl_prologue();
  const int b = blockIdx.y, L = a.seq_len;
  int off = 0, lmoff = 0;
  for (int bb = 0; bb < b; ++bb) { off += a.n_b[bb]; lmoff += a.nm_b[bb]; }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    a.row_off[b] = off; a.lm_off[b] = lmoff;
    if (b == a.batch - 1) {
      a.row_off[a.batch] = off + a.n_b[b]; a.lm_off[a.batch] = lmoff + a.nm_b[b];
      if (a.n_host) *a.n_host = off + a.n_b[b];
    }
  }
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < L; j += gridDim.x * blockDim.x) {
    const int rs = a.rank_s[(size_t)b * L + j];
    int slot = -1;
    if (rs >= 0) {
      slot = off + rs;
      a.sel_idx[slot] = j;
      a.row_seq[slot] = b;
      const int rl = a.rank_lm[(size_t)b * L + j];
      if (rl >= 0) a.lm_rows[lmoff + rl] = slot;
    }
    a.slot_of_pos[(size_t)b * L + j] = slot;
  }
}

int launch_select(const SelectArgs& a, cudaStream_t st) {
  if (a.batch <= 0) return D2C_OK;
  // a sequence of 65535 selected rows would overflow the packed 16-bit counters
  if (a.seq_len > 8192) { set_global_error("select: seq_len %d > 8192", a.seq_len); return D2C_ECAPACITY; }
  int P2 = 32;
  while (P2 < a.seq_len) P2 <<= 1;
  const size_t smem = (size_t)P2 * 8 + 2 * (size_t)a.seq_len;
  static PerDevice attr_set;
  if (attr_set.first()) {
    D2C_CUDA_OK(cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 8192 * 8 + 2 * 8192));
  }
  D2C_LAUNCH((select_kernel), a.batch, kSelThreads, smem, st, a, P2);
  if (a.batch > 1) {
    dim3 grid(ceil_div(a.seq_len, 256), a.batch);
    D2C_LAUNCH((select_finalize_kernel), grid, 256, 0, st, a);
  }
  return D2C_OK;
}

int build_phi_table(float sigma, uint32_t* tab, int len) {
  const double s = (double)sigma;
  int first_zero = len;
  for (int r = 0; r < len; ++r) {
    const double rr = (double)r;
    const double v = exp(-(rr * rr) / (2.0 * s * s)) * 1073741824.0;
    tab[r] = (uint32_t)floor(v + 0.5);
    if (tab[r] == 0 && first_zero == len) first_zero = r;
  }
  return first_zero;
}

}  // namespace d2c
