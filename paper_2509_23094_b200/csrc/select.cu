// Two-stage token selection of d2Cache (Section 4.1-4.2) and the compaction of the selected set.
//
// One CTA per sequence.  Every sum that decides an index is an integer sum, so the result does
// not depend on the order in which threads add:
//   stage 1 (Eq. 3-4): D(i) = sum over known j of phi(|i-j|), with phi tabulated as round(phi*2^30);
//                      key = fp32(D) * conf (one multiply); the k largest keys among masked positions
//                      (equal keys: lower position first).
//   stage 2 (after Eq. 9): candidates in the order (score c_j descending, position ascending); the shortest
//                      prefix whose mass sum floor(c_j*2^32) exceeds p times the total.
// Neither stage sorts.  Both are "take elements in that order until a running weight crosses a threshold"
// (weight 1 and threshold k for stage 1, the fixed-point mass and p * total for stage 2), which needs only the
// score value at which the crossing happens: four 8-bit radix passes over the fp32 bit patterns, each a
// 256-bin histogram of weights scanned from the top, find it exactly; elements above that value are taken,
// elements equal to it are taken in position order while the running weight has not crossed.  Up to 1024
// masked positions (every decoding step of the workloads) stage 1 skips even that and ranks each masked
// position against all others directly, one position per thread.
#include <math.h>

#include "common.cuh"

namespace d2c {

static constexpr int kSelThreads = 512;
static constexpr int kPhiMax = 512;              // phi entries kept in shared memory; a wider window reads the rest from global memory
static constexpr int kRankMax = 1024;            // stage 1 ranks by direct comparison up to this many masked positions
enum : uint8_t { F_SEL = 1, F_MSTAR = 2 };

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

// Shared scratch of the threshold search.
struct RadixScratch {
  // per digit: the weight sum of the members that carry it, kept as three 32-bit sums of 17-bit pieces of the
  // weights (weights stay below 2^51, 8192 positions x 2^17 below 2^32): 32-bit shared-memory atomics are native,
  // the 64-bit ones took about seven clocks per lane whatever the address (6700 of a 1024-position pass's clocks)
  uint32_t hist[3][256];
  unsigned long long warp_buf[32];
  unsigned long long total;
  unsigned long long above;
  int digit;                               // crossing digit of the pass, -1: the weight of all members does not cross
};

__device__ __forceinline__ unsigned long long shfl_up_u64(unsigned long long v, int o) {
  const uint32_t lo = __shfl_up_sync(0xffffffffu, (uint32_t)v, o), hi = __shfl_up_sync(0xffffffffu, (uint32_t)(v >> 32), o);
  return ((unsigned long long)hi << 32) | lo;
}
__device__ __forceinline__ unsigned long long shfl_xor_u64(unsigned long long v, int o) {
  const uint32_t lo = __shfl_xor_sync(0xffffffffu, (uint32_t)v, o), hi = __shfl_xor_sync(0xffffffffu, (uint32_t)(v >> 32), o);
  return ((unsigned long long)hi << 32) | lo;
}

// The shortest prefix, in the order (value bits descending, position ascending), of the positions j < L with
// member(j) whose running weight "crosses": crossed(w) must be monotone in w and false for w = 0.  Sets `mark`
// in flags for every position of that prefix; if the weight never crosses, for every member.
// weight(bits) is 1 (counting) or the fixed-point mass; all members with equal bits have equal weight.
// rs.hist must be zero on entry and is zero again on return.
// [vmin, vmax] bounds the members' value bits: leading digits on which the two agree need no pass.
template <typename Member, typename Weight, typename Crossed>
__device__ __forceinline__ void take_until_crossed(const uint32_t* vb, int L, Member member, Weight weight, Crossed crossed,
                                                   uint8_t* flags, uint8_t mark, RadixScratch& rs, uint32_t vmin, uint32_t vmax) {
  const int tid = threadIdx.x, lane = tid & 31, T = blockDim.x;
  uint32_t pref = 0;                                     // the high digits fixed so far
  unsigned long long above = 0;                          // weight of the members above the range still searched
  bool all = false;
  int pass0 = 0;
  while (pass0 < 3 && (vmin >> (24 - 8 * pass0)) == (vmax >> (24 - 8 * pass0))) ++pass0;
  if (pass0 > 0) pref = vmax >> (32 - 8 * pass0);
  for (int pass = pass0; pass < 4 && !all; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int base = 0; base < L; base += T) {
      const int j = base + tid;
      const bool m = j < L && member(j) && (pass == 0 || (vb[j] >> (shift + 8)) == pref);
      const unsigned act = __ballot_sync(0xffffffffu, m);
      if (act) {
        // a warp whose live lanes all carry the same digit (flat scores, the high digits) adds once; otherwise each lane adds
        const uint32_t d = m ? (vb[j] >> shift) & 255u : 0u;
        unsigned long long w = m ? weight(vb[j]) : 0ull;
        const int leader = __ffs(act) - 1;
        const uint32_t d0 = __shfl_sync(0xffffffffu, d, leader);
        const bool one_digit = __all_sync(0xffffffffu, !m || d == d0);
        if (one_digit)
          for (int o = 16; o > 0; o >>= 1) w += shfl_xor_u64(w, o);
        if (one_digit ? lane == leader : m) {
          // (a warp's sum of 32 weights may carry into bit 51 and above: the top piece takes all the high bits)
          const uint32_t w0 = (uint32_t)(w & 0x1FFFFull), w1 = (uint32_t)((w >> 17) & 0x1FFFFull), w2 = (uint32_t)(w >> 34);
          if (w0) atomicAdd(&rs.hist[0][d], w0);
          if (w1) atomicAdd(&rs.hist[1][d], w1);
          if (w2) atomicAdd(&rs.hist[2][d], w2);
        }
      }
    }
    __syncthreads();
    if (tid < 32) {
      // one warp walks the digits from the top: lane l owns digits 255 - 8 l down to 248 - 8 l
      unsigned long long w[8], sum = 0;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int bin = 255 - (8 * lane + k);
        w[k] = (unsigned long long)rs.hist[0][bin] + ((unsigned long long)rs.hist[1][bin] << 17) + ((unsigned long long)rs.hist[2][bin] << 34);
        rs.hist[0][bin] = 0; rs.hist[1][bin] = 0; rs.hist[2][bin] = 0;
        sum += w[k];
      }
      unsigned long long inc = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long up = shfl_up_u64(inc, o);
        if (lane >= o) inc += up;
      }
      unsigned long long run = above + inc - sum;        // weight above this lane's first digit
      int hit = -1; unsigned long long before = 0;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (hit < 0 && w[k] != 0 && crossed(run + w[k])) { hit = k; before = run; }
        run += w[k];
      }
      const unsigned found = __ballot_sync(0xffffffffu, hit >= 0);
      if (found == 0) {
        if (lane == 0) rs.digit = -1;
      } else if (lane == __ffs(found) - 1) {
        rs.digit = 255 - (8 * lane + hit);
        rs.above = before;
      }
    }
    __syncthreads();
    if (rs.digit < 0) {
      all = true;                                        // the weight of all members together does not cross
    } else {
      above = rs.above;
      pref = (pref << 8) | (uint32_t)rs.digit;
    }
    // (rs.digit is rewritten only behind the next pass's barrier)
  }
  // members above the crossing value are in; those equal to it, in position order, while the weight before them has not crossed
  const int per = (L + T - 1) / T;
  const int j0 = tid * per;
  unsigned long long ties = 0;
  if (!all)
    for (int e = 0; e < per; ++e) {
      const int j = j0 + e;
      if (j < L && member(j) && vb[j] == pref) ++ties;
    }
  unsigned long long r = all ? 0ull : block_exclusive_scan<unsigned long long>(ties, rs.warp_buf, &rs.total);
  const unsigned long long wstar = weight(pref);
  for (int e = 0; e < per; ++e) {
    const int j = j0 + e;
    if (j >= L || !member(j)) continue;
    bool in = all || vb[j] > pref;
    if (!all && vb[j] == pref) { in = !crossed(above + r * wstar); ++r; }
    if (in) flags[j] |= mark;
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kSelThreads) select_kernel(SelectArgs a) {
  pdl_prologue();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int b = blockIdx.x, L = a.seq_len, tid = threadIdx.x, lane = tid & 31;
  uint32_t* kb = reinterpret_cast<uint32_t*>(smem_raw);       // stage-1 key bits (0 outside the stage-1 set)
  uint32_t* cb = kb + L;                                       // stage-2 score bits
  uint8_t* flags = reinterpret_cast<uint8_t*>(cb + L);
  uint8_t* smask = flags + L;
  uint8_t* in1 = smask + L;                                    // 1: masked and inside the block (the set stage 1 ranks)
  __shared__ RadixScratch rsc;
  __shared__ unsigned long long mlist[kRankMax];               // stage-1 members: position, then (key bits << 32 | ~position)
  __shared__ int warp_buf32[32];
  __shared__ int s_total32, s_nm;
  __shared__ unsigned long long s_mass;
  __shared__ uint32_t s_lo, s_hi;
  __shared__ uint32_t s_phi[kPhiMax];                          // the non-zero head of the phi table (window +-65 at sigma 10)

  const uint8_t* mask = a.mask + (size_t)b * L;
  const float* conf = a.conf + (size_t)b * L;
  const float* cs = a.c + (size_t)b * L;
  const float* okey = a.override_key ? a.override_key + (size_t)b * L : nullptr;
  float* key_out = a.key + (size_t)b * L;

  // stage 1 may be confined to one block of positions (semi-autoregressive decoding); whole sequence otherwise
  const int blk_lo = a.block_hi > a.block_lo ? a.block_lo : 0, blk_hi = a.block_hi > a.block_lo ? a.block_hi : L;
  for (int i = tid; i < L; i += kSelThreads) {
    smask[i] = mask[i] ? 1 : 0; flags[i] = 0; kb[i] = 0;
    cb[i] = __float_as_uint(clean_score(cs[i]));
  }
  for (int r = tid; r < min(a.phi_len, kPhiMax); r += kSelThreads) s_phi[r] = a.phi_q30[r];
  for (int i = tid; i < 3 * 256; i += kSelThreads) (&rsc.hist[0][0])[i] = 0;
  if (tid == 0) { s_nm = 0; s_mass = 0; s_lo = 0xFFFFFFFFu; s_hi = 0u; }
  __syncthreads();

  // ---- the set stage 1 ranks: masked positions inside the block, listed in any order ----
  for (int base = 0; base < L; base += kSelThreads) {
    const int i = base + tid;
    const bool m1 = i < L && smask[i] && i >= blk_lo && i < blk_hi;
    if (i < L) { in1[i] = m1 ? 1 : 0; if (!m1) key_out[i] = 0.f; }
    const unsigned act = __ballot_sync(0xffffffffu, m1);
    if (act) {
      int slot0 = 0;
      if (lane == __ffs(act) - 1) slot0 = atomicAdd(&s_nm, __popc(act));
      slot0 = __shfl_sync(0xffffffffu, slot0, __ffs(act) - 1);
      const int slot = slot0 + __popc(act & ((1u << lane) - 1u));
      if (m1 && slot < kRankMax) mlist[slot] = (unsigned long long)i;
    }
  }
  __syncthreads();
  const int nm = s_nm;

  // ---- keys (Eq. 3-4): D(i) as an exact integer sum over the window, key = fp32(D) * confidence ----
  auto known_at = [&](int i, int r) {
    const int lo = i - r, hi = i + r;
    int known = 0;
    if (lo >= 0) known += 1 - smask[lo];
    if (hi < L) known += 1 - smask[hi];
    return (unsigned)known;
  };
  auto finish_key = [&](int i, unsigned long long dq, float cf) {
    float key;
    if (okey) {
      key = clean_score(okey[i]);
    } else {
      const float D = __ull2float_rn(dq) * 9.31322574615478515625e-10f;       // * 2^-30, exact
      key = clean_score(__fmul_rn(D, cf));
    }
    key_out[i] = key;
    kb[i] = __float_as_uint(key);
    return key;
  };
  if (nm <= kRankMax) {
    // a group of tpm lanes (a power of two, inside one warp) shares the window of one listed position
    int tpm = 1;
    while (tpm < 32 && 2 * tpm * nm <= kSelThreads) tpm <<= 1;
    const int sub = tid & (tpm - 1), groups = kSelThreads / tpm;
    for (int e0 = 0; e0 < nm; e0 += groups) {
      const int e = e0 + tid / tpm;
      const bool live = e < nm;
      const int i = live ? (int)mlist[e] : 0;
      const float cf = (live && sub == 0 && !okey) ? conf[i] : 0.f;       // in flight while the window is summed
      unsigned long long dq = 0;
      if (live && !okey)
        for (int r = 1 + sub; r < a.phi_len; r += tpm)
          dq += (unsigned long long)(r < kPhiMax ? s_phi[r] : a.phi_q30[r]) * known_at(i, r);
      for (int o = 1; o < tpm; o <<= 1) dq += shfl_xor_u64(dq, o);
      __syncwarp();
      if (live && sub == 0) {
        const float key = finish_key(i, dq, cf);
        mlist[e] = ((unsigned long long)__float_as_uint(key) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)i);
      }
    }
  } else {
    for (int i = tid; i < L; i += kSelThreads) {
      if (!in1[i]) continue;
      unsigned long long dq = 0;
      if (!okey)
        for (int r = 1; r < a.phi_len; ++r) dq += (unsigned long long)(r < kPhiMax ? s_phi[r] : a.phi_q30[r]) * known_at(i, r);
      finish_key(i, dq, okey ? 0.f : conf[i]);
    }
  }
  __syncthreads();

  // ---- stage 1: the k largest keys of the set, lower position first among equal keys ----
  {
    const int take = min(max(a.k, 0), nm);
    if (take == nm) {
      for (int i = tid; i < L; i += kSelThreads)
        if (in1[i]) flags[i] = F_SEL | F_MSTAR;
    } else if (take > 0 && nm <= kRankMax) {
      // rank of a listed position = how many others come before it; a group of tpe lanes (a power of two, inside
      // one warp) shares a position and each counts every tpe-th entry
      int tpe = 1;
      while (tpe < 32 && 2 * tpe * nm <= kSelThreads) tpe <<= 1;
      const int sub = tid & (tpe - 1), groups = kSelThreads / tpe;
      for (int e0 = 0; e0 < nm; e0 += groups) {
        const int e = e0 + tid / tpe;
        const bool live = e < nm;
        const unsigned long long mine = live ? mlist[e] : 0ull;
        int rank = 0;
        if (live)
          for (int f = sub; f < nm; f += tpe) rank += mlist[f] > mine ? 1 : 0;
        for (int o = 1; o < tpe; o <<= 1) rank += __shfl_xor_sync(0xffffffffu, rank, o);
        if (live && sub == 0 && rank < take) flags[0xFFFFFFFFu - (uint32_t)(mine & 0xFFFFFFFFull)] = F_SEL | F_MSTAR;
      }
    } else if (take > 0) {
      const unsigned long long want = (unsigned long long)take;
      take_until_crossed(kb, L, [&](int j) { return in1[j] != 0; }, [](uint32_t) { return 1ull; },
                         [&](unsigned long long w) { return w >= want; }, flags, (uint8_t)(F_SEL | F_MSTAR), rsc, 0u, 0xFFFFFFFFu);
    }
    __syncthreads();
  }

  // ---- stage 2: top-p over the candidates by influence score ----
  if (a.p > 0.f) {
    const bool mode1 = a.stage2_candidates != 0;
    auto cand = [&](int j) { return mode1 ? (flags[j] & F_MSTAR) == 0 : smask[j] == 0; };
    auto mass = [](uint32_t bits) { return (unsigned long long)__double2ull_rd((double)__uint_as_float(bits) * 4294967296.0); };
    unsigned long long local = 0;
    uint32_t lo = 0xFFFFFFFFu, hi = 0u;
    for (int j = tid; j < L; j += kSelThreads)
      if (cand(j)) { local += mass(cb[j]); lo = min(lo, cb[j]); hi = max(hi, cb[j]); }
    for (int o = 16; o > 0; o >>= 1) local += shfl_xor_u64(local, o);
    lo = __reduce_min_sync(0xffffffffu, lo); hi = __reduce_max_sync(0xffffffffu, hi);
    if (lane == 0) {
      if (local) atomicAdd(&s_mass, local);
      atomicMin(&s_lo, lo); atomicMax(&s_hi, hi);
    }
    __syncthreads();
    // (p above 1 selects every candidate, as p = 1 does: the total never exceeds itself)
    const double thr = __dmul_rn(fmin((double)a.p, 1.0), __ull2double_rn(s_mass));
    // The prefix's mass has crossed when double(mass) > thr.  double() is monotone, so that is mass >= T for the
    // smallest integer T whose double exceeds thr, and the search compares integers.  Below 2^52 every integer is
    // its own double: T = floor(thr) + 1; above, T lies within 2048 of floor(thr) (doubles are at most 1024 apart
    // below 2^63) and a bisection finds it.
    unsigned long long T;
    {
      const unsigned long long fl = __double2ull_rd(thr);
      if (thr < 4503599627370496.0) {
        T = fl + 1ull;
      } else {
        unsigned long long lo_t = fl - 2048ull, hi_t = fl + 2049ull;        // double(lo_t) <= thr < double(hi_t)
        while (hi_t - lo_t > 1ull) {
          const unsigned long long mid = lo_t + ((hi_t - lo_t) >> 1);
          if (__ull2double_rn(mid) > thr) hi_t = mid; else lo_t = mid;
        }
        T = hi_t;
      }
    }
    take_until_crossed(cb, L, cand, mass, [&](unsigned long long w) { return w >= T; }, flags, (uint8_t)F_SEL, rsc,
                       s_lo, max(s_hi, s_lo));
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
  const size_t smem = (size_t)a.seq_len * 11;               // two 32-bit words and three flag bytes per position
  static PerDevice attr_set;
  if (attr_set.first()) {
    D2C_CUDA_OK(cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 8192 * 11));
  }
  D2C_LAUNCH((select_kernel), a.batch, kSelThreads, smem, st, a);
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
