// Decoding-loop helper (Eq. 2): replaces masked positions by their predicted tokens.
// One CTA per sequence.  Eligible positions are those whose prediction the last step refreshed
// (selected and still masked).  Scores: confidence s^i, or the certainty prior D(i)*s^i of Section 4.1.
#include "common.cuh"

namespace d2c {

struct CommitArgs {
  int seq_len, d, rule; float threshold;
  const int32_t* slot_of_pos; const float* conf; const int32_t* pred; const uint32_t* phi_q30; int phi_len;
  const bf16* embed; bf16* h0; uint8_t* mask; int32_t* tokens; int32_t* committed;
};

__global__ void __launch_bounds__(256) commit_kernel(CommitArgs a) {
  pdl_prologue();
  extern __shared__ unsigned char take[];                       // [seq_len] 1 = commit this position
  __shared__ unsigned long long s_best[8];
  const int b = blockIdx.x, L = a.seq_len, tid = threadIdx.x;
  uint8_t* mask = a.mask + (size_t)b * L;
  unsigned long long best = 0;                                   // score bits << 32 | ~pos, 0 = none
  for (int j = tid; j < L; j += 256) {
    take[j] = 0;
    if (!mask[j] || a.slot_of_pos[(size_t)b * L + j] < 0) continue;
    const float s = a.conf[(size_t)b * L + j];
    float score = s;
    if (a.rule == 1) {
      unsigned long long dq = 0;
      for (int r = 1; r < a.phi_len; ++r) {
        int known = 0;
        if (j - r >= 0) known += 1 - (mask[j - r] ? 1 : 0);
        if (j + r < L) known += 1 - (mask[j + r] ? 1 : 0);
        dq += (unsigned long long)a.phi_q30[r] * (unsigned)known;
      }
      score = __fmul_rn(__ull2float_rn(dq) * 9.31322574615478515625e-10f, s);
    }
    score = (score > 0.f && score < INFINITY) ? fminf(score, 262144.f) : 0.f;
    const unsigned long long comp = ((unsigned long long)__float_as_uint(score) << 32) | (0xFFFFFFFFu - (unsigned)j);
    best = comp > best ? comp : best;
    if (a.rule == 2 && s > a.threshold) take[j] = 1;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
    best = other > best ? other : best;
  }
  if ((tid & 31) == 0) s_best[tid >> 5] = best;
  __syncthreads();                                               // also orders every read of mask before the writes below
  best = 0;
  for (int w = 0; w < 8; ++w) best = s_best[w] > best ? s_best[w] : best;
  const int best_pos = best ? (int)(0xFFFFFFFFu - (unsigned)(best & 0xFFFFFFFFull)) : -1;
  if (tid == 0) { a.committed[b] = best_pos; if (best_pos >= 0) take[best_pos] = 1; }
  __syncthreads();
  const int nv = a.d >> 3;
  for (int j = 0; j < L; ++j) {
    if (!take[j]) continue;                                      // uniform across the CTA
    const int tok = a.pred[(size_t)b * L + j];
    const uint4* src = reinterpret_cast<const uint4*>(a.embed + (size_t)tok * a.d);
    uint4* dst = reinterpret_cast<uint4*>(a.h0 + ((size_t)b * L + j) * a.d);
    for (int v = tid; v < nv; v += 256) dst[v] = src[v];
    if (tid == 0) { a.tokens[(size_t)b * L + j] = tok; mask[j] = 0; }
  }
}

int launch_commit(int batch, int seq_len, int d, int rule, float threshold, const int32_t* slot_of_pos,
                  const float* conf, const int32_t* pred, const uint32_t* phi, int phi_len, const bf16* embed,
                  bf16* h0, uint8_t* mask, int32_t* tokens, int32_t* committed, cudaStream_t st) {
  CommitArgs a{seq_len, d, rule, threshold, slot_of_pos, conf, pred, phi, phi_len, embed, h0, mask, tokens, committed};
  D2C_LAUNCH((commit_kernel), batch, 256, seq_len, st, a);
  return D2C_OK;
}

}  // namespace d2c
