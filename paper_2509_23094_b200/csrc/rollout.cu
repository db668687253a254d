// Attention rollout influence scores (Eq. 6-9) without the L x L matrices.
//
// c^T = 1^T W^(N) ... W^(1).  A row of W^(l) is e_i for an unselected position and (Abar_i + e_i)/2
// for a selected one (Abar rows sum to 1, so the row sum of Eq. 7 is 2).  Evaluated from the left
// this is one vector-matrix product per layer, last layer first:
//     u'_j = u_j * (j selected ? 1/2 : 1) + 1/2 * sum_{i selected} u_i * Abar^(l)[i][j]
// The column sums stream Abar once (HBM-bound); rows are split across CTAs and the partial sums are
// added in a fixed order, so the result is deterministic.
#include "common.cuh"

namespace d2c {
namespace {

__global__ void rollout_init_kernel(RolloutArgs a, uint8_t* insel) {
  pdl_prologue();
  const int b = blockIdx.y, L = a.seq_len;
  const int ro = a.row_off[b], nb = a.row_off[b + 1] - ro;
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < L; j += gridDim.x * blockDim.x) {
    a.u0[(size_t)b * L + j] = 1.f;
    insel[(size_t)b * L + j] = 0;
  }
  __syncthreads();
  // the grid covers every position once, so each CTA marks the selected positions inside the
  // range it has just cleared
  const int j0 = blockIdx.x * blockDim.x, j1 = min(L, j0 + (int)blockDim.x);
  for (int i = threadIdx.x; i < nb; i += blockDim.x) {
    const int pos = a.sel_idx[ro + i];
    if (pos >= j0 && pos < j1) insel[(size_t)b * L + pos] = 1;
  }
}

__global__ void __launch_bounds__(256)
rollout_partial_kernel(RolloutArgs a, const float* __restrict__ abar_l, const float* __restrict__ u) {
  pdl_prologue();
  const int b = blockIdx.z, s = blockIdx.y, L = a.seq_len;
  const int j = blockIdx.x * 256 + threadIdx.x;
  const int ro = a.row_off[b], nb = a.row_off[b + 1] - ro;
  if (nb <= 0) return;
  const int per = (nb + a.n_split - 1) / a.n_split;
  const int i0 = s * per, i1 = min(nb, i0 + per);
  float acc = 0.f;
  if (j < L) {
    const float* ub = u + (size_t)b * L;
    for (int i = i0; i < i1; ++i) {
      const float ui = ub[a.sel_idx[ro + i]];
      acc += ui * abar_l[(size_t)(ro + i) * L + j];
    }
    a.partial[((size_t)s * a.batch + b) * L + j] = acc;
  }
}

__global__ void __launch_bounds__(256)
rollout_combine_kernel(RolloutArgs a, const uint8_t* __restrict__ insel, const float* __restrict__ u,
                       float* __restrict__ out) {
  pdl_prologue();
  const int b = blockIdx.y, L = a.seq_len;
  const int j = blockIdx.x * 256 + threadIdx.x;
  if (j >= L || a.row_off[b + 1] - a.row_off[b] <= 0) return;
  float sum = 0.f;
  for (int s = 0; s < a.n_split; ++s) sum += a.partial[((size_t)s * a.batch + b) * L + j];
  const size_t o = (size_t)b * L + j;
  out[o] = u[o] * (insel[o] ? 0.5f : 1.f) + 0.5f * sum;
}
}  // namespace

int launch_rollout(const RolloutArgs& a, cudaStream_t st) {
  if (a.batch <= 0 || a.seq_len <= 0 || a.n_layers <= 0) return D2C_OK;
  const int L = a.seq_len;
  uint8_t* insel = reinterpret_cast<uint8_t*>(a.partial + (size_t)a.n_split * a.batch * L);
  D2C_LAUNCH((rollout_init_kernel), dim3(ceil_div(L, 256), a.batch), 256, 0, st, a, insel);
  const float* u = a.u0;
  float* bufs[2] = {a.u1, a.u0};
  for (int l = a.n_layers - 1; l >= 0; --l) {
    float* out = (l == 0) ? a.c : bufs[(a.n_layers - 1 - l) & 1];
    D2C_LAUNCH((rollout_partial_kernel), dim3(ceil_div(L, 256), a.n_split, a.batch), 256, 0, st, a, a.abar + (size_t)l * a.layer_stride, u);
    D2C_LAUNCH((rollout_combine_kernel), dim3(ceil_div(L, 256), a.batch), 256, 0, st, a, insel, u, out);
    u = out;
  }
  return D2C_OK;
}

}  // namespace d2c
