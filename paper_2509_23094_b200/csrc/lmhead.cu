// Eq. 1 from the per-tile statistics the LM-head GEMM leaves behind: for every row the running
// maximum, its column and sum exp(x - max) of each 128-column tile are merged into the arg-max
// token and its softmax probability 1 / sum_j exp(x_j - max).  The logits never reach HBM.
#include "common.cuh"

namespace d2c {

// One CTA per row.  lm_rows == null: results go to conf[r] / pred[r]; otherwise row lm_rows[r] of
// the step is looked up and the result is scattered to its (sequence, position).
__global__ void __launch_bounds__(256)
lm_reduce_kernel(const float* __restrict__ st_max, const float* __restrict__ st_sum,
                 const int32_t* __restrict__ st_arg, int n_tiles, const int32_t* __restrict__ n_rows,
                 const int32_t* __restrict__ lm_rows, const int32_t* __restrict__ sel_idx,
                 const int32_t* __restrict__ row_seq, int seq_len, float* __restrict__ conf,
                 int32_t* __restrict__ pred) {
  pdl_prologue();
  __shared__ float s_mx[8], s_sum[8];
  __shared__ int s_arg[8];
  const int n = *n_rows, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int r = blockIdx.x; r < n; r += gridDim.x) {
    const size_t base = (size_t)r * n_tiles;
    float mx = -INFINITY; int arg = 0x7fffffff;
    for (int t = threadIdx.x; t < n_tiles; t += 256) {
      const float v = st_max[base + t]; const int a2 = st_arg[base + t];
      if (v > mx || (v == mx && a2 < arg)) { mx = v; arg = a2; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float omx = __shfl_xor_sync(0xffffffffu, mx, o);
      const int oarg = __shfl_xor_sync(0xffffffffu, arg, o);
      if (omx > mx || (omx == mx && oarg < arg)) { mx = omx; arg = oarg; }
    }
    if (lane == 0) { s_mx[warp] = mx; s_arg[warp] = arg; }
    __syncthreads();
    mx = -INFINITY; arg = 0x7fffffff;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      const float v = s_mx[w]; const int a2 = s_arg[w];
      if (v > mx || (v == mx && a2 < arg)) { mx = v; arg = a2; }
    }
    float sum = 0.f;
    for (int t = threadIdx.x; t < n_tiles; t += 256) sum += st_sum[base + t] * __expf(st_max[base + t] - mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) s_sum[warp] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) tot += s_sum[w];                  // fixed order: deterministic
      size_t dst = (size_t)r;
      if (lm_rows) { const int row = lm_rows[r]; dst = (size_t)row_seq[row] * seq_len + sel_idx[row]; }
      conf[dst] = 1.f / tot;
      pred[dst] = arg;
    }
    __syncthreads();
  }
}

int launch_lm_reduce(const float* st_max, const float* st_sum, const int32_t* st_arg, int n_tiles,
                     const int32_t* n_rows, int max_rows, const int32_t* lm_rows, const int32_t* sel_idx,
                     const int32_t* row_seq, int seq_len, float* conf, int32_t* pred, cudaStream_t st) {
  if (max_rows <= 0) return D2C_OK;
  const int grid = max_rows < 148 * 4 ? max_rows : 148 * 4;
  D2C_LAUNCH((lm_reduce_kernel), grid, 256, 0, st, st_max, st_sum, st_arg, n_tiles, n_rows, lm_rows, sel_idx, row_seq, seq_len, conf, pred);
  return D2C_OK;
}

}  // namespace d2c
