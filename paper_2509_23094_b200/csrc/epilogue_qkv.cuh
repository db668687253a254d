// Fused epilogue of the QKV projection: bias, rotary embedding of the Q and K heads at the row's
// absolute position, Q written to the activation buffer, K and V written straight into the layer's
// cache row of (sequence, position).  Shared by the one-SM and the two-SM tcgen05 GEMM kernels; one
// thread owns one output row and walks the heads that fall into its tile.
#pragma once

#include "common.cuh"

namespace d2c {

// load_chunk(col, v) must deliver accumulator columns [col, col + 32) of this thread's row.
template <typename LoadChunk>
__device__ __forceinline__ void epilogue_qkv_rope(LoadChunk&& load_chunk, const GemmArgs& g, int row, bool row_ok, int n0,
                                                  int out_cols) {
  const int dh = g.q_dh, half_chunks = dh >> 6;               // 32-column chunks per half head: 1 (Dh 64) or 2 (Dh 128)
  int pos = 0, seq = 0;
  if (row_ok) { pos = g.q_sel_idx[row]; seq = g.q_row_seq[row]; }
  const float2* rt = g.q_rope + (size_t)pos * (dh >> 1);
  const size_t cache_row = ((size_t)seq * g.q_cache_seq + pos) * (size_t)(g.q_hkv * dh);
  for (int hc = 0; hc * dh < out_cols; ++hc) {                // heads inside this tile
    const int col_h = n0 + hc * dh;                           // first output column of the head
    if (col_h >= g.N) break;
    const int head = col_h / dh;
    const bool is_q = head < g.q_hq, is_k = !is_q && head < g.q_hq + g.q_hkv;
    bf16* dst;
    if (is_q) dst = g.C + (size_t)row * g.ldc + col_h;
    else if (is_k) dst = g.q_kc + cache_row + (size_t)(head - g.q_hq) * dh;
    else dst = g.q_vc + cache_row + (size_t)(head - g.q_hq - g.q_hkv) * dh;
#pragma unroll 1
    for (int c = 0; c < half_chunks; ++c) {
      uint32_t lo[32], hi[32];
      const int lc = hc * (dh >> 5) + c, hcx = lc + half_chunks;
      load_chunk(lc * 32, lo);
      load_chunk(hcx * 32, hi);
      if (!row_ok) continue;
      const int t0 = c * 32;                                  // index inside the half head
      union { uint4 u; __nv_bfloat162 h[4]; } olo, ohi;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int i = q * 8 + 2 * e;
          float l0 = __uint_as_float(lo[i]), l1 = __uint_as_float(lo[i + 1]);
          float h0 = __uint_as_float(hi[i]), h1 = __uint_as_float(hi[i + 1]);
          if (g.bias) {
            l0 += __bfloat162float(g.bias[col_h + t0 + i]); l1 += __bfloat162float(g.bias[col_h + t0 + i + 1]);
            h0 += __bfloat162float(g.bias[col_h + (dh >> 1) + t0 + i]); h1 += __bfloat162float(g.bias[col_h + (dh >> 1) + t0 + i + 1]);
          }
          if (is_q || is_k) {
            // the projection result is rounded to bf16 before the rotation, as the unfused path stores it
            l0 = __bfloat162float(__float2bfloat16_rn(l0)); l1 = __bfloat162float(__float2bfloat16_rn(l1));
            h0 = __bfloat162float(__float2bfloat16_rn(h0)); h1 = __bfloat162float(__float2bfloat16_rn(h1));
            const float2 cs0 = rt[t0 + i], cs1 = rt[t0 + i + 1];
            const float r0 = l0 * cs0.x - h0 * cs0.y, r1 = l1 * cs1.x - h1 * cs1.y;
            h0 = h0 * cs0.x + l0 * cs0.y; h1 = h1 * cs1.x + l1 * cs1.y;
            l0 = r0; l1 = r1;
          }
          olo.h[e] = __floats2bfloat162_rn(l0, l1);
          ohi.h[e] = __floats2bfloat162_rn(h0, h1);
        }
        reinterpret_cast<uint4*>(dst + t0)[q] = olo.u;
        reinterpret_cast<uint4*>(dst + (dh >> 1) + t0)[q] = ohi.u;
      }
    }
  }
}

}  // namespace d2c
