// Epilogues of the tcgen05 GEMM kernels, shared by the one-SM and the two-SM kernel.
//
// An epilogue warp owns 32 accumulator rows (its TMEM lane quarter) and receives them one row per lane,
// 32 columns at a time.  Written to global memory in that shape, every store instruction would touch 32
// different rows.  So each pair of 32-column chunks goes through an 8 KB per-warp staging buffer in shared
// memory and comes back transposed: a lane then holds 8 consecutive columns of a row, four lanes cover 64
// contiguous bytes of a row and one instruction covers 8 rows.  All element-wise work (bias, residual,
// SwiGLU, rotary embedding) happens in that layout, where its global reads are coalesced too.
#pragma once

#include "common.cuh"

namespace d2c {

constexpr int kEpiStageBytes = 8192;                          // per epilogue warp: two 32 x 32 fp32 sub-tiles

struct EpiWarp {
  uint32_t stage;                                             // shared-memory address of the warp's staging buffer
  int row0;                                                   // global row of the warp's first accumulator row
  int n;                                                      // live rows of the launch
  int lane;
};

union EpiPack8 { uint4 u; __nv_bfloat162 h[4]; };

// rsqrt(mean(x^2) + eps) of row `row` of the A operand, from the K / 32 partial sums of squares the GEMM that wrote
// x left behind (added here in chunk order: deterministic); 1 when the launch carries no folded RMSNorm.
__device__ __forceinline__ float folded_row_scale(const GemmArgs& g, int row, bool row_ok) {
  if (!g.in_ssq) return 1.f;
  float s = 0.f;
  if (row_ok) {
    const int chunks = g.K >> 5;
    const float* sp = g.in_ssq + (size_t)row * chunks;
    if ((chunks & 3) == 0) {
      for (int t = 0; t < chunks; t += 4) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(sp + t));
        s += (v.x + v.y) + (v.z + v.w);
      }
    } else {
      for (int t = 0; t < chunks; ++t) s += __ldcg(sp + t);
    }
  }
  return rsqrtf(s / (float)g.K + g.in_eps);
}

// Row `lane` of sub-tile `half` <- the 32 columns in v.  16-byte pieces are XOR-swizzled with the row so that
// neither this write (same piece, 32 rows) nor the transposed read (same row, 4 lanes) conflicts on banks.
__device__ __forceinline__ void epi_stage_put(const EpiWarp& w, int half, const uint32_t (&v)[32]) {
  const uint32_t base = w.stage + (uint32_t)half * 4096u + (uint32_t)w.lane * 128u;
#pragma unroll
  for (int q = 0; q < 8; ++q)
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(base + (uint32_t)((q ^ (w.lane & 7)) << 4)), "r"(v[4 * q]),
                 "r"(v[4 * q + 1]), "r"(v[4 * q + 2]), "r"(v[4 * q + 3])
                 : "memory");
}

// f <- columns [8 cg, 8 cg + 8) of row r of sub-tile `half`.
__device__ __forceinline__ void epi_stage_get(const EpiWarp& w, int half, int r, int cg, float (&f)[8]) {
  const uint32_t base = w.stage + (uint32_t)half * 4096u + (uint32_t)r * 128u;
#pragma unroll
  for (int k = 0; k < 2; ++k)
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(f[4 * k]), "=f"(f[4 * k + 1]), "=f"(f[4 * k + 2]), "=f"(f[4 * k + 3])
                 : "r"(base + (uint32_t)(((2 * cg + k) ^ (r & 7)) << 4))
                 : "memory");
}

__device__ __forceinline__ float epi_tanh(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint4 epi_pack(const float (&f)[8]) {
  EpiPack8 o;
#pragma unroll
  for (int e = 0; e < 4; ++e) o.h[e] = __floats2bfloat162_rn(f[2 * e], f[2 * e + 1]);
  return o.u;
}

// C[row][n0 .. n0 + out_cols) = acc (+ bias) or C += acc.  load_chunk(col, v) must deliver accumulator columns
// [col, col + 32) of the calling lane's row and must be called by the whole warp.  Only the 32-column chunks
// [c_begin, c_end) of the tile are handled (c_end < 0: all of them), which lets the parts of a split-K tile
// share one tile's epilogue.
template <int EPI, typename LoadChunk>
__device__ __forceinline__ void epilogue_rows(LoadChunk&& load_chunk, const GemmArgs& g, const EpiWarp& w, int n0, int out_cols,
                                              int c_begin = 0, int c_end = -1) {
  if (c_end < 0) c_end = out_cols >> 5;
  const int passes = (c_end - c_begin + 1) >> 1;              // up to 64 output columns per pass
  const bool vec = (g.ldc & 7) == 0;
  const int rsub = w.lane >> 2, cg = w.lane & 3;
  uint4 rc[8], rn[8];                                         // residual of this pass and of the next one
  auto load_res = [&](int p, uint4 (&r)[8]) {
    if (EPI == EPI_RESIDUAL && vec && p < passes) {
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int row = w.row0 + j * 8 + rsub, col = n0 + (c_begin + 2 * p + h) * 32 + cg * 8;
          if (row < w.n && c_begin + 2 * p + h < c_end && col + 8 <= g.N)
            r[j * 2 + h] = __ldcg(reinterpret_cast<const uint4*>(g.C + (size_t)row * g.ldc + col));
        }
    }
  };
  load_res(0, rc);
#pragma unroll 1
  for (int p = 0; p < passes; ++p) {
    load_res(p + 1, rn);
    const int c0 = c_begin + 2 * p;
    const bool two = c0 + 1 < c_end;
    {
      uint32_t v[32];
      load_chunk(c0 * 32, v);
      epi_stage_put(w, 0, v);
      if (two) {
        load_chunk(c0 * 32 + 32, v);
        epi_stage_put(w, 1, v);
      }
    }
    __syncwarp();
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int row = w.row0 + j * 8 + rsub, col = n0 + (c0 + h) * 32 + cg * 8;
        const bool live = row < w.n && col < g.N && (h == 0 || two);
        float sq = 0.f;                                       // this lane's share of the row's sum of squares in the chunk
        if (live) {
          float f[8];
          epi_stage_get(w, h, j * 8 + rsub, cg, f);
          bf16* dst = g.C + (size_t)row * g.ldc + col;
          if (vec && col + 8 <= g.N) {
            if (EPI == EPI_RESIDUAL) {
              EpiPack8 old; old.u = rc[j * 2 + h];
#pragma unroll
              for (int e = 0; e < 4; ++e) { const float2 of = __bfloat1622float2(old.h[e]); f[2 * e] += of.x; f[2 * e + 1] += of.y; }
            } else if (g.bias) {
#pragma unroll
              for (int e = 0; e < 8; ++e) f[e] += __bfloat162float(g.bias[col + e]);
            }
            EpiPack8 xr; xr.u = epi_pack(f);
            *reinterpret_cast<uint4*>(dst) = xr.u;
            if (EPI == EPI_RESIDUAL && g.nx_out) {
              // the next RMSNorm, folded: x * gain for the next GEMM, and the row's sum of squares, both from the stored bf16 x
              EpiPack8 gn, o; gn.u = __ldg(reinterpret_cast<const uint4*>(g.nx_gain + col));
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float2 xv = __bfloat1622float2(xr.h[e]), gv = __bfloat1622float2(gn.h[e]);
                sq += xv.x * xv.x + xv.y * xv.y;
                o.h[e] = __floats2bfloat162_rn(xv.x * gv.x, xv.y * gv.y);
              }
              *reinterpret_cast<uint4*>(g.nx_out + (size_t)row * g.ldc + col) = o.u;
            }
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              if (col + e < g.N) {
                float x = f[e];
                if (EPI == EPI_RESIDUAL) x += __bfloat162float(dst[e]);
                else if (g.bias) x += __bfloat162float(g.bias[col + e]);
                dst[e] = __float2bfloat16_rn(x);
              }
            }
          }
        }
        if (EPI == EPI_RESIDUAL && g.nx_ssq) {
          // the four lanes that share a row add their parts in a fixed order; one of them stores the chunk's sum
          sq += __shfl_xor_sync(0xffffffffu, sq, 1);
          sq += __shfl_xor_sync(0xffffffffu, sq, 2);
          if (cg == 0 && row < w.n && (h == 0 || two) && n0 + (c0 + h) * 32 < g.N)
            g.nx_ssq[(size_t)row * (size_t)(g.N >> 5) + (size_t)((n0 >> 5) + c0 + h)] = sq;
        }
      }
    __syncwarp();                                             // the staging buffer is rewritten by the next pass
#pragma unroll
    for (int i = 0; i < 8; ++i) rc[i] = rn[i];
  }
}

// C[row][n0 .. n0 + oc) = silu(gate) * up, gate in accumulator columns [0, oc) and up in [oc, 2 oc); oc is a
// multiple of 32.  Handles the 32-column chunks [c_begin, c_end) of the oc outputs (c_end < 0: all).
template <typename LoadChunk>
__device__ __forceinline__ void epilogue_swiglu(LoadChunk&& load_chunk, const GemmArgs& g, const EpiWarp& w, int n0, int oc,
                                                int c_begin = 0, int c_end = -1) {
  if (c_end < 0) c_end = oc >> 5;
  const bool vec = (g.ldc & 7) == 0;
  const int rsub = w.lane >> 2, cg = w.lane & 3;
#pragma unroll 1
  for (int c = c_begin; c < c_end; ++c) {
    {
      uint32_t v[32];
      load_chunk(c * 32, v);
      epi_stage_put(w, 0, v);
      load_chunk(oc + c * 32, v);
      epi_stage_put(w, 1, v);
    }
    __syncwarp();
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int row = w.row0 + j * 8 + rsub, col = n0 + c * 32 + cg * 8;
      if (row >= w.n || col >= g.N) continue;
      float gt[8], up[8];
      epi_stage_get(w, 0, j * 8 + rsub, cg, gt);
      epi_stage_get(w, 1, j * 8 + rsub, cg, up);
#pragma unroll
      for (int e = 0; e < 8; ++e) {                           // silu(x) = h tanh(h) + h, h = x / 2: one MUFU op
        const float hx = 0.5f * gt[e];
        gt[e] = fmaf(hx, epi_tanh(hx), hx) * up[e];
      }
      bf16* dst = g.C + (size_t)row * g.ldc + col;
      if (vec && col + 8 <= g.N) {
        *reinterpret_cast<uint4*>(dst) = epi_pack(gt);
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e)
          if (col + e < g.N) dst[e] = __float2bfloat16_rn(gt[e]);
      }
    }
    __syncwarp();
  }
}

// Fused epilogue of the QKV projection: bias, rotary embedding of the Q and K heads at the row's absolute
// position, Q written to the activation buffer, K and V written straight into the layer's cache row of
// (sequence, position).  The rotation pairs column i of a head with column i + Dh/2: the two 32-column
// chunks of a pass are the matching pieces of the lower and the upper half head.  The tile's passes are numbered
// head by head (out_cols / 64 of them); only passes [u_begin, u_end) are handled (u_end < 0: all).
template <typename LoadChunk>
__device__ __forceinline__ void epilogue_qkv_rope(LoadChunk&& load_chunk, const GemmArgs& g, const EpiWarp& w, int n0, int out_cols,
                                                  int u_begin = 0, int u_end = -1) {
  const int dh = g.q_dh, half_chunks = dh >> 6;               // 32-column chunks per half head: 1 (Dh 64) or 2 (Dh 128)
  if (u_end < 0) u_end = out_cols >> 6;
  const int rsub = w.lane >> 2, cg = w.lane & 3;
  int pos[4];
  size_t cache_row[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int row = w.row0 + j * 8 + rsub;
    pos[j] = 0; cache_row[j] = 0;
    if (row < w.n) {
      pos[j] = g.q_sel_idx[row];
      cache_row[j] = ((size_t)g.q_row_seq[row] * g.q_cache_seq + pos[j]) * (size_t)(g.q_hkv * dh);
    }
  }
  for (int hc = 0; hc * dh < out_cols; ++hc) {                // heads inside this tile
    const int col_h = n0 + hc * dh;                           // first output column of the head
    if (col_h >= g.N) break;
    const int head = col_h / dh;
    const bool is_q = head < g.q_hq, is_k = !is_q && head < g.q_hq + g.q_hkv;
#pragma unroll 1
    for (int c = 0; c < half_chunks; ++c) {
      const int unit = hc * half_chunks + c;
      if (unit < u_begin || unit >= u_end) continue;          // uniform across the warp
      const int lc = hc * (dh >> 5) + c;
      {
        uint32_t v[32];
        load_chunk(lc * 32, v);
        epi_stage_put(w, 0, v);
        load_chunk((lc + half_chunks) * 32, v);
        epi_stage_put(w, 1, v);
      }
      __syncwarp();
      const int t0 = c * 32 + cg * 8;                         // index inside the half head
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int row = w.row0 + j * 8 + rsub;
        if (row >= w.n) continue;
        float lo[8], hi[8];
        epi_stage_get(w, 0, j * 8 + rsub, cg, lo);
        epi_stage_get(w, 1, j * 8 + rsub, cg, hi);
        if (g.bias) {
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            lo[e] += __bfloat162float(g.bias[col_h + t0 + e]);
            hi[e] += __bfloat162float(g.bias[col_h + (dh >> 1) + t0 + e]);
          }
        }
        if (is_q || is_k) {
          const float4* rt = reinterpret_cast<const float4*>(g.q_rope + (size_t)pos[j] * (dh >> 1) + t0);   // (cos, sin) pairs
#pragma unroll
          for (int e2 = 0; e2 < 4; ++e2) {
            const float4 cs = __ldg(rt + e2);
#pragma unroll
            for (int k = 0; k < 2; ++k) {
              const int e = 2 * e2 + k;
              const float cx = k ? cs.z : cs.x, sx = k ? cs.w : cs.y;
              // the projection result is rounded to bf16 before the rotation, as the unfused path stores it
              const float l = __bfloat162float(__float2bfloat16_rn(lo[e])), h = __bfloat162float(__float2bfloat16_rn(hi[e]));
              lo[e] = l * cx - h * sx;
              hi[e] = h * cx + l * sx;
            }
          }
        }
        bf16* dst;
        if (is_q) dst = g.C + (size_t)row * g.ldc + col_h;
        else if (is_k) dst = g.q_kc + cache_row[j] + (size_t)(head - g.q_hq) * dh;
        else dst = g.q_vc + cache_row[j] + (size_t)(head - g.q_hq - g.q_hkv) * dh;
        *reinterpret_cast<uint4*>(dst + t0) = epi_pack(lo);
        *reinterpret_cast<uint4*>(dst + (dh >> 1) + t0) = epi_pack(hi);
      }
      __syncwarp();
    }
  }
}

}  // namespace d2c
