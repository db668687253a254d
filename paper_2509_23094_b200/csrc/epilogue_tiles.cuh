// Epilogues of the tcgen05 GEMM kernels, shared by the one-SM and the two-SM kernel.
//
// An epilogue warp owns 32 accumulator rows (its TMEM lane quarter) and receives them one row per lane,
// 32 columns at a time.  Everything element-wise happens in that shape, where a lane has the matching columns
// of its own row at hand: bias, residual, SwiGLU (gate and up chunk) and the rotary embedding (lower and upper
// half-head chunk).  Written to global memory in that shape, though, every store instruction would touch 32
// different rows (measured: about 3.5 clocks per lane and instruction, 4 us for a 128 x 256 tile).  So the
// finished chunk is rounded to bf16 first and the packed 32 x 32 sub-tile (2 KB) goes through a per-warp
// staging buffer in shared memory and comes back transposed: a lane then holds 8 consecutive columns of four
// rows, four lanes cover 64 contiguous bytes of a row and one store instruction covers 8 rows.  Two such
// buffers alternate, so a chunk needs one warp barrier.  Few instructions matter here: a warp that has a
// scheduler to itself issues one dependent instruction every four to five clocks.
#pragma once

#include "common.cuh"

namespace d2c {

constexpr int kEpiStageBytes = 4096;                          // per epilogue warp: two 32 x 32 bf16 sub-tiles

struct EpiWarp {
  uint32_t stage;                                             // shared-memory address of the warp's staging buffers
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

__device__ __forceinline__ float epi_tanh(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 32 fp32 values -> 32 bf16 (four 16-byte pieces), rounded to nearest even.
__device__ __forceinline__ void epi_pack32(const float (&f)[32], uint4 (&o)[4]) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    EpiPack8 pk;
#pragma unroll
    for (int e = 0; e < 4; ++e) pk.h[e] = __floats2bfloat162_rn(f[8 * q + 2 * e], f[8 * q + 2 * e + 1]);
    o[q] = pk.u;
  }
}

// The 32 x 32 bf16 sub-tile held one row per lane (o = this lane's 32 columns) comes back as t[i] = columns
// [8 (lane & 3), +8) of row 8 i + lane / 4.  Rows are 64 bytes apart in the buffer; the 16-byte pieces of a row
// are XOR-swizzled with bits 1-2 of the row so that neither the row-wise writes nor the transposed reads
// conflict on banks.  Consecutive calls must alternate `buf` (0, 1): the barrier inside then also separates a
// buffer's readers from its next writers.
__device__ __forceinline__ void epi_transpose(const EpiWarp& w, int buf, const uint4 (&o)[4], uint4 (&t)[4]) {
  const uint32_t base = w.stage + (uint32_t)buf * 2048u;
  const uint32_t wr = base + (uint32_t)w.lane * 64u, wsw = (uint32_t)((w.lane >> 1) & 3);
#pragma unroll
  for (int q = 0; q < 4; ++q)
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(wr + (((uint32_t)q ^ wsw) << 4)), "r"(o[q].x), "r"(o[q].y),
                 "r"(o[q].z), "r"(o[q].w)
                 : "memory");
  __syncwarp();
  const uint32_t r0 = (uint32_t)(w.lane >> 2), pc = (uint32_t)(w.lane & 3);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t r = r0 + 8u * i;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(t[i].x), "=r"(t[i].y), "=r"(t[i].z), "=r"(t[i].w)
                 : "r"(base + r * 64u + ((pc ^ ((r >> 1) & 3u)) << 4))
                 : "memory");
  }
}

// Stores a transposed sub-tile (see epi_transpose): piece i goes to dst_row(i, lr) + 8 (lane & 3) if row
// lr = 8 i + lane / 4 of the warp is live.  `cols_left` = valid columns from the sub-tile's first column on (>= 32: all).
template <typename RowPtr>
__device__ __forceinline__ void epi_store_t(const EpiWarp& w, const uint4 (&t)[4], bool vec, int cols_left, RowPtr&& dst_row) {
  const int cg8 = (w.lane & 3) * 8;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int lr = 8 * i + (w.lane >> 2);
    if (w.row0 + lr >= w.n) continue;
    bf16* dst = dst_row(i, lr) + cg8;
    if (vec && cg8 + 8 <= cols_left) {
      *reinterpret_cast<uint4*>(dst) = t[i];
    } else {
      EpiPack8 pk; pk.u = t[i];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (cg8 + 2 * e < cols_left) dst[2 * e] = __low2bfloat16(pk.h[e]);
        if (cg8 + 2 * e + 1 < cols_left) dst[2 * e + 1] = __high2bfloat16(pk.h[e]);
      }
    }
  }
}

// C[row][n0 .. n0 + out_cols) = acc (+ bias) or C += acc.  load_chunk(col, v) must deliver accumulator columns
// [col, col + 32) of the calling lane's row and must be called by the whole warp.  Only the 32-column chunks
// [c_begin, c_end) of the tile are handled (c_end < 0: all of them), which lets several warps, or the parts of a
// split-K tile, share one tile's epilogue.
template <int EPI, typename LoadChunk>
__device__ __forceinline__ void epilogue_rows(LoadChunk&& load_chunk, const GemmArgs& g, const EpiWarp& w, int n0, int out_cols,
                                              int c_begin = 0, int c_end = -1) {
  if (c_end < 0) c_end = out_cols >> 5;
  const bool vec = (g.ldc & 7) == 0;
  const bool bias_vec = (reinterpret_cast<uintptr_t>(g.bias) & 15) == 0;
  const int row = w.row0 + w.lane;
  const bool row_ok = row < w.n;
  bf16* crow = g.C + (size_t)row * g.ldc;                     // this lane's row (element-wise work)
  bf16* cwarp = g.C + (size_t)w.row0 * g.ldc;                 // the warp's first row (transposed stores)
  uint4 old[4], old_next[4];                                  // residual of this chunk and of the next one
  auto load_old = [&](int c, uint4 (&r)[4]) {
    const int col0 = n0 + c * 32;
    if (EPI == EPI_RESIDUAL && c < c_end && row_ok && vec && col0 + 32 <= g.N) {
#pragma unroll
      for (int q = 0; q < 4; ++q) r[q] = __ldcg(reinterpret_cast<const uint4*>(crow + col0) + q);
    }
  };
  load_old(c_begin, old);
#pragma unroll 1
  for (int c = c_begin; c < c_end; ++c) {
    const int col0 = n0 + c * 32;
    if (col0 >= g.N) break;                                   // uniform across the warp
    const bool full = vec && col0 + 32 <= g.N;
    load_old(c + 1, old_next);
    uint32_t v[32];
    load_chunk(c * 32, v);
    float f[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) f[i] = __uint_as_float(v[i]);
    if (row_ok) {
      if (EPI == EPI_RESIDUAL) {
        if (full) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            EpiPack8 o; o.u = old[q];
#pragma unroll
            for (int e = 0; e < 4; ++e) { const float2 of = __bfloat1622float2(o.h[e]); f[8 * q + 2 * e] += of.x; f[8 * q + 2 * e + 1] += of.y; }
          }
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (col0 + e < g.N) f[e] += __bfloat162float(crow[col0 + e]);
        }
      } else if (g.bias) {
        if (full && bias_vec) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            EpiPack8 b; b.u = __ldg(reinterpret_cast<const uint4*>(g.bias + col0) + q);
#pragma unroll
            for (int e = 0; e < 4; ++e) { const float2 bf = __bfloat1622float2(b.h[e]); f[8 * q + 2 * e] += bf.x; f[8 * q + 2 * e + 1] += bf.y; }
          }
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (col0 + e < g.N) f[e] += __bfloat162float(g.bias[col0 + e]);
        }
      }
    }
    uint4 o[4], t[4];
    epi_pack32(f, o);
    epi_transpose(w, (c - c_begin) & 1, o, t);
    epi_store_t(w, t, vec, g.N - col0, [&](int, int lr) { return cwarp + (size_t)lr * g.ldc + col0; });
    if (EPI == EPI_RESIDUAL && g.nx_out) {
      // the next RMSNorm, folded: x * gain for the next GEMM, and the row's sum of squares over the chunk, both
      // from the stored bf16 x
      float sq = 0.f, nx[32];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        EpiPack8 xr; xr.u = o[q];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 xv = __bfloat1622float2(xr.h[e]);
          const int col = col0 + 8 * q + 2 * e;
          const float g0 = col < g.N ? __bfloat162float(g.nx_gain[col]) : 0.f, g1 = col + 1 < g.N ? __bfloat162float(g.nx_gain[col + 1]) : 0.f;
          if (col < g.N) sq += xv.x * xv.x;
          if (col + 1 < g.N) sq += xv.y * xv.y;
          nx[8 * q + 2 * e] = xv.x * g0; nx[8 * q + 2 * e + 1] = xv.y * g1;
        }
      }
      if (g.nx_ssq && row_ok) g.nx_ssq[(size_t)row * (size_t)(g.N >> 5) + (size_t)(col0 >> 5)] = sq;
      uint4 on[4], tn[4];
      epi_pack32(nx, on);
      __syncwarp();                                           // the buffer used two calls ago is the one used next
      epi_transpose(w, ((c - c_begin) & 1) ^ 1, on, tn);
      __syncwarp();
      bf16* nwarp = g.nx_out + (size_t)w.row0 * g.ldc;
      epi_store_t(w, tn, vec, g.N - col0, [&](int, int lr) { return nwarp + (size_t)lr * g.ldc + col0; });
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) old[q] = old_next[q];
  }
}

// C[row][n0 .. n0 + oc) = silu(gate) * up, gate in accumulator columns [0, oc) and up in [oc, 2 oc); oc is a
// multiple of 32.  Handles the 32-column chunks [c_begin, c_end) of the oc outputs (c_end < 0: all).
template <typename LoadChunk>
__device__ __forceinline__ void epilogue_swiglu(LoadChunk&& load_chunk, const GemmArgs& g, const EpiWarp& w, int n0, int oc,
                                                int c_begin = 0, int c_end = -1) {
  if (c_end < 0) c_end = oc >> 5;
  const bool vec = (g.ldc & 7) == 0;
  bf16* cwarp = g.C + (size_t)w.row0 * g.ldc;
#pragma unroll 1
  for (int c = c_begin; c < c_end; ++c) {
    const int col0 = n0 + c * 32;
    if (col0 >= g.N) break;                                   // uniform across the warp
    uint32_t gt[32], up[32];
    load_chunk(c * 32, gt);
    load_chunk(oc + c * 32, up);
    float f[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) {                            // silu(x) = h tanh(h) + h, h = x / 2: one MUFU op
      const float hx = 0.5f * __uint_as_float(gt[e]);
      f[e] = fmaf(hx, epi_tanh(hx), hx) * __uint_as_float(up[e]);
    }
    uint4 o[4], t[4];
    epi_pack32(f, o);
    epi_transpose(w, (c - c_begin) & 1, o, t);
    epi_store_t(w, t, vec, g.N - col0, [&](int, int lr) { return cwarp + (size_t)lr * g.ldc + col0; });
  }
}

// Fused epilogue of the QKV projection: bias, rotary embedding of the Q and K heads at the row's absolute
// position, Q written to the activation buffer, K and V written straight into the layer's cache row of
// (sequence, position).  The rotation pairs column i of a head with column i + Dh/2: a unit of work is a
// 32-column chunk of the lower half head together with the matching chunk of the upper half.  The tile's units
// are numbered head by head (out_cols / 64 of them); only units [u_begin, u_end) are handled (u_end < 0: all).
template <typename LoadChunk>
__device__ __forceinline__ void epilogue_qkv_rope(LoadChunk&& load_chunk, const GemmArgs& g, const EpiWarp& w, int n0, int out_cols,
                                                  int u_begin = 0, int u_end = -1) {
  const int dh = g.q_dh, half_chunks = dh >> 6;               // 32-column chunks per half head: 1 (Dh 64) or 2 (Dh 128)
  if (u_end < 0) u_end = out_cols >> 6;
  const int row = w.row0 + w.lane;
  const bool row_ok = row < w.n;
  const bool bias_vec = (reinterpret_cast<uintptr_t>(g.bias) & 15) == 0;
  const int pos = row_ok ? g.q_sel_idx[row] : 0;              // this lane's row: position for the rotation
  size_t cache_row[4];                                        // the four rows this lane stores after the transposition
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = w.row0 + 8 * i + (w.lane >> 2);
    cache_row[i] = r < w.n ? ((size_t)g.q_row_seq[r] * g.q_cache_seq + g.q_sel_idx[r]) * (size_t)(g.q_hkv * dh) : 0;
  }
  bf16* cwarp = g.C + (size_t)w.row0 * g.ldc;
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
      const int t0 = c * 32;                                  // index inside the half head
      uint32_t vlo[32], vhi[32];
      load_chunk(lc * 32, vlo);
      load_chunk((lc + half_chunks) * 32, vhi);
      float lo[32], hi[32];
#pragma unroll
      for (int e = 0; e < 32; ++e) { lo[e] = __uint_as_float(vlo[e]); hi[e] = __uint_as_float(vhi[e]); }
      if (g.bias) {
        if (bias_vec) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            EpiPack8 bl, bh;
            bl.u = __ldg(reinterpret_cast<const uint4*>(g.bias + col_h + t0) + q);
            bh.u = __ldg(reinterpret_cast<const uint4*>(g.bias + col_h + (dh >> 1) + t0) + q);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 fl = __bfloat1622float2(bl.h[e]), fh = __bfloat1622float2(bh.h[e]);
              lo[8 * q + 2 * e] += fl.x; lo[8 * q + 2 * e + 1] += fl.y;
              hi[8 * q + 2 * e] += fh.x; hi[8 * q + 2 * e + 1] += fh.y;
            }
          }
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            lo[e] += __bfloat162float(g.bias[col_h + t0 + e]);
            hi[e] += __bfloat162float(g.bias[col_h + (dh >> 1) + t0 + e]);
          }
        }
      }
      if ((is_q || is_k) && row_ok) {
        const float4* rt = reinterpret_cast<const float4*>(g.q_rope + (size_t)pos * (dh >> 1) + t0);   // (cos, sin) pairs
#pragma unroll
        for (int e2 = 0; e2 < 16; ++e2) {
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
      const size_t head_off = is_q ? (size_t)col_h : (size_t)(head - g.q_hq - (is_k ? 0 : g.q_hkv)) * dh;
      auto dst_row = [&](int i, int lr) {
        if (is_q) return cwarp + (size_t)lr * g.ldc + head_off;
        return (is_k ? g.q_kc : g.q_vc) + cache_row[i] + head_off;
      };
      uint4 o[4], t[4];
      epi_pack32(lo, o);
      epi_transpose(w, 0, o, t);
      epi_store_t(w, t, true, 32, [&](int i, int lr) { return dst_row(i, lr) + t0; });
      epi_pack32(hi, o);
      epi_transpose(w, 1, o, t);
      epi_store_t(w, t, true, 32, [&](int i, int lr) { return dst_row(i, lr) + (dh >> 1) + t0; });
    }
  }
}

}  // namespace d2c
