// Portable tensor-core GEMM (mma.sync m16n8k16, bf16 in, fp32 accumulate) with the step's fused
// epilogues.  C[m][n] = sum_k A[m][k] * W[n][k].  The row count is read from device memory, so the
// grid is sized for the worst case and tiles past the live rows exit at once.
//
// This is the bring-up / cross-check implementation: the tcgen05 kernel in gemm_tc.cu is the one the
// step uses on B200; both share the argument block and must produce the same results.
//
// Tile 128 x 128 x 64, 8 warps (2 x 4), 3-stage cp.async pipeline, 128-byte rows XOR-swizzled in
// 16-byte chunks so that ldmatrix is conflict free.
#include "common.cuh"

namespace d2c {

namespace {
constexpr int BM = 128, BN = 128, BK = 64, STAGES = 3, THREADS = 256;
constexpr int STAGE_BYTES = (BM + BN) * BK * 2;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

// Column of the output that row r of the shared B tile holds.  For the SwiGLU epilogue a tile covers
// 64 output columns and interleaves gate and up rows in groups of 8, so that every thread ends up
// with the gate and the up value of the same column.
template <int EPI>
__device__ __forceinline__ void b_row_source(int r, int tile_n, int& col, bool& second) {
  if (EPI == EPI_SWIGLU) {
    const int warp_n = r >> 5, frag = (r >> 3) & 3, within = r & 7;
    second = frag & 1;
    col = tile_n * 64 + warp_n * 16 + (frag >> 1) * 8 + within;
  } else {
    second = false;
    col = tile_n * BN + r;
  }
}

template <int EPI>
__global__ void __launch_bounds__(THREADS, 2) gemm_mma_kernel(GemmArgs g) {
  pdl_prologue();
  extern __shared__ __align__(128) unsigned char smem[];
  const int n = *g.n_rows;
  const int m0 = blockIdx.y * BM;
  if (m0 >= n) return;
  const int tile_n = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int warp_m = warp >> 2, warp_n = warp & 3;
  const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);
  const int KT = g.K / BK;

  auto load_stage = [&](int stage, int kt) {
    const uint32_t sa = smem_base + stage * STAGE_BYTES, sb = sa + BM * BK * 2;
    const int k0 = kt * BK;
#pragma unroll
    for (int i = 0; i < (BM * 8) / THREADS; ++i) {
      const int idx = tid + i * THREADS, r = idx >> 3, ch = idx & 7;
      const int gr = m0 + r;
      const bool ok = gr < n;
      const bf16* src = g.A + (size_t)(ok ? gr : 0) * g.lda + k0 + ch * 8;
      cp_async16(sa + swz(r, ch), src, ok ? 16 : 0);
    }
#pragma unroll
    for (int i = 0; i < (BN * 8) / THREADS; ++i) {
      const int idx = tid + i * THREADS, r = idx >> 3, ch = idx & 7;
      int col; bool second;
      b_row_source<EPI>(r, tile_n, col, second);
      const bool ok = col < g.N;
      const bf16* w = second ? g.W2 : g.W;
      const bf16* src = w + (size_t)(ok ? col : 0) * g.K + k0 + ch * 8;
      cp_async16(sb + swz(r, ch), src, ok ? 16 : 0);
    }
  };

  float acc[4][4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < KT) load_stage(s, s);
    cp_async_commit();
  }
  for (int kt = 0; kt < KT; ++kt) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();
    if (kt + STAGES - 1 < KT) load_stage((kt + STAGES - 1) % STAGES, kt + STAGES - 1);
    cp_async_commit();
    const uint32_t sa = smem_base + (kt % STAGES) * STAGE_BYTES, sb = sa + BM * BK * 2;
#pragma unroll
    for (int kk = 0; kk < BK / 16; ++kk) {
      uint32_t af[4][4], bfr[2][4];
#pragma unroll
      for (int mi = 0; mi < 4; ++mi)
        ldmatrix_x4(af[mi], sa + swz(warp_m * 64 + mi * 16 + (lane & 15), kk * 2 + (lane >> 4)));
#pragma unroll
      for (int nj = 0; nj < 2; ++nj)
        ldmatrix_x4(bfr[nj], sb + swz(warp_n * 32 + nj * 16 + (lane & 7) + ((lane >> 4) << 3), kk * 2 + ((lane >> 3) & 1)));
#pragma unroll
      for (int mi = 0; mi < 4; ++mi)
#pragma unroll
        for (int ni = 0; ni < 4; ++ni)
          mma_bf16(acc[mi][ni], af[mi], bfr[ni >> 1][(ni & 1) * 2], bfr[ni >> 1][(ni & 1) * 2 + 1]);
    }
  }
  cp_async_wait<0>();

  // ---------------------------------------------------------------- epilogues
  const int qrow = lane >> 2, qcol = (lane & 3) * 2;
  if (EPI == EPI_STORE || EPI == EPI_RESIDUAL) {
#pragma unroll
    for (int mi = 0; mi < 4; ++mi)
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int row = m0 + warp_m * 64 + mi * 16 + qrow + hh * 8;
        if (row >= n) continue;
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) {
          const int col = tile_n * BN + warp_n * 32 + ni * 8 + qcol;
          if (col >= g.N) continue;                       // N is even, so col+1 < N as well
          float v0 = acc[mi][ni][hh * 2], v1 = acc[mi][ni][hh * 2 + 1];
          __nv_bfloat162* dst = reinterpret_cast<__nv_bfloat162*>(g.C + (size_t)row * g.ldc + col);
          if (EPI == EPI_STORE) {
            if (g.bias) { v0 += __bfloat162float(g.bias[col]); v1 += __bfloat162float(g.bias[col + 1]); }
          } else {
            const float2 old = __bfloat1622float2(*dst);
            v0 += old.x; v1 += old.y;
          }
          *dst = __floats2bfloat162_rn(v0, v1);
        }
      }
  } else if (EPI == EPI_SWIGLU) {
#pragma unroll
    for (int mi = 0; mi < 4; ++mi)
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int row = m0 + warp_m * 64 + mi * 16 + qrow + hh * 8;
        if (row >= n) continue;
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int col = tile_n * 64 + warp_n * 16 + q * 8 + qcol;
          if (col >= g.N) continue;
          const float g0 = acc[mi][2 * q][hh * 2], g1 = acc[mi][2 * q][hh * 2 + 1];
          const float u0 = acc[mi][2 * q + 1][hh * 2], u1 = acc[mi][2 * q + 1][hh * 2 + 1];
          const float o0 = g0 / (1.f + __expf(-g0)) * u0, o1 = g1 / (1.f + __expf(-g1)) * u1;
          *reinterpret_cast<__nv_bfloat162*>(g.C + (size_t)row * g.ldc + col) = __floats2bfloat162_rn(o0, o1);
        }
      }
  } else {  // EPI_LMSTATS
    __syncthreads();                                       // pipeline smem is free now
    float* s_max = reinterpret_cast<float*>(smem);         // [4 warps in n][128 rows]
    float* s_sum = s_max + 4 * BM;
    int* s_arg = reinterpret_cast<int*>(s_sum + 4 * BM);
#pragma unroll
    for (int mi = 0; mi < 4; ++mi)
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int lrow = warp_m * 64 + mi * 16 + qrow + hh * 8;
        const int row = m0 + lrow;
        float mx = -INFINITY; int arg = 0x7fffffff;
#pragma unroll
        for (int ni = 0; ni < 4; ++ni)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int col = tile_n * BN + warp_n * 32 + ni * 8 + qcol + e;
            const float v = acc[mi][ni][hh * 2 + e];
            if (col < g.N) {
              if (g.logits && row < n) g.logits[(size_t)row * g.N + col] = v;
              if (v > mx) { mx = v; arg = col; }           // columns ascend: first maximum wins
            }
          }
#pragma unroll
        for (int o = 1; o <= 2; o <<= 1) {
          const float omx = __shfl_xor_sync(0xffffffffu, mx, o);
          const int oarg = __shfl_xor_sync(0xffffffffu, arg, o);
          if (omx > mx || (omx == mx && oarg < arg)) { mx = omx; arg = oarg; }
        }
        float sum = 0.f;
#pragma unroll
        for (int ni = 0; ni < 4; ++ni)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int col = tile_n * BN + warp_n * 32 + ni * 8 + qcol + e;
            if (col < g.N) sum += __expf(acc[mi][ni][hh * 2 + e] - mx);
          }
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        if ((lane & 3) == 0) { s_max[warp_n * BM + lrow] = mx; s_sum[warp_n * BM + lrow] = sum; s_arg[warp_n * BM + lrow] = arg; }
      }
    __syncthreads();
    if (tid < BM && m0 + tid < n) {
      float mx = -INFINITY; int arg = 0x7fffffff;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const float v = s_max[w * BM + tid]; const int a2 = s_arg[w * BM + tid];
        if (v > mx || (v == mx && a2 < arg)) { mx = v; arg = a2; }
      }
      float sum = 0.f;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const float v = s_max[w * BM + tid];
        if (v > -INFINITY) sum += s_sum[w * BM + tid] * __expf(v - mx);
      }
      const size_t o = (size_t)(m0 + tid) * g.n_tiles + tile_n;
      g.st_max[o] = mx; g.st_sum[o] = sum; g.st_arg[o] = arg;
    }
  }
}

template <int EPI>
int launch_one(const GemmArgs& g, cudaStream_t st) {
  const int smem = STAGES * STAGE_BYTES;
  static PerDevice attr_set;
  if (attr_set.first()) {
    D2C_CUDA_OK(cudaFuncSetAttribute(gemm_mma_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  }
  const int n_tiles = EPI == EPI_SWIGLU ? ceil_div(g.N, 64) : ceil_div(g.N, BN);
  dim3 grid(n_tiles, ceil_div(g.max_rows, BM));
  D2C_LAUNCH((gemm_mma_kernel<EPI>), grid, THREADS, smem, st, g);
  return D2C_OK;
}
}  // namespace

int launch_gemm_mma(const GemmArgs& g, GemmEpilogue epi, cudaStream_t st) {
  if (g.max_rows <= 0 || g.N <= 0) return D2C_OK;
  if (g.K % BK != 0 || (g.N & 1)) { set_global_error("gemm: K=%d must be a multiple of 64 and N=%d even", g.K, g.N); return D2C_ESHAPE; }
  switch (epi) {
    case EPI_STORE: return launch_one<EPI_STORE>(g, st);
    case EPI_RESIDUAL: return launch_one<EPI_RESIDUAL>(g, st);
    case EPI_SWIGLU: return launch_one<EPI_SWIGLU>(g, st);
    case EPI_LMSTATS: return launch_one<EPI_LMSTATS>(g, st);
    default: break;
  }
  return D2C_EINVAL;
}

}  // namespace d2c
