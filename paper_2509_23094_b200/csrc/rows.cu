// Row-wise kernels of the step: gather of the selected hidden rows (Eq. 5) fused with the first
// RMSNorm, stand-alone RMSNorm, and rotary embedding fused with the K/V scatter into the cache.
// All are HBM-bound streaming kernels: 16-byte accesses, one CTA per row.
#include "common.cuh"

namespace d2c {

static constexpr int kRowThreads = 256;

__device__ __forceinline__ float block_sum(float v, float* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  if (lane == 0) sh[wid] = v;
  __syncthreads();
  float t = 0.f;
  const int nw = blockDim.x >> 5;
  for (int w = 0; w < nw; ++w) t += sh[w];        // same order in every thread: deterministic
  __syncthreads();
  return t;
}

union Pack8 { uint4 u; __nv_bfloat162 h[4]; };

// x[r] = src[src_row(r)], xn[r] = rmsnorm(x[r]) * gain.  `x` may be null (norm only).
template <bool kGather>
__global__ void __launch_bounds__(kRowThreads)
norm_rows_kernel(const bf16* __restrict__ src, const int32_t* __restrict__ sel_idx,
                 const int32_t* __restrict__ row_seq, const int32_t* __restrict__ row_map,
                 const int32_t* __restrict__ n_rows, int seq_len, int d, const bf16* __restrict__ gain,
                 float eps, bf16* __restrict__ x, bf16* __restrict__ xn) {
  pdl_prologue();
  __shared__ float sh[kRowThreads / 32];
  const int n = *n_rows;
  for (int r = blockIdx.x; r < n; r += gridDim.x) {
    size_t srow;
    if (kGather) srow = (size_t)row_seq[r] * seq_len + sel_idx[r];
    else srow = row_map ? (size_t)row_map[r] : (size_t)r;
    const uint4* in = reinterpret_cast<const uint4*>(src + srow * d);
    const int nv = d >> 3;
    float ss = 0.f;
    for (int v = threadIdx.x; v < nv; v += kRowThreads) {
      Pack8 p; p.u = in[v];
#pragma unroll
      for (int e = 0; e < 4; ++e) { const float2 f = __bfloat1622float2(p.h[e]); ss += f.x * f.x + f.y * f.y; }
      if (kGather && x) reinterpret_cast<uint4*>(x + (size_t)r * d)[v] = p.u;
    }
    const float tot = block_sum(ss, sh);
    const float rs = rsqrtf(tot / (float)d + eps);
    for (int v = threadIdx.x; v < nv; v += kRowThreads) {
      Pack8 p; p.u = in[v];
      Pack8 g; g.u = reinterpret_cast<const uint4*>(gain)[v];
      Pack8 o;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 f = __bfloat1622float2(p.h[e]);
        const float2 gg = __bfloat1622float2(g.h[e]);
        o.h[e] = __floats2bfloat162_rn(f.x * rs * gg.x, f.y * rs * gg.y);
      }
      reinterpret_cast<uint4*>(xn + (size_t)r * d)[v] = o.u;
    }
  }
}

static int row_grid(int max_rows) { return max_rows < 148 * 8 ? max_rows : 148 * 8; }

int launch_gather_norm(const bf16* h0, const int32_t* sel_idx, const int32_t* row_seq, const int32_t* n_rows,
                       int max_rows, int seq_len, int d, const bf16* gain, float eps, bf16* x, bf16* xn,
                       cudaStream_t st) {
  if (max_rows <= 0) return D2C_OK;
  D2C_LAUNCH((norm_rows_kernel<true>), row_grid(max_rows), kRowThreads, 0, st, h0, sel_idx, row_seq, nullptr, n_rows, seq_len, d, gain, eps, x, xn);
  return D2C_OK;
}

int launch_rmsnorm(const bf16* x, const int32_t* row_map, const int32_t* n_rows, int max_rows, int d,
                   const bf16* gain, float eps, bf16* xn, cudaStream_t st) {
  if (max_rows <= 0) return D2C_OK;
  D2C_LAUNCH((norm_rows_kernel<false>), row_grid(max_rows), kRowThreads, 0, st, x, nullptr, nullptr, row_map, n_rows, 0, d, gain, eps, nullptr, xn);
  return D2C_OK;
}

// tab[pos][t] = (cos, sin)(pos * base^(-2t/Dh)), evaluated in fp64 once at set-up.
__global__ void rope_table_kernel(float2* tab, int max_seq, int half, double base, int dh) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= max_seq * half) return;
  const int pos = i / half, t = i % half;
  const double ang = (double)pos * pow(base, -2.0 * (double)t / (double)dh);
  double s, c;
  sincos(ang, &s, &c);
  tab[i] = make_float2((float)c, (float)s);
}

int launch_rope_table(float2* tab, int max_seq, int head_dim, float base, cudaStream_t st) {
  const int half = head_dim / 2, n = max_seq * half;
  rope_table_kernel<<<ceil_div(n, 256), 256, 0, st>>>(tab, max_seq, half, (double)base, head_dim);
  D2C_LAUNCHED();
  return D2C_OK;
}

// One CTA per selected row.  Q heads are rotated in place inside the QKV buffer; K heads are rotated
// and written to the cache row of (sequence, position); V heads are copied there.  Each thread owns
// 8 consecutive dims of the low half and the matching 8 of the high half (16-byte loads and stores).
__global__ void __launch_bounds__(kRowThreads)
rope_scatter_kernel(bf16* __restrict__ qkv, const int32_t* __restrict__ sel_idx,
                    const int32_t* __restrict__ row_seq, const int32_t* __restrict__ n_rows, int hq, int hkv,
                    int dh, const float2* __restrict__ rope, bf16* __restrict__ kc, bf16* __restrict__ vc,
                    int cache_seq) {
  pdl_prologue();
  const int n = *n_rows;
  const int half = dh >> 1, chunks = half >> 3;            // 16-byte chunks per half head
  const int ld = (hq + 2 * hkv) * dh;
  for (int r = blockIdx.x; r < n; r += gridDim.x) {
    const int pos = sel_idx[r], b = row_seq[r];
    bf16* row = qkv + (size_t)r * ld;
    const size_t crow = ((size_t)b * cache_seq + pos) * (size_t)(hkv * dh);
    const float2* rt = rope + (size_t)pos * half;
    const int n_rot = (hq + hkv) * chunks;
    for (int w = threadIdx.x; w < n_rot; w += kRowThreads) {
      const int head = w / chunks, ch = w % chunks;
      bf16* base = row + (size_t)head * dh;
      Pack8 lo, hi, olo, ohi;
      lo.u = *reinterpret_cast<const uint4*>(base + ch * 8);
      hi.u = *reinterpret_cast<const uint4*>(base + half + ch * 8);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 l = __bfloat1622float2(lo.h[e]), h = __bfloat1622float2(hi.h[e]);
        const float2 cs0 = rt[ch * 8 + 2 * e], cs1 = rt[ch * 8 + 2 * e + 1];
        olo.h[e] = __floats2bfloat162_rn(l.x * cs0.x - h.x * cs0.y, l.y * cs1.x - h.y * cs1.y);
        ohi.h[e] = __floats2bfloat162_rn(h.x * cs0.x + l.x * cs0.y, h.y * cs1.x + l.y * cs1.y);
      }
      bf16* dst = head < hq ? base : kc + crow + (size_t)(head - hq) * dh;
      *reinterpret_cast<uint4*>(dst + ch * 8) = olo.u;
      *reinterpret_cast<uint4*>(dst + half + ch * 8) = ohi.u;
    }
    const int n_v = hkv * (dh >> 3);
    const bf16* vsrc = row + (size_t)(hq + hkv) * dh;
    for (int w = threadIdx.x; w < n_v; w += kRowThreads)
      *reinterpret_cast<uint4*>(vc + crow + (size_t)w * 8) = *reinterpret_cast<const uint4*>(vsrc + (size_t)w * 8);
  }
}

int launch_rope_scatter(bf16* qkv, const int32_t* sel_idx, const int32_t* row_seq, const int32_t* n_rows,
                        int max_rows, int hq, int hkv, int dh, const float2* rope, bf16* kc, bf16* vc,
                        int cache_seq, cudaStream_t st) {
  if (max_rows <= 0) return D2C_OK;
  D2C_LAUNCH((rope_scatter_kernel), row_grid(max_rows), kRowThreads, 0, st, qkv, sel_idx, row_seq, n_rows, hq, hkv, dh, rope, kc, vc, cache_seq);
  return D2C_OK;
}

}  // namespace d2c
