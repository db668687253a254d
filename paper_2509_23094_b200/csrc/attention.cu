// Selected-query bidirectional attention over the full KV cache (Section 4.2: the attention of the
// |y*| selected rows against all L keys), in two kernels:
//
//   attn_fwd_kernel   flash-style: O = softmax(Q K^T / sqrt(Dh)) V and the log-sum-exp of every
//                     (row, head), keys streamed in tiles of 64, nothing of size rows x L stored.
//   attn_abar_kernel  the head-averaged probabilities Abar[r][j] = 1/Hq sum_h exp(s_h[r][j] - lse_h[r])
//                     that the rollout (Eq. 6-9) consumes: one CTA per (64 rows x 64 keys) tile loops
//                     over the heads and adds in a fixed order, so the result is deterministic.
//
// Both use mma.sync m16n8k16 bf16 with fp32 accumulation; 4 warps, 16 query rows per warp.
#include "common.cuh"

namespace d2c {
namespace {

constexpr int QT = 64, KT = 64, ATHREADS = 128;
constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;

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
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Byte offset of (row, 16-byte chunk) in a tile whose rows hold DH bf16, chunks XOR-swizzled by row.
template <int DH>
__device__ __forceinline__ uint32_t toff(int row, int chunk) {
  return (uint32_t)(row * (DH * 2) + (((chunk & ~7) | ((chunk ^ row) & 7)) << 4));
}

// Copies `rows` x DH bf16 (row stride ld elements) into a swizzled tile; rows >= valid are zero-filled.
template <int DH>
__device__ __forceinline__ void load_tile(uint32_t sdst, const bf16* src, size_t ld, int valid, int rows) {
  constexpr int CH = DH / 8;
  for (int idx = threadIdx.x; idx < rows * CH; idx += ATHREADS) {
    const int r = idx / CH, ch = idx % CH;
    const bool ok = r < valid;
    cp_async16(sdst + toff<DH>(r, ch), src + (ok ? (size_t)r * ld + ch * 8 : 0), ok ? 16 : 0);
  }
}

template <int DH>
__global__ void __launch_bounds__(ATHREADS) attn_fwd_kernel(AttnArgs a) {
  pdl_prologue();
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int TILE = KT * DH * 2;
  const int b = blockIdx.z, h = blockIdx.y, g = h / (a.hq / a.hkv);
  const int r0 = a.row_off[b] + blockIdx.x * QT;
  const int nrows = min(QT, a.row_off[b + 1] - r0);
  if (nrows <= 0) return;
  const int L = a.seq_len, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t sq = (uint32_t)__cvta_generic_to_shared(smem);
  const uint32_t sk = sq + QT * DH * 2, sv = sk + 2 * TILE;
  const size_t kv_ld = (size_t)a.hkv * DH;
  const bf16* kbase = a.kc + (size_t)b * a.cache_seq * kv_ld + (size_t)g * DH;
  const bf16* vbase = a.vc + (size_t)b * a.cache_seq * kv_ld + (size_t)g * DH;
  const int T = (L + KT - 1) / KT;

  load_tile<DH>(sq, a.q + (size_t)r0 * a.ldq + (size_t)h * DH, a.ldq, nrows, QT);
  cp_async_commit();
  load_tile<DH>(sk, kbase, kv_ld, min(KT, L), KT);
  load_tile<DH>(sv, vbase, kv_ld, min(KT, L), KT);
  cp_async_commit();

  uint32_t qf[DH / 16][4];
  float o[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;     // rows lane/4 and lane/4 + 8 of this warp
  const float sc = kLog2e * rsqrtf((float)DH);

  for (int t = 0; t < T; ++t) {
    if (t + 1 < T) {
      const int k0 = (t + 1) * KT;
      load_tile<DH>(sk + ((t + 1) & 1) * TILE, kbase + (size_t)k0 * kv_ld, kv_ld, min(KT, L - k0), KT);
      load_tile<DH>(sv + ((t + 1) & 1) * TILE, vbase + (size_t)k0 * kv_ld, kv_ld, min(KT, L - k0), KT);
    }
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (t == 0) {
#pragma unroll
      for (int kk = 0; kk < DH / 16; ++kk)
        ldmatrix_x4(qf[kk], sq + toff<DH>(warp * 16 + (lane & 15), kk * 2 + (lane >> 4)));
    }
    const uint32_t skt = sk + (t & 1) * TILE, svt = sv + (t & 1) * TILE;
    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk) {
#pragma unroll
      for (int nj = 0; nj < 4; ++nj) {
        uint32_t kf[4];
        ldmatrix_x4(kf, skt + toff<DH>(nj * 16 + (lane & 7) + ((lane >> 4) << 3), kk * 2 + ((lane >> 3) & 1)));
        mma_bf16(s[2 * nj], qf[kk], kf[0], kf[1]);
        mma_bf16(s[2 * nj + 1], qf[kk], kf[2], kf[3]);
      }
    }
    // scale into the log2 domain, mask keys past the sequence end, online softmax
    const int kbase_idx = t * KT + (lane & 3) * 2;
    float mx0 = m0, mx1 = m1;
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = kbase_idx + i * 8 + (e & 1);
        const float v = key < L ? s[i][e] * sc : -INFINITY;
        s[i][e] = v;
        if (e < 2) mx0 = fmaxf(mx0, v); else mx1 = fmaxf(mx1, v);
      }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float c0 = exp2f(m0 - mx0), c1 = exp2f(m1 - mx1);   // first tile: exp2(-inf) = 0
    m0 = mx0; m1 = mx1;
    float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      s[i][0] = exp2f(s[i][0] - m0); s[i][1] = exp2f(s[i][1] - m0);
      s[i][2] = exp2f(s[i][2] - m1); s[i][3] = exp2f(s[i][3] - m1);
      rs0 += s[i][0] + s[i][1]; rs1 += s[i][2] + s[i][3];
    }
    l0 = l0 * c0 + rs0; l1 = l1 * c1 + rs1;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) { o[i][0] *= c0; o[i][1] *= c0; o[i][2] *= c1; o[i][3] *= c1; }
    // O += P V
#pragma unroll
    for (int j = 0; j < KT / 16; ++j) {
      uint32_t pf[4] = {pack_bf16(s[2 * j][0], s[2 * j][1]), pack_bf16(s[2 * j][2], s[2 * j][3]),
                        pack_bf16(s[2 * j + 1][0], s[2 * j + 1][1]), pack_bf16(s[2 * j + 1][2], s[2 * j + 1][3])};
#pragma unroll
      for (int dn = 0; dn < DH / 16; ++dn) {
        uint32_t vf[4];
        ldmatrix_x4_trans(vf, svt + toff<DH>(j * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, dn * 2 + (lane >> 4)));
        mma_bf16(o[2 * dn], pf, vf[0], vf[1]);
        mma_bf16(o[2 * dn + 1], pf, vf[2], vf[3]);
      }
    }
    __syncthreads();
  }
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const int lr0 = warp * 16 + (lane >> 2), lr1 = lr0 + 8;
  const float inv0 = 1.f / l0, inv1 = 1.f / l1;
  const size_t ldo = (size_t)a.hq * DH;
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) {
    const int col = h * DH + i * 8 + (lane & 3) * 2;
    if (lr0 < nrows) *reinterpret_cast<__nv_bfloat162*>(a.o + (size_t)(r0 + lr0) * ldo + col) = __floats2bfloat162_rn(o[i][0] * inv0, o[i][1] * inv0);
    if (lr1 < nrows) *reinterpret_cast<__nv_bfloat162*>(a.o + (size_t)(r0 + lr1) * ldo + col) = __floats2bfloat162_rn(o[i][2] * inv1, o[i][3] * inv1);
  }
  if ((lane & 3) == 0) {
    if (lr0 < nrows) a.lse[(size_t)(r0 + lr0) * a.hq + h] = (m0 + log2f(l0)) * kLn2;
    if (lr1 < nrows) a.lse[(size_t)(r0 + lr1) * a.hq + h] = (m1 + log2f(l1)) * kLn2;
  }
}

template <int DH>
__global__ void __launch_bounds__(ATHREADS) attn_abar_kernel(AttnArgs a) {
  pdl_prologue();
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int TILE = KT * DH * 2;
  const int b = blockIdx.z;
  const int r0 = a.row_off[b] + blockIdx.y * QT;
  const int nrows = min(QT, a.row_off[b + 1] - r0);
  const int k0 = blockIdx.x * KT, L = a.seq_len;
  if (nrows <= 0 || k0 >= L) return;
  const int nkeys = min(KT, L - k0);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t sq = (uint32_t)__cvta_generic_to_shared(smem);   // 2 stages of Q
  const uint32_t sk = sq + 2 * TILE;                               // 2 stages of K
  const size_t kv_ld = (size_t)a.hkv * DH;
  const int group = a.hq / a.hkv;
  const bf16* kbase = a.kc + ((size_t)b * a.cache_seq + k0) * kv_ld;
  const float sc = kLog2e * rsqrtf((float)DH);

  auto issue = [&](int h) {
    load_tile<DH>(sq + (h & 1) * TILE, a.q + (size_t)r0 * a.ldq + (size_t)h * DH, a.ldq, nrows, QT);
    if (h % group == 0) load_tile<DH>(sk + ((h / group) & 1) * TILE, kbase + (size_t)(h / group) * DH, kv_ld, nkeys, KT);
  };
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }
  const int lr0 = warp * 16 + (lane >> 2), lr1 = lr0 + 8;

  issue(0);
  cp_async_commit();
  for (int h = 0; h < a.hq; ++h) {
    if (h + 1 < a.hq) issue(h + 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    const uint32_t sqh = sq + (h & 1) * TILE, skh = sk + ((h / group) & 1) * TILE;
    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk) {
      uint32_t qf[4];
      ldmatrix_x4(qf, sqh + toff<DH>(warp * 16 + (lane & 15), kk * 2 + (lane >> 4)));
#pragma unroll
      for (int nj = 0; nj < 4; ++nj) {
        uint32_t kf[4];
        ldmatrix_x4(kf, skh + toff<DH>(nj * 16 + (lane & 7) + ((lane >> 4) << 3), kk * 2 + ((lane >> 3) & 1)));
        mma_bf16(s[2 * nj], qf, kf[0], kf[1]);
        mma_bf16(s[2 * nj + 1], qf, kf[2], kf[3]);
      }
    }
    const float e0 = lr0 < nrows ? a.lse[(size_t)(r0 + lr0) * a.hq + h] * kLog2e : 0.f;
    const float e1 = lr1 < nrows ? a.lse[(size_t)(r0 + lr1) * a.hq + h] * kLog2e : 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      acc[i][0] += exp2f(s[i][0] * sc - e0); acc[i][1] += exp2f(s[i][1] * sc - e0);
      acc[i][2] += exp2f(s[i][2] * sc - e1); acc[i][3] += exp2f(s[i][3] * sc - e1);
    }
    __syncthreads();
  }
  const float inv = 1.f / (float)a.hq;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int key = k0 + i * 8 + (lane & 3) * 2;
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      if (key + e < L) {
        if (lr0 < nrows) a.abar[(size_t)(r0 + lr0) * L + key + e] = acc[i][e] * inv;
        if (lr1 < nrows) a.abar[(size_t)(r0 + lr1) * L + key + e] = acc[i][2 + e] * inv;
      }
    }
  }
}

template <int DH>
int launch_dh(const AttnArgs& a, cudaStream_t st) {
  const int smem_fwd = QT * DH * 2 + 4 * KT * DH * 2, smem_ab = 4 * KT * DH * 2;
  static PerDevice attr_set;
  if (attr_set.first()) {
    D2C_CUDA_OK(cudaFuncSetAttribute(attn_fwd_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_fwd));
    D2C_CUDA_OK(cudaFuncSetAttribute(attn_abar_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_ab));
  }
  const int qtiles = ceil_div(a.max_rows_per_seq, QT);
  if (a.which != 2) {
    D2C_LAUNCH((attn_fwd_kernel<DH>), dim3(qtiles, a.hq, a.batch), ATHREADS, smem_fwd, st, a);
  }
  if (a.abar && a.which != 1) {
    D2C_LAUNCH((attn_abar_kernel<DH>), dim3(ceil_div(a.seq_len, KT), qtiles, a.batch), ATHREADS, smem_ab, st, a);
  }
  return D2C_OK;
}
}  // namespace

int launch_attention(const AttnArgs& a, cudaStream_t st) {
  if (a.batch <= 0 || a.seq_len <= 0 || a.max_rows_per_seq <= 0) return D2C_OK;
  if (a.hq % a.hkv != 0) { set_global_error("attention: %d query heads not a multiple of %d kv heads", a.hq, a.hkv); return D2C_ESHAPE; }
  if (!a.portable && attention_tc_supported(a)) return launch_attention_tc(a, st, a.status);
  if (a.dh == 64) return launch_dh<64>(a, st);
  if (a.dh == 128) return launch_dh<128>(a, st);
  set_global_error("attention: head_dim %d not supported (64 or 128)", a.dh);
  return D2C_ESHAPE;
}

}  // namespace d2c
