// Shared declarations of the d2c CUDA sources: error plumbing, small device helpers and the
// launchers each .cu file exposes to the C-ABI layer (d2c_api.cu).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "../../include/d2c.h"

typedef __nv_bfloat16 bf16;

namespace d2c {

// Text of the last error raised outside any context (thread local).
void set_global_error(const char* fmt, ...);
const char* global_error();
// Adds n to this thread's count of kernels launched by the library.
void count_launch(int n);

#define D2C_CUDA_OK(expr)                                                              \
  do {                                                                                 \
    cudaError_t e__ = (expr);                                                          \
    if (e__ != cudaSuccess) {                                                          \
      d2c::set_global_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__),   \
                            __FILE__, __LINE__);                                       \
      return D2C_ECUDA;                                                                \
    }                                                                                  \
  } while (0)
// Programmatic dependent launch: every kernel of the step is launched with the stream-serialisation
// attribute.  All but the GEMMs start with pdl_prologue(), which waits for the preceding kernel's results and
// then lets the following kernel begin its own launch, so launch latency overlaps the predecessor's tail.  The
// tcgen05 GEMMs let their successor launch first, set up barriers and TMEM, read the row count and request their
// first weight boxes, and wait only before they touch what the predecessor wrote.  That is sound because a
// pdl_prologue() kernel stands between the selection kernel, which writes the counts, and every GEMM: nothing
// behind that kernel can run before selection has completed.  (The same order in the attention kernels, whose
// loads all depend on the predecessor, measured no different and is not used.)
#ifdef __CUDACC__
__device__ __forceinline__ long long global_timer_ns() { long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
__device__ __forceinline__ void pdl_prologue() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args&&>(args)...);
}
#define D2C_LAUNCH(kernel, grid, block, smem, st, ...)                                      \
  do {                                                                                      \
    D2C_CUDA_OK(d2c::launch_pdl(kernel, grid, block, smem, st, __VA_ARGS__));               \
    d2c::count_launch(1);                                                                   \
  } while (0)
// After a kernel launch: checks the launch and counts it.
#define D2C_LAUNCHED() do { D2C_CUDA_OK(cudaGetLastError()); d2c::count_launch(1); } while (0)

// Per-device one-time set-up (function attributes, device properties): kernels' attributes belong to the
// device they were set on, so the "done" flags are kept per device ordinal, for the device that is current.
constexpr int kMaxDevices = 64;
struct PerDevice {
  bool done[kMaxDevices] = {};
  // true the first time it is called with this device current (and for ordinals beyond the table, every time)
  bool first() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return true;
    if (done[dev]) return false;
    done[dev] = true;
    return true;
  }
};
// Multiprocessor count of the current device (looked up once per device).
int sm_count_current();

static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- selection (select.cu) -------------------------------------------------------------------
struct SelectArgs {
  const uint8_t* mask; const float* conf; const float* c; const float* override_key;
  const int32_t* forced; const int32_t* forced_off;
  int batch, seq_len, k; float p; int stage2_candidates;
  int block_lo, block_hi;                        // stage 1 only looks at masked positions in [block_lo, block_hi); empty = all
  const uint32_t* phi_q30; int phi_len;          // phi table in 2^-30 fixed point, entries [0, phi_len)
  float* key; int32_t* sel_idx; int32_t* row_seq; int32_t* row_off; int32_t* lm_rows; int32_t* lm_off;
  int32_t* slot_of_pos;
  int32_t* rank_s; int32_t* rank_lm; int32_t* n_b; int32_t* nm_b;   // scratch [B][L],[B][L],[B],[B]
  int32_t* n_host;                               // optional: device-visible address of a host word that receives the total row count
};
int launch_select(const SelectArgs& a, cudaStream_t st);
// Fills tab[0..len) with floor(exp(-r^2/(2 sigma^2)) * 2^30 + 0.5); returns the first r whose entry is 0 (or len).
int build_phi_table(float sigma, uint32_t* tab, int len);

// ---- row kernels (rows.cu) -------------------------------------------------------------------
int launch_gather_norm(const bf16* h0, const int32_t* sel_idx, const int32_t* row_seq, const int32_t* n_rows,
                       int max_rows, int seq_len, int d, const bf16* gain, float eps, bf16* x, bf16* xn,
                       cudaStream_t st);
int launch_rmsnorm(const bf16* x, const int32_t* row_map, const int32_t* n_rows, int max_rows, int d,
                   const bf16* gain, float eps, bf16* xn, cudaStream_t st);
int launch_rope_table(float2* tab, int max_seq, int head_dim, float base, cudaStream_t st);
int launch_rope_scatter(bf16* qkv, const int32_t* sel_idx, const int32_t* row_seq, const int32_t* n_rows,
                        int max_rows, int hq, int hkv, int dh, const float2* rope, bf16* kc, bf16* vc,
                        int cache_seq, cudaStream_t st);

// ---- GEMMs (gemm_mma.cu, gemm_tc.cu) -----------------------------------------------------------
enum GemmEpilogue { EPI_STORE = 0, EPI_RESIDUAL = 1, EPI_SWIGLU = 2, EPI_LMSTATS = 3, EPI_QKV_ROPE = 4 };
struct GemmArgs {
  const bf16* A; int lda;            // [max_rows][K]
  const bf16* W; const bf16* W2;     // [N][K]; W2 = the "up" matrix for EPI_SWIGLU
  const bf16* bias;                  // [N] or null (EPI_STORE)
  bf16* C; int ldc;                  // output (EPI_STORE / EPI_RESIDUAL: C += ; EPI_SWIGLU: silu(AW^T)*(AW2^T))
  const int32_t* n_rows; int max_rows; int N; int K;
  // EPI_LMSTATS: per (row, 128-column tile) running max / sum of exp / arg-max, optional raw logits
  float* st_max; float* st_sum; int32_t* st_arg; float* logits; int n_tiles;
  // EPI_QKV_ROPE (tcgen05 kernels only): rotary embedding of Q/K and the K/V scatter into the cache fused into
  // the QKV projection; C/ldc is the QKV activation buffer (only its Q part is written)
  const int32_t* q_sel_idx; const int32_t* q_row_seq; const float2* q_rope; bf16* q_kc; bf16* q_vc;
  int q_cache_seq, q_hq, q_hkv, q_dh;
  // split-K scratch of the tcgen05 kernels (null: no split): sk_max_tiles partial tiles of 128 x 256 fp32
  // and twice as many zero-initialised counters
  float* sk_partials; int32_t* sk_counters; int sk_max_tiles;
  // RMSNorm folded into the GEMMs around it (tcgen05 kernels).  A residual epilogue that is given nx_out also writes
  // nx_out[row][col] = bf16(x_new[row][col] * nx_gain[col]) (same leading dimension as C) and, per (row, 32-column
  // chunk), the sum of squares of the new x into nx_ssq[row][N / 32].  A GEMM that is given in_ssq (K / 32 such
  // partial sums per row of A) multiplies accumulator row r by rsqrt(sum_t in_ssq[r][t] / K + in_eps) before its
  // own epilogue: the per-row scalar commutes with the contraction, so A = x * gain gives the same product as
  // A = rmsnorm(x) * gain.
  bf16* nx_out; const bf16* nx_gain; float* nx_ssq;
  const float* in_ssq; float in_eps;
  // optional (tcgen05 kernels): CTA 0 stores {clock64, globaltimer ns} at its start and its end, which gives the
  // SM clock the launch really ran at (a power-capped clock is not what a coarse NVML sample shows)
  long long* clock_probe;
};
static const int kSkMaxTiles = 160;
int launch_gemm_mma(const GemmArgs& g, GemmEpilogue epi, cudaStream_t st);

// ---- attention (attention.cu) ----------------------------------------------------------------
struct AttnArgs {
  const bf16* q; int ldq; const bf16* kc; const bf16* vc; const int32_t* row_off;
  int batch, seq_len, cache_seq, hq, hkv, dh; int max_rows_per_seq;
  bf16* o; float* lse; float* abar;      // abar may be null (layers outside the rollout)
  int q_rows;                            // rows the q buffer holds (bounds the TMA map)
  int portable;                          // 1: force the mma.sync kernels
  int* status;                           // device status word for bounded waits (may be null)
  int which;                             // 0: both kernels, 1: O/LSE only, 2: head-averaged probabilities only
  // optional scratch that lets the abar kernel split the heads over several CTAs when the problem has too few
  // (rows x keys) tiles to fill the GPU: partial sums [head group][rows][seq_len], added in a fixed order
  float* abar_partial; size_t abar_partial_floats; const int32_t* n_rows;
};
int launch_attention(const AttnArgs& a, cudaStream_t st);
bool attention_tc_supported(const AttnArgs& a);               // attention_tc.cu
int launch_attention_tc(const AttnArgs& a, cudaStream_t st, int* status);

// ---- LM head statistics (lmhead.cu) ------------------------------------------------------------
int launch_lm_reduce(const float* st_max, const float* st_sum, const int32_t* st_arg, int n_tiles,
                     const int32_t* n_rows, int max_rows, const int32_t* lm_rows, const int32_t* sel_idx,
                     const int32_t* row_seq, int seq_len, float* conf, int32_t* pred, cudaStream_t st);

// ---- rollout (rollout.cu) ----------------------------------------------------------------------
struct RolloutArgs {
  const float* abar; size_t layer_stride; int n_layers; const int32_t* sel_idx; const int32_t* row_off;
  int batch, seq_len; float* c; float* u0; float* u1; float* partial; int n_split;
};
int launch_rollout(const RolloutArgs& a, cudaStream_t st);
static const int kRolloutSplit = 16;

}  // namespace d2c

namespace d2c {
// ---- commit helper (commit.cu) -------------------------------------------------------------------
int launch_commit(int batch, int seq_len, int d, int rule, float threshold, const int32_t* slot_of_pos,
                  const float* conf, const int32_t* pred, const uint32_t* phi, int phi_len, const bf16* embed,
                  bf16* h0, uint8_t* mask, int32_t* tokens, int32_t* committed, cudaStream_t st);
// ---- tcgen05 GEMM (gemm_tc.cu) -------------------------------------------------------------------
// status: device int[4] that receives D2C_ETIMEOUT if a bounded wait runs out (null: a library-owned word).
int launch_gemm_tc(const GemmArgs& g, GemmEpilogue epi, cudaStream_t st, int* status = nullptr);
bool gemm_tc_supported(const GemmArgs& g);       // false: launch_gemm_tc would fall back to the mma.sync kernel
// ---- two-SM tcgen05 GEMM (gemm_tc2.cu): pairs of CTAs on 256-row tiles ---------------------------
bool gemm_tc2_supported(const GemmArgs& g);
int launch_gemm_tc2(const GemmArgs& g, GemmEpilogue epi, cudaStream_t st, int* status = nullptr);
}  // namespace d2c
