// C-ABI entry points of the stand-alone kernels (selection, GEMM, attention, LM head, rollout):
// argument checks and the split of caller-provided scratch.  Used to test and time each kernel alone.
#include <math.h>

#include <vector>

#include "common.cuh"

using namespace d2c;

static int bad(int code, const char* msg) { set_global_error("%s", msg); return code; }

extern "C" {

size_t d2c_op_select_scratch_bytes(int32_t batch, int32_t seq_len) {
  if (batch < 1 || seq_len < 1) return 0;
  const size_t R = (size_t)batch * seq_len;
  // rank_s, rank_lm, row_seq [R]; n_b, nm_b [batch]; phi table [seq_len]; each piece 256-byte aligned
  return 3 * align_up(R * 4, 256) + 2 * align_up((size_t)batch * 4, 256) + align_up((size_t)seq_len * 4, 256);
}

int d2c_op_select(const uint8_t* mask, const float* conf, const float* c, const float* override_key,
                  const int32_t* forced, const int32_t* forced_off, int32_t batch, int32_t seq_len,
                  int32_t k, float p, float sigma, int32_t stage2_candidates,
                  float* key, int32_t* sel_idx, int32_t* row_off, int32_t* lm_rows, int32_t* lm_off,
                  int32_t* slot_of_pos, void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (!mask || !conf || !c || !key || !sel_idx || !row_off || !lm_rows || !lm_off || !slot_of_pos || !scratch)
    return bad(D2C_EINVAL, "d2c_op_select: null pointer");
  if (batch < 1 || seq_len < 1 || k < 0 || isnan(p) || !(sigma > 0.f) || (stage2_candidates != 0 && stage2_candidates != 1))
    return bad(D2C_EINVAL, "d2c_op_select: bad batch / seq_len / k / p / sigma / stage2_candidates");
  if (seq_len > 8192) return bad(D2C_ECAPACITY, "d2c_op_select: seq_len > 8192");
  if ((forced == nullptr) != (forced_off == nullptr)) return bad(D2C_EINVAL, "d2c_op_select: forced and forced_off go together");
  if (scratch_bytes < d2c_op_select_scratch_bytes(batch, seq_len) || reinterpret_cast<uintptr_t>(scratch) % 256)
    return bad(D2C_ECAPACITY, "d2c_op_select: scratch too small or not 256-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t R = (size_t)batch * seq_len;
  char* sp = static_cast<char*>(scratch);
  SelectArgs a{};
  a.rank_s = reinterpret_cast<int32_t*>(sp); sp += align_up(R * 4, 256);
  a.rank_lm = reinterpret_cast<int32_t*>(sp); sp += align_up(R * 4, 256);
  a.row_seq = reinterpret_cast<int32_t*>(sp); sp += align_up(R * 4, 256);
  a.n_b = reinterpret_cast<int32_t*>(sp); sp += align_up((size_t)batch * 4, 256);
  a.nm_b = reinterpret_cast<int32_t*>(sp); sp += align_up((size_t)batch * 4, 256);
  uint32_t* phi = reinterpret_cast<uint32_t*>(sp);
  std::vector<uint32_t> tab(seq_len);
  const int phi_len = build_phi_table(sigma, tab.data(), seq_len);
  D2C_CUDA_OK(cudaMemcpyAsync(phi, tab.data(), tab.size() * 4, cudaMemcpyHostToDevice, st));
  D2C_CUDA_OK(cudaStreamSynchronize(st));       // pageable host table: the copy must finish before it dies
  a.mask = mask; a.conf = conf; a.c = c; a.override_key = override_key; a.forced = forced; a.forced_off = forced_off;
  a.batch = batch; a.seq_len = seq_len; a.k = k; a.p = p; a.stage2_candidates = stage2_candidates; a.block_lo = 0; a.block_hi = 0;
  a.phi_q30 = phi; a.phi_len = phi_len;
  a.key = key; a.sel_idx = sel_idx; a.row_off = row_off; a.lm_rows = lm_rows; a.lm_off = lm_off; a.slot_of_pos = slot_of_pos;
  return launch_select(a, st);
}

int d2c_op_gemm(const void* A, const void* W, const void* bias, void* C, const int32_t* n_rows,
                int32_t max_rows, int32_t N, int32_t K, int32_t impl, void* cuda_stream) {
  if (!A || !W || !C || !n_rows) return bad(D2C_EINVAL, "d2c_op_gemm: null pointer");
  if (max_rows < 1 || N < 2 || K < 64) return bad(D2C_EINVAL, "d2c_op_gemm: bad max_rows / N / K");
  GemmArgs g{};
  g.A = (const bf16*)A; g.lda = K; g.W = (const bf16*)W; g.bias = (const bf16*)bias; g.C = (bf16*)C; g.ldc = N;
  g.n_rows = n_rows; g.max_rows = max_rows; g.N = N; g.K = K;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (impl == 1) return launch_gemm_mma(g, EPI_STORE, st);
  if (impl == 0) return gemm_tc2_supported(g) ? launch_gemm_tc2(g, EPI_STORE, st) : launch_gemm_tc(g, EPI_STORE, st);
  if (impl == 2) return launch_gemm_tc(g, EPI_STORE, st);
  return bad(D2C_EINVAL, "d2c_op_gemm: impl must be 0 (tcgen05), 1 (mma.sync) or 2 (one-SM tcgen05)");
}

int d2c_op_attention(const void* q, int32_t q_rows, int32_t ldq, const void* kcache, const void* vcache,
                     const int32_t* row_off, int32_t batch, int32_t seq_len, int32_t cache_seq,
                     int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                     void* o, float* lse, float* abar, int32_t impl, void* cuda_stream) {
  if (!q || !kcache || !vcache || !row_off || !o || !lse) return bad(D2C_EINVAL, "d2c_op_attention: null pointer");
  if (batch < 1 || seq_len < 1 || cache_seq < seq_len || n_q_heads < 1 || n_kv_heads < 1 || ldq < n_q_heads * head_dim || (ldq & 7) ||
      q_rows < 1 || (impl != 0 && impl != 1))
    return bad(D2C_EINVAL, "d2c_op_attention: bad sizes");
  AttnArgs a{};
  a.q = (const bf16*)q; a.ldq = ldq; a.kc = (const bf16*)kcache; a.vc = (const bf16*)vcache; a.row_off = row_off;
  a.batch = batch; a.seq_len = seq_len; a.cache_seq = cache_seq; a.hq = n_q_heads; a.hkv = n_kv_heads; a.dh = head_dim;
  a.max_rows_per_seq = seq_len < q_rows ? seq_len : q_rows; a.o = (bf16*)o; a.lse = lse; a.abar = abar;
  a.q_rows = q_rows; a.portable = impl; a.status = nullptr;
  return launch_attention(a, static_cast<cudaStream_t>(cuda_stream));
}

size_t d2c_op_lm_head_scratch_bytes(int32_t max_rows, int32_t vocab) {
  if (max_rows < 1 || vocab < 2) return 0;
  return 3 * align_up((size_t)max_rows * ceil_div(vocab, 128) * 4, 256);
}

int d2c_op_lm_head(const void* x, const void* w_lm, const int32_t* n_rows, int32_t max_rows,
                   int32_t d, int32_t vocab, float* conf, int32_t* pred, float* logits,
                   void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (!x || !w_lm || !n_rows || !conf || !pred || !scratch) return bad(D2C_EINVAL, "d2c_op_lm_head: null pointer");
  if (max_rows < 1 || d < 64 || d % 64 || vocab < 2 || (vocab & 1)) return bad(D2C_EINVAL, "d2c_op_lm_head: bad sizes");
  if (scratch_bytes < d2c_op_lm_head_scratch_bytes(max_rows, vocab) || reinterpret_cast<uintptr_t>(scratch) % 256)
    return bad(D2C_ECAPACITY, "d2c_op_lm_head: scratch too small or not 256-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int nt = ceil_div(vocab, 128);
  const size_t piece = align_up((size_t)max_rows * nt * 4, 256);
  char* sp = static_cast<char*>(scratch);
  GemmArgs g{};
  g.A = (const bf16*)x; g.lda = d; g.W = (const bf16*)w_lm; g.n_rows = n_rows; g.max_rows = max_rows; g.N = vocab; g.K = d;
  g.st_max = reinterpret_cast<float*>(sp); g.st_sum = reinterpret_cast<float*>(sp + piece);
  g.st_arg = reinterpret_cast<int32_t*>(sp + 2 * piece); g.n_tiles = nt; g.logits = logits;
  int rc = launch_gemm_tc(g, EPI_LMSTATS, st);
  if (rc != D2C_OK) return rc;
  return launch_lm_reduce(g.st_max, g.st_sum, g.st_arg, nt, n_rows, max_rows, nullptr, nullptr, nullptr, 0, conf, pred, st);
}

size_t d2c_op_rollout_scratch_bytes(int32_t batch, int32_t seq_len) {
  if (batch < 1 || seq_len < 1) return 0;
  const size_t R = (size_t)batch * seq_len;
  return 2 * align_up(R * 4, 256) + align_up((size_t)kRolloutSplit * R * 4 + R, 256);
}

int d2c_op_rollout(const float* abar, size_t layer_stride, int32_t n_layers, const int32_t* sel_idx,
                   const int32_t* row_off, int32_t batch, int32_t seq_len, float* c,
                   void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (!abar || !sel_idx || !row_off || !c || !scratch) return bad(D2C_EINVAL, "d2c_op_rollout: null pointer");
  if (n_layers < 1 || batch < 1 || seq_len < 1) return bad(D2C_EINVAL, "d2c_op_rollout: bad sizes");
  if (scratch_bytes < d2c_op_rollout_scratch_bytes(batch, seq_len) || reinterpret_cast<uintptr_t>(scratch) % 256)
    return bad(D2C_ECAPACITY, "d2c_op_rollout: scratch too small or not 256-byte aligned");
  const size_t R = (size_t)batch * seq_len;
  char* sp = static_cast<char*>(scratch);
  RolloutArgs r{};
  r.abar = abar; r.layer_stride = layer_stride; r.n_layers = n_layers; r.sel_idx = sel_idx; r.row_off = row_off;
  r.batch = batch; r.seq_len = seq_len; r.c = c; r.n_split = kRolloutSplit;
  r.u0 = reinterpret_cast<float*>(sp); r.u1 = reinterpret_cast<float*>(sp + align_up(R * 4, 256));
  r.partial = reinterpret_cast<float*>(sp + 2 * align_up(R * 4, 256));
  return launch_rollout(r, static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"
