/*
 * d2c.h - C ABI of the d2Cache decode step for NVIDIA B200 (sm_100a).
 *
 * d2Cache ("Dual aDaptive Cache", arXiv 2509.23094) accelerates a bidirectional
 * diffusion LLM by recomputing, at every decoding step, only a selected subset
 * of rows and reusing the cached K/V of all others (Section 4).  One call of
 * d2c_step performs one such step:
 *
 *   1. stage-1 selection: certainty density D(i) (Eq. 3), key D(i)*s^i, top-k
 *      over the still-masked positions (Eq. 4);
 *   2. stage-2 selection: top-p over the remaining candidates by the attention
 *      rollout influence score c_j of the previous pass (Section 4.2, after Eq. 9);
 *   3. the transformer layers on the selected rows only (Eq. 5): gather, RMSNorm,
 *      QKV projection, rotary embedding, K/V written into the persistent
 *      per-layer cache, attention of the selected queries over ALL cached keys
 *      (the attention tensor of Section 4.2 has shape H x |y*| x L), output
 *      projection, SwiGLU feed-forward;
 *   4. LM head, arg-max token and its softmax probability (Eq. 1) for the
 *      selected rows that are still masked;
 *   5. attention rollout of this step's head-averaged attention (Eq. 6-9),
 *      giving c_j for the next step.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its name ends in _host or the
 *     comment says "host".  The library allocates no device memory: weights, the
 *     workspace and all outputs belong to the caller.
 *   - bf16 matrices are row-major [out_features][in_features].
 *   - All work is ordered on the stream given to d2c_create; calls return
 *     without synchronising unless stated.  d2c_step may run part of a step on
 *     two streams of its own (created by d2c_create, forked from and joined to
 *     the caller's stream by events inside the call), so work enqueued on the
 *     caller's stream after the call still sees the whole step; D2C_FLAG_SERIAL
 *     keeps every kernel on the caller's stream.  Either way a step can be captured
 *     into a CUDA graph from the caller's stream and replayed (the choice between
 *     kernel variants that follows an earlier step's row count is then frozen).
 *     One context per stream; a context is not re-entrant.
 *   - Return value: D2C_OK or a negative D2C_E* code; d2c_last_error() gives the
 *     text.  Nothing throws, aborts or traps.  Faults detected on the device
 *     (a bounded wait that ran out) are written to a status word that
 *     d2c_sync_status() reads.
 */
#ifndef D2C_H_
#define D2C_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define D2C_OK          0
#define D2C_EINVAL     (-1)  /* null pointer, NaN, negative count, ...            */
#define D2C_ESHAPE     (-2)  /* model dimensions the kernels do not support       */
#define D2C_ECAPACITY  (-3)  /* batch/seq_len beyond max_*, workspace too small   */
#define D2C_ECUDA      (-4)  /* a CUDA runtime call failed                        */
#define D2C_ETIMEOUT   (-5)  /* a bounded device-side wait gave up                */

typedef struct d2c_ctx d2c_ctx;

/* Model and policy, fixed at create.  Supported: head_dim 64 or 128;
 * d_model, n_q_heads*head_dim and d_ffn multiples of 64; n_q_heads a multiple
 * of n_kv_heads; max_seq <= 8192. */
typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
  int32_t max_batch, max_seq;
  float   rope_base;          /* rotary base; pairs (t, t + head_dim/2) rotate by pos * base^(-2t/head_dim) */
  float   rms_eps;
  float   sigma;              /* std-dev of the Gaussian in Eq. 3 (paper default 10)                      */
  int32_t qkv_bias;           /* 1: add bqkv after the QKV projection (Dream/Qwen2.5 shape)               */
  int32_t stage2_candidates;  /* 0: top-p runs over known (prompt/decoded) positions;
                                 1: over every position stage 1 did not take                             */
  int32_t rollout_layers;     /* 0: rollout over all layers (Eq. 8); n>0: only the first n layers        */
  int32_t flags;              /* D2C_FLAG_* bits                                                         */
} d2c_config;
#define D2C_FLAG_PORTABLE_GEMM 1        /* run the GEMMs on the mma.sync kernel instead of the tcgen05 one (cross-check) */
#define D2C_FLAG_PORTABLE_ATTENTION 2   /* same for the attention kernels                                                */
#define D2C_FLAG_ONE_SM_GEMM 4          /* keep the GEMMs on the one-SM tcgen05 kernel (no CTA pairs)                    */
#define D2C_FLAG_SERIAL 8               /* enqueue every kernel of a step on the caller's stream, one after the other    */
#define D2C_FLAG_FOLDED_NORMS 16        /* fold the layers' RMSNorms into the GEMM epilogues around them (x * gain and the row's sums of
                                           squares written by the residual epilogue, the row scale applied by the next projection)
                                           instead of running them as kernels of their own; measured slower at every workload          */

/* Weights.  The arrays of per-layer pointers are HOST arrays of n_layers DEVICE
 * pointers; they are copied at create, the device memory is borrowed for the
 * lifetime of the context. */
typedef struct {
  const void* const* wqkv;    /* [ (Hq+2*Hkv)*Dh ][ d ]  rows: all Q heads, then K heads, then V heads */
  const void* const* bqkv;    /* [ (Hq+2*Hkv)*Dh ] or NULL when qkv_bias == 0                          */
  const void* const* wo;      /* [ d ][ Hq*Dh ]                                                         */
  const void* const* w_gate;  /* [ F ][ d ]                                                             */
  const void* const* w_up;    /* [ F ][ d ]                                                             */
  const void* const* w_down;  /* [ d ][ F ]                                                             */
  const void* const* g_attn;  /* [ d ] RMSNorm gain before attention                                    */
  const void* const* g_ffn;   /* [ d ] RMSNorm gain before the feed-forward                             */
  const void* g_final;        /* [ d ] device pointer                                                   */
  const void* w_lm;           /* [ V ][ d ] device pointer                                              */
} d2c_weights;

/* Bytes of device workspace a context of this configuration needs (KV cache,
 * per-position state, attention store for the rollout, activations).  0 if the
 * configuration is not supported. */
size_t d2c_workspace_bytes(const d2c_config* cfg);

/* Builds a context over caller-owned memory.  `workspace` must be 256-byte
 * aligned device memory of at least d2c_workspace_bytes(cfg); it is zeroed
 * (cache, confidences and scores start at 0).  `cuda_stream` is a cudaStream_t
 * (NULL = default stream).  Synchronises the stream once. */
int d2c_create(const d2c_config* cfg, const d2c_weights* w, void* workspace, size_t workspace_bytes,
               void* cuda_stream, d2c_ctx** out);

typedef struct {
  int32_t batch, seq_len;          /* <= max_batch, <= max_seq                                            */
  const void*    h0;               /* bf16 [batch][seq_len][d]: input hidden states (embeddings of y_t)   */
  const uint8_t* mask;             /* [batch][seq_len], 1 = still [MASK] (the set M of Eq. 3-4)           */
  const int32_t* forced;           /* optional: extra positions to recompute (e.g. the token committed    */
  const int32_t* forced_off;       /*   after the last step); forced[forced_off[b] .. forced_off[b+1])    */
  int32_t k;                       /* Eq. 4's k (>= 0)                                                    */
  float   p;                       /* top-p threshold; <= 0 selects nothing, >= 1 every candidate         */
  const float* override_key;       /* optional [batch][seq_len]: use as stage-1 keys instead of D(i)*s^i  */
  const float* override_c;         /* optional [batch][seq_len]: use as stage-2 scores instead of state c */
  int32_t block_lo, block_hi;      /* semi-autoregressive decoding (blocks decoded left to right, Section 5.1):
                                      stage 1 only considers masked positions in [block_lo, block_hi);
                                      block_hi <= block_lo means the whole sequence                        */
} d2c_step_args;

typedef struct {
  int32_t* sel_idx;     /* optional [max_batch*max_seq]: selected positions, ascending per sequence       */
  int32_t* row_off;     /* optional [batch+1]: rows of sequence b are [row_off[b], row_off[b+1])          */
  void*    hidden_out;  /* optional bf16 [max_batch*max_seq][d]: residual stream of the selected rows
                           after the last layer (rows beyond row_off[batch] are not written)             */
  float*   logits;      /* optional f32 [rows with a masked position][V] in row order (debug, slow path)  */
  void*    layer_in;    /* optional bf16 [n_layers][batch*seq_len][d]: the residual stream of the selected
                           rows as it enters each layer (debug: lets a checker verify one layer at a time) */
} d2c_step_out;

/* One decoding step (see the top of this file).  Device pointers; enqueues only.
 * k >= #masked and p >= 1 recompute every row (the ordinary full forward, also
 * the way the cache is first filled); k == 0, p <= 0 and no forced rows change
 * nothing. */
int d2c_step(d2c_ctx* ctx, const d2c_step_args* args, const d2c_step_out* out);

/* The same step for callers whose data lives in HOST memory: h0, mask, forced,
 * forced_off and the override vectors are host pointers (pinned memory makes
 * the copies asynchronous); the outputs are host buffers: sel_idx_host
 * [batch*seq_len], row_off_host [batch+1], hidden_out_host bf16 [batch*seq_len][d] (the copy starts before the row
 * count is known, so the whole buffer may be written; rows beyond row_off_host[batch] are meaningless),
 * conf_host / pred_host [batch][seq_len] (any may be NULL).  Copies in, runs
 * d2c_step, copies out, and synchronises the stream before returning. */
typedef struct {
  int32_t* sel_idx_host; int32_t* row_off_host; void* hidden_out_host;
  float* conf_host; int32_t* pred_host;
} d2c_host_out;
int d2c_step_host(d2c_ctx* ctx, const d2c_step_args* host_args, const d2c_host_out* out);

/* Decoding-loop helper (Eq. 2): per sequence, among the masked positions whose
 * prediction was refreshed by the last step, commit the one with the highest
 * score - rule 0: confidence s^i; rule 1: certainty prior D(i)*s^i (Section 4.1).
 * Writes the predicted token into tokens[b][pos], clears mask[b][pos], copies
 * embed_table[token] into h0[b][pos] and records pos in committed[b] (-1 if the
 * sequence has nothing left).  rule 2 commits every such position whose
 * confidence exceeds `threshold` (parallel decoding), at least one per sequence;
 * committed then receives only the best one. */
int d2c_commit(d2c_ctx* ctx, int32_t batch, int32_t seq_len, const void* embed_table, void* h0,
               uint8_t* mask, int32_t* tokens, int32_t* committed, int32_t rule, float threshold);

/* Device pointers into the workspace (valid for the context's lifetime). */
typedef struct {
  void*    kcache;      /* bf16 [n_layers][max_batch][max_seq][Hkv][Dh], keys after rotary embedding */
  void*    vcache;      /* bf16, same layout                                                          */
  float*   conf;        /* [max_batch][max_seq] last confidence each position received (Eq. 1)       */
  int32_t* pred;        /* [max_batch][max_seq] last predicted token                                  */
  float*   c;           /* [max_batch][max_seq] rollout influence score (Eq. 9) of the last pass     */
  float*   key;         /* [max_batch][max_seq] stage-1 keys of the last step (0 for unmasked)       */
  int32_t* sel_idx;     /* [max_batch*max_seq]  selected positions of the last step                  */
  int32_t* row_off;     /* [max_batch+1]                                                              */
  int32_t* lm_rows;     /* [max_batch*max_seq]  row numbers that went through the LM head            */
  int32_t* lm_off;      /* [max_batch+1]                                                              */
  float*   abar;        /* f32 [n_layers][max_batch*max_seq][max_seq] head-averaged attention rows   */
  float*   lse;         /* f32 [max_batch*max_seq][Hq] log-sum-exp of the last layer's scores        */
  int32_t* status;      /* [4] device status word: [0] error code, [1] where                         */
  int64_t* gemm_clocks; /* [4] while d2c_profile is on: SM clock counter and global timer (ns) at the start
                           and at the end of CTA 0 of the last gate/up projection launch, i.e. the SM
                           clock that launch really ran at: ([2]-[0]) / ([3]-[1]) GHz                 */
} d2c_state;
/* The per-position vectors (conf, pred, c, key) are indexed [b*seq_len + pos] with the batch and
 * seq_len of the d2c_step calls; a context is used with one (batch, seq_len) from its first step on
 * (d2c_step and d2c_commit return D2C_EINVAL for any other pair).
 * abar: row r of layer l is at abar + l*max_batch*max_seq*max_seq + r*seq_len. */
int d2c_state_ptrs(d2c_ctx* ctx, d2c_state* out);

/* Synchronises the stream and returns the device status word's error code (D2C_OK, or what a kernel's
 * bounded wait recorded: D2C_ETIMEOUT with the wait's site number in the error text).  The word is sticky:
 * it keeps the first error until the caller writes zeros to status[0..3]. */
int d2c_sync_status(d2c_ctx* ctx);

/* Per-phase timing of d2c_step.  While enabled, d2c_step records one CUDA event at every phase
 * boundary on the context's stream (events are host objects; no device memory is allocated).
 * d2c_profile_read synchronises the stream and returns, accumulated since the last reset, the
 * milliseconds spent in each phase (phase_ms[D2C_N_PHASES]) and the number of kernels the library
 * launched in it (phase_launches[D2C_N_PHASES]); either may be NULL.  d2c_phase_name(i) names
 * phase i ("select", "gemm_qkv", ...). */
#define D2C_N_PHASES 13
int d2c_profile(d2c_ctx* ctx, int32_t enable);
int d2c_profile_read(d2c_ctx* ctx, float* phase_ms, int64_t* phase_launches, int32_t reset);
const char* d2c_phase_name(int32_t i);

/* Text of the last error on this context (host string, never NULL); with ctx == NULL the
 * last error of a failed d2c_create / stand-alone op on this thread. */
const char* d2c_last_error(const d2c_ctx* ctx);

int d2c_destroy(d2c_ctx* ctx);

/* ---------------------------------------------------------------------------
 * Stand-alone kernels of the step, exported so that each can be checked and
 * timed on its own.  Device pointers, enqueue on `cuda_stream`, no allocation:
 * scratch is passed in.
 * ------------------------------------------------------------------------- */

/* Bytes of scratch d2c_op_select needs. */
size_t d2c_op_select_scratch_bytes(int32_t batch, int32_t seq_len);

/* Both selection stages, the union and the compaction (Eq. 3-5), for `batch`
 * independent sequences.  conf: stored confidences, c: stored influence scores,
 * override_key / forced / forced_off optional (NULL).  Outputs: key [batch][seq_len];
 * sel_idx [batch*seq_len]; row_off [batch+1]; lm_rows [batch*seq_len] and lm_off
 * [batch+1]: global row numbers of the selected rows that are masked;
 * slot_of_pos [batch][seq_len]: row number of a selected position, else -1.
 * Unlike the other stand-alone kernels this call synchronises `cuda_stream` once before it enqueues its
 * kernels: it builds the phi table of Eq. 3 in host memory and copies it into the scratch first. */
int d2c_op_select(const uint8_t* mask, const float* conf, const float* c, const float* override_key,
                  const int32_t* forced, const int32_t* forced_off, int32_t batch, int32_t seq_len,
                  int32_t k, float p, float sigma, int32_t stage2_candidates,
                  float* key, int32_t* sel_idx, int32_t* row_off, int32_t* lm_rows, int32_t* lm_off,
                  int32_t* slot_of_pos, void* scratch, size_t scratch_bytes, void* cuda_stream);

/* C[m][n] = sum_k A[m][k] * W[n][k] (+ bias[n]) in bf16 with fp32 accumulation,
 * for the first *n_rows rows (n_rows is a DEVICE int32, <= max_rows).  A: [max_rows][K],
 * W: [N][K], C: [max_rows][N].  K a multiple of 64.  impl 0: tcgen05/TMEM kernels (CTA pairs where
 * the shape allows, else one SM per tile), impl 1: the portable mma.sync kernel, impl 2: the one-SM
 * tcgen05 kernel. */
int d2c_op_gemm(const void* A, const void* W, const void* bias, void* C, const int32_t* n_rows,
                int32_t max_rows, int32_t N, int32_t K, int32_t impl, void* cuda_stream);

/* Selected-query bidirectional attention of one layer (Section 4.2).
 * q: bf16 [q_rows][ldq] with head h at columns [h*Dh,(h+1)*Dh) (already rotated); q_rows >= row_off[batch];
 * kcache/vcache: bf16 [batch][cache_seq][Hkv][Dh] of this layer; rows of sequence b are
 * [row_off[b], row_off[b+1]) and attend to keys 0..seq_len-1 of that sequence.
 * Outputs: o bf16 [rows][Hq*Dh]; lse f32 [rows][Hq] (natural log); abar f32
 * [rows][seq_len] = mean over the Hq heads of the softmax probabilities (may be NULL).
 * impl 0: tcgen05 kernels where the shape allows (head_dim 128, q_rows >= 128), impl 1: mma.sync kernels. */
int d2c_op_attention(const void* q, int32_t q_rows, int32_t ldq, const void* kcache, const void* vcache,
                     const int32_t* row_off, int32_t batch, int32_t seq_len, int32_t cache_seq,
                     int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                     void* o, float* lse, float* abar, int32_t impl, void* cuda_stream);

/* Bytes of scratch d2c_op_lm_head needs for up to max_rows rows. */
size_t d2c_op_lm_head_scratch_bytes(int32_t max_rows, int32_t vocab);

/* Eq. 1 for the first *n_rows rows of x (bf16 [max_rows][d], already normalised):
 * logits = x * w_lm^T, conf[r] = max softmax probability, pred[r] = its token
 * (lowest id among equal logits).  logits (f32 [max_rows][V]) is optional. */
int d2c_op_lm_head(const void* x, const void* w_lm, const int32_t* n_rows, int32_t max_rows,
                   int32_t d, int32_t vocab, float* conf, int32_t* pred, float* logits,
                   void* scratch, size_t scratch_bytes, void* cuda_stream);

/* Bytes of scratch d2c_op_rollout needs. */
size_t d2c_op_rollout_scratch_bytes(int32_t batch, int32_t seq_len);

/* Eq. 6-9 as a vector chain: c = 1^T W^(N) ... W^(1).  abar: f32 [n_layers][layer_stride]
 * with layer l's rows at abar + l*layer_stride, row r at + r*seq_len; sel_idx / row_off as
 * produced by d2c_op_select.  Writes c [batch][seq_len] for sequences with at least one
 * selected row and leaves c of the others untouched. */
int d2c_op_rollout(const float* abar, size_t layer_stride, int32_t n_layers, const int32_t* sel_idx,
                   const int32_t* row_off, int32_t batch, int32_t seq_len, float* c,
                   void* scratch, size_t scratch_bytes, void* cuda_stream);

/* The library's bounded device-side wait, on its own.  Every pipeline wait of the tcgen05 kernels (on an
 * mbarrier that a TMA copy or a tensor-core commit completes) gives up after a cycle limit, records
 * D2C_ETIMEOUT in status[0] and the number of the wait that ran out in status[1], and lets the kernel drain
 * and return; d2c_sync_status then reports it.  This entry launches one small CTA that waits, with the given
 * limit (1e3 .. 2e9 SM clocks), on a barrier nothing arrives on: it returns after about that many clocks and
 * leaves status = {D2C_ETIMEOUT, 99, ...}.  status: device int32[4], zeroed by the caller.  It exists so that
 * the error path of section "Conventions" can be exercised without a fault; it has no counterpart in the paper. */
int d2c_op_wait_probe(int32_t* status, int64_t limit_cycles, void* cuda_stream);

/* d2c_op_rollout without a scratch argument.  (The paper has no counterpart for this entry point; it
 * exists for integration reasons only.)  It serves callers that cannot get device memory at the time
 * of the call, e.g. an inference server whose start-up handed every free byte of HBM to its cache
 * arena, or code on a latency-critical stream that may not go through cudaMalloc and its implicit
 * device synchronisation.  The scratch is a fixed array inside the library image (about 1.2 MB on every
 * GPU that loads the library, until the process exits), which limits the call to
 * batch * seq_len <= 16384; larger problems get D2C_ECAPACITY and should use d2c_op_rollout.
 * Arguments, outputs and results are those of d2c_op_rollout.  Calls no cudaMalloc / cudaFree and no
 * allocating library routine.  The first call on each device looks up the array's device address
 * (with that device current); make that first call outside any stream capture.  All calls on a device
 * share the one array: two calls whose kernels may overlap on the GPU (different streams, no ordering
 * between them) race on it, so order them.  Nothing in the array has to be cleared between calls:
 * every word that is read has been written earlier in the same call. */
int d2c_op_rollout_static(const float* abar, size_t layer_stride, int32_t n_layers, const int32_t* sel_idx,
                          const int32_t* row_off, int32_t batch, int32_t seq_len, float* c, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* D2C_H_ */
