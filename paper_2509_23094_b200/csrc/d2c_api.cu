// C-ABI layer of the d2Cache step: argument validation, the carve-up of the caller's workspace and
// the launch sequence of one step.  No device memory is allocated here.
#include <math.h>
#include <stdarg.h>
#include <string.h>

#include <new>
#include <vector>

#include "common.cuh"

namespace d2c {

static thread_local char g_err[512] = "";
void set_global_error(const char* fmt, ...) {
  va_list ap; va_start(ap, fmt); vsnprintf(g_err, sizeof(g_err), fmt, ap); va_end(ap);
}
const char* global_error() { return g_err; }

int sm_count_current() {
  static int count[kMaxDevices] = {};
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (dev >= 0 && dev < kMaxDevices && count[dev] > 0) return count[dev];
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  if (dev >= 0 && dev < kMaxDevices) count[dev] = n;
  return n;
}

static thread_local long long g_launches = 0;
void count_launch(int n) { g_launches += n; }

static const char* const kPhaseNames[D2C_N_PHASES] = {
    "select", "gather_norm", "rmsnorm", "gemm_qkv", "rope_scatter", "attention", "gemm_o",
    "gemm_gate_up", "gemm_down", "lm_head", "rollout", "copy_out", "attn_abar"};
enum Phase { PH_SELECT = 0, PH_GATHER, PH_NORM, PH_QKV, PH_ROPE, PH_ATTN, PH_O, PH_GATEUP, PH_DOWN, PH_LM, PH_ROLLOUT, PH_OUT, PH_ABAR };

// Hands out 256-byte aligned pieces of a buffer; with base == null it only measures.
struct Carver {
  char* base; size_t off = 0;
  explicit Carver(void* b) : base(static_cast<char*>(b)) {}
  template <typename T> T* take(size_t count) {
    off = align_up(off, 256);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

struct Buffers {
  bf16 *kcache, *vcache; float *conf, *c, *key; int32_t *pred, *status;
  int32_t *sel_idx, *row_seq, *row_off, *lm_rows, *lm_off, *slot_of_pos, *rank_s, *rank_lm, *n_b, *nm_b;
  uint32_t* phi; float2* rope;
  bf16 *x, *xn, *qkv, *o, *hmid, *xm; float *lse, *abar, *ssq;
  float *st_max, *st_sum; int32_t* st_arg;
  float *u0, *u1, *partial;
  float* sk_partials; int32_t* sk_counters; long long* gemm_clocks;
  float* abar_part; size_t abar_part_floats;
  bf16* h0_stage; uint8_t* mask_stage; int32_t *forced_stage, *forced_off_stage; float *okey_stage, *oc_stage;
  int32_t* committed_stage;
};

static int rollout_depth(const d2c_config& c) {
  return (c.rollout_layers > 0 && c.rollout_layers < c.n_layers) ? c.rollout_layers : c.n_layers;
}
static int lm_tiles(int vocab) { return ceil_div(vocab, 128); }

static size_t carve(const d2c_config& c, void* base, Buffers* out) {
  Carver w(base);
  Buffers b;
  const size_t B = c.max_batch, L = c.max_seq, R = B * L, d = c.d_model;
  const size_t kv = (size_t)c.n_kv_heads * c.head_dim, qkv_out = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  b.kcache = w.take<bf16>((size_t)c.n_layers * R * kv);
  b.vcache = w.take<bf16>((size_t)c.n_layers * R * kv);
  b.conf = w.take<float>(R); b.c = w.take<float>(R); b.key = w.take<float>(R);
  b.pred = w.take<int32_t>(R); b.status = w.take<int32_t>(4);
  b.sel_idx = w.take<int32_t>(R); b.row_seq = w.take<int32_t>(R); b.row_off = w.take<int32_t>(B + 1);
  b.lm_rows = w.take<int32_t>(R); b.lm_off = w.take<int32_t>(B + 1); b.slot_of_pos = w.take<int32_t>(R);
  b.rank_s = w.take<int32_t>(R); b.rank_lm = w.take<int32_t>(R); b.n_b = w.take<int32_t>(B); b.nm_b = w.take<int32_t>(B);
  b.phi = w.take<uint32_t>(L); b.rope = w.take<float2>(L * (c.head_dim / 2));
  b.x = w.take<bf16>(R * d); b.xn = w.take<bf16>(R * d); b.qkv = w.take<bf16>(R * qkv_out);
  b.o = w.take<bf16>(R * (size_t)c.n_q_heads * c.head_dim); b.hmid = w.take<bf16>(R * (size_t)c.d_ffn);
  b.xm = w.take<bf16>(R * d); b.lse = w.take<float>(R * (size_t)c.n_q_heads);
  b.ssq = w.take<float>(R * (d / 32));                      // per (row, 32 columns): sum of squares of the residual stream
  b.abar = w.take<float>((size_t)rollout_depth(c) * R * L);
  const size_t nt = lm_tiles(c.vocab);
  b.st_max = w.take<float>(R * nt); b.st_sum = w.take<float>(R * nt); b.st_arg = w.take<int32_t>(R * nt);
  b.u0 = w.take<float>(R); b.u1 = w.take<float>(R);
  b.partial = w.take<float>((size_t)kRolloutSplit * R + (R + 3) / 4);     // partial sums + selected-flag bytes
  b.sk_partials = w.take<float>((size_t)kSkMaxTiles * 128 * 256); b.sk_counters = w.take<int32_t>(2 * kSkMaxTiles);     // arrival and done counters
  b.gemm_clocks = w.take<long long>(4);
  // scratch for the head-split of the abar kernel: only worth having when the (rows x keys) grid is small
  const size_t tiles_worst = (size_t)ceil_div((int)L, 128) * ceil_div((int)L, 128) * B;
  b.abar_part_floats = tiles_worst < 2 * 160 ? (size_t)8 * R * L : 0;
  b.abar_part = w.take<float>(b.abar_part_floats);
  b.h0_stage = w.take<bf16>(R * d); b.mask_stage = w.take<uint8_t>(R);
  b.forced_stage = w.take<int32_t>(R); b.forced_off_stage = w.take<int32_t>(B + 1);
  b.okey_stage = w.take<float>(R); b.oc_stage = w.take<float>(R); b.committed_stage = w.take<int32_t>(B);
  if (out) *out = b;
  return align_up(w.off, 256);
}

static const char* check_config(const d2c_config* c) {
  if (!c) return "config is null";
  if (c->n_layers < 1 || c->d_model < 64 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->d_ffn < 64 || c->vocab < 2)
    return "non-positive model dimension";
  if (c->head_dim != 64 && c->head_dim != 128) return "head_dim must be 64 or 128";
  if (c->d_model % 64 || c->d_ffn % 64 || (c->n_q_heads * c->head_dim) % 64) return "d_model, d_ffn and n_q_heads*head_dim must be multiples of 64";
  if (c->n_q_heads % c->n_kv_heads) return "n_q_heads must be a multiple of n_kv_heads";
  if (c->vocab & 1) return "vocab must be even";
  if (c->max_batch < 1 || c->max_seq < 1 || c->max_seq > 8192) return "max_batch >= 1 and 1 <= max_seq <= 8192 required";
  if (!(c->rope_base > 1.f) || !(c->rms_eps >= 0.f) || !(c->sigma > 0.f)) return "rope_base > 1, rms_eps >= 0, sigma > 0 required";
  if (c->stage2_candidates != 0 && c->stage2_candidates != 1) return "stage2_candidates must be 0 or 1";
  if (c->rollout_layers < 0 || (c->flags & ~(D2C_FLAG_PORTABLE_GEMM | D2C_FLAG_PORTABLE_ATTENTION | D2C_FLAG_ONE_SM_GEMM | D2C_FLAG_SERIAL | D2C_FLAG_FOLDED_NORMS))) return "rollout_layers >= 0 and no unknown flag bits required";
  return nullptr;
}

}  // namespace d2c

using namespace d2c;

struct d2c_ctx {
  d2c_config cfg;
  std::vector<const bf16*> wqkv, bqkv, wo, w_gate, w_up, w_down, g_attn, g_ffn;
  const bf16 *g_final, *w_lm;
  cudaStream_t stream;
  Buffers buf;
  int phi_len;
  // Selected-row count of the previous step, which chooses between the GEMM kernels (both are correct for any
  // count, but they add fp32 partial sums in different orders).  The selection kernel writes the count into one
  // of two words of mapped host memory; the next step waits for the event recorded behind that kernel before it
  // reads the word, so the choice depends on the step sequence only, never on how far the host runs ahead.
  int32_t* hint_host[2] = {nullptr, nullptr};
  int32_t* hint_dev[2] = {nullptr, nullptr};
  cudaEvent_t ev_hint[2] = {nullptr, nullptr};
  long long hint_step[2] = {-1, -1};     // step number whose count the word holds
  long long step_no = 0;
  bool few_rows = false;                 // this step's regime: at most 128 rows expected
  bool one_sm_gemm = false;              // at most 384 rows expected: the projections run on the one-SM kernel
  int used_batch = 0, used_seq = 0;      // the (batch, seq_len) of the first step: the per-position state is laid out for it
  // d2c_step_host: the device-to-host copy of the hidden rows runs on its own stream, ordered after the
  // last layer by an event, so that it overlaps the LM head and the rollout
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t layers_done = nullptr;
  void* early_hidden_host = nullptr;     // set by d2c_step_host for the duration of one step
  // The head-averaged probabilities and the rollout feed only the next step's selection.  They run on a
  // low-priority stream beside the projections, the FFN and the LM head, filling the SMs those leave idle
  // (partial last waves); the rest of the step runs on a high-priority stream so that it wins every SM it
  // can use.  Both are forked from and joined to the caller's stream by events inside d2c_step.
  cudaStream_t work_stream = nullptr, side_stream = nullptr;
  cudaEvent_t ev_in = nullptr, ev_out = nullptr, ev_fwd = nullptr, ev_abar = nullptr, ev_side = nullptr;
  cudaStream_t run = nullptr;            // where the current step's critical path is enqueued
  char err[512];
  // optional per-phase timing: one event at every phase boundary, resolved by d2c_profile_read
  bool prof = false;
  std::vector<cudaEvent_t> ev;
  std::vector<int> ev_phase;      // phase that starts at event i, -1 = end of a step
  size_t ev_used = 0;
  double phase_ms[D2C_N_PHASES] = {0};
  long long phase_launches[D2C_N_PHASES] = {0};
  long long launch_mark = 0;
  int prof_phase = -1;
};

static void destroy_overlap(d2c_ctx* ctx) {
  if (ctx->work_stream) cudaStreamDestroy(ctx->work_stream);
  if (ctx->side_stream) cudaStreamDestroy(ctx->side_stream);
  for (cudaEvent_t* ev : {&ctx->ev_in, &ctx->ev_out, &ctx->ev_fwd, &ctx->ev_abar, &ctx->ev_side}) {
    if (*ev) cudaEventDestroy(*ev);
    *ev = nullptr;
  }
  ctx->work_stream = ctx->side_stream = nullptr;
}

// Marks the start of `phase` (or the end of the step with phase < 0) on the context's stream.
static int mark(d2c_ctx* ctx, int phase) {
  if (!ctx->prof) return D2C_OK;
  if (ctx->prof_phase >= 0) ctx->phase_launches[ctx->prof_phase] += g_launches - ctx->launch_mark;
  ctx->launch_mark = g_launches; ctx->prof_phase = phase;
  if (ctx->ev_used == ctx->ev.size()) {
    cudaEvent_t e;
    D2C_CUDA_OK(cudaEventCreate(&e));
    ctx->ev.push_back(e); ctx->ev_phase.push_back(-1);
  }
  ctx->ev_phase[ctx->ev_used] = phase;
  D2C_CUDA_OK(cudaEventRecord(ctx->ev[ctx->ev_used], ctx->stream));
  ctx->ev_used++;
  return D2C_OK;
}

static int fail(d2c_ctx* ctx, int code, const char* fmt, ...) {
  char tmp[512];
  va_list ap; va_start(ap, fmt); vsnprintf(tmp, sizeof(tmp), fmt, ap); va_end(ap);
  if (ctx) { strncpy(ctx->err, tmp, sizeof(ctx->err) - 1); ctx->err[sizeof(ctx->err) - 1] = 0; }
  set_global_error("%s", tmp);
  return code;
}
// Propagates an error raised by a launcher (its text is in the thread-local slot).
static int pass(d2c_ctx* ctx, int rc) {
  if (rc != D2C_OK && ctx) { strncpy(ctx->err, global_error(), sizeof(ctx->err) - 1); ctx->err[sizeof(ctx->err) - 1] = 0; }
  return rc;
}
// The step's GEMMs: tcgen05 kernel unless the context was created with D2C_FLAG_PORTABLE_GEMM.
static int gemm(d2c_ctx* ctx, const GemmArgs& g, GemmEpilogue epi) {
  if (ctx->cfg.flags & D2C_FLAG_PORTABLE_GEMM) return launch_gemm_mma(g, epi, ctx->run);
  // The LM head runs on few rows and is bound by the weight stream: the one-SM kernel sizes its A boxes to the
  // live rows, a pair would load a second, empty row tile.
  // Up to three 128-row tiles the one-SM kernel wins: its row tiles pad 257..384 rows to 384 where a pair tile pads
  // them to 512, and below 129 rows it streams weights with K split over the SMs.  Measured on one layer at
  // L = 1024 (step, ms): 204 rows 0.418 -> 0.398, 292 rows 0.456 -> 0.423, 381 rows 0.460 -> 0.427; from 470 rows
  // on the pairs win (0.461 against 0.481; 561 rows 0.529 against 0.540).
  if (!(ctx->cfg.flags & D2C_FLAG_ONE_SM_GEMM) && epi != EPI_LMSTATS && !ctx->one_sm_gemm && gemm_tc2_supported(g))
  {
    GemmArgs g2 = g;
    g2.sk_partials = ctx->buf.sk_partials; g2.sk_counters = ctx->buf.sk_counters; g2.sk_max_tiles = kSkMaxTiles;
    return launch_gemm_tc2(g2, epi, ctx->run, ctx->buf.status);
  }
  GemmArgs gs = g;
  gs.sk_partials = ctx->buf.sk_partials; gs.sk_counters = ctx->buf.sk_counters; gs.sk_max_tiles = kSkMaxTiles;
  return launch_gemm_tc(gs, epi, ctx->run, ctx->buf.status);
}
// A CUDA runtime call inside the step: its error text goes where launcher errors go.
static int cu(cudaError_t e) {
  if (e == cudaSuccess) return D2C_OK;
  set_global_error("d2c_step: %s", cudaGetErrorString(e));
  return D2C_ECUDA;
}
#define D2C_TRY(ctx, expr) do { int rc__ = (expr); if (rc__ != D2C_OK) return pass((ctx), rc__); } while (0)

extern "C" {

size_t d2c_workspace_bytes(const d2c_config* cfg) {
  if (check_config(cfg)) return 0;
  return carve(*cfg, nullptr, nullptr);
}

int d2c_create(const d2c_config* cfg, const d2c_weights* w, void* workspace, size_t workspace_bytes,
               void* cuda_stream, d2c_ctx** out) {
  if (!out) return fail(nullptr, D2C_EINVAL, "d2c_create: out is null");
  *out = nullptr;
  if (const char* why = check_config(cfg)) return fail(nullptr, cfg ? D2C_ESHAPE : D2C_EINVAL, "d2c_create: %s", why);
  if (!w || !workspace) return fail(nullptr, D2C_EINVAL, "d2c_create: weights or workspace is null");
  if (reinterpret_cast<uintptr_t>(workspace) % 256) return fail(nullptr, D2C_EINVAL, "d2c_create: workspace must be 256-byte aligned");
  const size_t need = carve(*cfg, nullptr, nullptr);
  if (workspace_bytes < need) return fail(nullptr, D2C_ECAPACITY, "d2c_create: workspace %zu bytes < %zu needed", workspace_bytes, need);
  if (!w->wqkv || !w->wo || !w->w_gate || !w->w_up || !w->w_down || !w->g_attn || !w->g_ffn || !w->g_final || !w->w_lm ||
      (cfg->qkv_bias && !w->bqkv))
    return fail(nullptr, D2C_EINVAL, "d2c_create: a weight pointer is null");
  d2c_ctx* ctx = new (std::nothrow) d2c_ctx();
  if (!ctx) return fail(nullptr, D2C_EINVAL, "d2c_create: out of host memory");
  ctx->cfg = *cfg; ctx->err[0] = 0;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  for (int l = 0; l < cfg->n_layers; ++l) {
    const void* ptrs[] = {w->wqkv[l], w->wo[l], w->w_gate[l], w->w_up[l], w->w_down[l], w->g_attn[l], w->g_ffn[l]};
    for (const void* p : ptrs)
      if (!p || reinterpret_cast<uintptr_t>(p) % 16) { delete ctx; return fail(nullptr, D2C_EINVAL, "d2c_create: layer %d weight pointer null or not 16-byte aligned", l); }
    ctx->wqkv.push_back((const bf16*)w->wqkv[l]); ctx->wo.push_back((const bf16*)w->wo[l]);
    ctx->w_gate.push_back((const bf16*)w->w_gate[l]); ctx->w_up.push_back((const bf16*)w->w_up[l]);
    ctx->w_down.push_back((const bf16*)w->w_down[l]); ctx->g_attn.push_back((const bf16*)w->g_attn[l]);
    ctx->g_ffn.push_back((const bf16*)w->g_ffn[l]);
    ctx->bqkv.push_back(cfg->qkv_bias ? (const bf16*)w->bqkv[l] : nullptr);
    if (cfg->qkv_bias && !w->bqkv[l]) { delete ctx; return fail(nullptr, D2C_EINVAL, "d2c_create: layer %d bias is null", l); }
  }
  ctx->g_final = (const bf16*)w->g_final; ctx->w_lm = (const bf16*)w->w_lm;
  carve(*cfg, workspace, &ctx->buf);
  {
    bool ok = cudaHostAlloc(reinterpret_cast<void**>(&ctx->hint_host[0]), 2 * sizeof(int32_t), cudaHostAllocMapped) == cudaSuccess;
    if (ok) {
      ctx->hint_host[1] = ctx->hint_host[0] + 1;
      ctx->hint_host[0][0] = ctx->hint_host[0][1] = 1 << 30;
      ok = cudaHostGetDevicePointer(reinterpret_cast<void**>(&ctx->hint_dev[0]), ctx->hint_host[0], 0) == cudaSuccess;
      ctx->hint_dev[1] = ctx->hint_dev[0] + 1;
      for (int i = 0; i < 2 && ok; ++i) ok = cudaEventCreateWithFlags(&ctx->ev_hint[i], cudaEventDisableTiming) == cudaSuccess;
    }
    if (!ok) {                                               // the step then always takes the many-row kernels
      for (int i = 0; i < 2; ++i) if (ctx->ev_hint[i]) { cudaEventDestroy(ctx->ev_hint[i]); ctx->ev_hint[i] = nullptr; }
      if (ctx->hint_host[0]) cudaFreeHost(ctx->hint_host[0]);
      ctx->hint_host[0] = ctx->hint_host[1] = nullptr; (void)cudaGetLastError();
    }
  }
  if (cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&ctx->layers_done, cudaEventDisableTiming) != cudaSuccess) {
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    ctx->copy_stream = nullptr; ctx->layers_done = nullptr; (void)cudaGetLastError();
  }
  ctx->run = ctx->stream;
  if (!(cfg->flags & D2C_FLAG_SERIAL)) {
    int least = 0, greatest = 0;
    bool ok = cudaDeviceGetStreamPriorityRange(&least, &greatest) == cudaSuccess && greatest < least &&
              cudaStreamCreateWithPriority(&ctx->work_stream, cudaStreamNonBlocking, greatest) == cudaSuccess &&
              cudaStreamCreateWithPriority(&ctx->side_stream, cudaStreamNonBlocking, least) == cudaSuccess;
    for (cudaEvent_t* ev : {&ctx->ev_in, &ctx->ev_out, &ctx->ev_fwd, &ctx->ev_abar, &ctx->ev_side})
      ok = ok && cudaEventCreateWithFlags(ev, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { destroy_overlap(ctx); (void)cudaGetLastError(); }      // the step then runs on the caller's stream alone
  }
  cudaError_t e = cudaMemsetAsync(workspace, 0, need, ctx->stream);
  if (e == cudaSuccess) {
    std::vector<uint32_t> tab(cfg->max_seq);
    ctx->phi_len = build_phi_table(cfg->sigma, tab.data(), cfg->max_seq);
    e = cudaMemcpyAsync(ctx->buf.phi, tab.data(), tab.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, ctx->stream);
    if (e == cudaSuccess) {
      int rc = launch_rope_table(ctx->buf.rope, cfg->max_seq, cfg->head_dim, cfg->rope_base, ctx->stream);
      if (rc != D2C_OK) { delete ctx; return rc; }
      e = cudaStreamSynchronize(ctx->stream);      // the host table above must outlive the copy
    }
  }
  if (e != cudaSuccess) { delete ctx; return fail(nullptr, D2C_ECUDA, "d2c_create: %s", cudaGetErrorString(e)); }
  *out = ctx;
  return D2C_OK;
}

int d2c_destroy(d2c_ctx* ctx) {
  if (!ctx) return D2C_EINVAL;
  for (cudaEvent_t e : ctx->ev) cudaEventDestroy(e);
  for (int i = 0; i < 2; ++i) if (ctx->ev_hint[i]) cudaEventDestroy(ctx->ev_hint[i]);
  if (ctx->hint_host[0]) cudaFreeHost(ctx->hint_host[0]);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  if (ctx->layers_done) cudaEventDestroy(ctx->layers_done);
  destroy_overlap(ctx);
  delete ctx;
  return D2C_OK;
}

const char* d2c_last_error(const d2c_ctx* ctx) { return ctx ? ctx->err : global_error(); }

int d2c_state_ptrs(d2c_ctx* ctx, d2c_state* out) {
  if (!ctx || !out) return D2C_EINVAL;
  const Buffers& b = ctx->buf;
  out->kcache = b.kcache; out->vcache = b.vcache; out->conf = b.conf; out->pred = b.pred; out->c = b.c; out->key = b.key;
  out->sel_idx = b.sel_idx; out->row_off = b.row_off; out->lm_rows = b.lm_rows; out->lm_off = b.lm_off;
  out->abar = b.abar; out->lse = b.lse; out->status = b.status; out->gemm_clocks = reinterpret_cast<int64_t*>(b.gemm_clocks);
  return D2C_OK;
}

int d2c_sync_status(d2c_ctx* ctx) {
  if (!ctx) return D2C_EINVAL;
  cudaError_t e = cudaStreamSynchronize(ctx->stream);
  if (e != cudaSuccess) return fail(ctx, D2C_ECUDA, "d2c_sync_status: %s", cudaGetErrorString(e));
  int32_t st[4];
  e = cudaMemcpy(st, ctx->buf.status, sizeof(st), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail(ctx, D2C_ECUDA, "d2c_sync_status: %s", cudaGetErrorString(e));
  if (st[0] != 0) return fail(ctx, st[0], "device status %d raised at site %d", st[0], st[1]);
  return D2C_OK;
}

static int check_step_args(d2c_ctx* ctx, const d2c_step_args* a) {
  if (!ctx) return D2C_EINVAL;
  if (!a) return fail(ctx, D2C_EINVAL, "d2c_step: args is null");
  if (a->batch < 1 || a->seq_len < 1) return fail(ctx, D2C_EINVAL, "d2c_step: batch %d / seq_len %d must be positive", a->batch, a->seq_len);
  if (a->batch > ctx->cfg.max_batch || a->seq_len > ctx->cfg.max_seq)
    return fail(ctx, D2C_ECAPACITY, "d2c_step: batch %d x seq_len %d exceeds the context's %d x %d", a->batch, a->seq_len, ctx->cfg.max_batch, ctx->cfg.max_seq);
  if (!a->h0 || !a->mask) return fail(ctx, D2C_EINVAL, "d2c_step: h0 or mask is null");
  if (a->k < 0) return fail(ctx, D2C_EINVAL, "d2c_step: k = %d is negative", a->k);
  if (isnan(a->p)) return fail(ctx, D2C_EINVAL, "d2c_step: p is NaN");
  if ((a->forced == nullptr) != (a->forced_off == nullptr)) return fail(ctx, D2C_EINVAL, "d2c_step: forced and forced_off must be given together");
  if (ctx->used_batch == 0) { ctx->used_batch = a->batch; ctx->used_seq = a->seq_len; }
  if (a->batch != ctx->used_batch || a->seq_len != ctx->used_seq)
    return fail(ctx, D2C_EINVAL, "d2c_step: batch %d x seq_len %d differs from the %d x %d this context was first used with",
                a->batch, a->seq_len, ctx->used_batch, ctx->used_seq);
  return D2C_OK;
}

int d2c_step(d2c_ctx* ctx, const d2c_step_args* a, const d2c_step_out* out) {
  D2C_TRY(ctx, check_step_args(ctx, a));
  const d2c_config& c = ctx->cfg;
  const Buffers& b = ctx->buf;
  // critical path on `st`, probabilities + rollout on `side` (the same stream while profiling or when serial)
  const bool overlap = ctx->work_stream != nullptr && !ctx->prof;
  cudaStream_t st = overlap ? ctx->work_stream : ctx->stream;
  cudaStream_t side = overlap ? ctx->side_stream : st;
  ctx->run = st;
  if (overlap) {
    D2C_TRY(ctx, cu(cudaEventRecord(ctx->ev_in, ctx->stream)));
    D2C_TRY(ctx, cu(cudaStreamWaitEvent(st, ctx->ev_in, 0)));
  }
  // The probabilities pass of a layer goes to the side stream when its CTAs cannot hold up the projections
  // that follow: in the weight-streaming regime (few rows: short CTAs, GEMMs bound by HBM) and for a single
  // layer (it then overlaps the LM head).  Otherwise a statically scheduled GEMM whose CTAs start late behind
  // side-stream CTAs loses more than the overlap gains (measured at 488 rows x 32 layers: +5 %).
  // regime of this step: the row count of the previous step, read behind that step's selection kernel
  bool capturing = false;
  {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(ctx->stream, &cs) != cudaSuccess) { (void)cudaGetLastError(); capturing = true; }
    else capturing = cs != cudaStreamCaptureStatusNone;
  }
  const bool track = ctx->hint_host[0] != nullptr && !capturing;
  const int slot = (int)(ctx->step_no & 1), prev = slot ^ 1;
  int expect_rows = 1 << 30;
  if (track && ctx->hint_step[prev] == ctx->step_no - 1) {
    D2C_TRY(ctx, cu(cudaEventSynchronize(ctx->ev_hint[prev])));
    expect_rows = *reinterpret_cast<volatile int32_t*>(ctx->hint_host[prev]);
  }
  ctx->few_rows = expect_rows <= 128;
  ctx->one_sm_gemm = expect_rows <= 384;
  const bool few_rows = ctx->few_rows;
  const bool abar_aside = overlap && (c.n_layers == 1 || few_rows);
  bool abar_pending = false, rollout_done = false;
  // Eq. 6-9 for the next step's stage 2: enqueued right after the last probabilities pass it needs
  RolloutArgs r{};
  r.abar = b.abar; r.layer_stride = (size_t)c.max_batch * c.max_seq * c.max_seq; r.n_layers = rollout_depth(c); r.sel_idx = b.sel_idx;
  r.row_off = b.row_off; r.batch = a->batch; r.seq_len = a->seq_len; r.c = b.c; r.u0 = b.u0; r.u1 = b.u1; r.partial = b.partial; r.n_split = kRolloutSplit;
  const int B = a->batch, L = a->seq_len, R = B * L, d = c.d_model;
  const int hq = c.n_q_heads, hkv = c.n_kv_heads, dh = c.head_dim;
  const int qkv_out = (hq + 2 * hkv) * dh;
  const size_t cache_layer = (size_t)c.max_batch * c.max_seq * hkv * dh;
  bf16* x = (out && out->hidden_out) ? static_cast<bf16*>(out->hidden_out) : b.x;
  if (reinterpret_cast<uintptr_t>(x) % 16 || reinterpret_cast<uintptr_t>(a->h0) % 16)
    return fail(ctx, D2C_EINVAL, "d2c_step: h0 and hidden_out must be 16-byte aligned");

  SelectArgs s{};
  s.mask = a->mask; s.conf = b.conf; s.c = a->override_c ? a->override_c : b.c; s.override_key = a->override_key;
  s.forced = a->forced; s.forced_off = a->forced_off; s.batch = B; s.seq_len = L; s.k = a->k; s.p = a->p;
  s.stage2_candidates = c.stage2_candidates; s.block_lo = a->block_lo; s.block_hi = a->block_hi; s.phi_q30 = b.phi; s.phi_len = ctx->phi_len < L ? ctx->phi_len : L;
  s.key = b.key; s.sel_idx = b.sel_idx; s.row_seq = b.row_seq; s.row_off = b.row_off; s.lm_rows = b.lm_rows;
  s.lm_off = b.lm_off; s.slot_of_pos = b.slot_of_pos; s.rank_s = b.rank_s; s.rank_lm = b.rank_lm; s.n_b = b.n_b; s.nm_b = b.nm_b;
  s.n_host = track ? ctx->hint_dev[slot] : nullptr;
  D2C_TRY(ctx, mark(ctx, PH_SELECT));
  D2C_TRY(ctx, launch_select(s, st));
  if (track) {
    D2C_TRY(ctx, cu(cudaEventRecord(ctx->ev_hint[slot], st)));
    ctx->hint_step[slot] = ctx->step_no;
  }
  ctx->step_no++;
  const int32_t* n_rows = b.row_off + B;
  const int32_t* n_lm = b.lm_off + B;

  D2C_TRY(ctx, mark(ctx, PH_GATHER));
  D2C_TRY(ctx, launch_gather_norm((const bf16*)a->h0, b.sel_idx, b.row_seq, n_rows, R, L, d, ctx->g_attn[0], c.rms_eps, x, b.xn, st));
  const int depth = rollout_depth(c);
  // on request the RMSNorms inside the layers ride in the tcgen05 GEMMs' epilogues (all four projections must run on
  // those kernels).  Off by default: the longer epilogues and the row scaling cost the GEMMs more than the two small
  // kernels per layer take (8.7 -> 9.2 ms per step at 488 rows x 32 layers, 420 -> 434 ms at 8 x 4096).
  bool fold = (c.flags & D2C_FLAG_FOLDED_NORMS) && !(c.flags & D2C_FLAG_PORTABLE_GEMM);
  {
    const int shapes[4][2] = {{qkv_out, d}, {d, hq * dh}, {c.d_ffn, d}, {d, c.d_ffn}};       // {N, K}
    const bf16* as[4] = {b.xn, b.o, b.xn, b.hmid};
    for (int i = 0; i < 4 && fold; ++i) {
      GemmArgs t{};
      t.A = as[i]; t.lda = shapes[i][1]; t.W = ctx->wqkv[0]; t.max_rows = R; t.N = shapes[i][0]; t.K = shapes[i][1];
      fold = gemm_tc_supported(t) && (d & 7) == 0;
    }
  }
  for (int l = 0; l < c.n_layers; ++l) {
    if (out && out->layer_in) {
      cudaError_t e = cudaMemcpyAsync(static_cast<bf16*>(out->layer_in) + (size_t)l * R * d, x, (size_t)R * d * sizeof(bf16),
                                      cudaMemcpyDeviceToDevice, st);
      if (e != cudaSuccess) return fail(ctx, D2C_ECUDA, "d2c_step: %s", cudaGetErrorString(e));
    }
    // RMSNorm folded into the projections (tcgen05 GEMMs): the residual epilogue before a norm leaves x * gain in xn
    // and the row's sums of squares in ssq, the projection after it scales its accumulator rows by rsqrt(mean + eps)
    if (l > 0 && !fold) {
      D2C_TRY(ctx, mark(ctx, PH_NORM));
      D2C_TRY(ctx, launch_rmsnorm(x, nullptr, n_rows, R, d, ctx->g_attn[l], c.rms_eps, b.xn, st));
    }
    D2C_TRY(ctx, mark(ctx, PH_QKV));
    if (abar_pending) {                                  // the previous layer's probabilities still read Q and the LSE
      D2C_TRY(ctx, cu(cudaStreamWaitEvent(st, ctx->ev_abar, 0)));
      abar_pending = false;
    }
    GemmArgs g{};
    g.A = b.xn; g.lda = d; g.W = ctx->wqkv[l]; g.bias = ctx->bqkv[l]; g.C = b.qkv; g.ldc = qkv_out;
    g.n_rows = n_rows; g.max_rows = R; g.N = qkv_out; g.K = d;
    if (fold && l > 0) { g.in_ssq = b.ssq; g.in_eps = c.rms_eps; }
    bf16* kc = b.kcache + (size_t)l * cache_layer; bf16* vc = b.vcache + (size_t)l * cache_layer;
    if (!(c.flags & D2C_FLAG_PORTABLE_GEMM) && gemm_tc_supported(g)) {
      // QKV projection with bias, rotary embedding and the K/V scatter in its epilogue
      g.q_sel_idx = b.sel_idx; g.q_row_seq = b.row_seq; g.q_rope = b.rope; g.q_kc = kc; g.q_vc = vc;
      g.q_cache_seq = c.max_seq; g.q_hq = hq; g.q_hkv = hkv; g.q_dh = dh;
      D2C_TRY(ctx, gemm(ctx, g, EPI_QKV_ROPE));
    } else {
      D2C_TRY(ctx, gemm(ctx, g, EPI_STORE));
      D2C_TRY(ctx, mark(ctx, PH_ROPE));
      D2C_TRY(ctx, launch_rope_scatter(b.qkv, b.sel_idx, b.row_seq, n_rows, R, hq, hkv, dh, b.rope, kc, vc, c.max_seq, st));
    }
    AttnArgs at{};
    at.q = b.qkv; at.ldq = qkv_out; at.kc = kc; at.vc = vc; at.row_off = b.row_off; at.batch = B; at.seq_len = L;
    at.cache_seq = c.max_seq; at.hq = hq; at.hkv = hkv; at.dh = dh; at.max_rows_per_seq = L;
    at.q_rows = R; at.portable = (c.flags & D2C_FLAG_PORTABLE_ATTENTION) ? 1 : 0; at.status = b.status;
    at.abar_partial = b.abar_part_floats ? b.abar_part : nullptr; at.abar_partial_floats = b.abar_part_floats; at.n_rows = n_rows;
    at.o = b.o; at.lse = b.lse; at.abar = l < depth ? b.abar + (size_t)l * c.max_batch * c.max_seq * c.max_seq : nullptr;
    D2C_TRY(ctx, mark(ctx, PH_ATTN));
    at.which = 1;
    D2C_TRY(ctx, launch_attention(at, st));
    if (at.abar) {
      D2C_TRY(ctx, mark(ctx, PH_ABAR));
      at.which = 2;
      if (abar_aside) {
        D2C_TRY(ctx, cu(cudaEventRecord(ctx->ev_fwd, st)));
        D2C_TRY(ctx, cu(cudaStreamWaitEvent(side, ctx->ev_fwd, 0)));
      }
      D2C_TRY(ctx, launch_attention(at, abar_aside ? side : st));
      if (abar_aside) {
        D2C_TRY(ctx, cu(cudaEventRecord(ctx->ev_abar, side)));
        abar_pending = true;
      }
      if (l == depth - 1) {
        D2C_TRY(ctx, mark(ctx, PH_ROLLOUT));
        if (overlap && !abar_aside) {                    // the side stream has followed nothing of this step yet
          D2C_TRY(ctx, cu(cudaEventRecord(ctx->ev_fwd, st)));
          D2C_TRY(ctx, cu(cudaStreamWaitEvent(side, ctx->ev_fwd, 0)));
        }
        D2C_TRY(ctx, launch_rollout(r, side));
        if (overlap) D2C_TRY(ctx, cu(cudaEventRecord(ctx->ev_side, side)));
        rollout_done = true;
      }
    }
    D2C_TRY(ctx, mark(ctx, PH_O));
    GemmArgs go{};
    go.A = b.o; go.lda = hq * dh; go.W = ctx->wo[l]; go.C = x; go.ldc = d; go.n_rows = n_rows; go.max_rows = R; go.N = d; go.K = hq * dh;
    if (fold) { go.nx_out = b.xn; go.nx_gain = ctx->g_ffn[l]; go.nx_ssq = b.ssq; }
    D2C_TRY(ctx, gemm(ctx, go, EPI_RESIDUAL));
    if (!fold) {
      D2C_TRY(ctx, mark(ctx, PH_NORM));
      D2C_TRY(ctx, launch_rmsnorm(x, nullptr, n_rows, R, d, ctx->g_ffn[l], c.rms_eps, b.xn, st));
    }
    D2C_TRY(ctx, mark(ctx, PH_GATEUP));
    GemmArgs gf{};
    gf.A = b.xn; gf.lda = d; gf.W = ctx->w_gate[l]; gf.W2 = ctx->w_up[l]; gf.C = b.hmid; gf.ldc = c.d_ffn;
    gf.n_rows = n_rows; gf.max_rows = R; gf.N = c.d_ffn; gf.K = d;
    gf.clock_probe = ctx->prof ? b.gemm_clocks : nullptr;
    if (fold) { gf.in_ssq = b.ssq; gf.in_eps = c.rms_eps; }
    D2C_TRY(ctx, gemm(ctx, gf, EPI_SWIGLU));
    GemmArgs gd{};
    gd.A = b.hmid; gd.lda = c.d_ffn; gd.W = ctx->w_down[l]; gd.C = x; gd.ldc = d; gd.n_rows = n_rows; gd.max_rows = R; gd.N = d; gd.K = c.d_ffn;
    if (fold && l + 1 < c.n_layers) { gd.nx_out = b.xn; gd.nx_gain = ctx->g_attn[l + 1]; gd.nx_ssq = b.ssq; }
    D2C_TRY(ctx, mark(ctx, PH_DOWN));
    D2C_TRY(ctx, gemm(ctx, gd, EPI_RESIDUAL));
  }
  if (ctx->early_hidden_host && ctx->copy_stream) {
    // the residual stream is final here: ship it to the host while the LM head and the rollout run
    // (the row count is not known on the host yet, so the worst case is copied)
    cudaError_t e = cudaEventRecord(ctx->layers_done, st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->copy_stream, ctx->layers_done, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->early_hidden_host, x, (size_t)R * d * sizeof(bf16), cudaMemcpyDeviceToHost, ctx->copy_stream);
    if (e != cudaSuccess) return fail(ctx, D2C_ECUDA, "d2c_step: %s", cudaGetErrorString(e));
  }
  // Eq. 1 on the selected rows that are still masked
  D2C_TRY(ctx, mark(ctx, PH_LM));
  D2C_TRY(ctx, launch_rmsnorm(x, b.lm_rows, n_lm, R, d, ctx->g_final, c.rms_eps, b.xm, st));
  GemmArgs gl{};
  gl.A = b.xm; gl.lda = d; gl.W = ctx->w_lm; gl.n_rows = n_lm; gl.max_rows = R; gl.N = c.vocab; gl.K = d;
  gl.st_max = b.st_max; gl.st_sum = b.st_sum; gl.st_arg = b.st_arg; gl.n_tiles = lm_tiles(c.vocab);
  gl.logits = out ? out->logits : nullptr;
  D2C_TRY(ctx, gemm(ctx, gl, EPI_LMSTATS));
  D2C_TRY(ctx, launch_lm_reduce(b.st_max, b.st_sum, b.st_arg, gl.n_tiles, n_lm, R, b.lm_rows, b.sel_idx, b.row_seq, L, b.conf, b.pred, st));
  if (!rollout_done) return fail(ctx, D2C_EINVAL, "d2c_step: no layer produced attention probabilities");
  if (overlap) D2C_TRY(ctx, cu(cudaStreamWaitEvent(st, ctx->ev_side, 0)));

  D2C_TRY(ctx, mark(ctx, PH_OUT));
  if (out && out->sel_idx) {
    cudaError_t e = cudaMemcpyAsync(out->sel_idx, b.sel_idx, (size_t)R * sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
    if (e != cudaSuccess) return fail(ctx, D2C_ECUDA, "d2c_step: %s", cudaGetErrorString(e));
  }
  if (out && out->row_off) {
    cudaError_t e = cudaMemcpyAsync(out->row_off, b.row_off, (size_t)(B + 1) * sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
    if (e != cudaSuccess) return fail(ctx, D2C_ECUDA, "d2c_step: %s", cudaGetErrorString(e));
  }
  D2C_TRY(ctx, mark(ctx, -1));
  if (overlap) {
    D2C_TRY(ctx, cu(cudaEventRecord(ctx->ev_out, st)));
    D2C_TRY(ctx, cu(cudaStreamWaitEvent(ctx->stream, ctx->ev_out, 0)));
  }
  ctx->run = ctx->stream;
  return D2C_OK;
}

int d2c_profile(d2c_ctx* ctx, int32_t enable) {
  if (!ctx) return D2C_EINVAL;
  ctx->prof = enable != 0;
  ctx->prof_phase = -1;
  return D2C_OK;
}

int d2c_profile_read(d2c_ctx* ctx, float* phase_ms, int64_t* phase_launches, int32_t reset) {
  if (!ctx) return D2C_EINVAL;
  cudaError_t e = cudaStreamSynchronize(ctx->stream);
  if (e != cudaSuccess) return fail(ctx, D2C_ECUDA, "d2c_profile_read: %s", cudaGetErrorString(e));
  for (size_t i = 0; i + 1 < ctx->ev_used; ++i) {
    if (ctx->ev_phase[i] < 0) continue;
    float ms = 0.f;
    e = cudaEventElapsedTime(&ms, ctx->ev[i], ctx->ev[i + 1]);
    if (e != cudaSuccess) return fail(ctx, D2C_ECUDA, "d2c_profile_read: %s", cudaGetErrorString(e));
    ctx->phase_ms[ctx->ev_phase[i]] += ms;
  }
  ctx->ev_used = 0;
  for (int i = 0; i < D2C_N_PHASES; ++i) {
    if (phase_ms) phase_ms[i] = (float)ctx->phase_ms[i];
    if (phase_launches) phase_launches[i] = ctx->phase_launches[i];
    if (reset) { ctx->phase_ms[i] = 0; ctx->phase_launches[i] = 0; }
  }
  return D2C_OK;
}

const char* d2c_phase_name(int32_t i) { return (i >= 0 && i < D2C_N_PHASES) ? kPhaseNames[i] : ""; }

int d2c_step_host(d2c_ctx* ctx, const d2c_step_args* h, const d2c_host_out* out) {
  D2C_TRY(ctx, check_step_args(ctx, h));
  const d2c_config& c = ctx->cfg;
  const Buffers& b = ctx->buf;
  cudaStream_t st = ctx->stream;
  const size_t B = h->batch, L = h->seq_len, R = B * L;
#define D2C_CP(dst, src, bytes, kind)                                                         \
  do { cudaError_t e__ = cudaMemcpyAsync((dst), (src), (bytes), (kind), st);                  \
       if (e__ != cudaSuccess) return fail(ctx, D2C_ECUDA, "d2c_step_host: %s", cudaGetErrorString(e__)); } while (0)
  d2c_step_args a = *h;
  D2C_CP(b.h0_stage, h->h0, R * c.d_model * sizeof(bf16), cudaMemcpyHostToDevice); a.h0 = b.h0_stage;
  D2C_CP(b.mask_stage, h->mask, R, cudaMemcpyHostToDevice); a.mask = b.mask_stage;
  if (h->forced) {
    int32_t n_forced = h->forced_off[B];
    if (n_forced < 0 || (size_t)n_forced > R) return fail(ctx, D2C_EINVAL, "d2c_step_host: %d forced rows", n_forced);
    D2C_CP(b.forced_off_stage, h->forced_off, (B + 1) * sizeof(int32_t), cudaMemcpyHostToDevice);
    if (n_forced) D2C_CP(b.forced_stage, h->forced, (size_t)n_forced * sizeof(int32_t), cudaMemcpyHostToDevice);
    a.forced = b.forced_stage; a.forced_off = b.forced_off_stage;
  }
  if (h->override_key) { D2C_CP(b.okey_stage, h->override_key, R * sizeof(float), cudaMemcpyHostToDevice); a.override_key = b.okey_stage; }
  if (h->override_c) { D2C_CP(b.oc_stage, h->override_c, R * sizeof(float), cudaMemcpyHostToDevice); a.override_c = b.oc_stage; }
  d2c_step_out dev_out{};
  const bool early = out && out->hidden_out_host && ctx->copy_stream;
  ctx->early_hidden_host = early ? out->hidden_out_host : nullptr;
  const int step_rc = d2c_step(ctx, &a, &dev_out);
  ctx->early_hidden_host = nullptr;
  if (step_rc != D2C_OK) { if (early) cudaStreamSynchronize(ctx->copy_stream); return step_rc; }
  // every result is copied without knowing the row count (worst-case sizes), then one synchronisation
  if (out) {
    if (out->row_off_host) D2C_CP(out->row_off_host, b.row_off, (B + 1) * sizeof(int32_t), cudaMemcpyDeviceToHost);
    if (out->sel_idx_host) D2C_CP(out->sel_idx_host, b.sel_idx, R * sizeof(int32_t), cudaMemcpyDeviceToHost);
    if (out->hidden_out_host && !early) D2C_CP(out->hidden_out_host, b.x, R * c.d_model * sizeof(bf16), cudaMemcpyDeviceToHost);
    if (out->conf_host) D2C_CP(out->conf_host, b.conf, R * sizeof(float), cudaMemcpyDeviceToHost);
    if (out->pred_host) D2C_CP(out->pred_host, b.pred, R * sizeof(int32_t), cudaMemcpyDeviceToHost);
  }
  cudaError_t e = cudaStreamSynchronize(st);
  if (e == cudaSuccess && early) e = cudaStreamSynchronize(ctx->copy_stream);
  if (e != cudaSuccess) return fail(ctx, D2C_ECUDA, "d2c_step_host: %s", cudaGetErrorString(e));
#undef D2C_CP
  return D2C_OK;
}

int d2c_commit(d2c_ctx* ctx, int32_t batch, int32_t seq_len, const void* embed_table, void* h0,
               uint8_t* mask, int32_t* tokens, int32_t* committed, int32_t rule, float threshold) {
  if (!ctx) return D2C_EINVAL;
  if (!embed_table || !h0 || !mask || !tokens || !committed) return fail(ctx, D2C_EINVAL, "d2c_commit: null pointer");
  if (batch < 1 || batch > ctx->cfg.max_batch || seq_len < 1 || seq_len > ctx->cfg.max_seq)
    return fail(ctx, D2C_ECAPACITY, "d2c_commit: batch %d x seq_len %d out of range", batch, seq_len);
  if (rule < 0 || rule > 2 || isnan(threshold)) return fail(ctx, D2C_EINVAL, "d2c_commit: rule %d / threshold", rule);
  if (ctx->used_batch != 0 && (batch != ctx->used_batch || seq_len != ctx->used_seq))
    return fail(ctx, D2C_EINVAL, "d2c_commit: batch %d x seq_len %d differs from the %d x %d of this context's steps", batch, seq_len, ctx->used_batch, ctx->used_seq);
  const Buffers& b = ctx->buf;
  D2C_TRY(ctx, launch_commit(batch, seq_len, ctx->cfg.d_model, rule, threshold, b.slot_of_pos, b.conf, b.pred, b.phi,
                             ctx->phi_len < seq_len ? ctx->phi_len : seq_len, (const bf16*)embed_table, (bf16*)h0, mask,
                             tokens, committed, ctx->stream));
  return D2C_OK;
}

}  // extern "C"
