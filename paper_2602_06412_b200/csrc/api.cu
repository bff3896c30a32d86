// C ABI of the SureLock step: context, per-step launch sequence, accessors (see include/surelock.h).
// The step is a fixed sequence of kernel launches on one stream; the number of active rows M lives in device
// memory and every kernel reads it there, so nothing in surelock_step waits for the GPU.
#include <math.h>
#include <string.h>

#include <new>
#include <vector>

#include "tc_common.cuh"

using namespace sl;

struct surelock_ctx {
  surelock_model_cfg cfg;
  int N = 0, B = 0, R = 0;            // R = B*N = capacity in packed rows
  size_t esz = 2;
  cudaStream_t st = nullptr;
  const void *tok_emb = nullptr, *lm_head = nullptr, *final_norm_g = nullptr;
  std::vector<const void*> attn_norm_g, wq, wk, wv, wo, ffn_norm_g, w_gate, w_up, w_down;
  std::vector<void*> allocs;
  char* kv = nullptr;                 // [L][2][R][H*dh]
  float* x = nullptr;                 // residual stream, fp32 [R][d]
  void *h = nullptr, *q = nullptr, *k = nullptr, *v = nullptr, *attn = nullptr, *act = nullptr;
  void* logits[2] = {nullptr, nullptr};
  float* lse[2] = {nullptr, nullptr};
  int32_t* row_of_pos[2] = {nullptr, nullptr};
  int32_t *idx = nullptr, *row_offsets = nullptr, *n_active = nullptr, *status = nullptr, *argmax = nullptr;
  float *kl = nullptr, *conf = nullptr;
  void* scratch = nullptr;
  float2* rope = nullptr;
  int32_t* st_tokens = nullptr;       // device staging for surelock_step_host
  uint8_t *st_mask = nullptr, *st_lock = nullptr;
  int cur = 0;
  bool have_prev = false;
  int launches = 0;
  int gemm_impl = 0;                  // 0 = tensor cores when possible, 1 = CUDA cores
  bool strict_tc = false;             // refuse (SL_EUNSUPPORTED) instead of falling back to the CUDA-core kernels
  int fallbacks = 0;                  // launches that fell back since the last reset
  int32_t* n_prev = nullptr;          // rows of the previous step's logits (copy of n_active taken at the end of a step)
  // Upper bound of M for choosing launch configurations on the host (M itself stays in device memory).  Every step
  // copies its row count into a page-locked word and records an event; a step first waits for the event of the step
  // BEFORE THE PREVIOUS ONE (normally long complete: the host may run two steps ahead, not more) and takes that count
  // as the bound: lock masks normally only grow, so the count two steps ago bounds this step's.  Always the same
  // step's count, whatever the timing, so that the choice of kernels, and with it every bit of the results, is
  // reproducible.  A bound that turns out too small only costs time (the kernels stay correct for any M).
  int32_t* h_m = nullptr;             // page-locked [2]
  cudaEvent_t ev_m[2] = {nullptr, nullptr};
  bool ev_m_valid[2] = {false, false};
  long long calls = 0;                // steps / layer steps since the last reset
  int row_bound_opt = 0;              // "row_bound" option: > 0 = the caller's bound, used instead
  // optional un-locking (App. "Optional Unlocking"); buffers exist once surelock_set_unlocking() switched it on
  bool unlocking = false;
  surelock_unlock_params up = {};
  int t_step = 0;                     // steps since the last reset (the step just taken is number t_step)
  void* frozen = nullptr;             // [R][V] storage dtype: logits of every position at the step it locked (p_{t*})
  float* frozen_lse = nullptr;        // [R]
  int32_t *frozen_rop = nullptr, *t_star = nullptr, *cool_until = nullptr;   // [R]: position (or -1), t*, last cool-down step
  uint8_t *relock = nullptr, *inv_lock = nullptr;                            // [R]
  int32_t *p_idx = nullptr, *p_offsets = nullptr, *p_n = nullptr, *p_argmax = nullptr, *n_unlocked = nullptr;
  float *p_kl = nullptr, *p_conf = nullptr, *p_lse = nullptr, *p_theta = nullptr;
  bool probe_mode = false;            // run_layer: queries only, nothing is written into the caches
  // "layer_chain" option: with few active rows the four contractions between two attention calls run as one persistent
  // kernel per layer (gemm_chain.cu): 1 (default) when the bound on M is at most 128, 0 never
  int layer_chain = 1;
  float *ch_ws = nullptr, *ssq_ffn = nullptr, *ssq_next = nullptr;
  unsigned* ch_bar = nullptr;
  unsigned ch_bar_base = 0;           // arrivals on ch_bar by all launches so far (host-side count)
  // "attn_split" option (default 1): with at most 128 active rows and few sequences, attention with the keys of a
  // (sequence, head) split over several CTAs (attention_split.cu)
  int attn_split = 1, att_S = 0;
  int chain_diag_skip = -1;           // "debug_chain_skip_barrier": one-shot, consumed by the next chain launch
  int paths = 0;                      // few-row kernels the current call has taken: 1 layer chain, 2 split-key attention
  float* att_ws = nullptr;
  unsigned long long* att_cnt = nullptr;
  bool gemm_stream = false;           // "gemm_stream" option: contractions of at most 128 rows on the weight-streaming kernel
  int m_bound = 0;                    // the bound the launches of the current call use
  bool last_gemm_tc = false;          // the last gemm() call went to the tensor-core kernel
  bool timing = false;                // per-kernel-class CUDA-event timing (off by default)
  std::vector<cudaEvent_t> ev;        // event pool, created when timing is switched on
  std::vector<int> ev_cls;            // class of the launch bracketed by events 2i, 2i+1
  int n_ev = 0;
  float gate_m = -1.f;                // confidence-gate percentile (Algorithm 1 line 21); < 0 = gate off
  float* theta = nullptr;             // [B] gate thresholds of the last step
  SplitWs split;                      // split-K workspace of the tensor-core GEMM (bf16 only)
  float4* lse_part = nullptr;         // [ceil(V/256)][R]: softmax statistics of the current logits, left by the LM head
  int* lse_valid = nullptr;           // set by the LM-head GEMM when it wrote them
  uint8_t* kv_valid = nullptr;        // [R] "check_cache": 1 = every layer's K/V of the position was written since the last reset
  bool check_cache = false;
  float* trace = nullptr;             // [2L+1][R][d]: slot 2l = input of block l, 2l+1 = after its attention sub-block, 2L = output

  size_t kv_layer_bytes() const { return (size_t)R * cfg.n_heads * cfg.head_dim * esz; }
  void* kcache(int l) const { return kv + (size_t)(2 * l) * kv_layer_bytes(); }
  void* vcache(int l) const { return kv + (size_t)(2 * l + 1) * kv_layer_bytes(); }
};

#define SL_TRY(expr)            \
  do {                          \
    int rc__ = (expr);          \
    if (rc__ != SL_OK) return rc__; \
  } while (0)

template <typename P>
static int dev_alloc(surelock_ctx* c, P** p, size_t bytes) {
  void* q = nullptr;
  if (bytes == 0) bytes = 16;
  if (cudaMalloc(&q, bytes) != cudaSuccess) {
    cudaGetLastError();
    return SL_ENOMEM;
  }
  c->allocs.push_back(q);
  *p = reinterpret_cast<P*>(q);
  return SL_OK;
}

// Kernel classes for the timing breakdown (order is part of the C ABI: surelock_kernel_times)
enum { K_COMPACT = 0, K_GATHER, K_RMSNORM, K_GEMM_QKV, K_ROPE, K_SCATTER, K_ATTN, K_GEMM_O, K_GEMM_GATEUP, K_GEMM_DOWN,
       K_GEMM_HEAD, K_SOFTMAX_KL, K_CONF_GATE, K_NUM };   // the cache check counts as K_COMPACT

static inline void tick(surelock_ctx* c, int cls) {
  if (c->timing && c->n_ev + 2 <= (int)c->ev.size()) {
    c->ev_cls[c->n_ev / 2] = cls;
    cudaEventRecord(c->ev[c->n_ev], c->st);
  }
}
static inline void tock(surelock_ctx* c) {
  if (c->timing && c->n_ev + 2 <= (int)c->ev.size()) {
    cudaEventRecord(c->ev[c->n_ev + 1], c->st);
    c->n_ev += 2;
  }
  ++c->launches;
}
#define SL_K(cls, expr) \
  do {                  \
    tick(c, cls);       \
    SL_TRY(expr);       \
    tock(c);            \
  } while (0)

namespace sl {
int launch_gemm_stream(const void* A, const void* W, const void* W2, void* C, const int32_t* n_active, int max_rows,
                       int m_bound, int n_out, int K, int epilogue, int32_t* status, bool prefetch_w, cudaStream_t st);   // gemm_stream.cu
int launch_gemm_stream_qkv(const void* A, const void* Wq, const void* Wk, const void* Wv, void* q_out, void* k_cache,
                           void* v_cache, const int32_t* idx, const float2* rope, const int32_t* n_active, int max_rows,
                           int m_bound, int n_seq, int hd, int dh, int K, int32_t* status, bool prefetch_w,
                           cudaStream_t st);                                                                          // gemm_stream.cu
int launch_gemm_tc(const void* A, const void* W, const void* W2, void* C, const int32_t* n_active, int max_rows,
                   int n_out, int K, int epilogue, int32_t* status, const SplitWs& sw, cudaStream_t st);   // gemm_tc.cu; SL_EUNSUPPORTED if the shape does not fit
int launch_gemm_tc_qkv(const void* A, const void* Wq, const void* Wk, const void* Wv, void* q_out, void* k_cache,
                       void* v_cache, const int32_t* idx, const float2* rope, const int32_t* n_active, int max_rows,
                       int n_seq, int hd, int dh, int K, int32_t* status, const SplitWs& sw, cudaStream_t st);   // gemm_tc.cu
int attention_split_plan(int B, int N, int H);
size_t attention_split_workspace_bytes(int head_dim);
int launch_attention_split(const void* q, const void* kc, const void* vc, const int32_t* row_offsets, int max_rows, int B,
                           int N, int H, int head_dim, int S, void* o, float* ws, unsigned long long* counters,
                           int32_t* status, int diag_skip, cudaStream_t st);
int launch_attention_tc(const void* q, const void* kc, const void* vc, const int32_t* row_offsets, int max_rows, int B,
                        int N, int H, int head_dim, void* o, int32_t* status, cudaStream_t st);   // attention_tc.cu
}

static int attention(surelock_ctx* c, int l) {
  const surelock_model_cfg& g = c->cfg;
  if (g.dtype == SL_BF16 && c->gemm_impl == 0 && c->attn_split && c->att_S >= 2 && !c->probe_mode && c->m_bound >= 1 &&
      c->m_bound <= 128) {
    const int rc = launch_attention_split(c->q, c->kcache(l), c->vcache(l), c->row_offsets, c->R, c->B, c->N, g.n_heads,
                                          g.head_dim, c->att_S, c->attn, c->att_ws, c->att_cnt, c->status, -1, c->st);
    if (rc == SL_OK) c->paths |= 2;
    if (rc != SL_EUNSUPPORTED) return rc;
  }
  if (g.dtype == SL_BF16 && c->gemm_impl == 0) {
    const int rc = launch_attention_tc(c->q, c->kcache(l), c->vcache(l), c->row_offsets, c->R, c->B, c->N, g.n_heads,
                                       g.head_dim, c->attn, c->status, c->st);
    if (rc != SL_EUNSUPPORTED || c->strict_tc) return rc;
    ++c->fallbacks;
  }
  return launch_attention_simt(c->q, c->kcache(l), c->vcache(l), c->idx, c->n_active, c->R, c->N, g.n_heads, g.head_dim,
                               c->attn, g.dtype, c->st);
}

// the bound on M for this call (see surelock_ctx::h_m)
static int begin_call(surelock_ctx* c) {
  const int slot = (int)(c->calls & 1);
  c->m_bound = c->R;
  c->paths = 0;
  if (c->ev_m_valid[slot]) {
    SL_CUDA_TRY(cudaEventSynchronize(c->ev_m[slot]));
    if (c->h_m[slot] >= 0 && c->h_m[slot] <= c->R) c->m_bound = c->h_m[slot];
  }
  if (c->row_bound_opt > 0) c->m_bound = c->row_bound_opt < c->R ? c->row_bound_opt : c->R;
  return SL_OK;
}
static int end_call(surelock_ctx* c) {
  const int slot = (int)(c->calls & 1);
  SL_CUDA_TRY(cudaMemcpyAsync(&c->h_m[slot], c->n_active, 4, cudaMemcpyDeviceToHost, c->st));
  SL_CUDA_TRY(cudaEventRecord(c->ev_m[slot], c->st));
  c->ev_m_valid[slot] = true;
  ++c->calls;
  return SL_OK;
}
static inline bool use_stream(const surelock_ctx* c) {
  return c->gemm_stream && c->cfg.dtype == SL_BF16 && c->gemm_impl == 0 && c->m_bound >= 1 && c->m_bound <= 128;
}

static int gemm(surelock_ctx* c, const void* A, const void* W, const void* W2, void* C, int n_out, int K, int epi) {
  c->last_gemm_tc = false;
  if (use_stream(c)) {
    const int rc = launch_gemm_stream(A, W, W2, C, c->n_active, c->R, c->m_bound, n_out, K, epi, c->status,
                                      c->split.prefetch_w, c->st);
    if (rc != SL_EUNSUPPORTED) return rc;          // (the weight-streaming kernel leaves no softmax statistics)
  }
  if (c->cfg.dtype == SL_BF16 && c->gemm_impl == 0) {
    const int rc = launch_gemm_tc(A, W, W2, C, c->n_active, c->R, n_out, K, epi, c->status, c->split, c->st);
    c->last_gemm_tc = rc == SL_OK;
    if (rc != SL_EUNSUPPORTED || c->strict_tc) return rc;
    ++c->fallbacks;
  }
  return launch_gemm_simt(A, W, W2, C, c->n_active, c->R, n_out, K, c->cfg.dtype, epi, c->st);
}

static inline bool use_chain(const surelock_ctx* c) {
  return c->layer_chain && c->ch_ws && !c->probe_mode && c->cfg.dtype == SL_BF16 && c->gemm_impl == 0 && c->m_bound >= 1 &&
         c->m_bound <= 128;
}

// Lines 10-11 of Algorithm 1 for few rows: xg = bf16(x * gain) + chunk sums of squares, then the chain kernel's Q/K/V
// phase (projection, row scale, rotary embedding, packed q, K/V into the cache rows) as its only phase.
static int layer_front_chain(surelock_ctx* c, int l, float* x) {
  const surelock_model_cfg& g = c->cfg;
  ChainLaunch L = {};
  L.attn = c->attn; L.wq = c->wq[l]; L.wk = c->wk[l]; L.wv = c->wv[l];
  L.x = x; L.xg = c->h; L.act = c->act;
  L.ssq_ffn = c->ssq_ffn; L.ssq_next = c->ssq_next;
  L.q = c->q; L.kc = c->kcache(l); L.vc = c->vcache(l);
  L.idx = c->idx; L.rope = c->rope; L.ws = c->ch_ws; L.bar = c->ch_bar; L.bar_base = &c->ch_bar_base;
  L.n_active = c->n_active; L.status = c->status;
  L.diag_skip = c->chain_diag_skip;
  c->chain_diag_skip = -1;
  L.max_rows = c->R; L.m_bound = c->m_bound; L.d = g.d_model; L.F = g.d_ff; L.hd = g.n_heads * g.head_dim; L.dh = g.head_dim;
  L.n_seq = c->N; L.rms_eps = g.rms_eps;
  SL_K(K_RMSNORM, launch_norm_prep(x, c->attn_norm_g[l], c->h, c->ssq_next, c->n_active, c->R, g.d_model, c->st));
  SL_K(K_GEMM_QKV, launch_gemm_chain(L, c->st));
  c->paths |= 1;
  return SL_OK;
}

// Algorithm 1 lines 10-13 for one layer on the packed rows in x (fp32 [M][d], updated in place): layer_front is lines
// 10-11 (norm, Q/K/V, rotary embedding, cache scatter), layer_back lines 12-13 (attention, output projection, FFN).
static int layer_front(surelock_ctx* c, int l, float* x) {
  const surelock_model_cfg& g = c->cfg;
  const int d = g.d_model, hd = g.n_heads * g.head_dim;
  if (use_chain(c)) {
    // few rows: the layer chain kernel with the Q/K/V phase alone (the norm folded in as in its other phases)
    const int rc = layer_front_chain(c, l, x);
    if (rc != SL_EUNSUPPORTED) return rc;
  }
  SL_K(K_RMSNORM, launch_rmsnorm(x, c->attn_norm_g[l], c->h, c->n_active, c->R, d, g.rms_eps, g.dtype, c->st));
  bool fused = false;
  if (c->probe_mode) {
    // the probe of un-locking: the rows are queries only; their k, v are not computed and the caches stay as they are
    SL_K(K_GEMM_QKV, gemm(c, c->h, c->wq[l], nullptr, c->q, hd, d, EPI_STORE));
    SL_K(K_ROPE, launch_rope(c->q, c->k, c->idx, c->n_active, c->R, c->N, g.n_heads, g.head_dim, c->rope, g.dtype, c->st));
    fused = true;
  } else if (g.dtype == SL_BF16 && c->gemm_impl == 0) {
    // one launch: Q, K, V projections + RoPE + K/V written straight into the cache rows of the active positions
    tick(c, K_GEMM_QKV);
    int rc = SL_EUNSUPPORTED;
    if (use_stream(c))
      rc = launch_gemm_stream_qkv(c->h, c->wq[l], c->wk[l], c->wv[l], c->q, c->kcache(l), c->vcache(l), c->idx, c->rope,
                                  c->n_active, c->R, c->m_bound, c->N, hd, g.head_dim, d, c->status, c->split.prefetch_w,
                                  c->st);
    if (rc == SL_EUNSUPPORTED)
      rc = launch_gemm_tc_qkv(c->h, c->wq[l], c->wk[l], c->wv[l], c->q, c->kcache(l), c->vcache(l), c->idx, c->rope,
                              c->n_active, c->R, c->N, hd, g.head_dim, d, c->status, c->split, c->st);
    if (rc == SL_OK) {
      tock(c);
      fused = true;
    } else if (rc != SL_EUNSUPPORTED || c->strict_tc) {
      return rc;
    } else {
      ++c->fallbacks;
    }
  }
  if (!fused) {
    SL_K(K_GEMM_QKV, gemm(c, c->h, c->wq[l], nullptr, c->q, hd, d, EPI_STORE));
    SL_K(K_GEMM_QKV, gemm(c, c->h, c->wk[l], nullptr, c->k, hd, d, EPI_STORE));
    SL_K(K_GEMM_QKV, gemm(c, c->h, c->wv[l], nullptr, c->v, hd, d, EPI_STORE));
    SL_K(K_ROPE, launch_rope(c->q, c->k, c->idx, c->n_active, c->R, c->N, g.n_heads, g.head_dim, c->rope, g.dtype, c->st));
    SL_K(K_SCATTER, launch_kv_scatter(c->k, c->v, c->idx, c->n_active, c->R, hd, c->kcache(l), c->vcache(l), g.dtype, c->st));
  }
  return SL_OK;
}

// Attention, then everything up to the next attention as one persistent kernel: output projection, SwiGLU FFN and,
// when `next` >= 0, the Q/K/V projections of layer `next` (Algorithm 1 lines 12-13, then 10-11 of the next block).
static int layer_back_chain(surelock_ctx* c, int l, float* x, int next) {
  const surelock_model_cfg& g = c->cfg;
  SL_K(K_ATTN, attention(c, l));
  ChainLaunch L = {};
  L.attn = c->attn; L.wo = c->wo[l]; L.wg = c->w_gate[l]; L.wu = c->w_up[l]; L.wd = c->w_down[l];
  if (next >= 0) { L.wq = c->wq[next]; L.wk = c->wk[next]; L.wv = c->wv[next]; }
  L.x = x; L.xg = c->h; L.act = c->act;
  L.gain_ffn = c->ffn_norm_g[l];
  L.gain_next = next >= 0 ? c->attn_norm_g[next] : nullptr;
  L.ssq_ffn = c->ssq_ffn; L.ssq_next = c->ssq_next;
  L.q = c->q;
  if (next >= 0) { L.kc = c->kcache(next); L.vc = c->vcache(next); }
  L.idx = c->idx; L.rope = c->rope; L.ws = c->ch_ws; L.bar = c->ch_bar; L.bar_base = &c->ch_bar_base;
  L.n_active = c->n_active; L.status = c->status;
  L.diag_skip = c->chain_diag_skip;
  c->chain_diag_skip = -1;
  if (c->trace && x == c->x) {
    L.trace_mid = c->trace + (size_t)(2 * l + 1) * c->R * g.d_model;
    L.trace_out = c->trace + (size_t)(2 * l + 2) * c->R * g.d_model;
  }
  L.max_rows = c->R; L.m_bound = c->m_bound; L.d = g.d_model; L.F = g.d_ff; L.hd = g.n_heads * g.head_dim; L.dh = g.head_dim;
  L.n_seq = c->N; L.rms_eps = g.rms_eps;
  SL_K(K_GEMM_GATEUP, launch_gemm_chain(L, c->st));
  c->paths |= 1;
  return SL_OK;
}

static int layer_back(surelock_ctx* c, int l, float* x) {
  const surelock_model_cfg& g = c->cfg;
  const int d = g.d_model, hd = g.n_heads * g.head_dim;
  SL_K(K_ATTN, attention(c, l));
  SL_K(K_GEMM_O, gemm(c, c->attn, c->wo[l], nullptr, x, d, hd, EPI_RESIDUAL));
  if (c->trace && x == c->x)
    SL_CUDA_TRY(cudaMemcpyAsync(c->trace + (size_t)(2 * l + 1) * c->R * d, x, (size_t)c->R * d * sizeof(float),
                                cudaMemcpyDeviceToDevice, c->st));
  SL_K(K_RMSNORM, launch_rmsnorm(x, c->ffn_norm_g[l], c->h, c->n_active, c->R, d, g.rms_eps, g.dtype, c->st));
  SL_K(K_GEMM_GATEUP, gemm(c, c->h, c->w_gate[l], c->w_up[l], c->act, g.d_ff, d, EPI_SWIGLU));
  SL_K(K_GEMM_DOWN, gemm(c, c->act, c->w_down[l], nullptr, x, d, g.d_ff, EPI_RESIDUAL));
  return SL_OK;
}

static int run_layer(surelock_ctx* c, int l, float* x) {
  SL_TRY(layer_front(c, l, x));
  if (use_chain(c)) {
    const int rc = layer_back_chain(c, l, x, -1);
    if (rc != SL_EUNSUPPORTED) return rc;
  }
  return layer_back(c, l, x);
}

extern "C" {

int surelock_init(surelock_ctx** out, const surelock_model_cfg* cfg, const surelock_weights* w, int N, int batch,
                  void* cuda_stream) {
  if (!out || !cfg || !w || N <= 0 || batch <= 0) return SL_EINVAL;
  *out = nullptr;
  if (cfg->n_layers <= 0 || cfg->d_model <= 0 || cfg->n_heads <= 0 || cfg->d_ff <= 0 || cfg->vocab < 0)
    return SL_EINVAL;
  if (cfg->dtype != SL_BF16 && cfg->dtype != SL_FP32) return SL_EINVAL;
  if (cfg->n_kv_heads != cfg->n_heads) return SL_EUNSUPPORTED;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return SL_EUNSUPPORTED;
  if (cfg->d_model % 8 || cfg->d_ff % 8 || cfg->vocab % 8) return SL_EUNSUPPORTED;
  if ((long long)N * batch >= (1ll << 31)) return SL_EINVAL;
  if (!w->attn_norm_g || !w->wq || !w->wk || !w->wv || !w->wo || !w->ffn_norm_g || !w->w_gate || !w->w_up ||
      !w->w_down)
    return SL_EINVAL;
  if (cfg->vocab > 0 && (!w->tok_emb || !w->lm_head || !w->final_norm_g)) return SL_EINVAL;
  for (int l = 0; l < cfg->n_layers; ++l)
    if (!w->attn_norm_g[l] || !w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->ffn_norm_g[l] ||
        !w->w_gate[l] || !w->w_up[l] || !w->w_down[l])
      return SL_EINVAL;

  surelock_ctx* c = new (std::nothrow) surelock_ctx();
  if (!c) return SL_ENOMEM;
  c->cfg = *cfg;
  c->N = N;
  c->B = batch;
  c->R = N * batch;
  c->esz = cfg->dtype == SL_BF16 ? 2 : 4;
  c->st = reinterpret_cast<cudaStream_t>(cuda_stream);
  c->tok_emb = w->tok_emb;
  c->lm_head = w->lm_head;
  c->final_norm_g = w->final_norm_g;
  const int L = cfg->n_layers;
  c->attn_norm_g.assign(w->attn_norm_g, w->attn_norm_g + L);
  c->wq.assign(w->wq, w->wq + L);
  c->wk.assign(w->wk, w->wk + L);
  c->wv.assign(w->wv, w->wv + L);
  c->wo.assign(w->wo, w->wo + L);
  c->ffn_norm_g.assign(w->ffn_norm_g, w->ffn_norm_g + L);
  c->w_gate.assign(w->w_gate, w->w_gate + L);
  c->w_up.assign(w->w_up, w->w_up + L);
  c->w_down.assign(w->w_down, w->w_down + L);

  const size_t R = c->R, d = cfg->d_model, hd = (size_t)cfg->n_heads * cfg->head_dim, F = cfg->d_ff, V = cfg->vocab;
  const size_t e = c->esz;
  int rc = SL_OK;
#define A_(p, bytes) if (rc == SL_OK) rc = dev_alloc(c, &(p), (bytes))
  A_(c->kv, 2 * (size_t)L * R * hd * e);
  A_(c->x, R * d * 4);
  A_(c->h, R * d * e);
  A_(c->q, R * hd * e);
  A_(c->k, R * hd * e);
  A_(c->v, R * hd * e);
  A_(c->attn, R * hd * e);
  A_(c->act, R * F * e);
  for (int i = 0; i < 2; ++i) {
    A_(c->logits[i], R * V * e);
    A_(c->lse[i], R * 4);
    A_(c->row_of_pos[i], R * 4);
  }
  A_(c->idx, R * 4);
  A_(c->row_offsets, ((size_t)batch + 1) * 4);
  A_(c->n_active, 16);
  A_(c->n_prev, 16);
  A_(c->status, 16);
  A_(c->argmax, R * 4);
  A_(c->kl, R * 4);
  A_(c->conf, R * 4);
  A_(c->scratch, compact_scratch_bytes((int64_t)R));
  A_(c->rope, (size_t)N * (cfg->head_dim / 2) * sizeof(float2));
  if (cfg->dtype == SL_BF16) {
    c->split.tiles = 4 * sm_count();
    c->split.prefetch_w = true;   // inside a step a GEMM never directly follows the kernel that writes n_active
    A_(c->split.ws, (size_t)c->split.tiles * SPLIT_TILE_BYTES);
    A_(c->split.counters, (size_t)c->split.tiles * 3 * sizeof(int));
    if (rc == SL_OK && cudaMemsetAsync(c->split.counters, 0, (size_t)c->split.tiles * 3 * sizeof(int), c->st) != cudaSuccess)
      rc = SL_ECUDA;
  }
  if (cfg->dtype == SL_BF16) {               // workspace of the layer-chain kernel (few active rows)
    A_(c->ch_ws, gemm_chain_workspace_bytes(128));
    A_(c->ssq_ffn, R * (d / 32 + 1) * sizeof(float));
    A_(c->ssq_next, R * (d / 32 + 1) * sizeof(float));
    A_(c->ch_bar, 16);
    if (rc == SL_OK && cudaMemsetAsync(c->ch_bar, 0, 16, c->st) != cudaSuccess) rc = SL_ECUDA;
    c->att_S = attention_split_plan(batch, N, cfg->n_heads);
    if (c->att_S >= 2) {                     // few sequences: attention with split keys for steps with few active rows
      A_(c->att_ws, attention_split_workspace_bytes(cfg->head_dim));
      A_(c->att_cnt, (size_t)batch * cfg->n_heads * sizeof(unsigned long long));
      if (rc == SL_OK &&
          cudaMemsetAsync(c->att_cnt, 0, (size_t)batch * cfg->n_heads * sizeof(unsigned long long), c->st) != cudaSuccess)
        rc = SL_ECUDA;
    }
  }
  if (cfg->dtype == SL_BF16 && V > 0) {
    A_(c->lse_part, ((V + 255) / 256) * R * sizeof(float4));
    A_(c->lse_valid, 16);
    if (rc == SL_OK && cudaMemsetAsync(c->lse_valid, 0, 16, c->st) != cudaSuccess) rc = SL_ECUDA;
  }
  if (rc == SL_OK && cudaMallocHost(reinterpret_cast<void**>(&c->h_m), 2 * sizeof(int32_t)) != cudaSuccess) rc = SL_ENOMEM;
  for (int i = 0; i < 2 && rc == SL_OK; ++i)
    if (cudaEventCreateWithFlags(&c->ev_m[i], cudaEventDisableTiming) != cudaSuccess) rc = SL_ECUDA;
  A_(c->theta, ((size_t)batch + 1) * 4);
  A_(c->st_tokens, R * 4);
  A_(c->st_mask, R);
  A_(c->st_lock, R);
#undef A_
  if (rc == SL_OK && cudaMemsetAsync(c->kv, 0, 2 * (size_t)L * R * hd * e, c->st) != cudaSuccess) rc = SL_ECUDA;
  if (rc == SL_OK) rc = build_rope_table(c->rope, N, cfg->head_dim, cfg->rope_theta, c->st);
  if (rc == SL_OK) rc = surelock_reset(c);
  if (rc == SL_OK && cudaStreamSynchronize(c->st) != cudaSuccess) rc = SL_ECUDA;
  if (rc != SL_OK) {
    surelock_destroy(c);
    return rc;
  }
  *out = c;
  return SL_OK;
}

int surelock_reset(surelock_ctx* c) {
  if (!c) return SL_EINVAL;
  c->have_prev = false;
  c->cur = 0;
  c->calls = 0;
  c->ev_m_valid[0] = c->ev_m_valid[1] = false;
  if (c->att_cnt)
    SL_CUDA_TRY(cudaMemsetAsync(c->att_cnt, 0, (size_t)c->B * c->cfg.n_heads * sizeof(unsigned long long), c->st));
  if (c->ch_bar) {                      // a chain kernel that gave up leaves the barrier count short: start over
    SL_CUDA_TRY(cudaMemsetAsync(c->ch_bar, 0, 16, c->st));
    c->ch_bar_base = 0;
  }
  c->t_step = 0;
  if (c->unlocking) {
    const size_t R = c->R;
    SL_CUDA_TRY(cudaMemsetAsync(c->frozen_rop, 0xff, R * 4, c->st));
    SL_CUDA_TRY(cudaMemsetAsync(c->t_star, 0xff, R * 4, c->st));
    SL_CUDA_TRY(cudaMemsetAsync(c->cool_until, 0xff, R * 4, c->st));
    SL_CUDA_TRY(cudaMemsetAsync(c->relock, 0, R, c->st));
  }
  for (int i = 0; i < 2; ++i) SL_CUDA_TRY(cudaMemsetAsync(c->row_of_pos[i], 0xff, (size_t)c->R * 4, c->st));
  SL_CUDA_TRY(cudaMemsetAsync(c->status, 0, 16, c->st));
  SL_CUDA_TRY(cudaMemsetAsync(c->n_active, 0, 16, c->st));
  SL_CUDA_TRY(cudaMemsetAsync(c->n_prev, 0, 16, c->st));
  c->fallbacks = 0;
  // a GEMM that gave up on a bounded wait leaves its tiles' hand-over counters half-way: start from zero again
  if (c->split.counters)
    SL_CUDA_TRY(cudaMemsetAsync(c->split.counters, 0, (size_t)c->split.tiles * 3 * sizeof(int), c->st));
  if (c->lse_valid) SL_CUDA_TRY(cudaMemsetAsync(c->lse_valid, 0, 16, c->st));
  if (c->kv_valid) SL_CUDA_TRY(cudaMemsetAsync(c->kv_valid, 0, (size_t)c->R, c->st));   // cache contents are undefined now
  return SL_OK;
}

int surelock_step(surelock_ctx* c, const int32_t* tokens, const uint8_t* mask_state, uint8_t* lock_mask, float kl_eps,
                  surelock_step_out* out) {
  if (!c || !tokens || !mask_state || !lock_mask) return SL_EINVAL;
  if (!(kl_eps >= 0.f)) return SL_EINVAL;   // also rejects NaN
  if (c->cfg.vocab <= 0) return SL_EUNSUPPORTED;
  const surelock_model_cfg& g = c->cfg;
  c->launches = 0;
  const int cur = c->cur, prv = cur ^ 1;
  c->n_ev = 0;
  SL_TRY(begin_call(c));
  ++c->t_step;
  if (c->check_cache) SL_K(K_COMPACT, launch_cache_check(lock_mask, c->kv_valid, c->R, c->status, c->st));
  SL_K(K_COMPACT, launch_compact(lock_mask, c->B, c->N, c->idx, c->row_offsets, c->n_active, c->row_of_pos[cur],
                                 c->scratch, c->status, c->st));
  SL_K(K_GATHER, launch_gather_rows(c->tok_emb, tokens, c->idx, c->n_active, c->R, g.d_model, g.vocab, c->x, g.dtype,
                                    c->status, c->st));
  const size_t xbytes = (size_t)c->R * g.d_model * sizeof(float);
  if (c->trace) SL_CUDA_TRY(cudaMemcpyAsync(c->trace, c->x, xbytes, cudaMemcpyDeviceToDevice, c->st));
  bool chained = false;                            // the Q/K/V of layer l were already done by layer l-1's chain kernel
  for (int l = 0; l < g.n_layers; ++l) {
    if (!chained) SL_TRY(layer_front(c, l, c->x));
    chained = false;
    int rc = SL_EUNSUPPORTED;
    if (use_chain(c)) {
      rc = layer_back_chain(c, l, c->x, l + 1 < g.n_layers ? l + 1 : -1);
      if (rc == SL_OK) chained = l + 1 < g.n_layers;
      else if (rc != SL_EUNSUPPORTED) return rc;
    }
    if (rc == SL_EUNSUPPORTED) {
      SL_TRY(layer_back(c, l, c->x));
      if (c->trace)
        SL_CUDA_TRY(cudaMemcpyAsync(c->trace + (size_t)(2 * l + 2) * c->R * g.d_model, c->x, xbytes,
                                    cudaMemcpyDeviceToDevice, c->st));
    }
  }
  SL_K(K_RMSNORM, launch_rmsnorm(c->x, c->final_norm_g, c->h, c->n_active, c->R, g.d_model, g.rms_eps, g.dtype, c->st));
  c->split.lse_part = c->lse_part;                 // the LM head leaves the rows' softmax statistics for the next kernel
  c->split.lse_rows = c->R;
  c->split.lse_valid = c->lse_valid;
  SL_K(K_GEMM_HEAD, gemm(c, c->h, c->lm_head, nullptr, c->logits[cur], g.vocab, g.d_model, EPI_STORE));
  c->split.lse_part = nullptr;
  c->split.lse_valid = nullptr;
  const bool head_tc = c->last_gemm_tc;            // only the tensor-core kernel writes the statistics (and their flag)
  SL_K(K_SOFTMAX_KL, launch_softmax_kl_sure(c->logits[cur], c->have_prev ? c->logits[prv] : nullptr, c->row_of_pos[prv],
                                            c->lse[prv], c->idx, c->n_active, c->R, g.vocab, g.dtype, mask_state,
                                            lock_mask, kl_eps, c->kl, c->conf, c->argmax, c->lse[cur], c->st,
                                            c->gate_m < 0.f && !c->unlocking, head_tc ? c->lse_part : nullptr,
                                            (g.vocab + 255) / 256, c->R, c->lse_valid));
  if (c->gate_m >= 0.f)
    SL_K(K_CONF_GATE, launch_conf_gate_lock(c->conf, c->kl, c->idx, c->row_offsets, c->B, c->N, mask_state, lock_mask,
                                            kl_eps, c->gate_m, c->theta, c->st, !c->unlocking));
  if (c->unlocking)   // per-position threshold and cool-down; rows that lock keep t* and their logits (p_{t*})
    SL_K(K_CONF_GATE, launch_lock_commit(c->kl, c->conf, c->lse[cur], c->idx, c->n_active, c->R, c->N, mask_state, lock_mask,
                                         kl_eps, c->up.rho, c->t_step, c->gate_m >= 0.f ? c->theta : nullptr,
                                         c->cool_until, c->relock, c->t_star, c->frozen_rop, c->frozen_lse,
                                         c->logits[cur], c->frozen, (size_t)g.vocab * c->esz, c->st));
  if (out) {
    out->active_idx = c->idx;
    out->row_offsets = c->row_offsets;
    out->n_active = c->n_active;
    out->logits = c->logits[cur];
    out->hidden = c->x;
    out->kl = c->kl;
    out->conf = c->conf;
    out->argmax = c->argmax;
  }
  // the row count of the logits the next step reads as "previous" (n_active itself is overwritten by other calls)
  SL_CUDA_TRY(cudaMemcpyAsync(c->n_prev, c->n_active, 4, cudaMemcpyDeviceToDevice, c->st));
  SL_TRY(end_call(c));
  c->cur = prv;
  c->have_prev = true;
  return SL_OK;
}

int surelock_step_host(surelock_ctx* c, const int32_t* tokens, const uint8_t* mask_state, uint8_t* lock_mask,
                       float kl_eps, int32_t* n_active, int32_t* active_idx, float* kl, float* conf, int32_t* argmax) {
  if (!c || !tokens || !mask_state || !lock_mask || !n_active) return SL_EINVAL;
  const size_t R = c->R;
  SL_CUDA_TRY(cudaMemcpyAsync(c->st_tokens, tokens, R * 4, cudaMemcpyHostToDevice, c->st));
  SL_CUDA_TRY(cudaMemcpyAsync(c->st_mask, mask_state, R, cudaMemcpyHostToDevice, c->st));
  SL_CUDA_TRY(cudaMemcpyAsync(c->st_lock, lock_mask, R, cudaMemcpyHostToDevice, c->st));
  SL_TRY(surelock_step(c, c->st_tokens, c->st_mask, c->st_lock, kl_eps, nullptr));
  SL_CUDA_TRY(cudaMemcpyAsync(lock_mask, c->st_lock, R, cudaMemcpyDeviceToHost, c->st));
  SL_CUDA_TRY(cudaMemcpyAsync(n_active, c->n_active, 4, cudaMemcpyDeviceToHost, c->st));
  if (active_idx) SL_CUDA_TRY(cudaMemcpyAsync(active_idx, c->idx, R * 4, cudaMemcpyDeviceToHost, c->st));
  if (kl) SL_CUDA_TRY(cudaMemcpyAsync(kl, c->kl, R * 4, cudaMemcpyDeviceToHost, c->st));
  if (conf) SL_CUDA_TRY(cudaMemcpyAsync(conf, c->conf, R * 4, cudaMemcpyDeviceToHost, c->st));
  if (argmax) SL_CUDA_TRY(cudaMemcpyAsync(argmax, c->argmax, R * 4, cudaMemcpyDeviceToHost, c->st));
  SL_CUDA_TRY(cudaStreamSynchronize(c->st));
  return SL_OK;
}

int surelock_layer_step(surelock_ctx* c, int layer, const void* hidden_in, const uint8_t* lock_mask, float* hidden_out,
                        surelock_step_out* out) {
  if (!c || !hidden_in || !lock_mask || !hidden_out) return SL_EINVAL;
  if (layer < 0 || layer >= c->cfg.n_layers) return SL_EINVAL;
  const surelock_model_cfg& g = c->cfg;
  c->launches = 0;
  c->n_ev = 0;
  SL_TRY(begin_call(c));
  SL_K(K_COMPACT, launch_compact(lock_mask, c->B, c->N, c->idx, c->row_offsets, c->n_active, nullptr, c->scratch,
                                 c->status, c->st));
  SL_K(K_GATHER, launch_gather_rows(hidden_in, nullptr, c->idx, c->n_active, c->R, g.d_model, c->R, hidden_out, g.dtype,
                                    c->status, c->st));
  SL_TRY(run_layer(c, layer, hidden_out));
  SL_TRY(end_call(c));
  if (out) {
    memset(out, 0, sizeof(*out));
    out->active_idx = c->idx;
    out->row_offsets = c->row_offsets;
    out->n_active = c->n_active;
    out->hidden = hidden_out;
  }
  return SL_OK;
}

int surelock_set_unlocking(surelock_ctx* c, const surelock_unlock_params* p) {
  if (!c) return SL_EINVAL;
  if (!p) {
    c->unlocking = false;
    return SL_OK;
  }
  if (p->period < 1 || !(p->eps_unlock >= 0.f) || p->d_interval < 0 || p->d_cool < 0 || !(p->rho >= 0.f) || p->rho > 1.f ||
      !(p->m_percent >= 0.f) || p->m_percent > 100.f)
    return SL_EINVAL;
  if (c->cfg.vocab <= 0) return SL_EUNSUPPORTED;
  if (!c->frozen) {
    const size_t R = c->R, V = c->cfg.vocab;
    int rc = SL_OK;
#define A_(p_, bytes) if (rc == SL_OK) rc = dev_alloc(c, &(p_), (bytes))
    A_(c->frozen, R * V * c->esz);
    A_(c->frozen_lse, R * 4);
    A_(c->frozen_rop, R * 4);
    A_(c->t_star, R * 4);
    A_(c->cool_until, R * 4);
    A_(c->relock, R);
    A_(c->inv_lock, R);
    A_(c->p_idx, R * 4);
    A_(c->p_offsets, ((size_t)c->B + 1) * 4);
    A_(c->p_n, 16);
    A_(c->n_unlocked, 16);
    A_(c->p_argmax, R * 4);
    A_(c->p_kl, R * 4);
    A_(c->p_conf, R * 4);
    A_(c->p_lse, R * 4);
    A_(c->p_theta, ((size_t)c->B + 1) * 4);
#undef A_
    if (rc != SL_OK) return rc;
  }
  c->up = *p;
  c->unlocking = true;
  return surelock_reset(c);          // t*, cool-down and the step counter start over
}

int surelock_probe_unlock(surelock_ctx* c, const int32_t* tokens, uint8_t* lock_mask, surelock_probe_out* out) {
  if (!c || !tokens || !lock_mask) return SL_EINVAL;
  if (!c->unlocking) return SL_EINVAL;
  const surelock_model_cfg& g = c->cfg;
  if (out) memset(out, 0, sizeof(*out));
  if (out) out->step = c->t_step;
  if (c->t_step < 1 || c->t_step % c->up.period != 0) return SL_OK;   // not a probe step
  const int done = c->cur ^ 1;       // the slot the step just taken wrote; slot c->cur is free until the next step
  const int scratch_slot = c->cur;
  // theta_t: per sequence the m-th percentile of u over the rows that were active in the step just taken
  SL_TRY(launch_conf_gate_lock(c->conf, c->kl, c->idx, c->row_offsets, c->B, c->N, lock_mask, lock_mask, 0.f,
                               c->up.m_percent, c->p_theta, c->st, false, true, INFINITY));
  // the locked rows, packed
  SL_TRY(launch_invert_mask(lock_mask, c->inv_lock, c->R, c->st));
  SL_TRY(launch_compact(c->inv_lock, c->B, c->N, c->p_idx, c->p_offsets, c->p_n, nullptr, c->scratch, c->status, c->st));
  // the forward of the step on those rows as queries only (Algorithm 1 lines 7, 10, 12, 15 without line 11)
  int32_t *s_idx = c->idx, *s_off = c->row_offsets, *s_n = c->n_active;
  const int s_bound = c->m_bound;
  c->idx = c->p_idx;
  c->row_offsets = c->p_offsets;
  c->n_active = c->p_n;
  c->m_bound = c->R;
  c->probe_mode = true;
  float* keep_trace = c->trace;
  c->trace = nullptr;
  int rc = launch_gather_rows(c->tok_emb, tokens, c->idx, c->n_active, c->R, g.d_model, g.vocab, c->x, g.dtype, c->status,
                              c->st);
  for (int l = 0; l < g.n_layers && rc == SL_OK; ++l) rc = run_layer(c, l, c->x);
  if (rc == SL_OK)
    rc = launch_rmsnorm(c->x, c->final_norm_g, c->h, c->n_active, c->R, g.d_model, g.rms_eps, g.dtype, c->st);
  if (rc == SL_OK) rc = gemm(c, c->h, c->lm_head, nullptr, c->logits[scratch_slot], g.vocab, g.d_model, EPI_STORE);
  // drift KL(p^_t || p_{t*}) against the frozen logits of each position, proxy confidence
  if (rc == SL_OK)
    rc = launch_softmax_kl_sure(c->logits[scratch_slot], c->frozen, c->frozen_rop, c->frozen_lse, c->idx, c->n_active, c->R,
                                g.vocab, g.dtype, lock_mask, lock_mask, 0.f, c->p_kl, c->p_conf, c->p_argmax, c->p_lse,
                                c->st, false);
  c->idx = s_idx;
  c->row_offsets = s_off;
  c->n_active = s_n;
  c->m_bound = s_bound;
  c->probe_mode = false;
  c->trace = keep_trace;
  (void)done;
  SL_TRY(rc);
  SL_CUDA_TRY(cudaMemsetAsync(c->n_unlocked, 0, 4, c->st));
  SL_TRY(launch_unlock(c->p_kl, c->p_conf, c->p_idx, c->p_n, c->R, c->N, c->p_theta, c->up.eps_unlock, c->up.d_interval,
                       c->up.d_cool, c->t_step, c->t_star, c->cool_until, c->relock, lock_mask, c->n_unlocked, c->st));
  if (out) {
    out->probed = 1;
    out->probed_idx = c->p_idx;
    out->n_probed = c->p_n;
    out->drift = c->p_kl;
    out->conf = c->p_conf;
    out->theta = c->p_theta;
    out->n_unlocked = c->n_unlocked;
    out->t_star = c->t_star;
    out->cool_until = c->cool_until;
  }
  return SL_OK;
}

int surelock_status_poll(surelock_ctx* c, int* device_status) {
  if (!c) return SL_EINVAL;
  int32_t s = 0;
  if (cudaStreamSynchronize(c->st) != cudaSuccess) return SL_ECUDA;
  if (cudaMemcpy(&s, c->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return SL_ECUDA;
  if (device_status) *device_status = s;
  return s ? SL_EDEVICE : SL_OK;
}

int surelock_kv_cache(surelock_ctx* c, int layer, void** k, void** v, size_t* row_stride_elems) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return SL_EINVAL;
  if (k) *k = c->kcache(layer);
  if (v) *v = c->vcache(layer);
  if (row_stride_elems) *row_stride_elems = (size_t)c->cfg.n_heads * c->cfg.head_dim;
  return SL_OK;
}

int surelock_prev_logits(surelock_ctx* c, void** buf, int32_t** row_of_pos) {
  if (!c) return SL_EINVAL;
  // the buffer the NEXT step reads as "previous" is the one the last step wrote
  const int prv = c->cur ^ 1;
  if (buf) *buf = c->logits[prv];
  if (row_of_pos) *row_of_pos = c->row_of_pos[prv];
  return SL_OK;
}

// ---- checkpoint / resume
struct StateHeader {
  uint64_t magic;                       // "SLKSTAT1"
  int32_t n_layers, d_model, n_heads, head_dim, d_ff, vocab, dtype, N, B;
  int32_t have_prev, rows_prev;         // rows of the previous step's logits that are stored
  // the row counts of the last two steps, from which the next two steps take their bound on M (so that a ctx that
  // imports the state chooses the same kernels as the one that went on): flags bit 0 / 1 = count 0 / 1 is there,
  // bit 2 = parity of the call counter
  int32_t m_flags, m_hist[2];
  int32_t reserved[2];
};
static const uint64_t STATE_MAGIC = 0x31544154534b4c53ull;

static void fill_header(const surelock_ctx* c, StateHeader* h) {
  memset(h, 0, sizeof(*h));
  h->magic = STATE_MAGIC;
  h->n_layers = c->cfg.n_layers; h->d_model = c->cfg.d_model; h->n_heads = c->cfg.n_heads; h->head_dim = c->cfg.head_dim;
  h->d_ff = c->cfg.d_ff; h->vocab = c->cfg.vocab; h->dtype = c->cfg.dtype; h->N = c->N; h->B = c->B;
}

size_t surelock_state_bytes(const surelock_ctx* c) {
  if (!c) return 0;
  const size_t R = c->R, V = c->cfg.vocab;
  return sizeof(StateHeader) + 2 * (size_t)c->cfg.n_layers * c->kv_layer_bytes() + R * V * c->esz + R * 4 + R * 4;
}

int surelock_state_export(surelock_ctx* c, void* host_dst, size_t capacity, size_t* written) {
  if (!c || !host_dst) return SL_EINVAL;
  SL_CUDA_TRY(cudaStreamSynchronize(c->st));
  const int prv = c->cur ^ 1;           // the slot the last step wrote
  StateHeader h;
  fill_header(c, &h);
  h.have_prev = c->have_prev ? 1 : 0;
  int32_t m_prev = 0;
  if (c->have_prev) SL_CUDA_TRY(cudaMemcpy(&m_prev, c->n_prev, 4, cudaMemcpyDeviceToHost));
  if (c->have_prev && m_prev == 0) m_prev = c->R;   // previous logits seeded by the caller ("have_prev"): keep every row
  if (m_prev < 0 || m_prev > c->R) return SL_EDEVICE;
  h.rows_prev = m_prev;
  h.m_flags = (c->ev_m_valid[0] ? 1 : 0) | (c->ev_m_valid[1] ? 2 : 0) | ((c->calls & 1) ? 4 : 0);
  h.m_hist[0] = c->h_m[0];                // (complete: the stream was synchronised above)
  h.m_hist[1] = c->h_m[1];
  const size_t kvb = 2 * (size_t)c->cfg.n_layers * c->kv_layer_bytes();
  const size_t lgb = (size_t)m_prev * c->cfg.vocab * c->esz, lsb = (size_t)m_prev * 4, rpb = (size_t)c->R * 4;
  const size_t need = sizeof(h) + kvb + lgb + lsb + rpb;
  if (capacity < need) return SL_EINVAL;
  char* p = static_cast<char*>(host_dst);
  memcpy(p, &h, sizeof(h));
  p += sizeof(h);
  SL_CUDA_TRY(cudaMemcpy(p, c->kv, kvb, cudaMemcpyDeviceToHost));
  p += kvb;
  if (lgb) SL_CUDA_TRY(cudaMemcpy(p, c->logits[prv], lgb, cudaMemcpyDeviceToHost));
  p += lgb;
  if (lsb) SL_CUDA_TRY(cudaMemcpy(p, c->lse[prv], lsb, cudaMemcpyDeviceToHost));
  p += lsb;
  SL_CUDA_TRY(cudaMemcpy(p, c->row_of_pos[prv], rpb, cudaMemcpyDeviceToHost));
  if (written) *written = need;
  return SL_OK;
}

int surelock_state_import(surelock_ctx* c, const void* host_src, size_t bytes) {
  if (!c || !host_src || bytes < sizeof(StateHeader)) return SL_EINVAL;
  StateHeader h, want;
  memcpy(&h, host_src, sizeof(h));
  fill_header(c, &want);
  if (h.magic != STATE_MAGIC || h.n_layers != want.n_layers || h.d_model != want.d_model || h.n_heads != want.n_heads ||
      h.head_dim != want.head_dim || h.d_ff != want.d_ff || h.vocab != want.vocab || h.dtype != want.dtype ||
      h.N != want.N || h.B != want.B || h.rows_prev < 0 || h.rows_prev > c->R)
    return SL_EINVAL;
  const size_t kvb = 2 * (size_t)c->cfg.n_layers * c->kv_layer_bytes();
  const size_t lgb = (size_t)h.rows_prev * c->cfg.vocab * c->esz, lsb = (size_t)h.rows_prev * 4, rpb = (size_t)c->R * 4;
  if (bytes < sizeof(h) + kvb + lgb + lsb + rpb) return SL_EINVAL;
  SL_CUDA_TRY(cudaStreamSynchronize(c->st));
  SL_TRY(surelock_reset(c));
  const int prv = c->cur ^ 1;
  const char* p = static_cast<const char*>(host_src) + sizeof(h);
  SL_CUDA_TRY(cudaMemcpyAsync(c->kv, p, kvb, cudaMemcpyHostToDevice, c->st));
  p += kvb;
  if (c->kv_valid) SL_CUDA_TRY(cudaMemsetAsync(c->kv_valid, 1, (size_t)c->R, c->st));   // an imported cache counts as filled
  if (lgb) SL_CUDA_TRY(cudaMemcpyAsync(c->logits[prv], p, lgb, cudaMemcpyHostToDevice, c->st));
  p += lgb;
  if (lsb) SL_CUDA_TRY(cudaMemcpyAsync(c->lse[prv], p, lsb, cudaMemcpyHostToDevice, c->st));
  p += lsb;
  SL_CUDA_TRY(cudaMemcpyAsync(c->row_of_pos[prv], p, rpb, cudaMemcpyHostToDevice, c->st));
  c->have_prev = h.have_prev != 0;
  const int32_t rows_prev = h.rows_prev;
  SL_CUDA_TRY(cudaMemcpyAsync(c->n_prev, &rows_prev, 4, cudaMemcpyHostToDevice, c->st));
  c->calls = (h.m_flags & 4) ? 1 : 0;
  for (int i = 0; i < 2; ++i) {
    if (!(h.m_flags & (1 << i)) || h.m_hist[i] < 0 || h.m_hist[i] > c->R) continue;
    c->h_m[i] = h.m_hist[i];
    SL_CUDA_TRY(cudaEventRecord(c->ev_m[i], c->st));
    c->ev_m_valid[i] = true;
  }
  SL_CUDA_TRY(cudaStreamSynchronize(c->st));
  return SL_OK;
}

int surelock_set_option(surelock_ctx* c, const char* name, int value) {
  if (!c || !name) return SL_EINVAL;
  if (!strcmp(name, "gemm_impl")) { c->gemm_impl = value; return SL_OK; }
  if (!strcmp(name, "strict_tc")) { c->strict_tc = value != 0; return SL_OK; }
  if (!strcmp(name, "gemm_stream")) { c->gemm_stream = value != 0; return SL_OK; }
  if (!strcmp(name, "debug_chain_skip_barrier")) { c->chain_diag_skip = value > 0 ? value - 1 : -1; return SL_OK; }
  if (!strcmp(name, "attn_split")) { c->attn_split = value != 0; return SL_OK; }
  if (!strcmp(name, "layer_chain")) {
    if (value < 0 || value > 1) return SL_EINVAL;
    c->layer_chain = value;
    return SL_OK;
  }
  if (!strcmp(name, "row_bound")) { c->row_bound_opt = value > 0 ? value : 0; return SL_OK; }
  if (!strcmp(name, "have_prev")) { c->have_prev = value != 0; return SL_OK; }
  if (!strcmp(name, "check_cache")) {
    if (value && !c->kv_valid) {
      const int rc = dev_alloc(c, &c->kv_valid, (size_t)c->R);
      if (rc != SL_OK) return rc;
    }
    if (value) SL_CUDA_TRY(cudaMemsetAsync(c->kv_valid, value == 2 ? 1 : 0, (size_t)c->R, c->st));
    c->check_cache = value != 0;
    return SL_OK;
  }
  if (!strcmp(name, "trace_layers")) {
    if (value && !c->trace) {
      const size_t bytes = (size_t)(2 * c->cfg.n_layers + 1) * c->R * c->cfg.d_model * sizeof(float);
      const int rc = dev_alloc(c, &c->trace, bytes);
      if (rc != SL_OK) return rc;
    }
    if (!value) c->trace = nullptr;   // the buffer stays allocated until destroy; tracing stops
    return SL_OK;
  }
  if (!strcmp(name, "time_kernels")) {
    if (value && c->ev.empty()) {
      const int n = 2 * (16 * c->cfg.n_layers + 16);
      c->ev.resize(n);
      c->ev_cls.assign(n / 2, 0);
      for (int i = 0; i < n; ++i)
        if (cudaEventCreate(&c->ev[i]) != cudaSuccess) return SL_ECUDA;
    }
    c->timing = value != 0;
    c->n_ev = 0;
    return SL_OK;
  }
  return SL_EINVAL;
}

int surelock_layer_trace(surelock_ctx* c, float** buf, size_t* layer_stride_elems) {
  if (!c || !buf) return SL_EINVAL;
  *buf = c->trace;
  if (layer_stride_elems) *layer_stride_elems = (size_t)c->R * c->cfg.d_model;
  return c->trace ? SL_OK : SL_EINVAL;
}

int surelock_set_confidence_gate(surelock_ctx* c, float m_percent, const float** theta) {
  if (!c) return SL_EINVAL;
  if (m_percent > 100.f) return SL_EINVAL;
  c->gate_m = (m_percent >= 0.f) ? m_percent : -1.f;     // negative or NaN: gate off
  if (theta) *theta = c->theta;
  return SL_OK;
}

int surelock_last_launch_count(surelock_ctx* c) { return c ? c->launches : SL_EINVAL; }

int surelock_last_fallback_count(surelock_ctx* c) { return c ? c->fallbacks : SL_EINVAL; }
int surelock_last_step_paths(surelock_ctx* c) { return c ? c->paths : SL_EINVAL; }

int surelock_kernel_times(surelock_ctx* c, float* ms, int32_t* launches, int n_classes) {
  if (!c || !ms || n_classes < K_NUM) return SL_EINVAL;
  for (int i = 0; i < n_classes; ++i) {
    ms[i] = 0.f;
    if (launches) launches[i] = 0;
  }
  if (!c->timing) return SL_OK;
  SL_CUDA_TRY(cudaStreamSynchronize(c->st));
  for (int i = 0; i + 1 < c->n_ev; i += 2) {
    float t = 0.f;
    SL_CUDA_TRY(cudaEventElapsedTime(&t, c->ev[i], c->ev[i + 1]));
    ms[c->ev_cls[i / 2]] += t;
    if (launches) ++launches[c->ev_cls[i / 2]];
  }
  return SL_OK;
}

void surelock_destroy(surelock_ctx* c) {
  if (!c) return;
  cudaStreamSynchronize(c->st);
  for (cudaEvent_t e : c->ev) cudaEventDestroy(e);
  for (int i = 0; i < 2; ++i)
    if (c->ev_m[i]) cudaEventDestroy(c->ev_m[i]);
  if (c->h_m) cudaFreeHost(c->h_m);
  for (void* p : c->allocs) cudaFree(p);
  delete c;
}

const char* surelock_strerror(int s) {
  switch (s) {
    case SL_OK: return "ok";
    case SL_EINVAL: return "invalid argument";
    case SL_ENOMEM: return "device allocation failed";
    case SL_ECUDA: return "CUDA runtime error";
    case SL_EDEVICE:
      return "a kernel reported an error through the status word (1 compaction wait, 2 GEMM wait, 3 attention wait ran "
             "out; 4 index out of range; 5 locked position without valid K/V)";
    case SL_EUNSUPPORTED: return "shape or type not supported";
    case SL_ELIMIT: return "size exceeds the fixed capacity of the allocation-free entry point";
    default: return "unknown status";
  }
}

// ---- single stages ------------------------------------------------------------------------------------------

size_t surelock_compact_scratch_bytes(int64_t total) { return compact_scratch_bytes(total); }

int surelock_compact(const uint8_t* lock_mask, int B, int N, int32_t* active_idx, int32_t* row_offsets, int32_t* n_active,
                     int32_t* row_of_pos, void* scratch, int32_t* dev_status, void* stream) {
  return launch_compact(lock_mask, B, N, active_idx, row_offsets, n_active, row_of_pos, scratch, dev_status,
                        (cudaStream_t)stream);
}

int surelock_compact_from_ticket(const uint8_t* lock_mask, int B, int N, int32_t* active_idx, int32_t* row_offsets,
                                 int32_t* n_active, int32_t* row_of_pos, void* scratch, uint32_t first_ticket,
                                 int32_t* dev_status, void* stream) {
  return launch_compact_from_ticket(lock_mask, B, N, active_idx, row_offsets, n_active, row_of_pos, scratch, first_ticket,
                                    dev_status, (cudaStream_t)stream);
}

int surelock_compact_noalloc(const uint8_t* lock_mask, int B, int N, int32_t* active_idx, int32_t* row_offsets,
                             int32_t* n_active, int32_t* row_of_pos, int32_t* dev_status, void* stream) {
  return launch_compact_noalloc(lock_mask, B, N, active_idx, row_offsets, n_active, row_of_pos, dev_status,
                                (cudaStream_t)stream);
}

int64_t surelock_compact_noalloc_max_flags(void) { return compact_noalloc_max_flags(); }

int surelock_kv_scatter(const void* k, const void* v, const int32_t* active_idx, const int32_t* n_active, int max_rows,
                        int row_elems, void* k_cache, void* v_cache, int dtype, void* stream) {
  if (!k || !v || !active_idx || !n_active || !k_cache || !v_cache || max_rows < 0 || row_elems <= 0) return SL_EINVAL;
  if (dtype != SL_BF16 && dtype != SL_FP32) return SL_EINVAL;
  return launch_kv_scatter(k, v, active_idx, n_active, max_rows, row_elems, k_cache, v_cache, dtype, (cudaStream_t)stream);
}

int surelock_softmax_kl_sure(const void* logits, const void* prev_logits, const int32_t* row_of_pos_prev,
                             const float* prev_lse, const int32_t* active_idx, const int32_t* n_active, int max_rows,
                             int vocab, int dtype, const uint8_t* mask_state, uint8_t* lock_mask, float kl_eps, float* kl,
                             float* conf, int32_t* argmax, float* lse_out, void* stream) {
  if (!logits || !n_active || !mask_state || !lock_mask || !kl || !conf || !argmax || max_rows < 0) return SL_EINVAL;
  if (!(kl_eps >= 0.f)) return SL_EINVAL;
  if (dtype != SL_BF16 && dtype != SL_FP32) return SL_EINVAL;
  return launch_softmax_kl_sure(logits, prev_logits, row_of_pos_prev, prev_lse, active_idx, n_active, max_rows, vocab,
                                dtype, mask_state, lock_mask, kl_eps, kl, conf, argmax, lse_out, (cudaStream_t)stream);
}

static size_t gemm_ws_tiles() { return 4 * (size_t)sm_count(); }
size_t surelock_gemm_workspace_bytes(void) { return gemm_ws_tiles() * (SPLIT_TILE_BYTES + 3 * sizeof(int)); }

int surelock_conf_gate_lock(const float* conf, const float* kl, const int32_t* active_idx, const int32_t* row_offsets,
                            int B, int N, const uint8_t* mask_state, uint8_t* lock_mask, float kl_eps, float m_percent,
                            float* theta_out, void* stream) {
  if (!conf || !kl || !active_idx || !row_offsets || !mask_state || !lock_mask || B <= 0 || N <= 0) return SL_EINVAL;
  if (!(kl_eps >= 0.f) || !(m_percent >= 0.f) || m_percent > 100.f) return SL_EINVAL;
  return launch_conf_gate_lock(conf, kl, active_idx, row_offsets, B, N, mask_state, lock_mask, kl_eps, m_percent,
                               theta_out, (cudaStream_t)stream);
}

int surelock_gemm(const void* A, const void* W, void* C, const int32_t* n_active, int max_rows, int n_out, int K,
                  int dtype, int impl, void* workspace, int32_t* dev_status, void* stream) {
  return surelock_gemm_fused(A, W, nullptr, C, n_active, max_rows, n_out, K, dtype, EPI_STORE, impl, workspace, dev_status,
                             stream);
}

int surelock_gemm_fused(const void* A, const void* W, const void* W2, void* C, const int32_t* n_active, int max_rows,
                        int n_out, int K, int dtype, int epilogue, int impl, void* workspace, int32_t* dev_status,
                        void* stream) {
  if (!A || !W || !C || !n_active || max_rows < 0 || n_out <= 0 || K <= 0) return SL_EINVAL;
  if (dtype != SL_BF16 && dtype != SL_FP32) return SL_EINVAL;
  if (epilogue != EPI_STORE && epilogue != EPI_RESIDUAL && epilogue != EPI_SWIGLU) return SL_EINVAL;
  if (epilogue == EPI_SWIGLU && !W2) return SL_EINVAL;
  if (epilogue != EPI_SWIGLU) W2 = nullptr;
  if (impl == 2)                                     // the weight-streaming kernel (bf16, at most 128 rows; no workspace)
    return dtype == SL_BF16 ? launch_gemm_stream(A, W, W2, C, n_active, max_rows, max_rows, n_out, K, epilogue, dev_status,
                                                 false, (cudaStream_t)stream)
                            : SL_EUNSUPPORTED;
  if (dtype == SL_BF16 && impl == 0) {
    SplitWs sw;
    if (workspace) {
      sw.tiles = (int)gemm_ws_tiles();
      sw.ws = reinterpret_cast<float*>(workspace);
      sw.counters = reinterpret_cast<int*>(reinterpret_cast<char*>(workspace) + gemm_ws_tiles() * SPLIT_TILE_BYTES);
    }
    const int rc = launch_gemm_tc(A, W, W2, C, n_active, max_rows, n_out, K, epilogue, dev_status, sw, (cudaStream_t)stream);
    if (rc != SL_EUNSUPPORTED) return rc;
  }
  return launch_gemm_simt(A, W, W2, C, n_active, max_rows, n_out, K, dtype, epilogue, (cudaStream_t)stream);
}

int surelock_update_mask(const float* conf, const int32_t* argmax, const int32_t* active_idx, const int32_t* row_offsets,
                         int B, int N, int lo, int hi, int k, int32_t mask_token, int32_t* tokens, uint8_t* mask_state,
                         int32_t* n_revealed, void* stream) {
  if (!conf || !argmax || !active_idx || !row_offsets || !tokens || !mask_state || B <= 0 || N <= 0 || lo < 0 ||
      hi < lo || hi > N || k < 0)
    return SL_EINVAL;
  return launch_update_mask(conf, argmax, active_idx, row_offsets, B, N, lo, hi, k, mask_token, tokens, mask_state,
                            n_revealed, (cudaStream_t)stream);
}

size_t surelock_attention_split_workspace_bytes(int B, int H, int head_dim) {
  if (B <= 0 || H <= 0 || head_dim <= 0) return 0;
  return (((size_t)B * H * sizeof(unsigned long long) + 255) & ~(size_t)255) + attention_split_workspace_bytes(head_dim);
}

int surelock_attention_split(const void* q, const void* k_cache, const void* v_cache, const int32_t* row_offsets,
                             int max_rows, int B, int N, int H, int head_dim, int splits, void* o, void* workspace,
                             int diag_skip, int32_t* dev_status, void* stream) {
  if (!q || !k_cache || !v_cache || !row_offsets || !o || !workspace || max_rows <= 0 || B <= 0 || N <= 0 || H <= 0 ||
      splits < 0)
    return SL_EINVAL;
  const int S = splits ? splits : attention_split_plan(B, N, H);
  if (S < 1) return SL_EUNSUPPORTED;
  if (diag_skip >= B * H * S) return SL_EINVAL;
  unsigned long long* counters = static_cast<unsigned long long*>(workspace);
  float* ws = reinterpret_cast<float*>(static_cast<char*>(workspace) +
                                       (((size_t)B * H * sizeof(unsigned long long) + 255) & ~(size_t)255));
  return launch_attention_split(q, k_cache, v_cache, row_offsets, max_rows, B, N, H, head_dim, S, o, ws, counters, dev_status,
                                diag_skip < 0 ? -1 : diag_skip, (cudaStream_t)stream);
}

int surelock_attention(const void* q, const void* k_cache, const void* v_cache, const int32_t* active_idx,
                       const int32_t* row_offsets, const int32_t* n_active, int max_rows, int B, int N, int H,
                       int head_dim, void* o, int dtype, int impl, int32_t* dev_status, void* stream) {
  if (!q || !k_cache || !v_cache || !active_idx || !n_active || !o || max_rows < 0 || B <= 0 || N <= 0 || H <= 0)
    return SL_EINVAL;
  if (dtype != SL_BF16 && dtype != SL_FP32) return SL_EINVAL;
  if (dtype == SL_BF16 && impl == 0 && row_offsets) {
    const int rc = launch_attention_tc(q, k_cache, v_cache, row_offsets, max_rows, B, N, H, head_dim, o, dev_status,
                                       (cudaStream_t)stream);
    if (rc != SL_EUNSUPPORTED) return rc;
  }
  return launch_attention_simt(q, k_cache, v_cache, active_idx, n_active, max_rows, N, H, head_dim, o, dtype,
                               (cudaStream_t)stream);
}

}  // extern "C"
