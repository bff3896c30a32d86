/*
 * surelock.h -- C ABI of the SureLock locked-forward hot path for NVIDIA B200 (sm_100a).
 *
 * SureLock ("Stopping Computation for Converged Tokens in Masked Diffusion-LM Decoding",
 * Algorithm 1) decodes a masked-diffusion LM while recomputing, at every step, only the M
 * positions of an N-token sequence that are not yet locked.  This library is one such step:
 * compaction of the active rows, RMSNorm / RoPE / QKV on those rows, scatter of their fresh
 * K/V into an N-length per-layer cache whose locked rows stay frozen, M x N bidirectional
 * attention, SwiGLU FFN and LM head on the M rows, and a fused softmax that computes each
 * active row's step-wise KL, applies the lock test and updates the lock mask.
 *
 * General rules
 *  - Every function returns 0 (SL_OK) or a negative surelock_status; nothing throws or exits.
 *  - "dev" pointers are CUDA device pointers, "host" pointers ordinary host memory.
 *  - Work is enqueued on the cudaStream_t passed (as void*) at init or to the call; calls do
 *    not synchronise with the host unless stated.
 *  - A device-side problem (a bounded wait that ran out, an index out of range) sets a sticky
 *    status word that surelock_status_poll() returns; kernels never trap.
 *  - There is no CPU fallback: every step of the path runs in the library's CUDA kernels.
 */
#ifndef SURELOCK_H
#define SURELOCK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SL_OK = 0,
  SL_EINVAL = -1,       /* null pointer, size out of range, negative or NaN threshold ...      */
  SL_ENOMEM = -2,       /* device allocation failed at init                                    */
  SL_ECUDA = -3,        /* a CUDA runtime call failed (sticky CUDA error)                      */
  SL_EDEVICE = -4,      /* a kernel reported a problem through the status word                 */
  SL_EUNSUPPORTED = -5, /* shape not supported by the kernels (e.g. head_dim not 64 or 128)    */
  SL_ELIMIT = -6        /* size beyond the fixed capacity of an allocation-free entry point    */
} surelock_status;

enum { SL_BF16 = 0, SL_FP32 = 1 };   /* storage type of weights, activations, caches and logits; accumulation is fp32 */

typedef struct surelock_ctx surelock_ctx;   /* opaque: owns caches, workspaces and previous logits */

/* Shape of the transformer (symbols of Sec. 2.3: L, d, H, d_h, H_kv, d_ff, vocabulary).
 * n_kv_heads must equal n_heads.  vocab may be 0: then there is no LM head and only
 * surelock_layer_step() can be used.  head_dim must be 64 or 128 and even. */
typedef struct {
  int32_t n_layers, d_model, n_heads, head_dim, n_kv_heads, d_ff, vocab;
  int32_t dtype;                 /* SL_BF16 or SL_FP32 */
  float rms_eps, rope_theta;
  int32_t mask_token_id;         /* informational; the caller writes it into `tokens` */
} surelock_model_cfg;

/* Weights: dev pointers, BORROWED (must outlive the ctx), element type cfg.dtype, every matrix row-major
 * [out_features][in_features].  The per-layer members are host arrays of n_layers dev pointers.
 * tok_emb [vocab][d], lm_head [vocab][d], norm gains [d], wq/wk/wv [H*d_h][d], wo [d][H*d_h],
 * w_gate/w_up [d_ff][d], w_down [d][d_ff].  With vocab == 0, tok_emb/lm_head/final_norm_g may be NULL. */
typedef struct {
  const void *tok_emb, *lm_head, *final_norm_g;
  const void *const *attn_norm_g, *const *wq, *const *wk, *const *wv, *const *wo;
  const void *const *ffn_norm_g, *const *w_gate, *const *w_up, *const *w_down;
} surelock_weights;

/* Results of a step: dev pointers into ctx-owned buffers, valid until the next step/reset/destroy.
 * Rows are PACKED: row r belongs to flat position active_idx[r] = b*N + i. */
typedef struct {
  const int32_t *active_idx;     /* [M] ascending flat positions of the unlocked rows (Algorithm 1 line 6)     */
  const int32_t *row_offsets;    /* [B+1] packed-row offset of each sequence; row_offsets[B] = M              */
  const int32_t *n_active;       /* [1] M                                                                      */
  const void *logits;            /* [M][vocab], cfg.dtype (Algorithm 1 line 15, before the softmax)            */
  const float *hidden;           /* [M][d] fp32, output of the last block (before the final norm)              */
  const float *kl;               /* [M] D = KL(p_t || p_{t-1}) in nats, +inf without a previous posterior      */
  const float *conf;             /* [M] max_v p_t(v) = 1 - u (Algorithm 1 line 18)                             */
  const int32_t *argmax;         /* [M] argmax_v p_t(v), lowest index on ties                                  */
} surelock_step_out;

/* ---- context ------------------------------------------------------------------------------------------- */

/* Allocate a context for sequences of exactly N tokens in batches of exactly `batch` sequences
 * (Algorithm 1 lines 1-2: lock-independent state = per-layer K/V caches and previous posteriors).
 * Allocates (cudaMalloc, on the current device) the K/V cache [L][2][B*N][H*d_h], packed workspaces for
 * M = B*N rows, two logit buffers [B*N][vocab] and index arrays; builds a rotary table.  The first call in a
 * process also raises kernel shared-memory limits.  Not asynchronous.  `cuda_stream` (a cudaStream_t, may be 0)
 * is the stream every later call of this ctx enqueues on. */
int surelock_init(surelock_ctx **out, const surelock_model_cfg *cfg, const surelock_weights *w,
                  int N, int batch, void *cuda_stream);

/* Forget the previous posteriors (p_{t-1} = None, so the next step's KL is +inf for every row: Algorithm 1
 * line 19), clear the device status word and the hand-over counters of the split-K GEMM (a kernel that gave up on a
 * bounded wait, device status 2, may have left them half-way), and zero the fallback count.  Cache contents are kept
 * (a caller may have pre-filled them). */
int surelock_reset(surelock_ctx *ctx);

/* One SureLock step (Algorithm 1 lines 6-15 and 18-24; the unmasking policy of line 16 is the caller's).
 *   tokens      dev int32 [B][N]   current sequence (mask positions hold the mask token id)
 *   mask_state  dev uint8 [B][N]   1 = masked.  The state the forward pass sees; a row can lock only if 0.
 *   lock_mask   dev uint8 [B][N]   in: locks entering the step (1 = locked; such rows are neither recomputed
 *                                  nor rewritten in the cache); out: rows passing D <= kl_eps are set to 1.
 *                                  Locking a row whose cache entries were never written is the caller's error.
 *   kl_eps      threshold eps >= 0 (not NaN)
 *   out         host struct filled with dev pointers (may be NULL)
 * Asynchronous; performs no allocation and never waits for the work it enqueues, nor for the previous step's.  (It
 * does wait for the step BEFORE the previous one to have finished, whose row count M, copied to the host, serves as
 * the upper bound of this step's M from which launch configurations are chosen: the host can run two steps ahead of
 * the GPU.  The bound affects speed only: every kernel reads M itself from device memory.) */
int surelock_step(surelock_ctx *ctx, const int32_t *tokens, const uint8_t *mask_state, uint8_t *lock_mask,
                  float kl_eps, surelock_step_out *out);

/* The same step for callers whose buffers live in HOST memory: copies tokens, mask_state and lock_mask to
 * ctx-owned device staging, runs surelock_step, copies back lock_mask (updated, [B][N]) and, for the M active
 * rows, kl / conf / argmax / active_idx (each array must have room for B*N entries; any may be NULL), stores
 * M in *n_active and synchronises the stream.  For best speed pass page-locked host memory. */
int surelock_step_host(surelock_ctx *ctx, const int32_t *tokens, const uint8_t *mask_state, uint8_t *lock_mask,
                       float kl_eps, int32_t *n_active, int32_t *active_idx, float *kl, float *conf,
                       int32_t *argmax);

/* One transformer block on the active rows (Algorithm 1 lines 6 and 10-13 for a single layer): compaction,
 * RMSNorm, QKV + RoPE, K/V scatter into this layer's cache, M x N attention, O-projection + residual,
 * RMSNorm, SwiGLU FFN + residual.
 *   hidden_in   dev [B][N][d] cfg.dtype; only rows of unlocked positions are read
 *   lock_mask   dev uint8 [B][N], read only
 *   hidden_out  dev fp32 [M][d] packed (room for B*N rows)
 *   out         host struct (may be NULL): active_idx, row_offsets, n_active are filled, the rest NULL
 * Asynchronous. */
int surelock_layer_step(surelock_ctx *ctx, int layer, const void *hidden_in, const uint8_t *lock_mask,
                        float *hidden_out, surelock_step_out *out);

/* ---- optional un-locking (paper App. "Optional Unlocking") ------------------------------------------------------
 * A locked position whose context has drifted may be returned to the active set.  Readings taken where the appendix
 * leaves a choice: the "budgeted proxy" is the step's own forward run on the LOCKED rows as queries against the caches
 * as they stand, without writing their K/V back; a position is un-locked when ALL three conditions of the printed
 * rule hold:  u~ > theta_t  AND  KL(p^_t || p_{t*}) > eps_unlock  AND  t - t* > d_interval,  where u~ = 1 - max p^_t,
 * p_{t*} is the posterior the position had in the step t* that locked it, and theta_t is, per sequence, the
 * m_percent-th percentile (linear interpolation) of u over the rows that were active in step t (a sequence without
 * active rows un-locks nothing).  An un-locked position is active from the next step on (its K/V are rewritten then),
 * cannot lock again for d_cool steps, and afterwards only under the threshold rho * kl_eps.  Positions the caller
 * locked by hand have no t* and are never un-locked. */
typedef struct {
  int period;          /* P: surelock_probe_unlock does its work after every P-th step, >= 1 */
  float eps_unlock;    /* drift threshold, >= 0 */
  int d_interval;      /* >= 0 */
  int d_cool;          /* >= 0 */
  float rho;           /* 0 <= rho <= 1 */
  float m_percent;     /* 0 ... 100 */
} surelock_unlock_params;

typedef struct {       /* dev pointers owned by the ctx, valid until the next probe; NULL when probed == 0 */
  int32_t step;                  /* t: number of the step just taken (1 = first step after a reset) */
  int32_t probed;                /* 1 if this call ran the probe (t is a multiple of P) */
  const int32_t *probed_idx;     /* [n] flat positions of the locked rows, ascending */
  const int32_t *n_probed;       /* [1] n */
  const float *drift;            /* [n] KL(p^_t || p_{t*}); +inf for a position without t* */
  const float *conf;             /* [n] max p^_t */
  const float *theta;            /* [B] theta_t */
  const int32_t *n_unlocked;     /* [1] */
  const int32_t *t_star;         /* [B*N] step that locked each position, -1 = none */
  const int32_t *cool_until;     /* [B*N] last step of the cool-down after an un-lock, -1 = none */
} surelock_probe_out;

/* Switch un-locking on (params != NULL) or off (NULL).  Switching it on allocates, once, a third logits buffer
 * [B*N][vocab] (the frozen posteriors p_{t*}, stored as logits; 3.1 GB at batch 8 x 1536 x vocab 126464) and a few
 * arrays of B*N entries, and calls surelock_reset().  While it is on, every surelock_step applies, per position, the
 * threshold rho * kl_eps after an earlier un-lock and the cool-down, and copies the logits of every row that locks
 * (one 2 * vocab byte row copy per lock).  Not part of surelock_state_export(). */
int surelock_set_unlocking(surelock_ctx *ctx, const surelock_unlock_params *params);

/* The probe, to be called after surelock_step (and after the caller has used that step's outputs: the packed
 * workspaces, `hidden` and the logits slot of the NEXT step are overwritten; kl / conf / argmax / active_idx of the
 * step stay valid).  Does nothing unless the number of the step just taken is a multiple of P.
 *   tokens     dev int32 [B][N]  the current sequence (after the caller's unmasking)
 *   lock_mask  dev uint8 [B][N]  in: the mask after the step's lock update; out: un-locked positions cleared
 * Asynchronous.  Costs one forward over the locked rows (queries only) plus two vocabulary sweeps per locked row. */
int surelock_probe_unlock(surelock_ctx *ctx, const int32_t *tokens, uint8_t *lock_mask, surelock_probe_out *out);

/* Synchronise the ctx stream and report: *device_status = 0, or the first code a kernel stored since the last
 * surelock_reset: 1 = the compaction's bounded look-back wait ran out, 2 = a bounded barrier wait of the tensor-core
 * GEMM ran out, 3 = the same in the attention kernel (in all three the kernel gave up and returned: the step's
 * results are invalid), 4 = a token id or row index read from device memory was out of range and was skipped,
 * 5 = with "check_cache" on, a position entered a step locked although its K/V were never written.
 * Returns SL_EDEVICE if non-zero, SL_ECUDA if the stream reported a CUDA error. */
int surelock_status_poll(surelock_ctx *ctx, int *device_status);

/* K/V cache of one layer (Algorithm 1 line 11: K^all / V^all): dev pointers to [B*N][H][d_h] arrays of
 * cfg.dtype, token-major (row b*N+i holds all heads of position i of sequence b, keys stored AFTER the rotary
 * embedding).  row_stride_elems = H*d_h.  For pre-filling and for parity checks. */
int surelock_kv_cache(surelock_ctx *ctx, int layer, void **k, void **v, size_t *row_stride_elems);

/* Previous-step logits (the stored form of p_{t-1}, Algorithm 1 line 2): *buf = dev [rows][vocab] cfg.dtype,
 * packed as the PREVIOUS step packed them; *row_of_pos = dev int32 [B*N], row of each flat position in *buf
 * or -1 when the position has no previous posterior.  Writing both lets a caller seed p_{t-1}. */
int surelock_prev_logits(surelock_ctx *ctx, void **buf, int32_t **row_of_pos);

/* Checkpoint / resume of a decoding run (the paper has no counterpart; the sampler state it lists in Algorithm 1's
 * "Require" and lines 1-3 is the lock mask, the cache C and p_{t-1}; the lock mask, tokens and mask state are the
 * caller's).  surelock_state_export writes what the ctx holds between two steps into a HOST buffer: a header (model
 * shape, N, batch, element type, rows of the last step, and the row counts of the last two steps, from which the next
 * two steps take the bound that selects their kernels), the K/V cache of every layer, and the previous step's logits,
 * their log-sum-exps and position -> row table.  surelock_state_import loads such a buffer into a ctx created with the
 * same model shape, N, batch and element type (weights are not part of the state); the next surelock_step then
 * continues bit for bit as the exporting ctx would have.  Both calls synchronise the ctx stream.
 *   surelock_state_bytes: capacity that always suffices for this ctx (the export usually writes less: only the rows
 *   of the last step's logits are stored).
 * Returns SL_EINVAL on NULL / too small a buffer / a buffer that is not a state of this shape, SL_ECUDA on a failed copy. */
size_t surelock_state_bytes(const surelock_ctx *ctx);
int surelock_state_export(surelock_ctx *ctx, void *host_dst, size_t capacity, size_t *written);
int surelock_state_import(surelock_ctx *ctx, const void *host_src, size_t bytes);

/* Optional confidence gate (Algorithm 1 lines 18, 21, 23; Sec. 2.2): with 0 <= m_percent <= 100 every later
 * surelock_step locks a candidate (active, unmasked row) only if, besides D <= kl_eps, its uncertainty
 * u = 1 - max_v p(v) is <= theta_m, the m-th percentile (linear interpolation between order statistics) of u over
 * the candidates of ITS sequence; a sequence without candidates locks nothing.  The paper's runs use m = 20.
 * A negative m_percent (or NaN) switches the gate off (the default: the KL criterion alone).  N must be <= 8192
 * while the gate is on.  *theta (may be NULL) receives a dev pointer to the B thresholds of the last step. */
int surelock_set_confidence_gate(surelock_ctx *ctx, float m_percent, const float **theta);

/* Tuning / test switches.  "gemm_impl": 0 = tensor-core GEMM and attention when the shape allows (default),
 * 1 = force the CUDA-core kernels.  "strict_tc": 1 = a bf16 contraction or attention whose shape the tensor-core
 * kernels do not take makes the step return SL_EUNSUPPORTED instead of running on the CUDA-core kernels (0, the
 * default, falls back and counts it: surelock_last_fallback_count()).  "time_kernels": 1 creates an event pool (once) and brackets every launch of
 * later steps with CUDA events for surelock_kernel_times().  "trace_layers": 1 allocates (once, here, not in the
 * step) a buffer [2L+1][B*N][d] fp32 and makes every later surelock_step copy the packed residual stream into it:
 * slot 2l = input of block l (slot 0 = the embeddings), slot 2l+1 = after the attention sub-block of block l,
 * slot 2L = output of the last block; for stage-wise parity checks.  "have_prev": 1 declares the buffers returned by surelock_prev_logits() valid
 * (after a caller seeded them), 0 forgets them.  "check_cache": checks, at the start of every later surelock_step, the
 * one precondition the host cannot see: a position that enters the step locked must have K/V in the caches (Algorithm 1
 * line 12 attends to them), i.e. it was active in an earlier step since the last reset / this call, or the caller
 * filled the caches.  1 = on, no position valid yet; 2 = on, every position declared valid (after a pre-fill through
 * surelock_kv_cache()); 0 = off (default).  A violation stores device status 5 and the step goes on; one small kernel
 * per step, one flag byte per position (allocated here).  surelock_reset() invalidates all positions,
 * surelock_state_import() validates all.  surelock_layer_step() neither checks nor marks.
 *  "gemm_stream": 1 = steps whose bound on the number of
 * active rows is at most 128 run their contractions on the weight-streaming kernel (see surelock_gemm, impl 2); 0
 * (default) = always the general kernel, which measured as fast or faster inside a step.  "layer_chain": with few active rows a bf16 step runs, per layer, the output projection, the SwiGLU
 * FFN and the next layer's Q/K/V projections as ONE persistent kernel that keeps the weight stream running across them
 * (RMSNorms folded in; cooperative launch, one CTA per SM): 1 (default) = when the bound on the number of active rows is
 * at most 128, 0 = never (one kernel per contraction).  "attn_split": 1 (default) = in a bf16 step whose bound on the
 * number of active rows is at most 128, and when batch x heads x 2 CTAs fit the GPU at one per SM, attention runs with the
 * keys of every (sequence, head) split over several CTAs, which meet in a workspace (allocated at init); 0 = never.  "row_bound": v > 0 = the
 * caller's upper bound of the number of active rows of later steps, used instead of the automatic one (the row count
 * two steps back); a bound that is too small costs time, never correctness (the weight-streaming kernel then makes
 * several passes over the weights); 0 = automatic (default).  "debug_chain_skip_barrier": v > 0 = failure-detection
 * diagnostic, consumed by the NEXT launch of the layer chain kernel only: CTA v - 1 does not arrive at that launch's
 * first grid barrier, so the bounded wait (about 1 s) of all other CTAs runs out, every role of every CTA leaves, the
 * kernel returns and device status 2 is reported; the step's results are invalid, nothing hangs or traps, and after
 * surelock_reset() the ctx works as before.  Unknown names return SL_EINVAL. */
int surelock_set_option(surelock_ctx *ctx, const char *name, int value);

/* The layer trace written by steps run with "trace_layers" on: *buf = dev fp32 [2L+1][B*N][d] (rows packed as in
 * that step), *layer_stride_elems = B*N*d.  SL_EINVAL if tracing was never switched on. */
int surelock_layer_trace(surelock_ctx *ctx, float **buf, size_t *layer_stride_elems);

/* Number of kernels the last surelock_step / surelock_layer_step call launched (host-side count). */
int surelock_last_launch_count(surelock_ctx *ctx);

/* Number of launches since the last surelock_reset in which a bf16 ctx with "gemm_impl" 0 ran a CUDA-core kernel
 * because the tensor-core kernel does not take the shape (host-side count; 0 for every benchmark configuration). */
int surelock_last_fallback_count(surelock_ctx *ctx);

/* Which of the kernels for few active rows the last surelock_step / surelock_layer_step call launched (host-side
 * flags): bit 0 = the layer chain kernel ("layer_chain"), bit 1 = attention with the keys of a (sequence, head) split
 * over several CTAs ("attn_split"). */
int surelock_last_step_paths(surelock_ctx *ctx);

/* Per-kernel-class device time of the LAST step, measured with CUDA events on the ctx stream; needs
 * surelock_set_option(ctx, "time_kernels", 1) before that step (events add a few microseconds per launch, so time
 * whole steps with the option off).  Synchronises the stream.  ms[i], launches[i] (may be NULL) for class i:
 * 0 compaction, 1 embedding/row gather, 2 RMSNorm, 3 QKV GEMM, 4 RoPE, 5 K/V scatter, 6 attention, 7 O-proj GEMM,
 * 8 gate/up GEMM + SwiGLU, 9 down GEMM, 10 LM-head GEMM, 11 softmax-KL-lock, 12 confidence gate.  n_classes >= 13. */
#define SURELOCK_KERNEL_CLASSES 13
int surelock_kernel_times(surelock_ctx *ctx, float *ms, int32_t *launches, int n_classes);

void surelock_destroy(surelock_ctx *ctx);
const char *surelock_strerror(int status);

/* ---- single stages (same kernels the step uses; for stage-wise parity and for timing them alone) -------- */

/* Bytes of zero-initialisable scratch surelock_compact needs for `total` flags. */
size_t surelock_compact_scratch_bytes(int64_t total);

/* Active-row compaction (Algorithm 1 line 6): A_t = { i : lock_i = 0 } for B sequences of N flags.
 *   lock_mask  dev uint8 [B*N]
 *   active_idx dev int32 [>= number of zeros]  ascending flat positions b*N+i
 *   row_offsets dev int32 [B+1]                exclusive per-sequence offsets, [B] = M
 *   n_active   dev int32 [1]                   M
 *   row_of_pos dev int32 [B*N] or NULL         packed row of each position, -1 for locked positions
 *   scratch    dev, surelock_compact_scratch_bytes(B*N) bytes; cleared by this call (cudaMemsetAsync)
 *   dev_status dev int32 [1] or NULL           set non-zero if a bounded wait ran out
 * B*N < 2^31.  Asynchronous on `stream`. */
int surelock_compact(const uint8_t *lock_mask, int B, int N, int32_t *active_idx, int32_t *row_offsets,
                     int32_t *n_active, int32_t *row_of_pos, void *scratch, int32_t *dev_status, void *stream);

/* Diagnostic for the failure-detection path of the compaction (no counterpart in the paper).  Same arguments as
 * surelock_compact plus `first_ticket`: the launch's chunk tickets start there instead of at 0, as if that many chunks
 * belonged to CTAs that never publish their counts.  With first_ticket = 1 every chunk that runs waits for chunk 0's
 * count, which nobody writes: each CTA polls up to its bound (about 70 ms), stores device status 1 in *dev_status
 * and returns; nothing hangs, faults or traps, outputs are left unspecified.  first_ticket = 0 is surelock_compact.
 * The mbarrier waits of the tensor-core kernels are bounded the same way (about 2 s; device status 2 / 3). */
int surelock_compact_from_ticket(const uint8_t *lock_mask, int B, int N, int32_t *active_idx, int32_t *row_offsets,
                                 int32_t *n_active, int32_t *row_of_pos, void *scratch, uint32_t first_ticket,
                                 int32_t *dev_status, void *stream);

/* Compaction for callers that must not allocate device memory.  (No counterpart in the paper: this is a
 * packaging variant of surelock_compact, same kernel, same results.)
 *
 * Who needs it: code that is handed its input and output buffers but may not call cudaMalloc itself -- a plug-in
 * running inside someone else's serving process whose memory was all reserved up front by that process's pool
 * allocator, or a latency-critical loop in which cudaMalloc's implicit device-wide synchronisation is not
 * acceptable.  Such a caller cannot provide the scratch words surelock_compact asks for, so here they live in a
 * fixed array that is part of the library image: 32,784 bytes of device memory on every GPU that loads the
 * library, held until the process exits.  That fixes the capacity: B*N <= 16,777,216 flags (4096 chunks of 4096);
 * larger inputs are refused with SL_ELIMIT and nothing is launched.
 *
 * Arguments and results are exactly those of surelock_compact minus `scratch`.  The call performs no cudaMalloc,
 * cudaFree or other allocating call; it enqueues one cudaMemsetAsync (the array keeps the previous call's
 * contents, so the words this call uses are cleared first) and one kernel on `stream`.
 * The FIRST call on each device also asks the CUDA runtime for the array's device address (with that device
 * current) and caches it for the life of the process; make that first call outside any stream capture.  The cached
 * address does not survive cudaDeviceReset() or the destruction of the device's primary context: a process that does
 * either must not call this entry point on that device afterwards.
 * All calls on a device share the one array: two calls whose kernels may overlap on the GPU (different streams,
 * or different host threads) race on it and give wrong results -- serialise them. */
int surelock_compact_noalloc(const uint8_t *lock_mask, int B, int N, int32_t *active_idx, int32_t *row_offsets,
                             int32_t *n_active, int32_t *row_of_pos, int32_t *dev_status, void *stream);

/* Capacity of surelock_compact_noalloc in flags (B*N). */
int64_t surelock_compact_noalloc_max_flags(void);

/* K/V cache scatter (Algorithm 1 line 11, K^all[A_t] <- K[A_t]): cache row active_idx[r] <- packed row r, for
 * r < *n_active; other cache rows are not touched.  k, v: dev [M][row_elems]; k_cache, v_cache: dev
 * [B*N][row_elems]; dtype SL_BF16 or SL_FP32; row_elems*sizeof(elem) must be a multiple of 16. */
int surelock_kv_scatter(const void *k, const void *v, const int32_t *active_idx, const int32_t *n_active,
                        int max_rows, int row_elems, void *k_cache, void *v_cache, int dtype, void *stream);

/* Fused softmax + step-wise KL + confidence + argmax + lock test + lock update (Algorithm 1 lines 15, 18-20,
 * 23-24 with the confidence gate off), for rows r < *n_active:
 *   p = softmax(logits[r]); conf[r] = max p; argmax[r]; pr = prev_row[...]:
 *   kl[r] = sum_v p(v) (log p(v) - log q(v)) with q = softmax(prev_logits[pr]), or +inf when pr < 0;
 *   if mask_state[pos] == 0 and kl[r] <= kl_eps: lock_mask[pos] = 1      (pos = active_idx[r])
 *   logits      dev [M][vocab] dtype        prev_logits dev [*][vocab] dtype
 *   row_of_pos_prev dev int32 [B*N]: row of position pos in prev_logits, or -1 (NULL: row r pairs with row r)
 *   prev_lse    dev fp32 [rows of prev_logits] log-sum-exp of each previous row as an earlier call's lse_out
 *               produced it, or NULL: then it is recomputed here from prev_logits
 *   active_idx  dev int32 [M] (NULL: pos = r)      mask_state dev uint8 [B*N]     lock_mask dev uint8 [B*N]
 *   kl, conf dev fp32 [M]; argmax dev int32 [M]; lse_out dev fp32 [M] or NULL (log-sum-exp of logits[r]).
 * vocab*sizeof(elem) must be a multiple of 16.  prev_logits == NULL means "no previous posterior at all". */
int surelock_softmax_kl_sure(const void *logits, const void *prev_logits, const int32_t *row_of_pos_prev,
                             const float *prev_lse, const int32_t *active_idx, const int32_t *n_active, int max_rows,
                             int vocab, int dtype, const uint8_t *mask_state, uint8_t *lock_mask, float kl_eps,
                             float *kl, float *conf, int32_t *argmax, float *lse_out, void *stream);

/* The confidence gate alone (the kernel surelock_step runs when the gate is on): for each of the B sequences,
 * theta = m-th percentile of u = 1 - conf over rows r in [row_offsets[b], row_offsets[b+1]) with
 * mask_state[active_idx[r]] == 0; then lock_mask[active_idx[r]] = 1 for those rows with u <= theta and
 * kl[r] <= kl_eps.  conf, kl: dev fp32 [M]; theta_out: dev fp32 [B] or NULL.  N <= 8192. */
int surelock_conf_gate_lock(const float *conf, const float *kl, const int32_t *active_idx, const int32_t *row_offsets,
                            int B, int N, const uint8_t *mask_state, uint8_t *lock_mask, float kl_eps, float m_percent,
                            float *theta_out, void *stream);

/* UpdateMASK (Algorithm 1 line 16) on the device: the confidence-ordered unmasking policy the paper describes for
 * masked-diffusion samplers (a fixed number of masked positions with the highest posterior probability become concrete
 * tokens each step), restricted to the semi-autoregressive block [lo, hi) (Sec. 4 set-up).  The Algorithm leaves the
 * policy to the sampler; this call is the one the decoding harness uses between two surelock_step calls, so that a
 * decoding loop needs no host round-trip.
 * For each of the B sequences: among the positions lo <= n < hi with mask_state == 1, the k with the largest conf
 * (ties: lowest position) get tokens[b][n] = argmax of that row (0 when that is mask_token) and mask_state[b][n] = 0.
 *   conf        dev fp32  [M]   max_v p(v) per packed row (surelock_step_out.conf)
 *   argmax      dev int32 [M]   (surelock_step_out.argmax)
 *   active_idx  dev int32 [M], row_offsets dev int32 [B+1]: the packing of the step that produced conf / argmax
 *   tokens      dev int32 [B][N], mask_state dev uint8 [B][N]: updated in place
 *   n_revealed  dev int32 [B] or NULL: how many positions of each sequence were revealed (< k when fewer were masked)
 * Masked positions are never locked, so every masked position of the block has a row.  0 <= lo <= hi <= N, k >= 0.
 * Returns SL_EINVAL on bad arguments, SL_ECUDA on a launch failure.  Asynchronous on `stream`. */
int surelock_update_mask(const float *conf, const int32_t *argmax, const int32_t *active_idx, const int32_t *row_offsets,
                         int B, int N, int lo, int hi, int k, int32_t mask_token, int32_t *tokens, uint8_t *mask_state,
                         int32_t *n_revealed, void *stream);

/* Bytes of workspace that lets surelock_gemm split K when M is small (see below). */
size_t surelock_gemm_workspace_bytes(void);

/* Dense contraction on packed rows, C[r][n] = sum_k A[r][k] * W[n][k] for r < *n_active (the projections of
 * Algorithm 1 lines 10, 12, 15; FLOP terms of Sec. 2.3).  A: dev [M][K]; W: dev [n_out][K]; C: dev [M][n_out];
 * A, W, C of `dtype`; fp32 accumulation.  impl: 0 = best available (tcgen05 tensor cores for SL_BF16 when the
 * shape allows), 1 = force the CUDA-core kernel, 2 = the weight-streaming tensor-core kernel for few rows (SL_BF16 and
 * max_rows <= 128 only, else SL_EUNSUPPORTED; weights on the 128-row side of the MMA, K split inside a thread-block
 * cluster; needs no workspace).
 * workspace: dev, surelock_gemm_workspace_bytes() bytes, ZERO-FILLED by the caller before its first use (the kernel
 * leaves it reusable, unless it gave up on a bounded wait: after device status 2 zero-fill it again), or NULL.  With a workspace and few output tiles (small M) the tensor-core kernel splits K
 * across SMs and sums the partial tiles in a fixed order (deterministic); without one it never splits.
 * dev_status as for surelock_compact. */
int surelock_gemm(const void *A, const void *W, void *C, const int32_t *n_active, int max_rows, int n_out, int K,
                  int dtype, int impl, void *workspace, int32_t *dev_status, void *stream);

/* The same contraction with the fused epilogues of the transformer block (Sec. 2.3: the output / down projections
 * feed the residual stream, the gate and up projections feed SwiGLU), for stage-wise parity checks and timing:
 *   epilogue 1: C is the fp32 residual stream, dev float [M][n_out]: C[r][n] += sum_k A[r][k] W[n][k]
 *   epilogue 2: C[r][n] = silu(sum_k A[r][k] W[n][k]) * (sum_k A[r][k] W2[n][k]), C of `dtype`; W2: dev [n_out][K]
 *   epilogue 0: surelock_gemm (W2 ignored)
 * Other arguments as for surelock_gemm; rows >= *n_active of C are not touched.  SL_EINVAL for an unknown epilogue or a
 * missing W2. */
int surelock_gemm_fused(const void *A, const void *W, const void *W2, void *C, const int32_t *n_active, int max_rows,
                        int n_out, int K, int dtype, int epilogue, int impl, void *workspace, int32_t *dev_status,
                        void *stream);

/* M x N bidirectional attention of the packed queries against the whole cache (Algorithm 1 line 12; Sec. 2.1: the
 * packed active queries attend to all N cached keys and values of their sequence): for packed row r at flat position
 * active_idx[r] = b*N+i and every head h, o[r][h] = softmax_j(q[r][h] . K[b*N+j][h] / sqrt(d_h)) V[b*N+j][h],
 * j = 0..N-1.  q, o: dev [M][H][d_h]; k_cache, v_cache: dev [B*N][H][d_h]; all of `dtype`. */
int surelock_attention(const void *q, const void *k_cache, const void *v_cache, const int32_t *active_idx,
                       const int32_t *row_offsets, const int32_t *n_active, int max_rows, int B, int N, int H,
                       int head_dim, void *o, int dtype, int impl, int32_t *dev_status, void *stream);

/* The same attention for FEW query rows (bf16; every sequence should have at most 128 packed rows, more cost further
 * passes), with the keys of every (sequence, head) split over `splits` CTAs that leave partial results in `workspace` and
 * meet there (see "attn_split" of surelock_set_option; this is the kernel a step then runs).  splits = 0 chooses the
 * number as a step would; B * H * splits must not exceed the number of SMs and splits must not exceed 8 nor the number of
 * 128-key blocks (SL_EUNSUPPORTED otherwise, also for head_dim other than 64 / 128 or pointers that are not 16-byte
 * aligned).  workspace: dev, surelock_attention_split_workspace_bytes(B, H, head_dim) bytes, ZEROED by the caller before
 * its first use (it begins with one 64-bit counter per (sequence, head) that only grows; calls with different numbers of
 * splits may follow one another on it) and not shared between streams.
 * diag_skip: -1 in normal use.  >= 0 is a failure-detection diagnostic: CTA number diag_skip (< B * H * splits) does not
 * arrive at the meeting of its (sequence, head), so the bounded wait (~0.2 s) of its siblings runs out: they store
 * device status 3 (see surelock_status_poll) in *dev_status and the kernel returns with o of that pair undefined; nothing hangs or traps; zero
 * the workspace again before the next use.  Asynchronous on `stream`. */
size_t surelock_attention_split_workspace_bytes(int B, int H, int head_dim);
int surelock_attention_split(const void *q, const void *k_cache, const void *v_cache, const int32_t *row_offsets,
                             int max_rows, int B, int N, int H, int head_dim, int splits, void *o, void *workspace,
                             int diag_skip, int32_t *dev_status, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SURELOCK_H */
