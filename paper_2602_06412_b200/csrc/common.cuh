// Shared declarations of the SureLock CUDA library (internal; the public interface is include/surelock.h).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "surelock.h"

// Device status codes stored (first writer wins) in the ctx status word.
enum {
  SL_DEV_OK = 0,
  SL_DEV_COMPACT_TIMEOUT = 1,   // decoupled look-back of the compaction gave up waiting for a predecessor chunk
  SL_DEV_GEMM_TIMEOUT = 2,      // an mbarrier wait in the tcgen05 GEMM ran out
  SL_DEV_ATTN_TIMEOUT = 3,      // an mbarrier wait in the tcgen05 attention ran out
  SL_DEV_BAD_INDEX = 4,         // an index read from device memory was out of range and was skipped
  SL_DEV_STALE_CACHE = 5        // "check_cache" is on and a position entered a step locked without valid K/V
};

// A failing CUDA runtime call makes the entry point return SL_ECUDA; with SURELOCK_DEBUG set in the environment the
// call site and the runtime's message are also written to stderr.
#define SL_CUDA_TRY(expr)                                                                              \
  do {                                                                                                 \
    cudaError_t e__ = (expr);                                                                          \
    if (e__ != cudaSuccess) {                                                                          \
      if (getenv("SURELOCK_DEBUG"))                                                                    \
        fprintf(stderr, "surelock: %s:%d: %s: %s\n", __FILE__, __LINE__, #expr, cudaGetErrorString(e__)); \
      return SL_ECUDA;                                                                                 \
    }                                                                                                  \
  } while (0)

namespace sl {

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// 2^x in one MUFU instruction (relative error 2^-22; flushes denormals)
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void set_status(int32_t* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

// ---- programmatic dependent launch ------------------------------------------------------------------------------------
// The kernels of a step run back to back on one stream.  Launched with the programmatic-serialization attribute, a
// kernel may start while its predecessor is still draining: everything it does before griddep_wait() (barrier set-up,
// tensor-memory allocation, in the GEMM the first weight copies, which depend on no earlier kernel) overlaps the
// predecessor's tail and the launch latency.  griddep_wait() returns once the predecessor grid has completed and its
// writes are visible; griddep_launch() (always after the wait, so at most two kernels are in flight) lets the successor
// start.  Both are no-ops in a kernel launched without the attribute.  SURELOCK_PDL=0 in the environment switches the
// attribute off.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

inline bool pdl_enabled() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("SURELOCK_PDL");
    v = (e && e[0] == '0') ? 0 : 1;
  }
  return v != 0;
}

// <<<grid, block, smem, st>>> with the programmatic-serialization attribute; only for kernels that call griddep_wait()
// before they touch anything an earlier kernel wrote.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

inline int sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (n <= 0) n = 148;
  }
  return n;
}

// ---- launchers (one per kernel family); all asynchronous on `st`, rows beyond *n_active are not touched ----

size_t compact_scratch_bytes(int64_t total);
int launch_compact(const uint8_t* lock, int B, int N, int32_t* idx, int32_t* row_offsets, int32_t* n_active,
                   int32_t* row_of_pos, void* scratch, int32_t* status, cudaStream_t st);

int launch_compact_from_ticket(const uint8_t* lock, int B, int N, int32_t* idx, int32_t* row_offsets, int32_t* n_active,
                               int32_t* row_of_pos, void* scratch, unsigned first_ticket, int32_t* status, cudaStream_t st);
long long compact_noalloc_max_flags();
int launch_compact_noalloc(const uint8_t* lock, int B, int N, int32_t* idx, int32_t* row_offsets, int32_t* n_active,
                           int32_t* row_of_pos, int32_t* status, cudaStream_t st);

// x[r] = table[tokens[idx[r]]] (embedding) or x[r] = src[idx[r]] (tokens == nullptr), widened to fp32
int launch_gather_rows(const void* table, const int32_t* tokens, const int32_t* idx, const int32_t* n_active,
                       int max_rows, int d, int table_rows, float* x, int dtype, int32_t* status, cudaStream_t st);
int launch_rmsnorm(const float* x, const void* gain, void* h, const int32_t* n_active, int max_rows, int d,
                   float eps, int dtype, cudaStream_t st);
// xg = bf16(x * gain) and ssq[r][d / 32] = sums of squares of x per 32-column chunk (bf16 models; rowops.cu)
int launch_norm_prep(const float* x, const void* gain, void* xg, float* ssq, const int32_t* n_active, int max_rows, int d,
                     cudaStream_t st);
int build_rope_table(float2* table, int N, int head_dim, float theta, cudaStream_t st);
// in-place rotation of q and k [M][H][dh] with position idx[r] % N
int launch_rope(void* q, void* k, const int32_t* idx, const int32_t* n_active, int max_rows, int N, int H,
                int head_dim, const float2* table, int dtype, cudaStream_t st);
int launch_kv_scatter(const void* k, const void* v, const int32_t* idx, const int32_t* n_active, int max_rows,
                      int row_elems, void* kc, void* vc, int dtype, cudaStream_t st);

enum GemmEpilogue {
  EPI_STORE = 0,      // C[T] = acc
  EPI_RESIDUAL = 1,   // Cf32 += acc
  EPI_SWIGLU = 2      // C[T] = silu(acc(W)) * acc(W2)
};
// C = A[M][K] . W[n_out][K]^T on CUDA cores (fp32 FMA); W2 only for EPI_SWIGLU
int launch_gemm_simt(const void* A, const void* W, const void* W2, void* C, const int32_t* n_active, int max_rows,
                     int n_out, int K, int dtype, int epilogue, cudaStream_t st);

int launch_attention_simt(const void* q, const void* kc, const void* vc, const int32_t* idx, const int32_t* n_active,
                          int max_rows, int N, int H, int head_dim, void* o, int dtype, cudaStream_t st);

int launch_softmax_kl_sure(const void* logits, const void* prev_logits, const int32_t* row_of_pos_prev,
                           const float* prev_lse, const int32_t* idx, const int32_t* n_active, int max_rows, int vocab,
                           int dtype, const uint8_t* mask_state, uint8_t* lock_mask, float kl_eps, float* kl,
                           float* conf, int32_t* argmax, float* lse_out, cudaStream_t st, bool apply_lock = true,
                           const float4* lse_part = nullptr, int part_tiles = 0, int part_rows = 0,
                           const int* lse_valid = nullptr);   // lse_part: per-tile softmax statistics left by the LM head
int launch_conf_gate_lock(const float* conf, const float* kl, const int32_t* idx, const int32_t* row_offsets, int B, int N,
                          const uint8_t* mask_state, uint8_t* lock_mask, float kl_eps, float m_percent, float* theta_out,
                          cudaStream_t st, bool apply_lock = true, bool all_rows = false, float empty_theta = -INFINITY);

// the contractions of a layer between two attention calls as one persistent kernel (gemm_chain.cu), bf16, few rows
struct ChainLaunch {
  const void *attn, *wo, *wg, *wu, *wd, *wq, *wk, *wv;   // wq == nullptr: no Q/K/V phase; wo == nullptr: ONLY that phase
  float* x;
  void *xg, *act;
  const void *gain_ffn, *gain_next;
  float *ssq_ffn, *ssq_next;
  void *q, *kc, *vc;
  const int32_t* idx;
  const float2* rope;
  float* ws;
  unsigned* bar;
  unsigned* bar_base;          // host-side count of launches since the barrier counter was last zeroed
  const int32_t* n_active;
  int32_t* status;
  int diag_skip;               // -1, or the CTA that skips its first grid barrier (failure-detection test)
  float *trace_mid, *trace_out;
  int max_rows, m_bound, d, F, hd, dh, n_seq;
  float rms_eps;
};
int launch_gemm_chain(const ChainLaunch& L, cudaStream_t st);   // SL_EUNSUPPORTED when the shapes do not fit
size_t gemm_chain_workspace_bytes(int np_max);

// optional un-locking (unlock.cu)
int launch_invert_mask(const uint8_t* lock, uint8_t* inv, int total, cudaStream_t st);
int launch_lock_commit(const float* kl, const float* conf, const float* lse, const int32_t* idx, const int32_t* n_active,
                       int max_rows, int N, const uint8_t* mask_state, uint8_t* lock_mask, float kl_eps, float rho, int t,
                       const float* theta, const int32_t* cool_until, const uint8_t* relock, int32_t* t_star,
                       int32_t* frozen_rop, float* frozen_lse, const void* logits, void* frozen, size_t row_bytes,
                       cudaStream_t st);
int launch_unlock(const float* drift, const float* conf, const int32_t* idx, const int32_t* n_probe, int max_rows, int N,
                  const float* theta, float eps_unlock, int d_interval, int d_cool, int t, const int32_t* t_star,
                  int32_t* cool_until, uint8_t* relock, uint8_t* lock_mask, int32_t* n_unlocked, cudaStream_t st);

// step precondition check (cache_check.cu): locked positions need kv_valid, active ones become valid
int launch_cache_check(const uint8_t* lock, uint8_t* kv_valid, int total, int32_t* status, cudaStream_t st);

int launch_update_mask(const float* conf, const int32_t* argmax, const int32_t* idx, const int32_t* row_offsets, int B,
                       int N, int lo, int hi, int k, int32_t mask_token, int32_t* tokens, uint8_t* mask_state,
                       int32_t* n_revealed, cudaStream_t st);

}  // namespace sl
