// Optional confidence gate of the lock test (Algorithm 1 lines 18, 21, 23; Sec. 2.2 "Optional: Confidence gate").
// u = 1 - max_v p(v).  Per sequence, theta_m = m-th percentile (linear interpolation between order statistics) of u
// over the locking candidates Z_t = active and unmasked rows of that sequence; a candidate locks when
// u <= theta_m and D <= eps.  One CTA per sequence: the candidates' u are gathered into shared memory, sorted there
// (bitonic network), theta is interpolated, and the lock mask is updated.  Runs after the softmax-KL kernel, which in
// this mode computes kl / conf but leaves the lock mask alone.
#include "common.cuh"

namespace sl {

constexpr int CG_THREADS = 1024;
constexpr int CG_MAX_N = 8192;    // rows of one sequence that fit the shared-memory sort

__global__ void __launch_bounds__(CG_THREADS)
conf_gate_lock_kernel(const float* __restrict__ conf, const float* __restrict__ kl, const int32_t* __restrict__ idx,
                      const int32_t* __restrict__ row_offsets, const uint8_t* __restrict__ mask_state,
                      uint8_t* __restrict__ lock_mask, float kl_eps, float m_percent, float* __restrict__ theta_out,
                      int apply_lock, int all_rows, float empty_theta) {
  // apply_lock = 0: only the thresholds are computed (the caller applies them).  all_rows = 1: the percentile is taken
  // over every active row of the sequence, masked or not (the reference uncertainty of the un-lock rule, App.
  // "Optional Unlocking"); empty_theta is what a sequence without any such row gets.
  extern __shared__ float s_u[];            // [pow2 >= candidates], padded with +inf
  __shared__ int s_n;
  __shared__ float s_theta;
  const int b = blockIdx.x;
  const int r0 = row_offsets[b], r1 = row_offsets[b + 1];
  const int rows = r1 - r0;
  if (threadIdx.x == 0) s_n = 0;
  __syncthreads();
  // gather u of the candidates (order is irrelevant: they get sorted)
  for (int i = threadIdx.x; i < rows; i += CG_THREADS) {
    const int r = r0 + i;
    if (all_rows || mask_state[idx[r]] == 0) s_u[atomicAdd(&s_n, 1)] = 1.f - conf[r];
  }
  __syncthreads();
  const int n = s_n;
  int p2 = 1;
  while (p2 < n) p2 <<= 1;
  for (int i = n + threadIdx.x; i < p2; i += CG_THREADS) s_u[i] = INFINITY;
  __syncthreads();
  for (int k = 2; k <= p2; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = threadIdx.x; i < p2; i += CG_THREADS) {
        const int ixj = i ^ j;
        if (ixj > i) {
          const float a = s_u[i], c = s_u[ixj];
          const bool up = (i & k) == 0;
          if ((a > c) == up) {
            s_u[i] = c;
            s_u[ixj] = a;
          }
        }
      }
      __syncthreads();
    }
  }
  if (threadIdx.x == 0) {
    float theta = empty_theta;               // no candidates (gate: -inf, nothing passes)
    if (n > 0) {
      const float h = (float)(n - 1) * (m_percent * 0.01f);
      int lo = (int)floorf(h);
      if (lo > n - 1) lo = n - 1;
      if (lo < 0) lo = 0;
      const int hi = lo + 1 < n ? lo + 1 : n - 1;
      theta = s_u[lo] + (h - (float)lo) * (s_u[hi] - s_u[lo]);
    }
    s_theta = theta;
    if (theta_out) theta_out[b] = theta;
  }
  __syncthreads();
  const float theta = s_theta;
  if (!apply_lock) return;
  for (int i = threadIdx.x; i < rows; i += CG_THREADS) {
    const int r = r0 + i, pos = idx[r];
    if (mask_state[pos] == 0 && (1.f - conf[r]) <= theta && kl[r] <= kl_eps) lock_mask[pos] = 1;
  }
}

int launch_conf_gate_lock(const float* conf, const float* kl, const int32_t* idx, const int32_t* row_offsets, int B, int N,
                          const uint8_t* mask_state, uint8_t* lock_mask, float kl_eps, float m_percent, float* theta_out,
                          cudaStream_t st, bool apply_lock, bool all_rows, float empty_theta) {
  if (N > CG_MAX_N) return SL_EUNSUPPORTED;
  int p2 = 1;
  while (p2 < N) p2 <<= 1;
  conf_gate_lock_kernel<<<B, CG_THREADS, (size_t)p2 * sizeof(float), st>>>(conf, kl, idx, row_offsets, mask_state, lock_mask,
                                                                          kl_eps, m_percent, theta_out, apply_lock ? 1 : 0,
                                                                          all_rows ? 1 : 0, empty_theta);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

}  // namespace sl
