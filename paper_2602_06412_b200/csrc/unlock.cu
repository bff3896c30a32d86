// Optional un-locking (paper App. "Optional Unlocking"): the small kernels around the probe.
//
// The probe itself is the ordinary forward of the step run on the LOCKED rows as queries against the caches, without
// writing their K/V back (see surelock_probe_unlock in api.cu); what lives here is
//   * the complement of the lock mask (so that the compaction kernel packs the locked rows),
//   * the lock update of a step while un-locking is enabled: per-position threshold (rho * eps for a position that was
//     un-locked before), no locking during the cool-down, optional confidence gate, and, for every row that locks, the
//     step number t* and a copy of its logits (the frozen posterior p_{t*} the drift is measured against),
//   * the un-lock rule  u~ > theta_t  AND  KL(p^_t || p_{t*}) > eps_unlock  AND  t - t* > D_interval.
#include "common.cuh"

namespace sl {

__global__ void __launch_bounds__(256)
invert_mask_kernel(const uint8_t* __restrict__ lock, uint8_t* __restrict__ inv, int total) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) inv[i] = lock[i] ? 0 : 1;
}

int launch_invert_mask(const uint8_t* lock, uint8_t* inv, int total, cudaStream_t st) {
  int g = (total + 255) / 256;
  g = g < 1 ? 1 : (g > 1024 ? 1024 : g);
  invert_mask_kernel<<<g, 256, 0, st>>>(lock, inv, total);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

// One CTA per active row (grid-stride).  Decision by thread 0, copy of the row by all threads.
__global__ void __launch_bounds__(256)
lock_commit_kernel(const float* __restrict__ kl, const float* __restrict__ conf, const float* __restrict__ lse,
                   const int32_t* __restrict__ idx, const int32_t* __restrict__ n_active, int N,
                   const uint8_t* __restrict__ mask_state, uint8_t* __restrict__ lock_mask, float kl_eps, float rho, int t,
                   const float* __restrict__ theta, const int32_t* __restrict__ cool_until,
                   const uint8_t* __restrict__ relock, int32_t* __restrict__ t_star, int32_t* __restrict__ frozen_rop,
                   float* __restrict__ frozen_lse, const uint4* __restrict__ logits, uint4* __restrict__ frozen,
                   long long row_vec) {
  __shared__ int s_pass;
  const int M = *n_active;
  for (int r = blockIdx.x; r < M; r += gridDim.x) {
    const int pos = idx[r];
    if (threadIdx.x == 0) {
      const float eps_i = relock[pos] ? rho * kl_eps : kl_eps;
      bool pass = mask_state[pos] == 0 && kl[r] <= eps_i && t > cool_until[pos];
      if (pass && theta) pass = (1.f - conf[r]) <= theta[pos / N];
      if (pass) {
        lock_mask[pos] = 1;
        t_star[pos] = t;
        frozen_rop[pos] = pos;
        frozen_lse[pos] = lse[r];
      }
      s_pass = pass ? 1 : 0;
    }
    __syncthreads();
    if (s_pass) {
      const uint4* src = logits + (long long)r * row_vec;
      uint4* dst = frozen + (long long)pos * row_vec;
      for (long long c = threadIdx.x; c < row_vec; c += blockDim.x) dst[c] = src[c];
    }
    __syncthreads();
  }
}

int launch_lock_commit(const float* kl, const float* conf, const float* lse, const int32_t* idx, const int32_t* n_active,
                       int max_rows, int N, const uint8_t* mask_state, uint8_t* lock_mask, float kl_eps, float rho, int t,
                       const float* theta, const int32_t* cool_until, const uint8_t* relock, int32_t* t_star,
                       int32_t* frozen_rop, float* frozen_lse, const void* logits, void* frozen, size_t row_bytes,
                       cudaStream_t st) {
  if (row_bytes % 16) return SL_EUNSUPPORTED;
  int g = max_rows < 1 ? 1 : (max_rows > 2 * sm_count() ? 2 * sm_count() : max_rows);
  lock_commit_kernel<<<g, 256, 0, st>>>(kl, conf, lse, idx, n_active, N, mask_state, lock_mask, kl_eps, rho, t, theta,
                                        cool_until, relock, t_star, frozen_rop, frozen_lse,
                                        reinterpret_cast<const uint4*>(logits), reinterpret_cast<uint4*>(frozen),
                                        (long long)(row_bytes / 16));
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

__global__ void __launch_bounds__(256)
unlock_kernel(const float* __restrict__ drift, const float* __restrict__ conf, const int32_t* __restrict__ idx,
              const int32_t* __restrict__ n_probe, int N, const float* __restrict__ theta, float eps_unlock,
              int d_interval, int d_cool, int t, const int32_t* __restrict__ t_star, int32_t* __restrict__ cool_until,
              uint8_t* __restrict__ relock, uint8_t* __restrict__ lock_mask, int32_t* __restrict__ n_unlocked) {
  const int n = *n_probe;
  for (int r = blockIdx.x * blockDim.x + threadIdx.x; r < n; r += gridDim.x * blockDim.x) {
    const int pos = idx[r];
    const int ts = t_star[pos];
    // a position the caller locked by hand (no recorded t*, no frozen posterior) is never un-locked here
    if (ts >= 0 && (1.f - conf[r]) > theta[pos / N] && drift[r] > eps_unlock && t - ts > d_interval) {
      lock_mask[pos] = 0;
      cool_until[pos] = t + d_cool;
      relock[pos] = 1;
      atomicAdd(n_unlocked, 1);
    }
  }
}

int launch_unlock(const float* drift, const float* conf, const int32_t* idx, const int32_t* n_probe, int max_rows, int N,
                  const float* theta, float eps_unlock, int d_interval, int d_cool, int t, const int32_t* t_star,
                  int32_t* cool_until, uint8_t* relock, uint8_t* lock_mask, int32_t* n_unlocked, cudaStream_t st) {
  int g = (max_rows + 255) / 256;
  g = g < 1 ? 1 : (g > 1024 ? 1024 : g);
  unlock_kernel<<<g, 256, 0, st>>>(drift, conf, idx, n_probe, N, theta, eps_unlock, d_interval, d_cool, t, t_star,
                                   cool_until, relock, lock_mask, n_unlocked);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

}  // namespace sl
