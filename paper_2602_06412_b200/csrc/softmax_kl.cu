// Fused softmax + step-wise KL + confidence + argmax + lock test + lock update for the packed active rows
// (Algorithm 1 lines 15, 18-20, 23-24; Sec. 2.2: D = KL(p_t || p_{t-1}), lock when D <= eps).
//
// One CTA per row.  Sweep 1 reads the current logits (and the previous ones unless their log-sum-exp was kept
// from the step that produced them) and forms max / sum-of-exponentials / argmax; sweep 2 re-reads both rows
// and accumulates the KL as a sum of NON-NEGATIVE terms
//     KL = sum_v p_v * g(r_v),   r_v = log p_v - log q_v,   g(r) = r - 1 + exp(-r) >= 0,
// which equals sum_v p_v r_v because sum p = sum q = 1.  The plain form cancels catastrophically in fp32 once
// KL is ~1e-7 (terms of size |r| summing to r^2/2); this one does not, is exactly 0 for identical rows, and is
// insensitive to first order to the rounding of the two log-sum-exps (d KL / d(lse_p - lse_q) = 1 - sum q = 0).
// g uses its Taylor series for |r| < 1/8 and r + (exp(-r) - 1) beyond.
#include "common.cuh"

namespace sl {

constexpr int KL_THREADS = 512;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

struct MaxSum {
  float m, s;
  int am;
};

__device__ __forceinline__ MaxSum combine(const MaxSum& a, const MaxSum& b) {
  MaxSum o;
  o.m = fmaxf(a.m, b.m);
  const float ea = a.m == -INFINITY ? 0.f : exp2f((a.m - o.m) * LOG2E);
  const float eb = b.m == -INFINITY ? 0.f : exp2f((b.m - o.m) * LOG2E);
  o.s = a.s * ea + b.s * eb;
  o.am = a.m > b.m ? a.am : (b.m > a.m ? b.am : (a.am < b.am ? a.am : b.am));
  return o;
}

__device__ __forceinline__ MaxSum block_combine(MaxSum v, MaxSum* s_ms) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    MaxSum t;
    t.m = __shfl_xor_sync(0xffffffffu, v.m, o);
    t.s = __shfl_xor_sync(0xffffffffu, v.s, o);
    t.am = __shfl_xor_sync(0xffffffffu, v.am, o);
    v = combine(v, t);
  }
  __syncthreads();
  if (lane == 0) s_ms[warp] = v;
  __syncthreads();
  MaxSum r = s_ms[0];
  for (int w = 1; w < KL_THREADS / 32; ++w) r = combine(r, s_ms[w]);
  return r;
}

template <typename T, int VEC>
__device__ __forceinline__ void unpack(const uint4& v, float (&f)[VEC]) {
  if constexpr (sizeof(T) == 2) {
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      f[2 * k] = __uint_as_float(w[k] << 16);
      f[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
  } else {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
}

template <int VEC>
__device__ __forceinline__ void accum_maxsum(const float (&f)[VEC], int c, MaxSum& st, bool track_arg) {
  float vmax = f[0];
#pragma unroll
  for (int k = 1; k < VEC; ++k) vmax = fmaxf(vmax, f[k]);
  if (vmax > st.m) {
    st.s *= exp2f((st.m - vmax) * LOG2E);   // st.m = -inf gives 0 * 0
    st.m = vmax;
    if (track_arg) {
      int a = VEC - 1;
#pragma unroll
      for (int k = VEC - 2; k >= 0; --k)
        if (f[k] == vmax) a = k;
      st.am = c + a;
    }
  }
  const float mb = st.m * LOG2E;
#pragma unroll
  for (int k = 0; k < VEC; ++k) st.s += exp2f(fmaf(f[k], LOG2E, -mb));
}

__device__ __forceinline__ float kl_g(float r) {
  // g(r) = r - 1 + exp(-r)
  if (fabsf(r) < 0.125f) {
    const float r2 = r * r;
    // r^2/2 - r^3/6 + r^4/24 - r^5/120 + r^6/720
    return r2 * (0.5f + r * (-1.f / 6.f + r * (1.f / 24.f + r * (-1.f / 120.f + r * (1.f / 720.f)))));
  }
  return r + (exp2f(-r * LOG2E) - 1.f);
}

template <typename T>
__global__ void __launch_bounds__(KL_THREADS)
softmax_kl_sure_kernel(const T* __restrict__ logits, const T* __restrict__ prev, const int32_t* __restrict__ row_of_pos_prev,
                       const float* __restrict__ prev_lse, const int32_t* __restrict__ idx,
                       const int32_t* __restrict__ n_active, int V, const uint8_t* __restrict__ mask_state,
                       uint8_t* __restrict__ lock_mask, float kl_eps, float* __restrict__ kl_out,
                       float* __restrict__ conf_out, int32_t* __restrict__ argmax_out, float* __restrict__ lse_out) {
  constexpr int VEC = 16 / sizeof(T);
  __shared__ MaxSum s_ms[KL_THREADS / 32];
  __shared__ double s_sum[KL_THREADS / 32];
  const int M = *n_active;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int r = blockIdx.x; r < M; r += gridDim.x) {
    const int pos = idx ? idx[r] : r;
    const int prow = row_of_pos_prev ? row_of_pos_prev[pos] : r;
    const T* z = logits + (long long)r * V;
    const T* y = (prev && prow >= 0) ? prev + (long long)prow * V : nullptr;
    const bool need_q = y && !prev_lse;

    MaxSum a{-INFINITY, 0.f, 0x7fffffff}, b{-INFINITY, 0.f, 0};
    for (int c = tid * VEC; c < V; c += KL_THREADS * VEC) {
      float f[VEC];
      unpack<T, VEC>(__ldg(reinterpret_cast<const uint4*>(z + c)), f);
      accum_maxsum<VEC>(f, c, a, true);
      if (need_q) {
        unpack<T, VEC>(__ldg(reinterpret_cast<const uint4*>(y + c)), f);
        accum_maxsum<VEC>(f, c, b, false);
      }
    }
    a = block_combine(a, s_ms);
    const float lse_p = a.m + log2f(a.s) * LN2;
    float lse_q = 0.f;
    if (need_q) {
      b = block_combine(b, s_ms);
      lse_q = b.m + log2f(b.s) * LN2;
    } else if (y) {
      lse_q = prev_lse[prow];
    }

    float kl = INFINITY;
    if (y) {
      const float dl = lse_p - lse_q;
      const float lp2 = lse_p * LOG2E;
      float acc = 0.f;
      for (int c = tid * VEC; c < V; c += KL_THREADS * VEC) {
        float fz[VEC], fy[VEC];
        unpack<T, VEC>(__ldg(reinterpret_cast<const uint4*>(z + c)), fz);
        unpack<T, VEC>(__ldg(reinterpret_cast<const uint4*>(y + c)), fy);
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
          const float rr = (fz[k] - fy[k]) - dl;
          const float p = exp2f(fmaf(fz[k], LOG2E, -lp2));
          acc = fmaf(p, kl_g(rr), acc);
        }
      }
      double d = (double)acc;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
      __syncthreads();
      if (lane == 0) s_sum[warp] = d;
      __syncthreads();
      d = 0.0;
      for (int w = 0; w < KL_THREADS / 32; ++w) d += s_sum[w];
      kl = (float)d;
    }
    if (tid == 0) {
      kl_out[r] = kl;
      conf_out[r] = 1.f / a.s;          // exp(max - lse)
      argmax_out[r] = a.am;
      if (lse_out) lse_out[r] = lse_p;
      if (mask_state[pos] == 0 && kl <= kl_eps) lock_mask[pos] = 1;
    }
  }
}

int launch_softmax_kl_sure(const void* logits, const void* prev_logits, const int32_t* row_of_pos_prev,
                           const float* prev_lse, const int32_t* idx, const int32_t* n_active, int max_rows, int vocab,
                           int dtype, const uint8_t* mask_state, uint8_t* lock_mask, float kl_eps, float* kl,
                           float* conf, int32_t* argmax, float* lse_out, cudaStream_t st) {
  const int vec = dtype == SL_BF16 ? 8 : 4;
  if (vocab <= 0 || vocab % vec) return SL_EUNSUPPORTED;
  int g = sm_count() * 2;
  if (g > max_rows) g = max_rows;
  if (g < 1) g = 1;
  if (dtype == SL_BF16)
    softmax_kl_sure_kernel<bf16><<<g, KL_THREADS, 0, st>>>((const bf16*)logits, (const bf16*)prev_logits, row_of_pos_prev,
                                                          prev_lse, idx, n_active, vocab, mask_state, lock_mask, kl_eps,
                                                          kl, conf, argmax, lse_out);
  else
    softmax_kl_sure_kernel<float><<<g, KL_THREADS, 0, st>>>((const float*)logits, (const float*)prev_logits,
                                                           row_of_pos_prev, prev_lse, idx, n_active, vocab, mask_state,
                                                           lock_mask, kl_eps, kl, conf, argmax, lse_out);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

}  // namespace sl
