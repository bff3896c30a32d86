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
#include <stdlib.h>

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
  const float ea = a.m == -INFINITY ? 0.f : fast_exp2((a.m - o.m) * LOG2E);
  const float eb = b.m == -INFINITY ? 0.f : fast_exp2((b.m - o.m) * LOG2E);
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
    st.s *= fast_exp2((st.m - vmax) * LOG2E);   // st.m = -inf gives 0 * 0
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
  for (int k = 0; k < VEC; ++k) st.s += fast_exp2(fmaf(f[k], LOG2E, -mb));
}

// g(r) = r - 1 + exp(-r) >= 0.  Series below 1/8 (relative error < 3e-7), exp beyond.
__device__ __forceinline__ float kl_g_series(float r) {
  const float r2 = r * r;   // r^2/2 - r^3/6 + r^4/24 - r^5/120 + r^6/720
  return r2 * (0.5f + r * (-1.f / 6.f + r * (1.f / 24.f + r * (-1.f / 120.f + r * (1.f / 720.f)))));
}
__device__ __forceinline__ float kl_g(float r) {
  return fabsf(r) < 0.125f ? kl_g_series(r) : r + (fast_exp2(-r * LOG2E) - 1.f);
}

constexpr int KL_UNROLL = 4;   // 128-bit loads in flight per thread and row: hides HBM latency at 1024 threads per SM

template <typename T>
__global__ void __launch_bounds__(KL_THREADS)
softmax_kl_sure_kernel(const T* __restrict__ logits, const T* __restrict__ prev, const int32_t* __restrict__ row_of_pos_prev,
                       const float* __restrict__ prev_lse, const int32_t* __restrict__ idx,
                       const int32_t* __restrict__ n_active, int V, const uint8_t* __restrict__ mask_state,
                       uint8_t* __restrict__ lock_mask, float kl_eps, float* __restrict__ kl_out,
                       float* __restrict__ conf_out, int32_t* __restrict__ argmax_out, float* __restrict__ lse_out,
                       int apply_lock) {
  constexpr int VEC = 16 / sizeof(T);
  __shared__ MaxSum s_ms[KL_THREADS / 32];
  __shared__ double s_sum[KL_THREADS / 32];
  const int M = *n_active;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = V / VEC;
  for (int r = blockIdx.x; r < M; r += gridDim.x) {
    const int pos = idx ? idx[r] : r;
    const int prow = row_of_pos_prev ? row_of_pos_prev[pos] : r;
    const uint4* z = reinterpret_cast<const uint4*>(logits + (long long)r * V);
    const uint4* y = (prev && prow >= 0) ? reinterpret_cast<const uint4*>(prev + (long long)prow * V) : nullptr;
    const bool need_q = y && !prev_lse;

    // sweep 1: max, sum of exponentials and argmax of the current row (and of the previous row if its lse is unknown)
    MaxSum a{-INFINITY, 0.f, 0x7fffffff}, b{-INFINITY, 0.f, 0};
    for (int v0 = tid; v0 < nvec; v0 += KL_THREADS * KL_UNROLL) {
      uint4 zz[KL_UNROLL], yy[KL_UNROLL];
#pragma unroll
      for (int k = 0; k < KL_UNROLL; ++k) {
        const int vi = v0 + k * KL_THREADS;
        if (vi < nvec) {
          zz[k] = __ldg(z + vi);
          if (need_q) yy[k] = __ldg(y + vi);
        }
      }
#pragma unroll
      for (int k = 0; k < KL_UNROLL; ++k) {
        const int vi = v0 + k * KL_THREADS;
        if (vi < nvec) {
          float f[VEC];
          unpack<T, VEC>(zz[k], f);
          accum_maxsum<VEC>(f, vi * VEC, a, true);
          if (need_q) {
            unpack<T, VEC>(yy[k], f);
            accum_maxsum<VEC>(f, vi * VEC, b, false);
          }
        }
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

    // sweep 2: KL as a sum of non-negative terms (the current row comes from L2)
    float kl = INFINITY;
    if (y) {
      const float dl = lse_p - lse_q;
      const float lp2 = lse_p * LOG2E;
      float acc = 0.f;
      for (int v0 = tid; v0 < nvec; v0 += KL_THREADS * KL_UNROLL) {
        uint4 zz[KL_UNROLL], yy[KL_UNROLL];
#pragma unroll
        for (int k = 0; k < KL_UNROLL; ++k) {
          const int vi = v0 + k * KL_THREADS;
          if (vi < nvec) {
            zz[k] = __ldg(z + vi);
            yy[k] = __ldg(y + vi);
          }
        }
#pragma unroll
        for (int k = 0; k < KL_UNROLL; ++k) {
          const int vi = v0 + k * KL_THREADS;
          if (vi < nvec) {
            float fz[VEC], fy[VEC], rr[VEC];
            unpack<T, VEC>(zz[k], fz);
            unpack<T, VEC>(yy[k], fy);
            float rmax = 0.f;
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
              rr[e] = (fz[e] - fy[e]) - dl;
              rmax = fmaxf(rmax, fabsf(rr[e]));
            }
            if (rmax < 0.125f) {          // whole vector in the series range: no per-element branch
#pragma unroll
              for (int e = 0; e < VEC; ++e) acc = fmaf(fast_exp2(fmaf(fz[e], LOG2E, -lp2)), kl_g_series(rr[e]), acc);
            } else {
#pragma unroll
              for (int e = 0; e < VEC; ++e) acc = fmaf(fast_exp2(fmaf(fz[e], LOG2E, -lp2)), kl_g(rr[e]), acc);
            }
          }
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
      if (apply_lock && mask_state[pos] == 0 && kl <= kl_eps) lock_mask[pos] = 1;
    }
  }
}

// ---- bf16 rows at full HBM rate -------------------------------------------------------------------------------
// Same computation as the generic kernel above, arranged for the instruction budget of a B200 SM: at the HBM rate a
// row pair (2 x V bf16) leaves ~20 issue slots per vocabulary entry, so the arithmetic runs on packed fp32x2
// instructions (two entries per FFMA2/FADD2/FMUL2), the row maximum is taken on packed bf16 pairs, the series/exp
// choice of g is made per 8-entry vector from sum(r^2), and the next vectors are loaded while the current ones are
// processed.
constexpr int KLF_THREADS = 256;

// The current row is read twice (sweep 1 from HBM, sweep 2 from L2): ask L2 to keep it; the previous row is read
// once: mark it evict-first so that it does not push current rows out.
__device__ __forceinline__ uint64_t l2_policy_keep() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_stream() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint4 ld_hint(const uint4* p, uint64_t pol) {
  uint4 v;
  asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(pol));
  return v;
}

__device__ __forceinline__ float2 unpack_pair(unsigned w) {   // (low bf16, high bf16) -> two floats
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ float vec_max_bf16(const uint4& v) {
  const __nv_bfloat162 a = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&v.x), *reinterpret_cast<const __nv_bfloat162*>(&v.y));
  const __nv_bfloat162 b = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&v.z), *reinterpret_cast<const __nv_bfloat162*>(&v.w));
  const __nv_bfloat162 m = __hmax2(a, b);
  const unsigned w = *reinterpret_cast<const unsigned*>(&m);
  return fmaxf(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

struct MaxSum2 {
  float m;
  float2 s;   // two partial sums (even / odd entries), added at the end
  int am;
};

__device__ __forceinline__ void accum_maxsum_bf16(const uint4& v, int c, MaxSum2& st, bool track_arg) {
  const float vmax = vec_max_bf16(v);
  if (vmax > st.m) {
    const float sc = fast_exp2((st.m - vmax) * LOG2E);   // st.m = -inf: 0
    st.s.x *= sc;
    st.s.y *= sc;
    st.m = vmax;
    if (track_arg) {
      const unsigned w[4] = {v.x, v.y, v.z, v.w};
      int a = 7;
#pragma unroll
      for (int k = 3; k >= 0; --k) {
        if (__uint_as_float(w[k] & 0xffff0000u) == vmax) a = 2 * k + 1;
        if (__uint_as_float(w[k] << 16) == vmax) a = 2 * k;
      }
      st.am = c + a;
    }
  }
  const float mb = -st.m * LOG2E;
  const float2 l2 = make_float2(LOG2E, LOG2E), mb2 = make_float2(mb, mb);
  const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float2 t = __ffma2_rn(unpack_pair(w[k]), l2, mb2);
    st.s = __fadd2_rn(st.s, make_float2(fast_exp2(t.x), fast_exp2(t.y)));
  }
}

// sum_v p_v g(r_v) over the 8 entries of one vector pair
__device__ __forceinline__ float2 kl_vec_bf16(const uint4& zv, const uint4& yv, float dl, float lp2, float2 acc) {
  const unsigned zw[4] = {zv.x, zv.y, zv.z, zv.w}, yw[4] = {yv.x, yv.y, yv.z, yv.w};
  const float2 ndl = make_float2(-dl, -dl), l2 = make_float2(LOG2E, LOG2E), nlp = make_float2(-lp2, -lp2);
  const float2 neg1 = make_float2(-1.f, -1.f);
  float2 z[4], r[4], r2[4];
  float2 ss = make_float2(0.f, 0.f);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    z[k] = unpack_pair(zw[k]);
    const float2 y = unpack_pair(yw[k]);
    r[k] = __fadd2_rn(__ffma2_rn(y, neg1, z[k]), ndl);     // (z - y) - dl
    r2[k] = __fmul2_rn(r[k], r[k]);
    ss = __fadd2_rn(ss, r2[k]);
  }
  if (ss.x + ss.y < 0.015625f) {                             // every |r| < 1/8: series, two entries per instruction
    const float2 c2 = make_float2(0.5f, 0.5f), c3 = make_float2(-1.f / 6.f, -1.f / 6.f);
    const float2 c4 = make_float2(1.f / 24.f, 1.f / 24.f), c5 = make_float2(-1.f / 120.f, -1.f / 120.f);
    const float2 c6 = make_float2(1.f / 720.f, 1.f / 720.f);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float2 h = __ffma2_rn(r[k], c6, c5);
      h = __ffma2_rn(r[k], h, c4);
      h = __ffma2_rn(r[k], h, c3);
      h = __ffma2_rn(r[k], h, c2);
      const float2 t = __ffma2_rn(z[k], l2, nlp);
      const float2 p = make_float2(fast_exp2(t.x), fast_exp2(t.y));
      acc = __ffma2_rn(p, __fmul2_rn(r2[k], h), acc);
    }
  } else if (ss.x + ss.y < 0.25f) {                          // every |r| < 1/2: series up to r^9 (relative error < 3e-9)
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float2 h = __ffma2_rn(r[k], make_float2(-1.f / 362880.f, -1.f / 362880.f), make_float2(1.f / 40320.f, 1.f / 40320.f));
      h = __ffma2_rn(r[k], h, make_float2(-1.f / 5040.f, -1.f / 5040.f));
      h = __ffma2_rn(r[k], h, make_float2(1.f / 720.f, 1.f / 720.f));
      h = __ffma2_rn(r[k], h, make_float2(-1.f / 120.f, -1.f / 120.f));
      h = __ffma2_rn(r[k], h, make_float2(1.f / 24.f, 1.f / 24.f));
      h = __ffma2_rn(r[k], h, make_float2(-1.f / 6.f, -1.f / 6.f));
      h = __ffma2_rn(r[k], h, make_float2(0.5f, 0.5f));
      const float2 t = __ffma2_rn(z[k], l2, nlp);
      const float2 p = make_float2(fast_exp2(t.x), fast_exp2(t.y));
      acc = __ffma2_rn(p, __fmul2_rn(r2[k], h), acc);
    }
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float2 t = __ffma2_rn(z[k], l2, nlp);
      acc.x = fmaf(fast_exp2(t.x), kl_g(r[k].x), acc.x);
      acc.y = fmaf(fast_exp2(t.y), kl_g(r[k].y), acc.y);
    }
  }
  return acc;
}

__global__ void __launch_bounds__(KLF_THREADS, 3)
softmax_kl_sure_bf16_kernel(const bf16* __restrict__ logits, const bf16* __restrict__ prev,
                            const int32_t* __restrict__ row_of_pos_prev, const float* __restrict__ prev_lse,
                            const int32_t* __restrict__ idx, const int32_t* __restrict__ n_active, int V,
                            const uint8_t* __restrict__ mask_state, uint8_t* __restrict__ lock_mask, float kl_eps,
                            float* __restrict__ kl_out, float* __restrict__ conf_out, int32_t* __restrict__ argmax_out,
                            float* __restrict__ lse_out, int apply_lock, const float4* __restrict__ lse_part,
                            int part_tiles, int part_rows, const int* __restrict__ lse_valid) {
  __shared__ float s_m[KLF_THREADS / 32], s_s[KLF_THREADS / 32];
  __shared__ int s_a[KLF_THREADS / 32];
  __shared__ double s_sum[KLF_THREADS / 32];
  const int M = *n_active;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = V >> 3;
  constexpr int STEP = 2 * KLF_THREADS;   // two vectors per thread and iteration
  // the LM head may have left the current rows' softmax statistics per 256-column tile: then sweep 1 is a reduction
  // of part_tiles small records instead of a pass over the row
  const bool have_part = lse_part != nullptr && *lse_valid != 0;
  const uint64_t pol_keep = l2_policy_keep(), pol_stream = l2_policy_stream();

  auto block_maxsum = [&](MaxSum2 st) -> MaxSum {
    MaxSum v{st.m, st.s.x + st.s.y, st.am};
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      MaxSum t;
      t.m = __shfl_xor_sync(0xffffffffu, v.m, o);
      t.s = __shfl_xor_sync(0xffffffffu, v.s, o);
      t.am = __shfl_xor_sync(0xffffffffu, v.am, o);
      v = combine(v, t);
    }
    __syncthreads();
    if (lane == 0) { s_m[warp] = v.m; s_s[warp] = v.s; s_a[warp] = v.am; }
    __syncthreads();
    MaxSum r{s_m[0], s_s[0], s_a[0]};
    for (int w = 1; w < KLF_THREADS / 32; ++w) r = combine(r, MaxSum{s_m[w], s_s[w], s_a[w]});
    return r;
  };

  for (int r = blockIdx.x; r < M; r += gridDim.x) {
    const int pos = idx ? idx[r] : r;
    const int prow = row_of_pos_prev ? row_of_pos_prev[pos] : r;
    const uint4* z = reinterpret_cast<const uint4*>(logits + (long long)r * V);
    const uint4* y = (prev && prow >= 0) ? reinterpret_cast<const uint4*>(prev + (long long)prow * V) : nullptr;
    const bool need_q = y && !prev_lse;

    // sweep 1 (current row; the previous row only if its log-sum-exp was not kept), next vectors prefetched
    MaxSum2 a{-INFINITY, make_float2(0.f, 0.f), 0x7fffffff}, b{-INFINITY, make_float2(0.f, 0.f), 0};
    if (have_part) {
      MaxSum acc{-INFINITY, 0.f, 0x7fffffff};
      for (int t = tid; t < part_tiles; t += KLF_THREADS) {
        const float4 p = __ldcs(lse_part + (size_t)t * part_rows + r);
        acc = combine(acc, MaxSum{p.x, p.y, __float_as_int(p.z)});
      }
      a.m = acc.m;
      a.s = make_float2(acc.s, 0.f);
      a.am = acc.am;
      if (need_q) {
        for (int v0 = tid; v0 < nvec; v0 += KLF_THREADS) accum_maxsum_bf16(ld_hint(y + v0, pol_stream), v0 * 8, b, false);
      }
    } else {
      const uint4 zero = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);   // eight times -inf
      uint4 c0 = tid < nvec ? ld_hint(z + tid, pol_keep) : zero;
      uint4 c1 = tid + KLF_THREADS < nvec ? ld_hint(z + tid + KLF_THREADS, pol_keep) : zero;
      for (int v0 = tid; v0 < nvec; v0 += STEP) {
        const int n0 = v0 + STEP, n1 = n0 + KLF_THREADS;
        const uint4 p0 = n0 < nvec ? ld_hint(z + n0, pol_keep) : zero;
        const uint4 p1 = n1 < nvec ? ld_hint(z + n1, pol_keep) : zero;
        accum_maxsum_bf16(c0, v0 * 8, a, true);
        if (v0 + KLF_THREADS < nvec) accum_maxsum_bf16(c1, (v0 + KLF_THREADS) * 8, a, true);
        c0 = p0;
        c1 = p1;
      }
      if (need_q) {
        for (int v0 = tid; v0 < nvec; v0 += KLF_THREADS) accum_maxsum_bf16(ld_hint(y + v0, pol_stream), v0 * 8, b, false);
      }
    }
    const MaxSum ra = block_maxsum(a);
    const float lse_p = ra.m + log2f(ra.s) * LN2;
    float lse_q = 0.f;
    if (need_q) {
      const MaxSum rb = block_maxsum(b);
      lse_q = rb.m + log2f(rb.s) * LN2;
    } else if (y) {
      lse_q = prev_lse[prow];
    }

    // sweep 2: KL as a sum of non-negative terms (the current row comes back from L2)
    float kl = INFINITY;
    if (y) {
      const float dl = lse_p - lse_q, lp2 = lse_p * LOG2E;
      float2 acc = make_float2(0.f, 0.f);
      const uint4 zero = make_uint4(0, 0, 0, 0);
      uint4 cz0 = tid < nvec ? ld_hint(z + tid, pol_keep) : zero, cy0 = tid < nvec ? ld_hint(y + tid, pol_stream) : zero;
      uint4 cz1 = zero, cy1 = zero;
      if (tid + KLF_THREADS < nvec) { cz1 = ld_hint(z + tid + KLF_THREADS, pol_keep); cy1 = ld_hint(y + tid + KLF_THREADS, pol_stream); }
      for (int v0 = tid; v0 < nvec; v0 += STEP) {
        const int n0 = v0 + STEP, n1 = n0 + KLF_THREADS;
        uint4 pz0 = zero, py0 = zero, pz1 = zero, py1 = zero;
        if (n0 < nvec) { pz0 = ld_hint(z + n0, pol_keep); py0 = ld_hint(y + n0, pol_stream); }
        if (n1 < nvec) { pz1 = ld_hint(z + n1, pol_keep); py1 = ld_hint(y + n1, pol_stream); }
        acc = kl_vec_bf16(cz0, cy0, dl, lp2, acc);
        if (v0 + KLF_THREADS < nvec) acc = kl_vec_bf16(cz1, cy1, dl, lp2, acc);
        cz0 = pz0; cy0 = py0; cz1 = pz1; cy1 = py1;
      }
      double d = (double)acc.x + (double)acc.y;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
      __syncthreads();
      if (lane == 0) s_sum[warp] = d;
      __syncthreads();
      d = 0.0;
      for (int w = 0; w < KLF_THREADS / 32; ++w) d += s_sum[w];
      kl = (float)d;
    }
    if (tid == 0) {
      kl_out[r] = kl;
      conf_out[r] = 1.f / ra.s;          // exp(max - lse)
      argmax_out[r] = ra.am;
      if (lse_out) lse_out[r] = lse_p;
      if (apply_lock && mask_state[pos] == 0 && kl <= kl_eps) lock_mask[pos] = 1;
    }
  }
}

int launch_softmax_kl_sure(const void* logits, const void* prev_logits, const int32_t* row_of_pos_prev,
                           const float* prev_lse, const int32_t* idx, const int32_t* n_active, int max_rows, int vocab,
                           int dtype, const uint8_t* mask_state, uint8_t* lock_mask, float kl_eps, float* kl,
                           float* conf, int32_t* argmax, float* lse_out, cudaStream_t st, bool apply_lock,
                           const float4* lse_part, int part_tiles, int part_rows, const int* lse_valid) {
  const int vec = dtype == SL_BF16 ? 8 : 4;
  if (vocab <= 0 || vocab % vec) return SL_EUNSUPPORTED;
  int g = sm_count() * 2;
  if (g > max_rows) g = max_rows;
  if (g < 1) g = 1;
  if (dtype == SL_BF16) {
    static int per_sm = 0;
    if (!per_sm) {
      const char* e = getenv("SURELOCK_KL_CTAS_PER_SM");   // tuning aid
      per_sm = e ? atoi(e) : 3;
      if (per_sm < 1 || per_sm > 3) per_sm = 3;
    }
    int gb = sm_count() * per_sm;
    if (gb > max_rows) gb = max_rows;
    if (gb < 1) gb = 1;
    softmax_kl_sure_bf16_kernel<<<gb, KLF_THREADS, 0, st>>>((const bf16*)logits, (const bf16*)prev_logits, row_of_pos_prev,
                                                             prev_lse, idx, n_active, vocab, mask_state, lock_mask, kl_eps,
                                                             kl, conf, argmax, lse_out, apply_lock ? 1 : 0, lse_part,
                                                             part_tiles, part_rows, lse_valid);
  } else
    softmax_kl_sure_kernel<float><<<g, KL_THREADS, 0, st>>>((const float*)logits, (const float*)prev_logits,
                                                           row_of_pos_prev, prev_lse, idx, n_active, vocab, mask_state,
                                                           lock_mask, kl_eps, kl, conf, argmax, lse_out, apply_lock ? 1 : 0);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

}  // namespace sl
