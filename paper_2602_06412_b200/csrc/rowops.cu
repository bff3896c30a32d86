// Row-wise, HBM-bound stages of the locked forward: block-input gather (Algorithm 1 line 7), RMSNorm ("LN" of
// line 10), rotary embedding on q and k with the ORIGINAL position index, and the K/V cache scatter (line 11).
// All kernels are grid-stride over packed rows and read the row count M from device memory, so a step needs no
// host synchronisation.  Rows move as 128-bit words.
#include "common.cuh"

namespace sl {

static inline int row_grid(int max_rows, int ctas_per_sm) {
  int g = sm_count() * ctas_per_sm;
  if (g > max_rows) g = max_rows;
  return g < 1 ? 1 : g;
}

// ------------------------------------------------------------------------------------------------ gather
template <typename T>
__global__ void __launch_bounds__(256)
gather_rows_kernel(const T* __restrict__ table, const int32_t* __restrict__ tokens, const int32_t* __restrict__ idx,
                   const int32_t* __restrict__ n_active, int d, int table_rows, float* __restrict__ x,
                   int32_t* status) {
  griddep_wait();
  griddep_launch();
  const int M = *n_active;
  constexpr int VEC = 16 / sizeof(T);
  for (int r = blockIdx.x; r < M; r += gridDim.x) {
    const int pos = idx[r];
    const long long src = tokens ? (long long)tokens[pos] : (long long)pos;
    if (src < 0 || src >= table_rows) {
      if (threadIdx.x == 0) set_status(status, SL_DEV_BAD_INDEX);
      continue;
    }
    const T* s = table + src * d;
    float* o = x + (long long)r * d;
    for (int c = threadIdx.x * VEC; c < d; c += blockDim.x * VEC) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(s + c));
      const T* e = reinterpret_cast<const T*>(&v);
      float f[VEC];
#pragma unroll
      for (int k = 0; k < VEC; ++k) f[k] = to_f(e[k]);
#pragma unroll
      for (int k = 0; k < VEC; k += 4)
        *reinterpret_cast<float4*>(o + c + k) = make_float4(f[k], f[k + 1], f[k + 2], f[k + 3]);
    }
  }
}

int launch_gather_rows(const void* table, const int32_t* tokens, const int32_t* idx, const int32_t* n_active,
                       int max_rows, int d, int table_rows, float* x, int dtype, int32_t* status, cudaStream_t st) {
  const int g = row_grid(max_rows, 8);
  if (dtype == SL_BF16) {
    if (d % 8) return SL_EUNSUPPORTED;
    SL_CUDA_TRY(launch_pdl(gather_rows_kernel<bf16>, dim3(g), dim3(256), 0, st, (const bf16*)table, tokens, idx, n_active, d, table_rows, x, status));
  } else {
    if (d % 4) return SL_EUNSUPPORTED;
    SL_CUDA_TRY(launch_pdl(gather_rows_kernel<float>, dim3(g), dim3(256), 0, st, (const float*)table, tokens, idx, n_active, d, table_rows, x, status));
  }
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

// ------------------------------------------------------------------------------------------------ RMSNorm
// h = x * rsqrt(mean(x^2) + eps) * g; x fp32 residual stream, h in the storage type (the GEMM operand).
// One CTA per row.  For d <= 8192 the row is read once and kept in registers (REGS float4 per thread) between the
// sum of squares and the scaling, and the CTA's NEXT row is already on its way while this one is reduced and
// written (the loads of a persistent CTA otherwise stop during the two barriers and the stores: 0.66 -> 0.75 of
// the copy rate at 6587 rows of 4096); longer rows fall back to a second read.
template <typename T, int REGS>
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const float* __restrict__ x, const T* __restrict__ gain, T* __restrict__ h,
               const int32_t* __restrict__ n_active, int d, float eps) {
  __shared__ float s_part[8];
  // nothing is written and nothing but the gain is read before the wait: the successor (a GEMM that first streams
  // weights) may launch at once
  griddep_launch();
  griddep_wait();
  const int M = *n_active;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nv = d >> 2;                                   // float4 per row
  float4 nxt[REGS > 0 ? REGS : 1];                        // the row after this one, in flight while this one is reduced
  auto fetch = [&](int r) {
    const float4* xr = reinterpret_cast<const float4*>(x + (long long)r * d);
#pragma unroll
    for (int k = 0; k < (REGS > 0 ? REGS : 1); ++k) {
      const int c = threadIdx.x + k * 256;
      nxt[k] = c < nv ? __ldcs(xr + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  if (REGS > 0 && (int)blockIdx.x < M) fetch(blockIdx.x);
  for (int r = blockIdx.x; r < M; r += gridDim.x) {
    const float4* xr = reinterpret_cast<const float4*>(x + (long long)r * d);
    float4 v[REGS > 0 ? REGS : 1];
    float ss = 0.f;
    if (REGS > 0) {
#pragma unroll
      for (int k = 0; k < REGS; ++k) {
        v[k] = nxt[k];
        ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
      }
      if (r + (int)gridDim.x < M) fetch(r + gridDim.x);
    } else {
      for (int c = threadIdx.x; c < nv; c += 256) {
        const float4 t = xr[c];
        ss += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    __syncthreads();   // s_part reuse across rows
    if (lane == 0) s_part[warp] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += s_part[w];
    const float rstd = rsqrtf(tot / (float)d + eps);
    T* hr = h + (long long)r * d;
    auto emit = [&](int c, const float4& t) {
      const int e = c << 2;
      const float o0 = t.x * rstd * to_f(gain[e]), o1 = t.y * rstd * to_f(gain[e + 1]);
      const float o2 = t.z * rstd * to_f(gain[e + 2]), o3 = t.w * rstd * to_f(gain[e + 3]);
      if constexpr (sizeof(T) == 2) {
        __nv_bfloat162 a = __floats2bfloat162_rn(o0, o1), b2 = __floats2bfloat162_rn(o2, o3);
        uint2 pk;
        pk.x = *reinterpret_cast<unsigned*>(&a);
        pk.y = *reinterpret_cast<unsigned*>(&b2);
        *reinterpret_cast<uint2*>(hr + e) = pk;
      } else {
        *reinterpret_cast<float4*>(hr + e) = make_float4(o0, o1, o2, o3);
      }
    };
    if (REGS > 0) {
#pragma unroll
      for (int k = 0; k < REGS; ++k) {
        const int c = threadIdx.x + k * 256;
        if (c < nv) emit(c, v[k]);
      }
    } else {
      for (int c = threadIdx.x; c < nv; c += 256) emit(c, xr[c]);   // second read hits L1/L2
    }
  }
}

// Input of a contraction with the RMSNorm folded in (the layer chain kernel): xg = bf16(x * gain) and, per row and
// 32-column chunk, the sum of squares of x; the contraction's epilogue scales row r by rsqrt(mean x_r^2 + eps).
// One CTA per row, one thread per chunk.
__global__ void __launch_bounds__(128)
norm_prep_kernel(const float* __restrict__ x, const bf16* __restrict__ gain, bf16* __restrict__ xg, float* __restrict__ ssq,
                 const int32_t* __restrict__ n_active, int d) {
  griddep_launch();
  griddep_wait();
  const int M = *n_active, chunks = d >> 5;
  for (int r = blockIdx.x; r < M; r += gridDim.x) {
    for (int ch = threadIdx.x; ch < chunks; ch += 128) {
      const float4* xr = reinterpret_cast<const float4*>(x + (size_t)r * d + ch * 32);
      float4 v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = xr[k];
      float ss = 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
        const uint2 g2 = *reinterpret_cast<const uint2*>(gain + ch * 32 + 4 * k);
        const float2 g01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&g2.x));
        const float2 g23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&g2.y));
        const __nv_bfloat162 a = __floats2bfloat162_rn(v[k].x * g01.x, v[k].y * g01.y);
        const __nv_bfloat162 b = __floats2bfloat162_rn(v[k].z * g23.x, v[k].w * g23.y);
        uint2 pk;
        pk.x = *reinterpret_cast<const unsigned*>(&a);
        pk.y = *reinterpret_cast<const unsigned*>(&b);
        *reinterpret_cast<uint2*>(xg + (size_t)r * d + ch * 32 + 4 * k) = pk;
      }
      ssq[(size_t)r * chunks + ch] = ss;
    }
  }
}

int launch_norm_prep(const float* x, const void* gain, void* xg, float* ssq, const int32_t* n_active, int max_rows, int d,
                     cudaStream_t st) {
  if (d % 32) return SL_EUNSUPPORTED;
  const int g = max_rows < 1 ? 1 : (max_rows > 4 * sm_count() ? 4 * sm_count() : max_rows);
  SL_CUDA_TRY(launch_pdl(norm_prep_kernel, dim3(g), dim3(128), 0, st, x, (const bf16*)gain, (bf16*)xg, ssq, n_active, d));
  return SL_OK;
}

template <typename T>
static int launch_rms_t(const float* x, const void* gain, void* h, const int32_t* n_active, int g, int d, float eps,
                         cudaStream_t st) {
  const int nv = d >> 2;
  if (nv <= 256 * 2) SL_CUDA_TRY(launch_pdl(rmsnorm_kernel<T, 2>, dim3(g), dim3(256), 0, st, x, (const T*)gain, (T*)h, n_active, d, eps));
  else if (nv <= 256 * 4) SL_CUDA_TRY(launch_pdl(rmsnorm_kernel<T, 4>, dim3(g), dim3(256), 0, st, x, (const T*)gain, (T*)h, n_active, d, eps));
  else if (nv <= 256 * 8) SL_CUDA_TRY(launch_pdl(rmsnorm_kernel<T, 8>, dim3(g), dim3(256), 0, st, x, (const T*)gain, (T*)h, n_active, d, eps));
  else SL_CUDA_TRY(launch_pdl(rmsnorm_kernel<T, 0>, dim3(g), dim3(256), 0, st, x, (const T*)gain, (T*)h, n_active, d, eps));
  return SL_OK;
}

int launch_rmsnorm(const float* x, const void* gain, void* h, const int32_t* n_active, int max_rows, int d, float eps,
                   int dtype, cudaStream_t st) {
  if (d % 4) return SL_EUNSUPPORTED;
  const int g = row_grid(max_rows, 4);   // 52 registers with the next row in flight: four CTAs per SM
  const int rc = dtype == SL_BF16 ? launch_rms_t<bf16>(x, gain, h, n_active, g, d, eps, st)
                                  : launch_rms_t<float>(x, gain, h, n_active, g, d, eps, st);
  if (rc != SL_OK) return rc;
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

// ------------------------------------------------------------------------------------------------ RoPE
// table[pos][j] = (cos, sin)(pos * theta^(-2j/d_h)), built once in double precision.
__global__ void rope_table_kernel(float2* table, int N, int half, double theta) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N * half) return;
  const int pos = i / half, j = i % half;
  const double ang = (double)pos * pow(theta, -(double)j / (double)half);
  double s, c;
  sincos(ang, &s, &c);
  table[i] = make_float2((float)c, (float)s);
}

int build_rope_table(float2* table, int N, int head_dim, float theta, cudaStream_t st) {
  const int half = head_dim / 2, n = N * half;
  rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(table, N, half, (double)theta);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

// pair (j, j + d_h/2) of every head of q and k rotated by the angle of position idx[r] % N
template <typename T>
__global__ void __launch_bounds__(256)
rope_kernel(T* __restrict__ q, T* __restrict__ k, const int32_t* __restrict__ idx, const int32_t* __restrict__ n_active,
            int N, int H, int dh, const float2* __restrict__ table) {
  const int M = *n_active;
  const int half = dh >> 1, pairs = H * half;
  for (int r = blockIdx.x; r < M; r += gridDim.x) {
    const int pos = idx[r] % N;
    const float2* tr = table + (long long)pos * half;
    for (int p = threadIdx.x; p < 2 * pairs; p += blockDim.x) {
      T* base = (p < pairs ? q : k) + (long long)r * H * dh;
      const int pp = p < pairs ? p : p - pairs;
      const int h = pp / half, j = pp % half;
      const float2 cs = tr[j];
      T* e = base + h * dh + j;
      const float lo = to_f(e[0]), hi = to_f(e[half]);
      e[0] = from_f<T>(lo * cs.x - hi * cs.y);
      e[half] = from_f<T>(hi * cs.x + lo * cs.y);
    }
  }
}

int launch_rope(void* q, void* k, const int32_t* idx, const int32_t* n_active, int max_rows, int N, int H,
                int head_dim, const float2* table, int dtype, cudaStream_t st) {
  const int g = row_grid(max_rows, 8);
  if (dtype == SL_BF16)
    rope_kernel<bf16><<<g, 256, 0, st>>>((bf16*)q, (bf16*)k, idx, n_active, N, H, head_dim, table);
  else
    rope_kernel<float><<<g, 256, 0, st>>>((float*)q, (float*)k, idx, n_active, N, H, head_dim, table);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

// ------------------------------------------------------------------------------------------------ K/V scatter
// cache row idx[r] <- packed row r, for K and V.  Token-major cache: one row = all heads of one position, so
// both the read and the write of a row are contiguous 128-bit streams.  One warp moves one (row, K|V) pair.
__global__ void __launch_bounds__(256)
kv_scatter_kernel(const uint4* __restrict__ k, const uint4* __restrict__ v, const int32_t* __restrict__ idx,
                  const int32_t* __restrict__ n_active, int row_vec, uint4* __restrict__ kc, uint4* __restrict__ vc) {
  const int M = *n_active;
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  for (int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < 2 * M; w += warps) {
    const int r = w >> 1;
    const uint4* src = ((w & 1) ? v : k) + (long long)r * row_vec;
    uint4* dst = ((w & 1) ? vc : kc) + (long long)idx[r] * row_vec;
    for (int c = lane; c < row_vec; c += 32) dst[c] = __ldg(src + c);
  }
}

int launch_kv_scatter(const void* k, const void* v, const int32_t* idx, const int32_t* n_active, int max_rows,
                      int row_elems, void* kc, void* vc, int dtype, cudaStream_t st) {
  const size_t row_bytes = (size_t)row_elems * (dtype == SL_BF16 ? 2 : 4);
  if (row_bytes % 16) return SL_EUNSUPPORTED;
  int g = (2 * max_rows + 7) / 8;
  const int cap = sm_count() * 8;
  if (g > cap) g = cap;
  if (g < 1) g = 1;
  kv_scatter_kernel<<<g, 256, 0, st>>>((const uint4*)k, (const uint4*)v, idx, n_active, (int)(row_bytes / 16),
                                       (uint4*)kc, (uint4*)vc);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

}  // namespace sl
