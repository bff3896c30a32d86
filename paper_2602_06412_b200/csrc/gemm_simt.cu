// CUDA-core GEMM on packed rows: C[r][n] = sum_k A[r][k] W[n][k], r < M (M read from device memory).
// This is the fp32 path (tiny fp32 model) and the fallback for shapes the tcgen05 kernel does not take; the
// bf16 LLaDA-shaped contractions run on the tensor-core kernel in gemm_tc.cu.  64x64x16 tiles, 4x4 per thread,
// fp32 FMA; the three epilogues match the tensor-core kernel's (store, residual add into the fp32 stream,
// SwiGLU over a gate/up weight pair).
#include "common.cuh"

namespace sl {

constexpr int GS_BM = 64, GS_BN = 64, GS_BK = 16, GS_LD = 68;

template <typename T>
__device__ __forceinline__ void load4(const T* p, bool ok, float (&f)[4]) {
  if (!ok) {
    f[0] = f[1] = f[2] = f[3] = 0.f;
    return;
  }
  if constexpr (sizeof(T) == 2) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&v.x);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&v.y);
    f[0] = __low2float(a); f[1] = __high2float(a); f[2] = __low2float(b); f[3] = __high2float(b);
  } else {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
}

template <typename T, int EPI>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const T* __restrict__ A, const T* __restrict__ W, const T* __restrict__ W2, void* __restrict__ Cv,
                 const int32_t* __restrict__ n_active, int n_out, int K) {
  __shared__ __align__(16) float As[GS_BK][GS_LD];
  __shared__ __align__(16) float Bs[GS_BK][GS_LD];
  __shared__ __align__(16) float B2s[EPI == EPI_SWIGLU ? GS_BK : 1][GS_LD];
  const int M = *n_active;
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  const int lrow = t >> 2, lk = (t & 3) * 4;
  const int n0 = blockIdx.x * GS_BN;
  for (int mt = blockIdx.y; mt * GS_BM < M; mt += gridDim.y) {
    const int m0 = mt * GS_BM;
    float acc[4][4] = {}, acc2[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += GS_BK) {
      float fa[4], fb[4], fb2[4];
      const bool kok = k0 + lk < K;
      load4(A + (long long)(m0 + lrow) * K + k0 + lk, kok && (m0 + lrow) < M, fa);
      load4(W + (long long)(n0 + lrow) * K + k0 + lk, kok && (n0 + lrow) < n_out, fb);
      if (EPI == EPI_SWIGLU) load4(W2 + (long long)(n0 + lrow) * K + k0 + lk, kok && (n0 + lrow) < n_out, fb2);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        As[lk + i][lrow] = fa[i];
        Bs[lk + i][lrow] = fb[i];
        if (EPI == EPI_SWIGLU) B2s[lk + i][lrow] = fb2[i];
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < GS_BK; ++kk) {
        const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
        const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
        const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        if (EPI == EPI_SWIGLU) {
          const float4 b2 = *reinterpret_cast<const float4*>(&B2s[kk][tx * 4]);
          const float b2v[4] = {b2.x, b2.y, b2.z, b2.w};
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc2[i][j] = fmaf(av[i], b2v[j], acc2[i][j]);
        }
      }
      __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = m0 + ty * 4 + i;
      if (r >= M) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = n0 + tx * 4 + j;
        if (c >= n_out) continue;
        const long long o = (long long)r * n_out + c;
        if (EPI == EPI_STORE) {
          reinterpret_cast<T*>(Cv)[o] = from_f<T>(acc[i][j]);
        } else if (EPI == EPI_RESIDUAL) {
          reinterpret_cast<float*>(Cv)[o] += acc[i][j];
        } else {
          const float g = acc[i][j];
          reinterpret_cast<T*>(Cv)[o] = from_f<T>(g / (1.f + __expf(-g)) * acc2[i][j]);
        }
      }
    }
  }
}

template <typename T>
static int launch_t(const void* A, const void* W, const void* W2, void* C, const int32_t* n_active, int max_rows,
                    int n_out, int K, int epilogue, cudaStream_t st) {
  dim3 grid((n_out + GS_BN - 1) / GS_BN, (max_rows + GS_BM - 1) / GS_BM);
  const int cap = (4 * sm_count() + (int)grid.x - 1) / (int)grid.x;   // enough CTAs to fill the GPU, then loop
  if ((int)grid.y > cap) grid.y = cap;
  if (grid.y < 1) grid.y = 1;
  const T *a = (const T*)A, *w = (const T*)W, *w2 = (const T*)W2;
  switch (epilogue) {
    case EPI_STORE: gemm_simt_kernel<T, EPI_STORE><<<grid, 256, 0, st>>>(a, w, w2, C, n_active, n_out, K); break;
    case EPI_RESIDUAL: gemm_simt_kernel<T, EPI_RESIDUAL><<<grid, 256, 0, st>>>(a, w, w2, C, n_active, n_out, K); break;
    case EPI_SWIGLU: gemm_simt_kernel<T, EPI_SWIGLU><<<grid, 256, 0, st>>>(a, w, w2, C, n_active, n_out, K); break;
    default: return SL_EINVAL;
  }
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

int launch_gemm_simt(const void* A, const void* W, const void* W2, void* C, const int32_t* n_active, int max_rows,
                     int n_out, int K, int dtype, int epilogue, cudaStream_t st) {
  if (K % 4) return SL_EUNSUPPORTED;
  return dtype == SL_BF16 ? launch_t<bf16>(A, W, W2, C, n_active, max_rows, n_out, K, epilogue, st)
                          : launch_t<float>(A, W, W2, C, n_active, max_rows, n_out, K, epilogue, st);
}

}  // namespace sl
