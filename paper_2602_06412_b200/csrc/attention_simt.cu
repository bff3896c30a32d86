// CUDA-core M x N attention (Algorithm 1 line 12; Sec. 2.1: packed queries of the active rows against the full
// K/V tables of their sequence, no mask).  One warp owns one (packed row, head) pair and streams all N keys of
// that row's sequence in blocks of 32 with an online softmax.  This is the fp32 path and the fallback; the bf16
// LLaDA-shaped attention runs on the tensor-core kernel.
#include "common.cuh"

namespace sl {

template <typename T, int DH>
__global__ void __launch_bounds__(128)
attention_simt_kernel(const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc,
                      const int32_t* __restrict__ idx, const int32_t* __restrict__ n_active, int N, int H,
                      T* __restrict__ o, float scale) {
  __shared__ float s_q[4][DH];
  __shared__ float s_p[4][32];
  constexpr int VEC = 16 / sizeof(T);
  constexpr int E = DH / 32;
  const int M = *n_active;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long total = (long long)M * H;
  const long long row_stride = (long long)H * DH;
  for (long long w = (long long)blockIdx.x * 4 + warp; w < total; w += (long long)gridDim.x * 4) {
    const int r = (int)(w / H), h = (int)(w % H);
    const int b = idx[r] / N;
    const T* qp = q + ((long long)r * H + h) * DH;
    for (int c = lane; c < DH; c += 32) s_q[warp][c] = to_f(qp[c]) * scale;
    __syncwarp();
    const T* Kb = kc + ((long long)b * N * H + h) * DH;
    const T* Vb = vc + ((long long)b * N * H + h) * DH;
    float m = -INFINITY, l = 0.f, acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    for (int j0 = 0; j0 < N; j0 += 32) {
      const int j = j0 + lane;
      float s = -INFINITY;
      if (j < N) {
        const T* kr = Kb + (long long)j * row_stride;
        s = 0.f;
#pragma unroll
        for (int c = 0; c < DH; c += VEC) {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(kr + c));
          const T* e = reinterpret_cast<const T*>(&v);
#pragma unroll
          for (int k = 0; k < VEC; ++k) s = fmaf(s_q[warp][c + k], to_f(e[k]), s);
        }
      }
      float mx = s;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      const float m_new = fmaxf(m, mx);
      const float p = j < N ? __expf(s - m_new) : 0.f;
      const float corr = __expf(m - m_new);
      float ps = p;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
      l = l * corr + ps;
#pragma unroll
      for (int e = 0; e < E; ++e) acc[e] *= corr;
      s_p[warp][lane] = p;
      __syncwarp();
      const int nj = N - j0 < 32 ? N - j0 : 32;
      for (int jj = 0; jj < nj; ++jj) {
        const float pj = s_p[warp][jj];
        const T* vr = Vb + (long long)(j0 + jj) * row_stride;
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = fmaf(pj, to_f(vr[lane + 32 * e]), acc[e]);
      }
      __syncwarp();
      m = m_new;
    }
    T* op = o + ((long long)r * H + h) * DH;
    const float inv = 1.f / l;
#pragma unroll
    for (int e = 0; e < E; ++e) op[lane + 32 * e] = from_f<T>(acc[e] * inv);
    __syncwarp();
  }
}

int launch_attention_simt(const void* q, const void* kc, const void* vc, const int32_t* idx, const int32_t* n_active,
                          int max_rows, int N, int H, int head_dim, void* o, int dtype, cudaStream_t st) {
  long long warps = (long long)max_rows * H;
  int g = (int)((warps + 3) / 4);
  const int cap = sm_count() * 16;
  if (g > cap) g = cap;
  if (g < 1) g = 1;
  const float scale = 1.0f / sqrtf((float)head_dim);
#define SL_ATT(T, DH) \
  attention_simt_kernel<T, DH><<<g, 128, 0, st>>>((const T*)q, (const T*)kc, (const T*)vc, idx, n_active, N, H, (T*)o, scale)
  if (dtype == SL_BF16 && head_dim == 128) SL_ATT(bf16, 128);
  else if (dtype == SL_BF16 && head_dim == 64) SL_ATT(bf16, 64);
  else if (dtype == SL_FP32 && head_dim == 128) SL_ATT(float, 128);
  else if (dtype == SL_FP32 && head_dim == 64) SL_ATT(float, 64);
  else return SL_EUNSUPPORTED;
#undef SL_ATT
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

}  // namespace sl
