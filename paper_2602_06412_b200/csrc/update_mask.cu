// UpdateMASK on the device (Algorithm 1 line 16): the confidence-ordered unmasking policy, restricted to one
// semi-autoregressive block.  One CTA per sequence.  Per sequence, among the positions lo <= n < hi that are still
// masked (they are always active rows, so they have a posterior), the k with the largest conf = max_v p(v) (ties:
// lowest position) take their argmax token and become unmasked.  k rounds of a block-wide arg-max over the sequence's
// packed rows; a revealed position drops out of the next round because its mask flag is cleared.
#include "common.cuh"

namespace sl {

constexpr int UM_THREADS = 256;

__global__ void __launch_bounds__(UM_THREADS)
update_mask_kernel(const float* __restrict__ conf, const int32_t* __restrict__ argmax, const int32_t* __restrict__ idx,
                   const int32_t* __restrict__ row_offsets, int N, int lo, int hi, int k, int32_t mask_token,
                   int32_t* __restrict__ tokens, uint8_t* __restrict__ mask_state, int32_t* __restrict__ n_revealed) {
  __shared__ float s_conf[UM_THREADS / 32];
  __shared__ int s_row[UM_THREADS / 32];
  __shared__ int s_first, s_last;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r0 = row_offsets[b], r1 = row_offsets[b + 1];
  const long long base = (long long)b * N;
  // the rows of this sequence are sorted by position: narrow [r0, r1) to the block [lo, hi) once
  if (tid == 0) {
    int a = r0, z = r1;
    while (a < z) {                                    // first row with position >= lo
      const int m = (a + z) >> 1;
      if (idx[m] - base < lo) a = m + 1; else z = m;
    }
    s_first = a;
    z = r1;
    while (a < z) {                                    // first row with position >= hi
      const int m = (a + z) >> 1;
      if (idx[m] - base < hi) a = m + 1; else z = m;
    }
    s_last = a;
  }
  __syncthreads();
  const int f = s_first, l = s_last;
  int revealed = 0;
  for (int round = 0; round < k; ++round) {
    float best = -1.f;                                 // conf >= 0; -1 = none
    int best_row = -1;
    for (int r = f + tid; r < l; r += UM_THREADS) {    // rows ascend with position: the first maximum wins ties
      if (mask_state[idx[r]] == 1) {
        const float c = conf[r];
        if (c > best) {
          best = c;
          best_row = r;
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float oc = __shfl_down_sync(0xffffffffu, best, o);
      const int orow = __shfl_down_sync(0xffffffffu, best_row, o);
      if (orow >= 0 && (oc > best || (oc == best && (best_row < 0 || orow < best_row)))) {
        best = oc;
        best_row = orow;
      }
    }
    if (lane == 0) {
      s_conf[warp] = best;
      s_row[warp] = best_row;
    }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < UM_THREADS / 32; ++w) {
        const float oc = s_conf[w];
        const int orow = s_row[w];
        if (orow >= 0 && (oc > best || (oc == best && (best_row < 0 || orow < best_row)))) {
          best = oc;
          best_row = orow;
        }
      }
      if (best_row >= 0) {
        const int pos = idx[best_row];
        const int32_t tok = argmax[best_row];
        tokens[pos] = tok == mask_token ? 0 : tok;     // a sampler never emits the mask token
        mask_state[pos] = 0;
        ++revealed;
      }
      s_row[0] = best_row;
    }
    __syncthreads();                                   // the cleared flag is visible to the next round
    if (s_row[0] < 0) break;                           // nothing left to reveal in this block
    __syncthreads();
  }
  if (tid == 0 && n_revealed) n_revealed[b] = revealed;
}

int launch_update_mask(const float* conf, const int32_t* argmax, const int32_t* idx, const int32_t* row_offsets, int B,
                       int N, int lo, int hi, int k, int32_t mask_token, int32_t* tokens, uint8_t* mask_state,
                       int32_t* n_revealed, cudaStream_t st) {
  update_mask_kernel<<<B, UM_THREADS, 0, st>>>(conf, argmax, idx, row_offsets, N, lo, hi, k, mask_token, tokens,
                                               mask_state, n_revealed);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

}  // namespace sl
