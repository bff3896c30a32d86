// Optional precondition check of a step: a position that enters the step locked must have valid K/V in every
// layer's cache, i.e. it was an active row of an earlier step since the last reset, or the caller declared the caches
// filled (Algorithm 1 line 12 reads the frozen K/V of the locked rows; nothing else can tell whether they were ever
// written).  One flag byte per position; a violation records SL_DEV_STALE_CACHE in the status word and the step goes
// on.  Positions that are active in this step become valid (line 11 writes their K/V).
#include "common.cuh"

namespace sl {

__global__ void __launch_bounds__(256)
cache_check_kernel(const uint8_t* __restrict__ lock, uint8_t* __restrict__ kv_valid, int total, int32_t* status) {
  bool bad = false;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    if (lock[i]) {
      bad |= kv_valid[i] == 0;
    } else {
      kv_valid[i] = 1;
    }
  }
  if (__syncthreads_or(bad) && threadIdx.x == 0) set_status(status, SL_DEV_STALE_CACHE);
}

int launch_cache_check(const uint8_t* lock, uint8_t* kv_valid, int total, int32_t* status, cudaStream_t st) {
  if (total <= 0) return SL_OK;
  int grid = (total + 255) / 256;
  if (grid > 4 * sm_count()) grid = 4 * sm_count();
  cache_check_kernel<<<grid, 256, 0, st>>>(lock, kv_valid, total, status);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

}  // namespace sl
