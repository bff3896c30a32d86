// Active-row compaction (Algorithm 1, line 6): A_t = { i : lock_i = 0 }, ascending, for a batch of sequences.
//
// The flat index b*N + i is row-major over [B][N], so the whole batch is ONE stream compaction over B*N flags;
// row_offsets[b] is the exclusive count at flat position b*N.  Single pass: every CTA takes a chunk of 4096
// flags (a ticket fixes the chunk order, so a chunk's predecessors have always started), scans it with warp
// shuffles, and obtains its global offset by decoupled look-back over 64-bit (status,value) words.  The
// look-back wait is bounded; when it runs out the CTA records SL_DEV_COMPACT_TIMEOUT and returns.
#include <mutex>

#include "common.cuh"

namespace sl {

constexpr int CP_THREADS = 256;
constexpr int CP_FPT = 16;                        // flags per thread, one 128-bit load
constexpr int CP_CHUNK = CP_THREADS * CP_FPT;     // 4096 flags per CTA
constexpr unsigned CP_SPIN_LIMIT = 1u << 20;      // polls of ~64 ns

struct CompactScratch {
  unsigned int ticket;
  unsigned int pad[3];
  unsigned long long state[1];                    // [chunks]: (status << 32) | value; status 0 empty, 1 aggregate, 2 inclusive
};

size_t compact_scratch_bytes(int64_t total) {
  int64_t chunks = (total + CP_CHUNK - 1) / CP_CHUNK;
  if (chunks < 1) chunks = 1;
  return 16 + 8 * (size_t)chunks;
}

__device__ __forceinline__ unsigned long long ld_relaxed(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__global__ void __launch_bounds__(CP_THREADS)
compact_kernel(const uint8_t* __restrict__ lock, int total, int N, int B, int32_t* __restrict__ idx,
               int32_t* __restrict__ row_offsets, int32_t* __restrict__ n_active, int32_t* __restrict__ row_of_pos,
               CompactScratch* s, int32_t* status) {
  __shared__ unsigned s_chunk;
  __shared__ int s_warp[CP_THREADS / 32];
  __shared__ int s_excl, s_total, s_fail;
  __shared__ int s_out[CP_CHUNK];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    s_chunk = atomicAdd(&s->ticket, 1u);
    s_fail = 0;
  }
  __syncthreads();
  const unsigned chunk = s_chunk;
  if (chunk >= gridDim.x) return;                 // only when the ticket did not start at zero (the diagnostic entry point)
  const long long base = (long long)chunk * CP_CHUNK + (long long)tid * CP_FPT;

  unsigned bits = 0;   // bit k set <=> flag base+k is 0 (active)
  if (base + CP_FPT <= total && ((reinterpret_cast<uintptr_t>(lock) & 15) == 0)) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(lock + base));
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int b = 0; b < 4; ++b)
        if (((w[j] >> (8 * b)) & 0xffu) == 0) bits |= 1u << (4 * j + b);
  } else {
    for (int k = 0; k < CP_FPT; ++k)
      if (base + k < total && lock[base + k] == 0) bits |= 1u << k;
  }
  const int cnt = __popc(bits);
  int inc = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();

  if (warp == 0) {
    int w = lane < CP_THREADS / 32 ? s_warp[lane] : 0;
    int winc = w;
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    const int block_total = __shfl_sync(0xffffffffu, winc, CP_THREADS / 32 - 1);
    if (lane < CP_THREADS / 32) s_warp[lane] = winc - w;   // exclusive prefix of each warp
    if (lane == 0) {
      s_total = block_total;
      st_relaxed(&s->state[chunk], ((chunk == 0 ? 2ull : 1ull) << 32) | (unsigned)block_total);
    }
    int excl = 0, fail = 0;
    if (chunk > 0) {
      long long look = (long long)chunk - 1;
      unsigned spins = 0;
      while (true) {
        const long long j = look - lane;
        const unsigned long long v = j >= 0 ? ld_relaxed(&s->state[j]) : (2ull << 32);   // "inclusive 0" before chunk 0
        const unsigned stt = (unsigned)(v >> 32);
        const unsigned inc_mask = __ballot_sync(0xffffffffu, stt == 2);
        const unsigned empty_mask = __ballot_sync(0xffffffffu, stt == 0);
        const int first_inc = inc_mask ? __ffs(inc_mask) - 1 : 32;
        const unsigned need = first_inc >= 31 ? 0xffffffffu : ((2u << first_inc) - 1u);   // lanes 0..first_inc
        if (empty_mask & need) {
          if (++spins > CP_SPIN_LIMIT) { fail = 1; break; }
          __nanosleep(64);
          continue;
        }
        int val = ((need >> lane) & 1u) ? (int)(unsigned)(v & 0xffffffffull) : 0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) val += __shfl_xor_sync(0xffffffffu, val, o);
        excl += val;
        if (first_inc < 32) break;
        look -= 32;
      }
      if (lane == 0 && !fail) st_relaxed(&s->state[chunk], (2ull << 32) | (unsigned)(excl + block_total));
    }
    if (lane == 0) {
      s_excl = excl;
      s_fail = fail;
    }
  }
  __syncthreads();
  if (s_fail) {
    if (tid == 0) set_status(status, SL_DEV_COMPACT_TIMEOUT);
    return;
  }
  const int chunk_excl = s_excl;
  const int local = s_warp[warp] + (inc - cnt);   // rank of this thread's first active flag inside the chunk

  {
    int o = local;
#pragma unroll
    for (int k = 0; k < CP_FPT; ++k)
      if ((bits >> k) & 1u) s_out[o++] = (int)(base + k);
  }
  if (row_of_pos) {
    if (base + CP_FPT <= total && ((reinterpret_cast<uintptr_t>(row_of_pos) & 15) == 0)) {
      int r[CP_FPT];
      int o = chunk_excl + local;
#pragma unroll
      for (int k = 0; k < CP_FPT; ++k) r[k] = ((bits >> k) & 1u) ? o++ : -1;
      int4* dst = reinterpret_cast<int4*>(row_of_pos + base);
#pragma unroll
      for (int j = 0; j < 4; ++j) dst[j] = make_int4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
    } else {
      int o = chunk_excl + local;
      for (int k = 0; k < CP_FPT; ++k)
        if (base + k < total) row_of_pos[base + k] = ((bits >> k) & 1u) ? o++ : -1;
    }
  }
  // sequence boundaries inside this thread's 16 flags: row_offsets[b] = active rows before flat position b*N
  if (base < total) {
    long long p = ((base + N - 1) / N) * (long long)N;
    for (; p < base + CP_FPT && p < total; p += N) {
      const int k = (int)(p - base);
      row_offsets[p / N] = chunk_excl + local + __popc(bits & ((1u << k) - 1u));
    }
  }
  __syncthreads();
  const int block_total = s_total;
  for (int i = tid; i < block_total; i += CP_THREADS) idx[chunk_excl + i] = s_out[i];
  if (chunk == gridDim.x - 1 && tid == 0) {
    const int M = chunk_excl + block_total;
    *n_active = M;
    row_offsets[B] = M;
  }
}

int launch_compact(const uint8_t* lock, int B, int N, int32_t* idx, int32_t* row_offsets, int32_t* n_active,
                   int32_t* row_of_pos, void* scratch, int32_t* status, cudaStream_t st) {
  if (!lock || !idx || !row_offsets || !n_active || !scratch || B <= 0 || N <= 0) return SL_EINVAL;
  const long long total = (long long)B * N;
  if (total >= (1ll << 31)) return SL_EINVAL;
  const int chunks = (int)((total + CP_CHUNK - 1) / CP_CHUNK);
  SL_CUDA_TRY(cudaMemsetAsync(scratch, 0, compact_scratch_bytes(total), st));
  compact_kernel<<<chunks, CP_THREADS, 0, st>>>(lock, (int)total, N, B, idx, row_offsets, n_active, row_of_pos,
                                                 reinterpret_cast<CompactScratch*>(scratch), status);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

// Diagnostic: the same launch with the ticket counter starting at `first_ticket` instead of 0, as if that many chunks
// had been taken by CTAs that never publish their counts.  Every CTA that does run finds the words of the chunks
// before it empty, polls up to its bound (CP_SPIN_LIMIT polls of 64 ns, about 70 ms), records
// SL_DEV_COMPACT_TIMEOUT and returns: the give-up path of the look-back, reached without hanging or faulting anything.
int launch_compact_from_ticket(const uint8_t* lock, int B, int N, int32_t* idx, int32_t* row_offsets, int32_t* n_active,
                               int32_t* row_of_pos, void* scratch, unsigned first_ticket, int32_t* status, cudaStream_t st) {
  if (!lock || !idx || !row_offsets || !n_active || !scratch || B <= 0 || N <= 0) return SL_EINVAL;
  const long long total = (long long)B * N;
  if (total >= (1ll << 31)) return SL_EINVAL;
  const int chunks = (int)((total + CP_CHUNK - 1) / CP_CHUNK);
  SL_CUDA_TRY(cudaMemsetAsync(scratch, 0, compact_scratch_bytes(total), st));
  SL_CUDA_TRY(cudaMemcpyAsync(scratch, &first_ticket, sizeof(unsigned), cudaMemcpyHostToDevice, st));
  compact_kernel<<<chunks, CP_THREADS, 0, st>>>(lock, (int)total, N, B, idx, row_offsets, n_active, row_of_pos,
                                                 reinterpret_cast<CompactScratch*>(scratch), status);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

// ---- allocation-free variant ---------------------------------------------------------------------------------
// The look-back words live in a fixed array inside the library image instead of caller-provided scratch.
constexpr long long CP_NOALLOC_MAX_FLAGS = 1ll << 24;                                    // 4096 chunks
constexpr size_t CP_NOALLOC_BYTES = 16 + 8 * (size_t)(CP_NOALLOC_MAX_FLAGS / CP_CHUNK);  // 32,784 bytes
static __device__ __align__(256) unsigned char g_compact_scratch[CP_NOALLOC_BYTES];

constexpr int CP_MAX_DEVICES = 64;
static void* g_scratch_addr[CP_MAX_DEVICES];   // device address of g_compact_scratch, per device, filled on first use
static std::mutex g_scratch_mu;

long long compact_noalloc_max_flags() { return CP_NOALLOC_MAX_FLAGS; }

int launch_compact_noalloc(const uint8_t* lock, int B, int N, int32_t* idx, int32_t* row_offsets, int32_t* n_active,
                           int32_t* row_of_pos, int32_t* status, cudaStream_t st) {
  if (!lock || !idx || !row_offsets || !n_active || B <= 0 || N <= 0) return SL_EINVAL;
  const long long total = (long long)B * N;
  if (total > CP_NOALLOC_MAX_FLAGS) return SL_ELIMIT;
  int dev = -1;
  SL_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= CP_MAX_DEVICES) return SL_EUNSUPPORTED;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> g(g_scratch_mu);
    if (!g_scratch_addr[dev]) {
      // In host code the array's name is only a handle; the address a kernel can use comes from the runtime,
      // for the device that is current now.
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_compact_scratch) != cudaSuccess || !p) return SL_ECUDA;
      g_scratch_addr[dev] = p;
    }
    scratch = g_scratch_addr[dev];
  }
  const int chunks = (int)((total + CP_CHUNK - 1) / CP_CHUNK);
  // the array keeps the previous call's words: the ticket and this call's chunk words must start at zero
  SL_CUDA_TRY(cudaMemsetAsync(scratch, 0, 16 + 8 * (size_t)chunks, st));
  compact_kernel<<<chunks, CP_THREADS, 0, st>>>(lock, (int)total, N, B, idx, row_offsets, n_active, row_of_pos,
                                                 reinterpret_cast<CompactScratch*>(scratch), status);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

}  // namespace sl
