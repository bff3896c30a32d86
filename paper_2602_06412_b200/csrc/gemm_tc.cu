// Tensor-core GEMM for the packed active rows on sm_100a: C[r][n] = sum_k A[r][k] W[n][k], bf16 in, fp32 accumulate
// (the Q/K/V, output, SwiGLU and LM-head contractions of Algorithm 1 lines 10, 12 and 15).
//
// Persistent, warp-specialised CTAs, one per SM:
//   warp 0   TMA producer: cp.async.bulk.tensor loads of a 128x64 A tile and two 128x64 W tiles per stage into
//            128-byte-swizzled shared memory, completion counted on an mbarrier (no multicast);
//   warp 1   allocates tensor memory and issues tcgen05.mma (128 x BN x 16, cta_group::1) from one thread, operands
//            described by shared-memory matrix descriptors; tcgen05.commit hands smem stages back to the producer
//            and finished accumulators to the epilogue;
//   warps 2-5 epilogue: tcgen05.ld the fp32 accumulator (one row per thread), apply the fused operation
//            (store bf16 | add into the fp32 residual stream | silu(gate)*up | QKV: rotary embedding on q and k with
//            the row's ORIGINAL position, q stored packed, k and v written straight into the cache row of that
//            position, which is Algorithm 1 line 11 done in the epilogue) and write with 128-bit stores.
// Two accumulators live in tensor memory so the epilogue of tile i overlaps the main loop of tile i+1.
// The number of rows M is read from device memory: tiles whose first row is >= M are never scheduled, TMA zero-fills
// rows beyond the allocation, and the epilogue stores only rows < M.  Every mbarrier wait is bounded: when it runs out
// the CTA records SL_DEV_GEMM_TIMEOUT, all roles leave their loops, tensor memory is freed and the kernel returns.
#include <mutex>
#include <unordered_map>

#include "tc_common.cuh"

namespace sl {

constexpr int TC_BM = 128, TC_BK = 64, TC_THREADS = 192;
constexpr int EPI_QKV = 3;   // three weight matrices side by side; epilogue = RoPE + packed q + K/V cache scatter

struct QkvArgs {
  bf16 *q, *kc, *vc;          // q packed [M][hd]; caches [B*N][hd]
  const int32_t* idx;         // [M] flat position of each packed row
  const float2* rope;         // [n_seq][dh/2] (cos, sin)
  int n_seq, hd, dh;
};

// ----------------------------------------------------------------------------------------------- kernel
template <int EPI, int BN, int STAGES>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2, void* __restrict__ Cv,
               const int32_t* __restrict__ n_active, int n_out, int K, int32_t* status, const QkvArgs qkv) {
  constexpr int A_BYTES = TC_BM * TC_BK * 2;              // 16 KB
  constexpr int B_BYTES = BN * TC_BK * 2;                 // 32 KB (two 128-row halves)
  constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr int OUT_BN = EPI == EPI_SWIGLU ? BN / 2 : BN; // output columns per tile
  constexpr uint32_t TMEM_COLS = 2 * BN;                  // two accumulators
  static_assert(TMEM_COLS == 512 || TMEM_COLS == 256, "tensor memory allocation must be a power of two");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  // bars: full[STAGES], empty[STAGES], acc_full[2], acc_empty[2]
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto accf_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
  auto acce_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accf_bar(a), 1);
      mbar_init(acce_bar(a), 4);
    }
    *s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) tc_alloc(smem_u32(s_tmem), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;

  const int M = *n_active;
  const int m_tiles = (M + TC_BM - 1) / TC_BM;
  const int n_tiles = (n_out + OUT_BN - 1) / OUT_BN;
  const int total = m_tiles * n_tiles;
  const int num_kb = (K + TC_BK - 1) / TC_BK;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
        const int m0 = (t % m_tiles) * TC_BM, n0 = (t / m_tiles) * OUT_BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1, s_abort))) break;
          const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES), sb = sa + A_BYTES;
          mbar_expect_tx(full_bar(stage), STAGE_BYTES);
          tma_load_2d(sa, &tmA, kb * TC_BK, m0, full_bar(stage));
          if (EPI == EPI_SWIGLU) {
            tma_load_2d(sb, &tmB0, kb * TC_BK, n0, full_bar(stage));
            tma_load_2d(sb + B_BYTES / 2, &tmB1, kb * TC_BK, n0, full_bar(stage));
          } else if (EPI == EPI_QKV) {
            const int src = n0 / qkv.hd, ln0 = n0 - src * qkv.hd;      // a tile never straddles two matrices
            const CUtensorMap* mp = src == 0 ? &tmB0 : (src == 1 ? &tmB1 : &tmB2);
#pragma unroll
            for (int hb = 0; hb < BN / 128; ++hb)
              tma_load_2d(sb + hb * (B_BYTES / (BN / 128)), mp, kb * TC_BK, ln0 + hb * 128, full_bar(stage));
          } else {
#pragma unroll
            for (int hb = 0; hb < BN / 128; ++hb)
              tma_load_2d(sb + hb * (B_BYTES / (BN / 128)), &tmB0, kb * TC_BK, n0 + hb * 128, full_bar(stage));
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_m128(BN);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x, ++it) {
        const int acc = it & 1;
        const uint32_t use = (uint32_t)(it >> 1);
        if (!(ok = mbar_wait(acce_bar(acc), (use & 1) ^ 1, s_abort))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!(ok = mbar_wait(full_bar(stage), phase, s_abort))) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES), sb = sa + A_BYTES;
          const uint64_t adesc = smem_desc_k_sw128(sa), bdesc = smem_desc_k_sw128(sb);
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k)   // 16 bf16 = 32 bytes along K inside the 128-byte swizzle row
            tc_mma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (kb | k) != 0);
          tc_commit(empty_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) tc_commit(accf_bar(acc));
      }
    }
  } else {
    const int quarter = warp & 3;             // tensor-memory lanes 32*quarter .. 32*quarter+31
    bool ok = true;
    int it = 0;
    for (int t = blockIdx.x; t < total && ok; t += gridDim.x, ++it) {
      const int acc = it & 1;
      const uint32_t use = (uint32_t)(it >> 1);
      const int m0 = (t % m_tiles) * TC_BM, n0 = (t / m_tiles) * OUT_BN;
      ok = mbar_wait(accf_bar(acc), use & 1, s_abort);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = m0 + quarter * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
      if (EPI == EPI_QKV) {
        const int src = n0 / qkv.hd, ln0 = n0 - src * qkv.hd;
        const bool live = row < M;
        const int pos = live ? qkv.idx[row] : 0;
        bf16* drow = src == 0 ? qkv.q + (long long)row * qkv.hd
                              : (src == 1 ? qkv.kc : qkv.vc) + (long long)pos * qkv.hd;
        if (src == 2) {
#pragma unroll 1
          for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t v[32];
            tc_ld32(taddr + c0, v);
            tc_wait_ld();
            if (live) {
#pragma unroll
              for (int j = 0; j < 32; j += 8)
                *reinterpret_cast<uint4*>(drow + ln0 + c0 + j) =
                    make_uint4(pack_bf16(__uint_as_float(v[j]), __uint_as_float(v[j + 1])),
                               pack_bf16(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3])),
                               pack_bf16(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5])),
                               pack_bf16(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7])));
            }
          }
        } else {
          const int half = qkv.dh >> 1;
          const float2* tr = qkv.rope + (long long)(pos % qkv.n_seq) * half;
#pragma unroll 1
          for (int hh = 0; hh < BN; hh += qkv.dh) {            // heads inside this tile
#pragma unroll 1
            for (int cc = 0; cc < half; cc += 32) {              // pair (j, j + dh/2), 32 pairs at a time
              uint32_t lo[32], hi[32];
              tc_ld32(taddr + hh + cc, lo);
              tc_ld32(taddr + hh + half + cc, hi);
              tc_wait_ld();
              if (live) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  const float2 cs = __ldg(tr + cc + j);
                  const float a = __uint_as_float(lo[j]), b = __uint_as_float(hi[j]);
                  lo[j] = __float_as_uint(a * cs.x - b * cs.y);
                  hi[j] = __float_as_uint(b * cs.x + a * cs.y);
                }
                bf16* d0 = drow + ln0 + hh + cc;
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                  *reinterpret_cast<uint4*>(d0 + j) =
                      make_uint4(pack_bf16(__uint_as_float(lo[j]), __uint_as_float(lo[j + 1])),
                                 pack_bf16(__uint_as_float(lo[j + 2]), __uint_as_float(lo[j + 3])),
                                 pack_bf16(__uint_as_float(lo[j + 4]), __uint_as_float(lo[j + 5])),
                                 pack_bf16(__uint_as_float(lo[j + 6]), __uint_as_float(lo[j + 7])));
                  *reinterpret_cast<uint4*>(d0 + half + j) =
                      make_uint4(pack_bf16(__uint_as_float(hi[j]), __uint_as_float(hi[j + 1])),
                                 pack_bf16(__uint_as_float(hi[j + 2]), __uint_as_float(hi[j + 3])),
                                 pack_bf16(__uint_as_float(hi[j + 4]), __uint_as_float(hi[j + 5])),
                                 pack_bf16(__uint_as_float(hi[j + 6]), __uint_as_float(hi[j + 7])));
                }
              }
            }
          }
        }
      } else
#pragma unroll 1
      for (int c0 = 0; c0 < OUT_BN; c0 += 32) {
        uint32_t v[32];
        tc_ld32(taddr + c0, v);
        if (EPI == EPI_SWIGLU) {
          uint32_t u[32];
          tc_ld32(taddr + OUT_BN + c0, u);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float g = __uint_as_float(v[j]);
            v[j] = __float_as_uint(g / (1.f + __expf(-g)) * __uint_as_float(u[j]));
          }
        } else {
          tc_wait_ld();
        }
        const int col = n0 + c0;
        if (row < M && col < n_out) {
          if (EPI == EPI_RESIDUAL) {
            float* dst = reinterpret_cast<float*>(Cv) + (long long)row * n_out + col;
            if (col + 32 <= n_out) {
#pragma unroll
              for (int j = 0; j < 32; j += 4) {
                float4 o = *reinterpret_cast<float4*>(dst + j);
                o.x += __uint_as_float(v[j]); o.y += __uint_as_float(v[j + 1]);
                o.z += __uint_as_float(v[j + 2]); o.w += __uint_as_float(v[j + 3]);
                *reinterpret_cast<float4*>(dst + j) = o;
              }
            } else {
              for (int j = 0; j < 32 && col + j < n_out; ++j) dst[j] += __uint_as_float(v[j]);
            }
          } else {
            bf16* dst = reinterpret_cast<bf16*>(Cv) + (long long)row * n_out + col;
            if (col + 32 <= n_out) {
#pragma unroll
              for (int j = 0; j < 32; j += 8) {
                uint4 o;
                o.x = pack_bf16(__uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                o.y = pack_bf16(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                o.z = pack_bf16(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5]));
                o.w = pack_bf16(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7]));
                *reinterpret_cast<uint4*>(dst + j) = o;
              }
            } else {
              for (int j = 0; j < 32 && col + j < n_out; ++j) dst[j] = __float2bfloat16_rn(__uint_as_float(v[j]));
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acce_bar(acc));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *s_abort) set_status(status, SL_DEV_GEMM_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tc_dealloc(tmem_base, TMEM_COLS);
  }
}

// ----------------------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

struct MapKey {
  const void* ptr;
  long long rows, cols;
  int box_rows;
  bool operator==(const MapKey& o) const { return ptr == o.ptr && rows == o.rows && cols == o.cols && box_rows == o.box_rows; }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    return std::hash<const void*>()(k.ptr) ^ (std::hash<long long>()(k.rows) * 31) ^ (std::hash<long long>()(k.cols) * 131) ^
           (size_t)k.box_rows;
  }
};

// 2-D bf16 row-major [rows][cols] tensor, box = box_rows x 64 elements, 128-byte swizzle, zero fill out of bounds
int get_tensor_map_2d(const void* ptr, long long rows, long long cols, int box_rows, CUtensorMap* out) {
  static std::mutex mu;
  static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
  const MapKey key{ptr, rows, cols, box_rows};
  std::lock_guard<std::mutex> g(mu);
  auto it = cache.find(key);
  if (it != cache.end()) {
    *out = it->second;
    return SL_OK;
  }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return SL_ECUDA;
  CUtensorMap m;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return SL_ECUDA;
  if (cache.size() > 4096) cache.clear();
  cache.emplace(key, m);
  *out = m;
  return SL_OK;
}

template <int EPI, int BN, int STAGES>
static int launch_cfg(const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1, const CUtensorMap& b2, void* C,
                      const int32_t* n_active, int max_rows, int n_out, int K, int32_t* status, const QkvArgs& qkv,
                      cudaStream_t st) {
  constexpr int SMEM = STAGES * (TC_BM * TC_BK * 2 + BN * TC_BK * 2) + 1024 + 256;
  static bool attr_set = false;
  if (!attr_set) {
    SL_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<EPI, BN, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM));
    attr_set = true;
  }
  constexpr int OUT_BN = EPI == EPI_SWIGLU ? BN / 2 : BN;
  const long long tiles = (long long)((max_rows + TC_BM - 1) / TC_BM) * ((n_out + OUT_BN - 1) / OUT_BN);
  int grid = sm_count();
  if (tiles < grid) grid = (int)tiles;
  if (grid < 1) grid = 1;
  gemm_tc_kernel<EPI, BN, STAGES><<<grid, TC_THREADS, SMEM, st>>>(a, b0, b1, b2, C, n_active, n_out, K, status, qkv);
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

int launch_gemm_tc(const void* A, const void* W, const void* W2, void* C, const int32_t* n_active, int max_rows,
                   int n_out, int K, int epilogue, int32_t* status, cudaStream_t st) {
  // TMA needs 16-byte aligned bases and row strides; the epilogue's 128-bit stores need n_out % 8 == 0
  if (K % 8 || n_out % 8 || max_rows < 1) return SL_EUNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(W2) |
       reinterpret_cast<uintptr_t>(C)) & 15)
    return SL_EUNSUPPORTED;
  if (epilogue == EPI_SWIGLU && !W2) return SL_EINVAL;
  CUtensorMap a, b0, b1;
  {
    int rc = get_tensor_map_2d(A, max_rows, K, TC_BM, &a);
    if (rc != SL_OK) return rc;
    rc = get_tensor_map_2d(W, n_out, K, 128, &b0);
    if (rc != SL_OK) return rc;
    b1 = b0;
    if (W2) {
      rc = get_tensor_map_2d(W2, n_out, K, 128, &b1);
      if (rc != SL_OK) return rc;
    }
  }
  switch (epilogue) {
    case EPI_STORE: return launch_cfg<EPI_STORE, 256, 4>(a, b0, b1, b1, C, n_active, max_rows, n_out, K, status, QkvArgs{}, st);
    case EPI_RESIDUAL: return launch_cfg<EPI_RESIDUAL, 256, 4>(a, b0, b1, b1, C, n_active, max_rows, n_out, K, status, QkvArgs{}, st);
    case EPI_SWIGLU: return launch_cfg<EPI_SWIGLU, 256, 4>(a, b0, b1, b1, C, n_active, max_rows, n_out, K, status, QkvArgs{}, st);
    default: return SL_EINVAL;
  }
}

// Q/K/V projections in one launch with RoPE and the cache scatter in the epilogue (Algorithm 1 lines 10-11).
int launch_gemm_tc_qkv(const void* A, const void* Wq, const void* Wk, const void* Wv, void* q_out, void* k_cache,
                       void* v_cache, const int32_t* idx, const float2* rope, const int32_t* n_active, int max_rows,
                       int n_seq, int hd, int dh, int K, int32_t* status, cudaStream_t st) {
  if (K % 8 || hd % 256 || (dh != 64 && dh != 128) || max_rows < 1) return SL_EUNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(Wq) | reinterpret_cast<uintptr_t>(Wk) |
       reinterpret_cast<uintptr_t>(Wv) | reinterpret_cast<uintptr_t>(q_out) | reinterpret_cast<uintptr_t>(k_cache) |
       reinterpret_cast<uintptr_t>(v_cache)) & 15)
    return SL_EUNSUPPORTED;
  CUtensorMap a, b0, b1, b2;
  int rc = get_tensor_map_2d(A, max_rows, K, TC_BM, &a);
  if (rc == SL_OK) rc = get_tensor_map_2d(Wq, hd, K, 128, &b0);
  if (rc == SL_OK) rc = get_tensor_map_2d(Wk, hd, K, 128, &b1);
  if (rc == SL_OK) rc = get_tensor_map_2d(Wv, hd, K, 128, &b2);
  if (rc != SL_OK) return rc;
  QkvArgs qa{(bf16*)q_out, (bf16*)k_cache, (bf16*)v_cache, idx, rope, n_seq, hd, dh};
  return launch_cfg<EPI_QKV, 256, 4>(a, b0, b1, b2, nullptr, n_active, max_rows, 3 * hd, K, status, qa, st);
}

}  // namespace sl
