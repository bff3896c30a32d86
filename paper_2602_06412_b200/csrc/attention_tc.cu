// Tensor-core M x N attention on sm_100a (Algorithm 1 line 12; Sec. 2.1: the packed queries of the active rows
// attend to ALL N cached keys/values of their sequence, bidirectional, no mask).
//
// Work item = (sequence b, head h, tile of up to 128 consecutive packed rows of that sequence); items never
// straddle sequences.  Persistent CTAs take items round-robin; the q-tile index runs fastest so CTAs working at the
// same time read the same K/V head through L2.  Per item the keys are streamed in blocks of 128:
//   warp 0    TMA producer: Q tile once, then K and V blocks (two stages each), token-major cache rows, 128-byte swizzle;
//   warp 1    one thread issues S = Q K^T (tcgen05.mma, 128x128xd_h, accumulator in tensor memory, two S buffers so
//             S of block j+1 is computed while block j is in the softmax) and O += P V (V is the MN-major operand);
//   warps 2-9 softmax: two threads share one query row, 64 of the block's 128 scores each (the exponentials of a block
//             are bound by the SM's 16 special-function results per clock, so all four schedulers carry two softmax
//             warps): tcgen05.ld the scores, online max / sum in fp32 with the 1/sqrt(d_h) scale folded into an exp2
//             (each thread also reads its partner's 64 scores for the row maximum: cheaper than an exchange),
//             P written as bf16 into swizzled shared memory.
//             O stays in tensor memory; it is rescaled (tcgen05.ld / st) only when a row's running maximum grows by
//             more than 2^8, so after the first blocks the correction is almost never taken.  The final O / l is
//             stored as bf16.
// Keys beyond N in the last block are masked to -inf.  All waits are bounded (SL_DEV_ATTN_TIMEOUT).
#include <stdio.h>

#include "tc_common.cuh"

namespace sl {

constexpr int AT_THREADS = 320;   // TMA warp, MMA warp, 8 softmax warps (two per tensor-memory lane quarter)
constexpr int AT_BQ = 128, AT_BKV = 128;
constexpr int AT_MAX_B = 1024;

template <int DH>
__global__ void __launch_bounds__(AT_THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const int32_t* __restrict__ row_offsets, int B, int N, int H,
                    bf16* __restrict__ o, float scale_log2, int32_t* status, unsigned long long* prof) {
  constexpr int SLABS = DH / 64;                       // 64-element (128-byte) column blocks per row
  constexpr int SLAB_BYTES = 128 * 128;                // 128 rows x 128 bytes
  constexpr int Q_BYTES = SLABS * SLAB_BYTES;
  constexpr int KV_BYTES = SLABS * SLAB_BYTES;         // one K or V block of 128 keys
  constexpr int P_BYTES = 2 * SLAB_BYTES;              // 128 queries x 128 keys, bf16
  constexpr uint32_t TMEM_COLS = 512;                  // S0 [0,128) S1 [128,256) O [256,256+DH)
  constexpr uint32_t O_COL = 256;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + Q_BYTES;                          // 2 stages
  uint8_t* sV = sK + 2 * KV_BYTES;                     // 2 stages
  uint8_t* sP = sV + 2 * KV_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sP + P_BYTES);
  // q_full, q_free, k_full[2], k_free[2], v_full[2], v_free[2], s_full[2], s_free[2], p_full, p_free, o_free,
  // x_sum (the two threads of a row add their partial sums here; an mbarrier, so that this wait is bounded too)
  enum { Q_FULL = 0, Q_FREE, K_FULL, K_FREE = K_FULL + 2, V_FULL = K_FREE + 2, V_FREE = V_FULL + 2, S_FULL = V_FREE + 2,
         S_FREE = S_FULL + 2, P_FULL = S_FREE + 2, P_FREE, O_FREE, X_SUM, NUM_BARS };
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  float* s_xsum = reinterpret_cast<float*>(s_tmem + 2);    // [2 halves][128 rows] partial row sums at the end of an item
  int* s_prefix = reinterpret_cast<int*>(s_xsum + 256);  // [B+1] work-item prefix per sequence

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto bar = [&](int i) { return bar0 + 8u * i; };

  if (threadIdx.x == 0) {
    for (int i = 0; i < NUM_BARS; ++i) {
      uint32_t cnt = 1;
      if (i == S_FREE || i == S_FREE + 1 || i == O_FREE) cnt = 8;
      if (i == P_FULL || i == X_SUM) cnt = 8;   // one elected arrival per softmax warp
      mbar_init(bar(i), cnt);
    }
    *s_abort = 0;
    fence_mbar_init();
    int acc = 0;
    s_prefix[0] = 0;
    for (int b = 0; b < B; ++b) {
      const int mb = row_offsets[b + 1] - row_offsets[b];
      acc += ((mb + AT_BQ - 1) / AT_BQ) * H;
      s_prefix[b + 1] = acc;
    }
  }
  if (warp == 1) tc_alloc(smem_u32(s_tmem), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const int total = s_prefix[B];
  const int nblk = (N + AT_BKV - 1) / AT_BKV;

  // item -> (b, h, first packed row, rows in tile)
  auto decode = [&](int w, int& b, int& h, int& row0, int& nrows) {
    int lo = 0, hi = B;                                 // largest b with prefix[b] <= w
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_prefix[mid] <= w) lo = mid; else hi = mid;
    }
    b = lo;
    const int r0 = row_offsets[b], mb = row_offsets[b + 1] - r0;
    const int tiles = (mb + AT_BQ - 1) / AT_BQ;
    const int local = w - s_prefix[b];
    h = local / tiles;
    const int qt = local % tiles;
    row0 = r0 + qt * AT_BQ;
    nrows = mb - qt * AT_BQ < AT_BQ ? mb - qt * AT_BQ : AT_BQ;
  };

  if (warp == 0) {
    if (lane == 0) {
      uint32_t kcnt = 0, qcnt = 0;
      bool ok = true;
      for (int w = blockIdx.x; w < total && ok; w += gridDim.x, ++qcnt) {
        int b, h, row0, nrows;
        decode(w, b, h, row0, nrows);
        if (!(ok = mbar_wait(bar(Q_FREE), (qcnt & 1) ^ 1, s_abort))) break;
        mbar_expect_tx(bar(Q_FULL), Q_BYTES);
#pragma unroll
        for (int s = 0; s < SLABS; ++s) tma_load_2d(smem_u32(sQ + s * SLAB_BYTES), &tmQ, h * DH + 64 * s, row0, bar(Q_FULL));
        for (int j = 0; j < nblk; ++j, ++kcnt) {
          const int st = kcnt & 1;
          const uint32_t ph = (kcnt >> 1) & 1;
          const int key0 = b * N + j * AT_BKV;
          if (!(ok = mbar_wait(bar(K_FREE + st), ph ^ 1, s_abort))) break;
          mbar_expect_tx(bar(K_FULL + st), KV_BYTES);
#pragma unroll
          for (int s = 0; s < SLABS; ++s)
            tma_load_2d(smem_u32(sK + st * KV_BYTES + s * SLAB_BYTES), &tmK, h * DH + 64 * s, key0, bar(K_FULL + st));
          if (!(ok = mbar_wait(bar(V_FREE + st), ph ^ 1, s_abort))) break;
          mbar_expect_tx(bar(V_FULL + st), KV_BYTES);
#pragma unroll
          for (int s = 0; s < SLABS; ++s)
            tma_load_2d(smem_u32(sV + st * KV_BYTES + s * SLAB_BYTES), &tmV, h * DH + 64 * s, key0, bar(V_FULL + st));
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16_m128(AT_BKV, false);
      constexpr uint32_t idesc_o = idesc_bf16_m128(DH, true);
      uint32_t g = 0, it = 0;
      bool ok = true;
      // S(gi) = Q K^T for global block gi into S buffer gi & 1
      auto issue_s = [&](uint32_t gi) -> bool {
        const int st = gi & 1;
        const uint32_t ph = (gi >> 1) & 1;
        if (!mbar_wait(bar(K_FULL + st), ph, s_abort)) return false;
        if (!mbar_wait(bar(S_FREE + st), ph ^ 1, s_abort)) return false;
        tc_fence_after();
        const uint32_t qa = smem_u32(sQ), ka = smem_u32(sK + st * KV_BYTES);
#pragma unroll
        for (int kk = 0; kk < DH / 16; ++kk) {
          const uint32_t off = (kk >> 2) * SLAB_BYTES + (kk & 3) * 32;
          tc_mma_bf16(tmem_base + st * 128, smem_desc_k_sw128(qa + off), smem_desc_k_sw128(ka + off), idesc_s, kk != 0);
        }
        tc_commit(bar(K_FREE + st));
        tc_commit(bar(S_FULL + st));
        return true;
      };
      for (int w = blockIdx.x; w < total && ok; w += gridDim.x, ++it) {
        if (!(ok = mbar_wait(bar(Q_FULL), it & 1, s_abort))) break;
        if (!(ok = issue_s(g))) break;
        for (int j = 0; j < nblk && ok; ++j) {
          const uint32_t gj = g + j;
          if (j + 1 < nblk) {
            if (!(ok = issue_s(gj + 1))) break;
          } else {
            tc_commit(bar(Q_FREE));                      // every S MMA of this item has been issued
          }
          const int st = gj & 1;
          const uint32_t ph = (gj >> 1) & 1;
          if (!(ok = mbar_wait(bar(P_FULL), gj & 1, s_abort))) break;
          if (!(ok = mbar_wait(bar(V_FULL + st), ph, s_abort))) break;
          if (j == 0 && !(ok = mbar_wait(bar(O_FREE), (it & 1) ^ 1, s_abort))) break;
          tc_fence_after();
          const uint32_t pa = smem_u32(sP), va = smem_u32(sV + st * KV_BYTES);
#pragma unroll
          for (int kk = 0; kk < AT_BKV / 16; ++kk) {
            const uint64_t ad = smem_desc_k_sw128(pa + (kk >> 2) * SLAB_BYTES + (kk & 3) * 32);
            const uint64_t bd = smem_desc_mn_sw128(va + kk * 16 * 128, SLAB_BYTES);
            tc_mma_bf16(tmem_base + O_COL, ad, bd, idesc_o, (j | kk) != 0);
          }
          tc_commit(bar(V_FREE + st));
          tc_commit(bar(P_FREE));
        }
        g += nblk;
      }
    }
  } else {
    const int quarter = warp & 3;
    const int half = (warp - 2) >> 2;                    // which 64 of the block's 128 keys (and which half of O)
    const int trow = quarter * 32 + lane;                // query row of this thread inside the tile
    const uint32_t tlane = (uint32_t)(quarter * 32) << 16;
    constexpr int OH = DH / 2;                           // O columns per thread
    uint32_t g = 0, it = 0;
    bool ok = true;
#ifdef ATT_PROFILE
    unsigned long long tp[8] = {0, 0, 0, 0, 0, 0, 0, 0}, t0 = clock64(), t1;
#define ATT_T(i) { t1 = clock64(); tp[i] += t1 - t0; t0 = t1; }
#else
#define ATT_T(i)
#endif
    for (int w = blockIdx.x; w < total && ok; w += gridDim.x, ++it) {
      int b, h, row0, nrows;
      decode(w, b, h, row0, nrows);
      float m_used = 0.f, l = 0.f;
      for (int j = 0; j < nblk; ++j) {
        const uint32_t gj = g + j;
        const int sb = gj & 1;
        const uint32_t ph = (gj >> 1) & 1;
        ATT_T(0)
        ok = __all_sync(0xffffffffu, mbar_wait(bar(S_FULL + sb), ph, s_abort));
        if (!ok) break;
        ATT_T(1)
        tc_fence_after();
        // this thread's 64 scores, and the partner's 64 as well: the row maximum needs all 128, and reading them from
        // tensor memory in the same batch is cheaper than an exchange through shared memory
        uint32_t s[64], t[64];
        tc_ld32(tmem_base + tlane + sb * 128 + half * 64, s);
        tc_ld32(tmem_base + tlane + sb * 128 + half * 64 + 32, s + 32);
        tc_ld32(tmem_base + tlane + sb * 128 + (half ^ 1) * 64, t);
        tc_ld32(tmem_base + tlane + sb * 128 + (half ^ 1) * 64 + 32, t + 32);
        tc_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(S_FREE + sb));
        ATT_T(2)
        const int nvalid = N - j * AT_BKV - half * 64;   // keys of this thread's 64 that exist
        if (nvalid < 64) {
#pragma unroll
          for (int c = 0; c < 64; ++c)
            if (c >= nvalid) s[c] = 0xff800000u;         // -inf
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four independent chains
#pragma unroll
        for (int c = 0; c < 64; c += 4) {
          mx4[0] = fmaxf(mx4[0], __uint_as_float(s[c]));
          mx4[1] = fmaxf(mx4[1], __uint_as_float(s[c + 1]));
          mx4[2] = fmaxf(mx4[2], __uint_as_float(s[c + 2]));
          mx4[3] = fmaxf(mx4[3], __uint_as_float(s[c + 3]));
        }
        {
          const int ovalid = N - j * AT_BKV - (half ^ 1) * 64;
          if (ovalid >= 64) {
#pragma unroll
            for (int c = 0; c < 64; c += 4) {
              mx4[0] = fmaxf(mx4[0], __uint_as_float(t[c]));
              mx4[1] = fmaxf(mx4[1], __uint_as_float(t[c + 1]));
              mx4[2] = fmaxf(mx4[2], __uint_as_float(t[c + 2]));
              mx4[3] = fmaxf(mx4[3], __uint_as_float(t[c + 3]));
            }
          } else {
#pragma unroll
            for (int c = 0; c < 64; ++c)
              if (c < ovalid) mx4[c & 3] = fmaxf(mx4[c & 3], __uint_as_float(t[c]));
          }
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2;
        ATT_T(3)
        bool need = false;
        float corr = 1.f;
        if (j == 0) {
          m_used = mx;
        } else if (mx > m_used + 8.f) {
          need = true;
          corr = fast_exp2(m_used - mx);
          m_used = mx;
          l *= corr;
        }
        float2 sum2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        uint32_t pk[32];
        const float2 sc2 = make_float2(scale_log2, scale_log2), nm2 = make_float2(-m_used, -m_used);
#pragma unroll
        for (int c = 0; c < 64; c += 2) {
          const float2 t = __ffma2_rn(make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2, nm2);
          const float2 p = make_float2(fast_exp2(t.x), fast_exp2(t.y));
          sum2[(c >> 1) & 1] = __fadd2_rn(sum2[(c >> 1) & 1], p);
          pk[c >> 1] = pack_bf16(p.x, p.y);
        }
        l += (sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y);
        ATT_T(4)
        if (gj > 0) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar(P_FREE), (gj - 1) & 1, s_abort));   // P V of the previous block done
          if (!ok) break;
        }
        ATT_T(5)
        if (j > 0 && __any_sync(0xffffffffu, need)) {      // both threads of a row take the same decision
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < OH; c += 32) {
            uint32_t ov[32];
            tc_ld32(tmem_base + tlane + O_COL + half * OH + c, ov);
            tc_wait_ld();
#pragma unroll
            for (int k = 0; k < 32; ++k) ov[k] = __float_as_uint(__uint_as_float(ov[k]) * corr);
            tc_st32(tmem_base + tlane + O_COL + half * OH + c, ov);
          }
          tc_wait_st();
        }
        // P row -> shared memory, 128-byte swizzle: 16-byte chunk c of row r sits at chunk position c ^ (r & 7);
        // this thread's 64 keys are exactly one 128-byte row of slab `half`
        {
          uint8_t* prow = sP + half * SLAB_BYTES + (trow >> 3) * 1024 + (trow & 7) * 128;
#pragma unroll
          for (int c = 0; c < 8; ++c)
            *reinterpret_cast<uint4*>(prow + ((c ^ (trow & 7)) << 4)) =
                make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
        }
        fence_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(P_FULL));
        ATT_T(6)
      }
      if (!ok) break;
      g += nblk;
      // row sum: add the partner's half
      s_xsum[half * 128 + trow] = l;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(X_SUM));
      ok = __all_sync(0xffffffffu, mbar_wait(bar(X_SUM), it & 1, s_abort));
      if (!ok) break;
      l += s_xsum[(half ^ 1) * 128 + trow];
      ok = __all_sync(0xffffffffu, mbar_wait(bar(P_FREE), (g - 1) & 1, s_abort));       // last P V of the item done
      if (!ok) break;
      tc_fence_after();
      const float inv = 1.f / l;
      bf16* orow = o + ((long long)(row0 + trow) * H + h) * DH + half * OH;
#pragma unroll 1
      for (int c = 0; c < OH; c += 32) {
        uint32_t ov[32];
        tc_ld32(tmem_base + tlane + O_COL + half * OH + c, ov);
        tc_wait_ld();
        if (trow < nrows) {
#pragma unroll
          for (int k = 0; k < 32; k += 8) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(ov[k]) * inv, __uint_as_float(ov[k + 1]) * inv);
            v.y = pack_bf16(__uint_as_float(ov[k + 2]) * inv, __uint_as_float(ov[k + 3]) * inv);
            v.z = pack_bf16(__uint_as_float(ov[k + 4]) * inv, __uint_as_float(ov[k + 5]) * inv);
            v.w = pack_bf16(__uint_as_float(ov[k + 6]) * inv, __uint_as_float(ov[k + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + c + k) = v;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(O_FREE));
      ATT_T(7)
    }
#ifdef ATT_PROFILE
    if (prof && blockIdx.x == 0 && warp == 2 && lane == 0)
      for (int i = 0; i < 8; ++i) prof[i] = tp[i];
#endif
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *s_abort) set_status(status, SL_DEV_ATTN_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tc_dealloc(tmem_base, TMEM_COLS);
  }
}

template <int DH>
static int launch_dh(const CUtensorMap& q, const CUtensorMap& k, const CUtensorMap& v, const int32_t* row_offsets,
                     int max_rows, int B, int N, int H, void* o, int32_t* status, cudaStream_t st) {
  constexpr int SLABS = DH / 64;
  const int smem = 5 * SLABS * 128 * 128 + 2 * 128 * 128 + 1024 + 512 + 3072 + 4 * (B + 2);
  static int attr_smem = 0;
  if (smem > attr_smem) {
    SL_CUDA_TRY(cudaFuncSetAttribute(attention_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    attr_smem = smem;
  }
  long long items = (long long)H * ((max_rows + AT_BQ - 1) / AT_BQ + B);
  int grid = sm_count();
  if (items < grid) grid = (int)items;
  if (grid < 1) grid = 1;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
  unsigned long long* prof = nullptr;
#ifdef ATT_PROFILE
  static unsigned long long* d_prof = nullptr;
  if (!d_prof) cudaMalloc(&d_prof, 64);
  prof = d_prof;
#endif
  attention_tc_kernel<DH><<<grid, AT_THREADS, smem, st>>>(q, k, v, row_offsets, B, N, H, (bf16*)o, scale_log2, status, prof);
#ifdef ATT_PROFILE
  {
    unsigned long long h[8];
    cudaMemcpy(h, d_prof, 64, cudaMemcpyDeviceToHost);
    fprintf(stderr, "ATT_PROFILE cycles: loop %llu waitS %llu ldS %llu max+xchg %llu exp %llu waitPV %llu writeP %llu epi %llu\n",
            h[0], h[1], h[2], h[3], h[4], h[5], h[6], h[7]);
  }
#endif
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

int launch_attention_tc1(const void* q, const void* kc, const void* vc, const int32_t* row_offsets, int max_rows, int B,
                        int N, int H, int head_dim, void* o, int32_t* status, cudaStream_t st) {
  if ((head_dim != 64 && head_dim != 128) || B > AT_MAX_B || max_rows < 1 || !row_offsets) return SL_EUNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(kc) | reinterpret_cast<uintptr_t>(vc) |
       reinterpret_cast<uintptr_t>(o)) & 15)
    return SL_EUNSUPPORTED;
  CUtensorMap tq, tk, tv;
  const long long cols = (long long)H * head_dim;
  int rc = get_tensor_map_2d(q, max_rows, cols, 128, &tq);
  if (rc != SL_OK) return rc;
  rc = get_tensor_map_2d(kc, (long long)B * N, cols, 128, &tk);
  if (rc != SL_OK) return rc;
  rc = get_tensor_map_2d(vc, (long long)B * N, cols, 128, &tv);
  if (rc != SL_OK) return rc;
  return head_dim == 128 ? launch_dh<128>(tq, tk, tv, row_offsets, max_rows, B, N, H, o, status, st)
                         : launch_dh<64>(tq, tk, tv, row_offsets, max_rows, B, N, H, o, status, st);
}

}  // namespace sl
