// M x N attention for FEW query rows (Algorithm 1 line 12; Sec. 2.1: the packed queries of the active rows attend to ALL N
// cached keys/values of their sequence, bidirectional, no mask), with the KEYS of a (sequence, head) split over several
// CTAs.
//
// With at most 128 active rows per sequence a (sequence, head) pair is ONE query tile: the general kernel then runs on
// B x H CTAs (32 of 148 SMs for one sequence) and walks through all key blocks one after the other.  Here CTA
// (b, h, s) takes the s-th of S contiguous ranges of 128-key blocks, so that B x H x S CTAs (at most one per SM) share
// the key loop, and leaves an unnormalised partial result (fp32 O, running maximum m, sum l) in a workspace.  The S
// CTAs of a pair then meet on a counter (bounded wait; all of them are resident: the launch is cooperative and the
// grid no larger than the number of SMs) and each combines its share of the rows: o = sum_i w_i O_i / sum_i w_i l_i, w_i = 2^(m_i - max m), in
// split order (deterministic).  With S = 1 the result is written directly.
//   warp 0     TMA producer: Q once per query tile, then K and V blocks (two stages each), 128-byte swizzle;
//   warp 1     one thread issues S = Q K^T and O += P V (P read from tensor memory as the A operand, V the MN-major
//              shared-memory operand), in that order per block, so a finished S implies the previous P V is done;
//   warps 2-5  one thread per query row: scores from tensor memory, running max / sum in fp32 with 1/sqrt(d_h) folded
//              into an exp2, P written back as packed bf16 over columns 64..127 of the S tile; O is rescaled when the
//              running maximum grows by more than 2^8.
// Tensor memory (256 columns): S [0,128), O [128, 128 + d_h).  All waits are bounded.
#include <stdio.h>

#include "tc_common.cuh"

namespace sl {

namespace {

constexpr int AS_THREADS = 192;
constexpr int AS_BQ = 128, AS_BKV = 128;
constexpr int AS_MAX_SPLITS = 8;
constexpr unsigned long long AS_MEET_CYCLES = 400000000ull;   // bound of the wait for the other splits: ~0.2 s

// D[tmem] (+)= A[tmem] * B[smem]: A = 128 lanes x 8 columns, two bf16 per column (K = 16)
__device__ __forceinline__ void as_mma_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accum)
      : "memory");
}

__device__ __forceinline__ unsigned long long as_ld_acquire(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
// One meeting of the S splits of a (sequence, head) adds AS_MEET_QUANTUM to the pair's 64-bit counter whatever S is (each
// split adds AS_MEET_QUANTUM / S; S <= 8 divides it), so the counter only grows, never wraps in practice, and launches
// with different numbers of splits can share a workspace.
constexpr unsigned long long AS_MEET_QUANTUM = 840;

}  // namespace

template <int DH>
__global__ void __launch_bounds__(AS_THREADS, 1)
attention_split_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV, const int32_t* __restrict__ row_offsets, int B, int N, int H,
                       int S, bf16* __restrict__ o, float scale_log2, float* __restrict__ ws_o, float2* __restrict__ ws_ml,
                       unsigned long long* __restrict__ counters, int32_t* status, int diag_skip) {
  constexpr int SLABS = DH / 64;                       // 64-element (128-byte) column blocks per row
  constexpr int SLAB_BYTES = 128 * 128;                // 128 rows x 128 bytes
  constexpr int Q_BYTES = SLABS * SLAB_BYTES;
  constexpr int KV_BYTES = SLABS * SLAB_BYTES;
  constexpr uint32_t TMEM_COLS = 256;
  constexpr uint32_t O_COL = 128;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + Q_BYTES;                          // 2 stages
  uint8_t* sV = sK + 2 * KV_BYTES;                     // 2 stages
  uint64_t* bars = reinterpret_cast<uint64_t*>(sV + 2 * KV_BYTES);
  enum { Q_FULL = 0, Q_FREE = 1, K_FULL = 2, K_FREE = 4, V_FULL = 6, V_FREE = 8, S_FULL = 10, P_FULL = 11, O_FULL = 12,
         O_FREE = 13, NUM_BARS = 14 };
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  volatile int* s_meet = reinterpret_cast<volatile int*>(s_tmem + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto bar = [&](int i) { return bar0 + 8u * i; };

  if (threadIdx.x == 0) {
    for (int i = 0; i < NUM_BARS; ++i) mbar_init(bar(i), (i == P_FULL || i == O_FREE) ? 4 : 1);   // one arrival per softmax warp
    *s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) tc_alloc(smem_u32(s_tmem), TMEM_COLS);
  // everything above overlaps the tail of the previous kernel; nothing below may run before it has completed
  griddep_wait();
  griddep_launch();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;

  const int s = (int)blockIdx.x % S, bh = (int)blockIdx.x / S, h = bh % H, b = bh / H;
  const int r0 = row_offsets[b], mb = row_offsets[b + 1] - r0;
  const int n_qt = (mb + AS_BQ - 1) / AS_BQ;                      // query tiles (one, unless the caller's bound was too small)
  const int nblk = (N + AS_BKV - 1) / AS_BKV, per = (nblk + S - 1) / S;
  const int j0 = s * per < nblk ? s * per : nblk, j1 = j0 + per < nblk ? j0 + per : nblk;
  const int nj = j1 - j0;                                         // key blocks of this split (0: nothing to add)

  if (warp == 0) {
    if (lane == 0) {
      uint32_t kcnt = 0;
      bool ok = true;
      const uint64_t once = l2_policy_evict_first();    // every K / V block is read by exactly one CTA per step
      for (int qt = 0; qt < n_qt && ok && nj > 0; ++qt) {
        if (!(ok = mbar_wait(bar(Q_FREE), (qt & 1) ^ 1, s_abort))) break;
        mbar_expect_tx(bar(Q_FULL), Q_BYTES);
#pragma unroll
        for (int sl = 0; sl < SLABS; ++sl)
          tma_load_2d(smem_u32(sQ + sl * SLAB_BYTES), &tmQ, h * DH + 64 * sl, r0 + qt * AS_BQ, bar(Q_FULL));
        for (int j = j0; j < j1; ++j, ++kcnt) {
          const int st = kcnt & 1;
          const uint32_t ph = (kcnt >> 1) & 1;
          const int key0 = b * N + j * AS_BKV;
          if (!(ok = mbar_wait(bar(K_FREE + st), ph ^ 1, s_abort))) break;
          mbar_expect_tx(bar(K_FULL + st), KV_BYTES);
#pragma unroll
          for (int sl = 0; sl < SLABS; ++sl)
            tma_load_2d_hint(smem_u32(sK + st * KV_BYTES + sl * SLAB_BYTES), &tmK, h * DH + 64 * sl, key0, bar(K_FULL + st), once);
          if (!(ok = mbar_wait(bar(V_FREE + st), ph ^ 1, s_abort))) break;
          mbar_expect_tx(bar(V_FULL + st), KV_BYTES);
#pragma unroll
          for (int sl = 0; sl < SLABS; ++sl)
            tma_load_2d_hint(smem_u32(sV + st * KV_BYTES + sl * SLAB_BYTES), &tmV, h * DH + 64 * sl, key0, bar(V_FULL + st), once);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16_m128(AS_BKV, false);
      constexpr uint32_t idesc_o = idesc_bf16_m128(DH, true);
      uint32_t kc = 0;                                  // key blocks so far
      bool ok = true;
      // O (+)= P V for block number blk (counted over the whole kernel), jb = its index inside the query tile
      auto issue_pv = [&](uint32_t blk, int jb, int qt) -> bool {
        const int st = blk & 1;
        const uint32_t va = smem_u32(sV + st * KV_BYTES);
        if (!mbar_wait(bar(V_FULL + st), (blk >> 1) & 1, s_abort)) return false;
        if (!mbar_wait(bar(P_FULL), blk & 1, s_abort)) return false;
        if (jb == 0 && !mbar_wait(bar(O_FREE), (qt & 1) ^ 1, s_abort)) return false;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < AS_BKV / 16; ++kk)
          as_mma_ta(tmem_base + O_COL, tmem_base + 64 + kk * 8, smem_desc_mn_sw128(va + kk * 16 * 128, SLAB_BYTES), idesc_o,
                    (jb | kk) != 0);
        tc_commit(bar(V_FREE + st));
        return true;
      };
      for (int qt = 0; qt < n_qt && ok && nj > 0; ++qt) {
        if (!(ok = mbar_wait(bar(Q_FULL), qt & 1, s_abort))) break;
        for (int jb = 0; jb < nj && ok; ++jb) {
          if (jb > 0 && !(ok = issue_pv(kc + jb - 1, jb - 1, qt))) break;
          const int st = (kc + jb) & 1;
          if (!(ok = mbar_wait(bar(K_FULL + st), ((kc + jb) >> 1) & 1, s_abort))) break;
          tc_fence_after();
          const uint32_t qa = smem_u32(sQ), ka = smem_u32(sK + st * KV_BYTES);
#pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {
            const uint32_t off = (kk >> 2) * SLAB_BYTES + (kk & 3) * 32;
            tc_mma_bf16(tmem_base, smem_desc_k_sw128(qa + off), smem_desc_k_sw128(ka + off), idesc_s, kk != 0);
          }
          tc_commit(bar(S_FULL));
          tc_commit(bar(K_FREE + st));
        }
        if (!ok) break;
        tc_commit(bar(Q_FREE));                          // every S product of this tile has been issued
        if (!(ok = issue_pv(kc + nj - 1, nj - 1, qt))) break;
        tc_commit(bar(O_FULL));
        kc += nj;
      }
    }
  } else {
    const int quarter = warp & 3;                        // tensor-memory lane quarter this warp may access
    const int trow = quarter * 32 + lane;                // query row of this thread inside the tile
    const int e_tid = (warp - 2) * 32 + lane;
    const uint32_t tlane = (uint32_t)(quarter * 32) << 16;
    const uint32_t s_addr = tmem_base + tlane, o_addr = tmem_base + tlane + O_COL;
    uint32_t g = 0;                                      // key blocks so far
    bool ok = true;
    auto rescale_o = [&](float corr) {
#pragma unroll 1
      for (int c = 0; c < DH; c += 32) {
        uint32_t ov[32];
        tc_ld32(o_addr + c, ov);
        tc_wait_ld();
#pragma unroll
        for (int k = 0; k < 32; ++k) ov[k] = __float_as_uint(__uint_as_float(ov[k]) * corr);
        tc_st32(o_addr + c, ov);
      }
      tc_wait_st();
    };
    // the S splits of this (sequence, head) meet: every meeting adds one quantum to the pair's counter, which only grows
    auto meet = [&]() -> bool {
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (e_tid == 0 && (int)blockIdx.x == diag_skip) {
        *s_meet = 1;                                     // diagnostic: this CTA does not arrive, so its siblings' wait runs out
      } else if (e_tid == 0) {
        __threadfence();                                 // release: the CTA's stores (ordered before by the bar.sync)
        const unsigned long long ticket = atomicAdd(counters + bh, AS_MEET_QUANTUM / (unsigned long long)S);
        const unsigned long long target = (ticket / AS_MEET_QUANTUM + 1ull) * AS_MEET_QUANTUM;
        const unsigned long long t0 = clock64();
        int good = 1;
        while (as_ld_acquire(counters + bh) < target) {
          if (*s_abort || clock64() - t0 > AS_MEET_CYCLES) {
            *s_abort = 1;
            good = 0;
            break;
          }
        }
        *s_meet = good;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      return *s_meet != 0;
    };
    for (int qt = 0; qt < n_qt && ok; ++qt) {
      const int rows_t = mb - qt * AS_BQ < AS_BQ ? mb - qt * AS_BQ : AS_BQ;
      const int row_first = r0 + qt * AS_BQ;
      float m_used = -INFINITY, l = 0.f;
      for (int jb = 0; jb < nj && ok; ++jb) {
        if (!__all_sync(0xffffffffu, mbar_wait(bar(S_FULL), (g + jb) & 1, s_abort))) {
          ok = false;
          break;
        }
        tc_fence_after();
        uint32_t sc[128];
        tc_ld32(s_addr, sc);
        tc_ld32(s_addr + 32, sc + 32);
        tc_ld32(s_addr + 64, sc + 64);
        tc_ld32(s_addr + 96, sc + 96);
        tc_wait_ld();
        const int nvalid = N - (j0 + jb) * AS_BKV;        // keys of this block that exist
        if (nvalid < AS_BKV) {
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (c >= nvalid) sc[c] = 0xff800000u;        // -inf
        }
        float mx = __uint_as_float(sc[0]);
#pragma unroll
        for (int c = 1; c < 128; ++c) mx = fmaxf(mx, __uint_as_float(sc[c]));
        mx *= scale_log2;
        // the running maximum is replaced only when it grows by more than 2^8
        bool need = false;
        float corr = 1.f;
        if (jb == 0) {
          m_used = mx;
        } else if (mx > m_used + 8.f) {
          need = true;
          corr = fast_exp2(m_used - mx);
          m_used = mx;
          l *= corr;
        }
        // S of this block is complete, so the previous block's P V is too, and this block's has not been issued
        if (jb > 0 && __any_sync(0xffffffffu, need)) rescale_o(corr);
        float sum = 0.f;
#pragma unroll
        for (int c = 0; c < 128; c += 2) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(sc[c]), scale_log2, -m_used));
          const float p1 = fast_exp2(fmaf(__uint_as_float(sc[c + 1]), scale_log2, -m_used));
          sum += p0 + p1;
          sc[c >> 1] = pack_bf16(p0, p1);                // packed P over the registers whose scores are spent
        }
        l += sum;
        // P: keys 2c, 2c+1 in column 64 + c of the S tile (whose scores are all in registers by now)
        tc_st32(s_addr + 64, sc);
        tc_st32(s_addr + 96, sc + 32);
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(P_FULL));
      }
      g += nj;
      if (ok && nj > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar(O_FULL), qt & 1, s_abort));   // last P V of the tile done
        tc_fence_after();
      }
      if (S > 1) ok = epilogue_warps_agree(ok);           // nobody is left alone at the meeting below
      if (!ok) break;
      if (S == 1) {
        const float inv = 1.f / l;
        bf16* orow = o + ((long long)(row_first + trow) * H + h) * DH;
#pragma unroll 1
        for (int c = 0; c < DH; c += 32) {
          uint32_t ov[32];
          tc_ld32(o_addr + c, ov);
          tc_wait_ld();
          if (trow < rows_t) {
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
        continue;
      }
      // partial result of this split: unnormalised O, running maximum (in the exp2 domain) and sum
      float* po = ws_o + ((size_t)blockIdx.x * AS_BQ + trow) * DH;
      if (nj > 0) {
#pragma unroll 1
        for (int c = 0; c < DH; c += 32) {
          uint32_t ov[32];
          tc_ld32(o_addr + c, ov);
          tc_wait_ld();
          if (trow < rows_t) {
#pragma unroll
            for (int k = 0; k < 32; k += 4)
              __stcg(reinterpret_cast<float4*>(po + c + k),
                     make_float4(__uint_as_float(ov[k]), __uint_as_float(ov[k + 1]), __uint_as_float(ov[k + 2]),
                                 __uint_as_float(ov[k + 3])));
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(O_FREE));
      }
      if (trow < rows_t) __stcg(ws_ml + (size_t)blockIdx.x * AS_BQ + trow, make_float2(m_used, l));
      if (!(ok = meet())) break;
      // this split's share of the rows, (row, four features) items over the 128 threads
      const int ra = (int)((long long)s * rows_t / S), rb = (int)((long long)(s + 1) * rows_t / S);
      constexpr int G8 = DH / 8;
      const size_t first = (size_t)bh * S;               // first split's slot
      for (int it = ra * G8 + e_tid; it < rb * G8; it += 128) {
        const int r = it / G8, c8 = (it - r * G8) * 8;
        // all loads of a round are issued before anything is computed: two L2 round trips per item
        float2 ml[AS_MAX_SPLITS];
        float4 v[AS_MAX_SPLITS][2];
#pragma unroll
        for (int i = 0; i < AS_MAX_SPLITS; ++i) {
          ml[i] = make_float2(-INFINITY, 0.f);
          if (i < S) {
            ml[i] = __ldcg(ws_ml + (first + i) * AS_BQ + r);
            const float4* src = reinterpret_cast<const float4*>(ws_o + ((first + i) * AS_BQ + r) * DH + c8);
            v[i][0] = __ldcg(src);
            v[i][1] = __ldcg(src + 1);
          }
        }
        float mmax = -INFINITY;
#pragma unroll
        for (int i = 0; i < AS_MAX_SPLITS; ++i) mmax = fmaxf(mmax, ml[i].x);
        float L = 0.f, acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int i = 0; i < AS_MAX_SPLITS; ++i) {
          if (i < S && ml[i].y > 0.f) {                  // a split without keys leaves l = 0 and no O
            const float w = fast_exp2(ml[i].x - mmax);
            L = fmaf(w, ml[i].y, L);
            acc[0] = fmaf(w, v[i][0].x, acc[0]); acc[1] = fmaf(w, v[i][0].y, acc[1]);
            acc[2] = fmaf(w, v[i][0].z, acc[2]); acc[3] = fmaf(w, v[i][0].w, acc[3]);
            acc[4] = fmaf(w, v[i][1].x, acc[4]); acc[5] = fmaf(w, v[i][1].y, acc[5]);
            acc[6] = fmaf(w, v[i][1].z, acc[6]); acc[7] = fmaf(w, v[i][1].w, acc[7]);
          }
        }
        const float inv = 1.f / L;
        uint4 pk;
        pk.x = pack_bf16(acc[0] * inv, acc[1] * inv);
        pk.y = pack_bf16(acc[2] * inv, acc[3] * inv);
        pk.z = pack_bf16(acc[4] * inv, acc[5] * inv);
        pk.w = pack_bf16(acc[6] * inv, acc[7] * inv);
        *reinterpret_cast<uint4*>(o + ((long long)(row_first + r) * H + h) * DH + c8) = pk;
      }
      // another query tile would overwrite the slots: not before every split has read them
      if (qt + 1 < n_qt && !(ok = meet())) break;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *s_abort) set_status(status, SL_DEV_ATTN_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tc_dealloc(tmem_base, TMEM_COLS);
  }
}

// Number of key splits for this problem, 0 = the general kernel is the better choice: every split gets at least one key
// block, and B x H x S CTAs fit the GPU at one per SM (which the meeting of the splits relies on).
int attention_split_plan(int B, int N, int H) {
  const int nblk = (N + AS_BKV - 1) / AS_BKV;
  int S = sm_count() / (B * H);
  if (S > AS_MAX_SPLITS) S = AS_MAX_SPLITS;
  if (S > nblk) S = nblk;
  while (S > 1 && ((nblk + S - 1) / S) * (S - 1) >= nblk) --S;   // no empty split
  return S >= 2 ? S : 0;
}

size_t attention_split_workspace_bytes(int head_dim) {
  return (size_t)sm_count() * AS_BQ * ((size_t)head_dim * sizeof(float) + sizeof(float2));
}

template <int DH>
static int launch_split_dh(const CUtensorMap& q, const CUtensorMap& k, const CUtensorMap& v, const int32_t* row_offsets, int B,
                           int N, int H, int S, void* o, float* ws, unsigned long long* counters, int32_t* status, int diag_skip,
                           cudaStream_t st) {
  constexpr int SLABS = DH / 64;
  const int smem = 5 * SLABS * 128 * 128 + 1024 + 512;
  static bool attr_set = false;
  if (!attr_set) {
    SL_CUDA_TRY(cudaFuncSetAttribute(attention_split_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    attr_set = true;
  }
  float* ws_o = ws;
  float2* ws_ml = reinterpret_cast<float2*>(ws + (size_t)sm_count() * AS_BQ * DH);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
  // The splits wait for one another, so with S > 1 the launch is cooperative: every CTA of the grid is resident at the
  // same time whatever else runs on the device (the grid was checked against one CTA per SM).  Programmatic dependent
  // launch on top of it where the driver takes the combination.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(B * H * S);
  cfg.blockDim = dim3(AS_THREADS);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  int n_at = 0;
  if (S > 1) {
    at[n_at].id = cudaLaunchAttributeCooperative;
    at[n_at].val.cooperative = 1;
    ++n_at;
  }
  static int with_pdl = -1;                            // -1: not tried yet
  if (with_pdl < 0) with_pdl = pdl_enabled() ? 1 : 0;
  const int n_base = n_at;
  if (with_pdl) {
    at[n_at].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n_at].val.programmaticStreamSerializationAllowed = 1;
    ++n_at;
  }
  cfg.attrs = at;
  cfg.numAttrs = n_at;
  bf16* op = (bf16*)o;
  cudaError_t e = cudaLaunchKernelEx(&cfg, attention_split_kernel<DH>, q, k, v, row_offsets, B, N, H, S, op, scale_log2, ws_o,
                                     ws_ml, counters, status, diag_skip);
  if (e != cudaSuccess && with_pdl && n_base > 0) {    // the combination of the two attributes is refused: cooperative only
    cudaGetLastError();
    with_pdl = 0;
    cfg.numAttrs = n_base;
    e = cudaLaunchKernelEx(&cfg, attention_split_kernel<DH>, q, k, v, row_offsets, B, N, H, S, op, scale_log2, ws_o, ws_ml,
                           counters, status, diag_skip);
  }
  SL_CUDA_TRY(e);
  return SL_OK;
}

// ws: attention_split_workspace_bytes(head_dim) bytes; counters: B x H 64-bit words, zero before the first launch.
// diag_skip >= 0: CTA diag_skip does not arrive at the meeting of its (sequence, head) (failure-detection test: the other
// splits' bounded wait runs out and the kernel reports SL_DEV_ATTN_TIMEOUT); -1 otherwise.
// SL_EUNSUPPORTED when the problem does not fit (the caller then takes the general kernel).
int launch_attention_split(const void* q, const void* kc, const void* vc, const int32_t* row_offsets, int max_rows, int B,
                           int N, int H, int head_dim, int S, void* o, float* ws, unsigned long long* counters, int32_t* status,
                           int diag_skip, cudaStream_t st) {
  if ((head_dim != 64 && head_dim != 128) || max_rows < 1 || !row_offsets || !ws || !counters) return SL_EUNSUPPORTED;
  if (S < 1 || S > AS_MAX_SPLITS || (long long)B * H * S > sm_count()) return SL_EUNSUPPORTED;
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
  return head_dim == 128 ? launch_split_dh<128>(tq, tk, tv, row_offsets, B, N, H, S, o, ws, counters, status, diag_skip, st)
                         : launch_split_dh<64>(tq, tk, tv, row_offsets, B, N, H, S, o, ws, counters, status, diag_skip, st);
}

}  // namespace sl
