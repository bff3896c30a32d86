// Tensor-core M x N attention on sm_100a, two query tiles per CTA (Algorithm 1 line 12; Sec. 2.1: the packed queries of
// the active rows attend to ALL N cached keys/values of their sequence, bidirectional, no mask).
//
// Work item = (sequence b, head h, up to 256 consecutive packed rows of that sequence = two tiles of 128; one tile
// when that spreads a small problem over more SMs); items never straddle sequences.  Persistent CTAs take items
// round-robin, the row-tile index fastest, so CTAs working at the same time read the same K/V head through L2.  Keys
// are streamed in blocks of 128.  Two modes, chosen on the device from the row counts of the sequences:
//  * PAIRS (dense active sets): the two tiles of an item share every K/V block (two stages each);
//  * STREAMS (at least as many lone tiles as pairs, e.g. every sequence has <= 128 active rows): a CTA runs two
//    independent streams of one-tile items (stream CTA + t * grid), each with its own Q tile, ONE K and ONE V buffer and
//    its own producer warp, so that any two tiles share an SM; every tile of a launch takes the same number of key
//    blocks, so the streams advance in step.  (K/V blocks are then copied once per tile, which costs 3-9 % when the
//    tiles could have shared them: hence the two modes.)
//   warp 0     TMA producer (of stream 0; warp 10 of stream 1): Q once per item, then K and V blocks, token-major
//              cache rows, 128-byte swizzle;
//   warp 1     one thread issues, per key block and tile t: O_t += P_t V (previous block; P_t is read from TENSOR
//              MEMORY as the A operand, V is the MN-major shared-memory operand) and then S_t = Q_t K^T;
//   warps 2-5  softmax of tile 0, warps 6-9 softmax of tile 1: ONE thread per query row (no exchange between
//              threads): tcgen05.ld the 128 scores, running max / sum in fp32 with 1/sqrt(d_h) folded into an exp2,
//              P written back as packed bf16 over the last 64 columns of the S tile (tcgen05.st), in two halves so
//              that the first half of P V runs under the second half of the exponentials.
// The two tiles alternate: while the softmax warps of one tile work, the tensor pipe runs the other tile's two
// products, and each scheduler's special-function unit always has one of its two softmax warps to feed.
// O stays in tensor memory and is rescaled only when a row's running maximum grows by more than 2^8; O / l is stored
// as bf16 at the end of the item.  Keys beyond N in the last block are masked to -inf.  All waits are bounded
// (SL_DEV_ATTN_TIMEOUT).
//
// Tensor memory (512 columns): S0 [0,128)  S1 [128,256)  O0 [256,256+d_h)  O1 [256+d_h, 256+2 d_h).
#include <stdio.h>
#include <type_traits>

#include "tc_common.cuh"

namespace sl {

namespace {

constexpr int PP_THREADS = 352;   // TMA warp, MMA warp, 4 softmax warps per tile, second TMA warp (STREAMS mode)
constexpr int PP_BQ = 128, PP_BKV = 128, PP_ITEM_ROWS = 256;
constexpr int PP_MAX_B = 1024;

// D[tmem] (+)= A[tmem] * B[smem]: A = 128 lanes x 8 columns, two bf16 per column (K = 16)
__device__ __forceinline__ void tc_mma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accum)
      : "memory");
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

}  // namespace

template <int DH>
__global__ void __launch_bounds__(PP_THREADS, 1)
attention_pp_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const int32_t* __restrict__ row_offsets, int B, int N, int H,
                    bf16* __restrict__ o, float scale_log2, int32_t* status) {
  constexpr int SLABS = DH / 64;                       // 64-element (128-byte) column blocks per row
  constexpr int SLAB_BYTES = 128 * 128;                // 128 rows x 128 bytes
  constexpr int Q_BYTES = SLABS * SLAB_BYTES;          // one Q tile
  constexpr int KV_BYTES = SLABS * SLAB_BYTES;         // one K or V block of 128 keys
  constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t O_COL = 256;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                                  // 2 tiles
  uint8_t* sK = sQ + 2 * Q_BYTES;                      // 2 stages
  uint8_t* sV = sK + 2 * KV_BYTES;                     // 2 stages
  uint64_t* bars = reinterpret_cast<uint64_t*>(sV + 2 * KV_BYTES);
  // every barrier name has two slots: per K/V stage or per tile in PAIRS mode (Q: slot 0), per stream in STREAMS mode
  enum { Q_FULL = 0, Q_FREE = 2, K_FULL = 4, K_FREE = 6, V_FULL = 8, V_FREE = 10, S_FULL = 12, P_HALF = 14, P_FULL = 16,
         O_FULL = 18, O_FREE = 20, NUM_BARS = 22 };
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  int* s_item_rows = reinterpret_cast<int*>(s_tmem + 2);
  int* s_streams = reinterpret_cast<int*>(s_tmem + 3);
  int* s_prefix = reinterpret_cast<int*>(s_tmem + 4);  // [B+1] work-item prefix per sequence

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto bar = [&](int i) { return bar0 + 8u * i; };

  if (threadIdx.x == 0) {
    for (int i = 0; i < NUM_BARS; ++i) {
      const bool per_warp = (i >= P_HALF && i < P_FULL + 2) || (i >= O_FREE && i < O_FREE + 2);
      mbar_init(bar(i), per_warp ? 4 : 1);             // one elected arrival per softmax warp of the tile
    }
    *s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) tc_alloc(smem_u32(s_tmem), TMEM_COLS);
  // everything above overlaps the tail of the previous kernel; nothing below may run before it has completed
  griddep_wait();
  griddep_launch();
  if (threadIdx.x == 0) {
    // STREAMS when lone tiles (a sequence's odd tile) are at least as many as tile pairs
    int lone = 0, pairs = 0;
    for (int b = 0; b < B; ++b) {
      const int tb = (row_offsets[b + 1] - row_offsets[b] + PP_BQ - 1) / PP_BQ;
      lone += tb & 1;
      pairs += tb >> 1;
    }
    const int streams = lone >= pairs;
    *s_streams = streams;
    // PAIRS: items of two tiles, unless one-tile items finish sooner: a one-tile item takes about 0.8 of the time of a
    // two-tile item (its softmax warps and the tensor pipe alternate instead of overlapping), so they win when they
    // spread over idle SMs, i.e. when 4 * rounds(one-tile) < 5 * rounds(two-tile).  STREAMS: one-tile items.
    int rows = streams ? PP_BQ : PP_ITEM_ROWS, rounds2 = 0;
    for (int pass = streams ? 2 : 0; pass < 3; ++pass) {
      int acc = 0;
      s_prefix[0] = 0;
      for (int b = 0; b < B; ++b) {
        const int mb = row_offsets[b + 1] - row_offsets[b];
        acc += ((mb + rows - 1) / rows) * H;
        s_prefix[b + 1] = acc;
      }
      const int rounds = (acc + (int)gridDim.x - 1) / (int)gridDim.x;
      if (pass == 0) {
        rounds2 = rounds;
        rows = PP_BQ;                                    // try one-tile items
      } else if (pass == 1) {
        if (4 * rounds < 5 * rounds2) break;             // keep one-tile items
        rows = PP_ITEM_ROWS;                             // back to two-tile items
      } else {
        break;
      }
    }
    *s_item_rows = rows;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const int total = s_prefix[B];
  const int item_rows = *s_item_rows;
  const bool streams = *s_streams != 0;
  const int nstream = 2 * (int)gridDim.x;
  const int nblk = (N + PP_BKV - 1) / PP_BKV;

  // item -> (b, h, first packed row, rows in the item (1..256))
  auto decode = [&](int w, int& b, int& h, int& row0, int& nrows) {
    int lo = 0, hi = B;                                 // largest b with prefix[b] <= w
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_prefix[mid] <= w) lo = mid; else hi = mid;
    }
    b = lo;
    const int r0 = row_offsets[b], mb = row_offsets[b + 1] - r0;
    const int parts = (mb + item_rows - 1) / item_rows;
    const int local = w - s_prefix[b];
    h = local / parts;
    const int qt = local % parts;
    row0 = r0 + qt * item_rows;
    nrows = mb - qt * item_rows < item_rows ? mb - qt * item_rows : item_rows;
  };

  if (streams) {
    if (warp == 0 || warp == 10) {
      if (lane == 0) {
        const int t = warp == 0 ? 0 : 1;                   // stream of this producer
        uint32_t kcnt = 0, qcnt = 0;
        bool ok = true;
        for (int w = (int)blockIdx.x + t * (int)gridDim.x; w < total && ok; w += nstream, ++qcnt) {
          int b, h, row0, nrows;
          decode(w, b, h, row0, nrows);
          if (!(ok = mbar_wait(bar(Q_FREE + t), (qcnt & 1) ^ 1, s_abort))) break;
          mbar_expect_tx(bar(Q_FULL + t), Q_BYTES);
  #pragma unroll
          for (int s = 0; s < SLABS; ++s)
            tma_load_2d(smem_u32(sQ + t * Q_BYTES + s * SLAB_BYTES), &tmQ, h * DH + 64 * s, row0, bar(Q_FULL + t));
          for (int j = 0; j < nblk; ++j, ++kcnt) {
            const uint32_t ph = kcnt & 1;
            const int key0 = b * N + j * PP_BKV;
            if (!(ok = mbar_wait(bar(K_FREE + t), ph ^ 1, s_abort))) break;
            mbar_expect_tx(bar(K_FULL + t), KV_BYTES);
  #pragma unroll
            for (int s = 0; s < SLABS; ++s)
              tma_load_2d(smem_u32(sK + t * KV_BYTES + s * SLAB_BYTES), &tmK, h * DH + 64 * s, key0, bar(K_FULL + t));
            if (!(ok = mbar_wait(bar(V_FREE + t), ph ^ 1, s_abort))) break;
            mbar_expect_tx(bar(V_FULL + t), KV_BYTES);
  #pragma unroll
            for (int s = 0; s < SLABS; ++s)
              tma_load_2d(smem_u32(sV + t * KV_BYTES + s * SLAB_BYTES), &tmV, h * DH + 64 * s, key0, bar(V_FULL + t));
          }
        }
      }
    } else if (warp == 1) {
      if (lane == 0) {
        constexpr uint32_t idesc_s = idesc_bf16_m128(PP_BKV, false);
        constexpr uint32_t idesc_o = idesc_bf16_m128(DH, true);
        uint32_t g = 0, it = 0;                            // key blocks and tiles so far (the same for both streams)
        bool ok = true;
        // S_t = Q_t K^T for the key block in the stream's K buffer
        auto issue_s = [&](int t) {
          const uint32_t qa = smem_u32(sQ + t * Q_BYTES), ka = smem_u32(sK + t * KV_BYTES);
  #pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {
            const uint32_t off = (kk >> 2) * SLAB_BYTES + (kk & 3) * 32;
            tc_mma_bf16(tmem_base + t * 128, smem_desc_k_sw128(qa + off), smem_desc_k_sw128(ka + off), idesc_s, kk != 0);
          }
          tc_commit(bar(S_FULL + t));
          tc_commit(bar(K_FREE + t));
        };
        // O_t (+)= P_t V for key block jb of the tile (global block number g + jb), V in the stream's V buffer
        auto issue_pv = [&](int t, int jb) -> bool {
          const uint32_t va = smem_u32(sV + t * KV_BYTES);
          const uint32_t par = (g + jb) & 1;
          if (!mbar_wait(bar(V_FULL + t), par, s_abort)) return false;
          if (!mbar_wait(bar(P_HALF + t), par, s_abort)) return false;
          if (jb == 0 && !mbar_wait(bar(O_FREE + t), (it & 1) ^ 1, s_abort)) return false;
          tc_fence_after();
  #pragma unroll
          for (int kk = 0; kk < PP_BKV / 32; ++kk)
            tc_mma_bf16_ta(tmem_base + O_COL + t * DH, tmem_base + t * 128 + 64 + kk * 8,
                           smem_desc_mn_sw128(va + kk * 16 * 128, SLAB_BYTES), idesc_o, (jb | kk) != 0);
          if (!mbar_wait(bar(P_FULL + t), par, s_abort)) return false;
          tc_fence_after();
  #pragma unroll
          for (int kk = PP_BKV / 32; kk < PP_BKV / 16; ++kk)
            tc_mma_bf16_ta(tmem_base + O_COL + t * DH, tmem_base + t * 128 + 64 + kk * 8,
                           smem_desc_mn_sw128(va + kk * 16 * 128, SLAB_BYTES), idesc_o, 1);
          tc_commit(bar(V_FREE + t));
          return true;
        };
        // the two streams take their tiles in step: round `it` is tile CTA + t * grid + it * nstream of stream t
        for (int w0 = (int)blockIdx.x; w0 < total && ok; w0 += nstream, ++it) {
          const int nt = w0 + (int)gridDim.x < total ? 2 : 1;   // streams that still have a tile
          for (int t = 0; t < nt && ok; ++t) ok = mbar_wait(bar(Q_FULL + t), it & 1, s_abort);
          for (int j = 0; j < nblk && ok; ++j) {
            for (int t = 0; t < nt && ok; ++t) {
              if (j > 0) ok = issue_pv(t, j - 1);
              if (!ok) break;
              if (!(ok = mbar_wait(bar(K_FULL + t), (g + j) & 1, s_abort))) break;
              tc_fence_after();
              issue_s(t);
            }
          }
          if (!ok) break;
          for (int t = 0; t < nt; ++t) tc_commit(bar(Q_FREE + t));   // every S product of these tiles has been issued
          for (int t = 0; t < nt && ok; ++t) {
            ok = issue_pv(t, nblk - 1);
            if (ok) tc_commit(bar(O_FULL + t));
          }
          g += nblk;
        }
      }
    }
  } else {
    if (warp == 0) {
      if (lane == 0) {
        uint32_t kcnt = 0, qcnt = 0;
        bool ok = true;
        for (int w = blockIdx.x; w < total && ok; w += gridDim.x, ++qcnt) {
          int b, h, row0, nrows;
          decode(w, b, h, row0, nrows);
          const int ntile = nrows > PP_BQ ? 2 : 1;
          if (!(ok = mbar_wait(bar(Q_FREE), (qcnt & 1) ^ 1, s_abort))) break;
          mbar_expect_tx(bar(Q_FULL), ntile * Q_BYTES);
          for (int t = 0; t < ntile; ++t)
  #pragma unroll
            for (int s = 0; s < SLABS; ++s)
              tma_load_2d(smem_u32(sQ + t * Q_BYTES + s * SLAB_BYTES), &tmQ, h * DH + 64 * s, row0 + t * PP_BQ, bar(Q_FULL));
          for (int j = 0; j < nblk; ++j, ++kcnt) {
            const int st = kcnt & 1;
            const uint32_t ph = (kcnt >> 1) & 1;
            const int key0 = b * N + j * PP_BKV;
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
        constexpr uint32_t idesc_s = idesc_bf16_m128(PP_BKV, false);
        constexpr uint32_t idesc_o = idesc_bf16_m128(DH, true);
        uint32_t kc = 0, it = 0;
        uint32_t gt[2] = {0, 0}, itt[2] = {0, 0};          // per tile: key blocks and items so far
        bool ok = true;
        // S_t = Q_t K^T for the key block in stage kst
        auto issue_s = [&](int t, int kst) {
          const uint32_t qa = smem_u32(sQ + t * Q_BYTES), ka = smem_u32(sK + kst * KV_BYTES);
  #pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) {
            const uint32_t off = (kk >> 2) * SLAB_BYTES + (kk & 3) * 32;
            tc_mma_bf16(tmem_base + t * 128, smem_desc_k_sw128(qa + off), smem_desc_k_sw128(ka + off), idesc_s, kk != 0);
          }
          tc_commit(bar(S_FULL + t));
        };
        // O_t (+)= P_t V for the key block in stage vst; jb = index of that block inside the item
        auto issue_pv = [&](int t, int vst, int jb) -> bool {
          const uint32_t va = smem_u32(sV + vst * KV_BYTES);
          if (!mbar_wait(bar(P_HALF + t), (gt[t] + jb) & 1, s_abort)) return false;
          if (jb == 0 && !mbar_wait(bar(O_FREE + t), (itt[t] & 1) ^ 1, s_abort)) return false;
          tc_fence_after();
  #pragma unroll
          for (int kk = 0; kk < PP_BKV / 32; ++kk)
            tc_mma_bf16_ta(tmem_base + O_COL + t * DH, tmem_base + t * 128 + 64 + kk * 8,
                           smem_desc_mn_sw128(va + kk * 16 * 128, SLAB_BYTES), idesc_o, (jb | kk) != 0);
          if (!mbar_wait(bar(P_FULL + t), (gt[t] + jb) & 1, s_abort)) return false;
          tc_fence_after();
  #pragma unroll
          for (int kk = PP_BKV / 32; kk < PP_BKV / 16; ++kk)
            tc_mma_bf16_ta(tmem_base + O_COL + t * DH, tmem_base + t * 128 + 64 + kk * 8,
                           smem_desc_mn_sw128(va + kk * 16 * 128, SLAB_BYTES), idesc_o, 1);
          return true;
        };
        for (int w = blockIdx.x; w < total && ok; w += gridDim.x, ++it) {
          int b, h, row0, nrows;
          decode(w, b, h, row0, nrows);
          const int ntile = nrows > PP_BQ ? 2 : 1;
          if (!(ok = mbar_wait(bar(Q_FULL), it & 1, s_abort))) break;
          for (int j = 0; j < nblk && ok; ++j) {
            const int kst = (kc + j) & 1;
            if (!(ok = mbar_wait(bar(K_FULL + kst), ((kc + j) >> 1) & 1, s_abort))) break;
            const int vst = (kc + j - 1) & 1;
            if (j > 0 && !(ok = mbar_wait(bar(V_FULL + vst), ((kc + j - 1) >> 1) & 1, s_abort))) break;
            for (int t = 0; t < ntile && ok; ++t) {
              if (j > 0) ok = issue_pv(t, vst, j - 1);
              if (!ok) break;
              tc_fence_after();
              issue_s(t, kst);
            }
            if (!ok) break;
            tc_commit(bar(K_FREE + kst));
            if (j > 0) tc_commit(bar(V_FREE + vst));
          }
          if (!ok) break;
          tc_commit(bar(Q_FREE));                          // every S product of this item has been issued
          const int vst = (kc + nblk - 1) & 1;
          if (!(ok = mbar_wait(bar(V_FULL + vst), ((kc + nblk - 1) >> 1) & 1, s_abort))) break;
          for (int t = 0; t < ntile && ok; ++t) {
            ok = issue_pv(t, vst, nblk - 1);
            if (ok) tc_commit(bar(O_FULL + t));
          }
          if (!ok) break;
          tc_commit(bar(V_FREE + vst));
          kc += nblk;
          for (int t = 0; t < ntile; ++t) {
            gt[t] += nblk;
            ++itt[t];
          }
        }
      }
    }
  }
  if (warp >= 2 && warp < 10) {
    const int t = (warp - 2) >> 2;                       // tile of this warp
    const int quarter = warp & 3;                        // tensor-memory lane quarter this warp may access
    const int trow = quarter * 32 + lane;                // query row of this thread inside the tile
    const uint32_t tlane = (uint32_t)(quarter * 32) << 16;
    const uint32_t s_addr = tmem_base + tlane + t * 128;
    const uint32_t o_addr = tmem_base + tlane + O_COL + t * DH;
    uint32_t g = 0, it = 0;
    bool ok = true;
    // O row *= corr (whole warp; rows whose maximum did not move pass 1)
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
    // PAIRS: tile t of every item of this CTA; STREAMS: every item of stream t
    const int w_first = (int)blockIdx.x + (streams ? t * (int)gridDim.x : 0), w_step = streams ? nstream : (int)gridDim.x;
    const int t_off = streams ? 0 : t * PP_BQ;
    for (int w = w_first; w < total && ok; w += w_step) {
      int b, h, row0, nrows;
      decode(w, b, h, row0, nrows);
      const int rows_t = nrows - t_off;                  // rows of this tile (<= 0: the item has no second tile)
      if (rows_t <= 0) continue;
      float m_used = 0.f, l = 0.f;
      // one key block of this tile; MASKED only for a last block that reaches beyond key N (kept apart so that the
      // common path is free of branches and the compiler can interleave loads, maxima and exponentials)
      auto block = [&](int j, auto masked_tag) -> bool {
        constexpr bool MASKED = decltype(masked_tag)::value;
        if (!__all_sync(0xffffffffu, mbar_wait(bar(S_FULL + t), (g + j) & 1, s_abort))) return false;
        tc_fence_after();
        uint32_t s[128];
        tc_ld32(s_addr, s);
        tc_ld32(s_addr + 32, s + 32);
        tc_ld32(s_addr + 64, s + 64);
        tc_ld32(s_addr + 96, s + 96);
        tc_wait_ld();
        if (MASKED) {
          const int nvalid = N - j * PP_BKV;             // keys of this block that exist
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (c >= nvalid) s[c] = 0xff800000u;         // -inf
        }
        float mx8[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) mx8[c] = __uint_as_float(s[c]);
#pragma unroll
        for (int c = 8; c < 120; c += 16) {
#pragma unroll
          for (int k = 0; k < 8; ++k) mx8[k] = max3(mx8[k], __uint_as_float(s[c + 2 * k]), __uint_as_float(s[c + 2 * k + 1]));
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) mx8[k] = max3(mx8[k], __uint_as_float(s[120 + 2 * k]), __uint_as_float(s[121 + 2 * k]));
        const float mx = max3(max3(mx8[0], mx8[1], mx8[2]), max3(mx8[3], mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])) * scale_log2;
        // the running maximum is replaced only when it grows by more than 2^8
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
        // S of this block is complete, so the previous block's P V is too, and this block's has not been issued
        if (j > 0 && __any_sync(0xffffffffu, need)) rescale_o(corr);
        const float2 sc2 = make_float2(scale_log2, scale_log2), nm2 = make_float2(-m_used, -m_used);
        float2 sum2[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#define PP_EXP32(c0)                                                                                                   \
  _Pragma("unroll") for (int c = (c0); c < (c0) + 32; c += 2) {                                                        \
    const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2, nm2);              \
    const float2 p = make_float2(fast_exp2(x.x), fast_exp2(x.y));                                                      \
    sum2[(c >> 1) & 3] = __fadd2_rn(sum2[(c >> 1) & 3], p);                                                            \
    s[c >> 1] = pack_bf16(p.x, p.y);                     /* packed P over the registers whose scores are spent */      \
  }
        PP_EXP32(0)
        PP_EXP32(32)
        // P: keys 2c, 2c+1 in column 64 + c of the S tile (whose scores are all in registers by now)
        tc_st32(s_addr + 64, s);                         // keys 0..63
        PP_EXP32(64)
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(P_HALF + t));     // the first half of P V can start
        PP_EXP32(96)
        tc_st32(s_addr + 96, s + 32);                    // keys 64..127
        sum2[0] = __fadd2_rn(__fadd2_rn(sum2[0], sum2[1]), __fadd2_rn(sum2[2], sum2[3]));
        l += sum2[0].x + sum2[0].y;
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(P_FULL + t));
        return true;
      };
      const int nfast = (N % PP_BKV) ? nblk - 1 : nblk;
      for (int j = 0; j < nfast && ok; ++j) ok = block(j, std::false_type{});
      if (ok && nfast < nblk) ok = block(nblk - 1, std::true_type{});
      if (!ok) break;
      g += nblk;
      ok = __all_sync(0xffffffffu, mbar_wait(bar(O_FULL + t), it & 1, s_abort));   // last P V of the item done
      if (!ok) break;
      ++it;
      tc_fence_after();
      const float inv = 1.f / l;
      bf16* orow = o + ((long long)(row0 + t_off + trow) * H + h) * DH;
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
      if (lane == 0) mbar_arrive(bar(O_FREE + t));
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

template <int DH>
static int launch_pp_dh(const CUtensorMap& q, const CUtensorMap& k, const CUtensorMap& v, const int32_t* row_offsets,
                        int max_rows, int B, int N, int H, void* o, int32_t* status, cudaStream_t st) {
  constexpr int SLABS = DH / 64;
  const int smem = 6 * SLABS * 128 * 128 + 1024 + 512 + 4 * (B + 4);
  static int attr_smem = 0;
  if (smem > attr_smem) {
    SL_CUDA_TRY(cudaFuncSetAttribute(attention_pp_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    attr_smem = smem;
  }
  long long items = (long long)H * ((max_rows + PP_BQ - 1) / PP_BQ + B);
  int grid = sm_count();
  if (items < grid) grid = (int)items;
  if (grid < 1) grid = 1;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)DH);
  SL_CUDA_TRY(launch_pdl(attention_pp_kernel<DH>, dim3(grid), dim3(PP_THREADS), (size_t)smem, st, q, k, v, row_offsets, B, N, H,
                         (bf16*)o, scale_log2, status));
  SL_CUDA_TRY(cudaGetLastError());
  return SL_OK;
}

int launch_attention_tc(const void* q, const void* kc, const void* vc, const int32_t* row_offsets, int max_rows, int B,
                         int N, int H, int head_dim, void* o, int32_t* status, cudaStream_t st) {
  if ((head_dim != 64 && head_dim != 128) || B > PP_MAX_B || max_rows < 1 || !row_offsets) return SL_EUNSUPPORTED;
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
  return head_dim == 128 ? launch_pp_dh<128>(tq, tk, tv, row_offsets, max_rows, B, N, H, o, status, st)
                         : launch_pp_dh<64>(tq, tk, tv, row_offsets, max_rows, B, N, H, o, status, st);
}

}  // namespace sl
