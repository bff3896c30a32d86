// Tensor-core GEMM for the packed active rows on sm_100a: C[r][n] = sum_k A[r][k] W[n][k], bf16 in, fp32 accumulate
// (the Q/K/V, output, SwiGLU and LM-head contractions of Algorithm 1 lines 10, 12 and 15).
//
// Persistent, warp-specialised CTAs, one per SM:
//   warp 0   TMA producer: cp.async.bulk.tensor loads of an A tile (128, 64 or 32 rows x 64) and a W tile (BN rows x 64,
//            as one 256-row box when BN = 256) per stage into 128-byte-swizzled shared memory, completion counted on
//            an mbarrier (no multicast); 4 to 16 stages in 216 KB, the stage size follows the tile;
//   warp 1   allocates tensor memory and issues tcgen05.mma (128 x BN x 16, cta_group::1) from one thread, operands
//            described by shared-memory matrix descriptors; tcgen05.commit hands smem stages back to the producer
//            and finished accumulators to the epilogue;
//   warps 2-5 epilogue: tcgen05.ld the fp32 accumulator (one row per thread), apply the fused operation
//            (store bf16 | add into the fp32 residual stream, as 128-byte bulk reductions performed by the L2 from a
//            per-thread staging slot wherever the stages leave 18 KB of shared memory, so that the epilogue never
//            waits for a load of x | silu(gate)*up | QKV: rotary embedding on q and k with
//            the row's ORIGINAL position, q stored packed, k and v written straight into the cache row of that
//            position, which is Algorithm 1 line 11 done in the epilogue) and write with 128-bit stores.
// Two accumulators live in tensor memory so the epilogue of tile i overlaps the main loop of tile i+1.
// At large M the whole launch takes the CTA-pair path (run_pair below: cluster of two, cta_group::2, 256 x 256 tiles).
// At small M the K dimension is split over several CTAs; they meet in a workspace (see the epilogue).  The kernel is
// launched with programmatic stream serialization: set-up, and inside a step the first weight copies, run while the
// previous kernel drains.
// The number of rows M is read from device memory: tiles whose first row is >= M are never scheduled, TMA zero-fills
// rows beyond the allocation, and the epilogue stores only rows < M.  Every mbarrier wait is bounded: when it runs out
// the CTA records SL_DEV_GEMM_TIMEOUT, all roles leave their loops, tensor memory is freed and the kernel returns.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <unordered_map>

#include "tc_common.cuh"

namespace sl {

constexpr int TC_BM = 128, TC_BK = 64, TC_THREADS = 192;
constexpr int TC_MAX_STAGES = 16;
constexpr unsigned long long SPLIT_HELP_CYCLES = 200000ull;   // how long a split waits for its siblings before leaving (~0.1 ms)
constexpr int TC_DATA_BYTES = 216 * 1024;   // operand stages: 4 x 48 KB (128 rows of A + a 256-wide weight tile) ... 16 x 12 KB

constexpr int EPI_QKV = 3;   // three weight matrices side by side; epilogue = RoPE + packed q + K/V cache scatter

struct QkvArgs {
  bf16 *q, *kc, *vc;          // q packed [M][hd]; caches [B*N][hd]
  const int32_t* idx;         // [M] flat position of each packed row
  const float2* rope;         // [n_seq][dh/2] (cos, sin)
  int n_seq, hd, dh;
  // EPI_STORE only (the LM head): per (256-column tile, row) the running maximum, sum of exp(x - max) and arg-max of the
  // stored (bf16-rounded) values, [n_tiles][lse_rows] float4 (m, s, index as int bits, 0); *lse_valid = 1 when this
  // launch wrote them (256-wide tiles without K split).  nullptr: not wanted.
  float4* lse_part;
  int lse_rows;
  int* lse_valid;
};

struct RowStat {
  float m, s;
  int am;
};

// ----------------------------------------------------------------------------------------------- kernel
// Source of accumulator values for the epilogue: tensor memory (one tile computed by this CTA), or the sum of the
// fp32 partial tiles that the K-splits of a tile left in the workspace (summed in split order: deterministic).
struct TmemSrc {
  uint32_t taddr;
  __device__ __forceinline__ void load(int col, uint32_t* v) const {
    tc_ld32(taddr + col, v);
    tc_wait_ld();
  }
  __device__ __forceinline__ void load2(int col0, uint32_t* v0, int col1, uint32_t* v1) const {
    tc_ld32(taddr + col0, v0);
    tc_ld32(taddr + col1, v1);
    tc_wait_ld();
  }
};
// Partial tiles are stored column-group-major: element (r, c) of a tile at float ((c / 4) * 128 + r) * 4 + c % 4, so
// that the 32 rows of a warp write (and the finisher's threads read) 512 contiguous bytes per float4.
struct WsSrc {
  const float* base;      // partial tile of split 0
  int r;                  // row inside the tile
  size_t split_stride;    // floats between consecutive splits of the same tile
  int S;
  // sum over the splits in split order (deterministic), four splits' loads in flight at a time
  __device__ __forceinline__ void load(int col, uint32_t* v) const {
    float acc[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) acc[j] = 0.f;
    const float* p0 = base + ((size_t)(col >> 2) * TC_BM + r) * 4;
    for (int s0 = 0; s0 < S; s0 += 4) {
      float4 t[4][8];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (s0 + q < S) {
          const float* p = p0 + (size_t)(s0 + q) * split_stride;
#pragma unroll
          for (int j = 0; j < 8; ++j) t[q][j] = __ldcg(reinterpret_cast<const float4*>(p + (size_t)j * TC_BM * 4));
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (s0 + q < S) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            acc[4 * j] += t[q][j].x; acc[4 * j + 1] += t[q][j].y; acc[4 * j + 2] += t[q][j].z; acc[4 * j + 3] += t[q][j].w;
          }
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(acc[j]);
  }
  __device__ __forceinline__ void load2(int col0, uint32_t* v0, int col1, uint32_t* v1) const {
    load(col0, v0);
    load(col1, v1);
  }
};

// STREAM: the output is not read again soon (logits, the SwiGLU activations of a large step): stored with the
// streaming hint so that it does not push the activation tiles, which every column tile re-reads, out of L2
template <bool STREAM = false>
__device__ __forceinline__ void store_bf16x32(bf16* dst, const uint32_t* v) {
#pragma unroll
  for (int j = 0; j < 32; j += 8) {
    const uint4 t = make_uint4(pack_bf16(__uint_as_float(v[j]), __uint_as_float(v[j + 1])),
                                                    pack_bf16(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3])),
                                                    pack_bf16(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5])),
                                                    pack_bf16(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7])));
    if (STREAM) __stcs(reinterpret_cast<uint4*>(dst + j), t);
    else *reinterpret_cast<uint4*>(dst + j) = t;
  }
}

// One 32-column unit of the LM head: store as bf16 and fold the stored values into the row's running softmax statistics
// (Algorithm 1 line 15: the posterior's normaliser, and the arg-max / confidence of line 18, taken where the logits are
// still in registers so that the softmax-KL kernel need not read the current row twice).
template <typename Src>
__device__ __forceinline__ void store_unit_with_stats(const Src& src, int row, bool live, int u, int n0, int n_out,
                                                      void* __restrict__ Cv, RowStat& rs) {
  const int c0 = u * 32, col = n0 + c0;
  uint32_t v[32];
  src.load(c0, v);
  if (!live || col >= n_out) return;
  float f[32];
  float lm = -INFINITY;
  int li = 0;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    f[j] = col + j < n_out ? __bfloat162float(__float2bfloat16_rn(__uint_as_float(v[j]))) : -INFINITY;
    if (f[j] > lm) {                                   // strict: the lowest index wins a tie
      lm = f[j];
      li = j;
    }
  }
  if (lm > rs.m) {
    rs.s *= fast_exp2((rs.m - lm) * 1.4426950408889634f);   // rs.m = -inf: 0
    rs.m = lm;
    rs.am = col + li;
  }
  const float nb = -rs.m * 1.4426950408889634f;
  float2 acc = make_float2(0.f, 0.f);
#pragma unroll
  for (int j = 0; j < 32; j += 2) {
    const float2 t = __ffma2_rn(make_float2(f[j], f[j + 1]), make_float2(1.4426950408889634f, 1.4426950408889634f),
                                make_float2(nb, nb));
    acc = __fadd2_rn(acc, make_float2(fast_exp2(t.x), fast_exp2(t.y)));
  }
  rs.s += acc.x + acc.y;
  bf16* dst = reinterpret_cast<bf16*>(Cv) + (long long)row * n_out + col;
  if (col + 32 <= n_out) {
    store_bf16x32<true>(dst, v);
  } else {
    for (int j = 0; j < 32 && col + j < n_out; ++j) dst[j] = __float2bfloat16_rn(__uint_as_float(v[j]));
  }
}

// The epilogue works in UNITS of one row: 32 output columns (64 for a rotated q/k pair block).  A 128 x bn tile has
// units_per_row() units per row; unit u of row `row` is finished by epilogue_unit().  Reading the accumulator from
// tensor memory ties a thread to its row (lane); reading summed partial tiles from the workspace does not, so the
// split-K finisher spreads (row, unit) pairs over all epilogue threads.
template <int EPI>
__device__ __forceinline__ int units_per_row(int bn, int n0, const QkvArgs& qkv) {
  if (EPI == EPI_SWIGLU) return bn >> 6;
  if (EPI == EPI_QKV && n0 / qkv.hd != 2) return bn >> 6;   // (head, 32-pair block): bn/dh * (dh/2)/32
  return bn >> 5;
}

template <int EPI, typename Src, bool STREAM_OUT = false>
__device__ __forceinline__ void epilogue_unit(const Src& src, int bn, int row, bool live, int u, int n0, int n_out,
                                              void* __restrict__ Cv, const QkvArgs& qkv, uint32_t red_slot = 0) {
  if (EPI == EPI_QKV) {
    const int srcm = n0 / qkv.hd, ln0 = n0 - srcm * qkv.hd;
    const int pos = live ? qkv.idx[row] : 0;
    bf16* drow = srcm == 0 ? qkv.q + (long long)row * qkv.hd : (srcm == 1 ? qkv.kc : qkv.vc) + (long long)pos * qkv.hd;
    if (srcm == 2) {
      uint32_t v[32];
      src.load(u * 32, v);
      if (live) store_bf16x32(drow + ln0 + u * 32, v);
    } else {
      const int half = qkv.dh >> 1, per_head = half >> 5;
      const int hh = (u / per_head) * qkv.dh, cc = (u % per_head) * 32;     // head offset, pair block
      const float2* tr = qkv.rope + (long long)(pos % qkv.n_seq) * half;
      uint32_t lo[32], hi[32];
      src.load2(hh + cc, lo, hh + half + cc, hi);
      if (live) {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float2 cs = __ldg(tr + cc + j);
          const float a = __uint_as_float(lo[j]), b = __uint_as_float(hi[j]);
          lo[j] = __float_as_uint(a * cs.x - b * cs.y);
          hi[j] = __float_as_uint(b * cs.x + a * cs.y);
        }
        store_bf16x32(drow + ln0 + hh + cc, lo);
        store_bf16x32(drow + ln0 + hh + half + cc, hi);
      }
    }
    return;
  }
  const int out_bn = EPI == EPI_SWIGLU ? bn >> 1 : bn;
  const int c0 = u * 32;
  uint32_t v[32];
  if (EPI == EPI_SWIGLU) {
    uint32_t g2[32];
    src.load2(c0, v, out_bn + c0, g2);
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const float g = __uint_as_float(v[j]);
      v[j] = __float_as_uint(g / (1.f + __expf(-g)) * __uint_as_float(g2[j]));
    }
  } else {
    src.load(c0, v);
  }
  const int col = n0 + c0;
  if (live && col < n_out) {
    if (EPI == EPI_RESIDUAL) {
      float* dst = reinterpret_cast<float*>(Cv) + (long long)row * n_out + col;
      if (col + 32 <= n_out && red_slot) {
        // residual add done by the L2: the 128 bytes of this row go through the thread's staging slot into one bulk
        // reduction, so the epilogue never waits for a load of x
        bulk_wait_read0();                       // the previous unit's reduction has read the slot
#pragma unroll
        for (int j = 0; j < 32; j += 4) st_shared_f4(red_slot + 4 * j, v[j], v[j + 1], v[j + 2], v[j + 3]);
        fence_async_smem();
        bulk_reduce_add_f32(dst, red_slot, 128);
        bulk_commit();
      } else if (col + 32 <= n_out) {
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
        store_bf16x32<STREAM_OUT>(dst, v);
      } else {
        for (int j = 0; j < 32 && col + j < n_out; ++j) dst[j] = __float2bfloat16_rn(__uint_as_float(v[j]));
      }
    }
  }
}

// Tile width and K-split for this launch, derived on the device from M so that every role of every CTA agrees.
// Enough 256-wide tiles to fill the grid (large M): 256-wide, no split, the tensor-pipe-bound configuration.
// A single row tile (M <= 128, the weight-streaming regime): the widest tiles that, split at most four ways, fill one
// round of the grid.  A few row tiles: width and split with the least estimated time.  Splits meet in the workspace;
// the partial tiles are summed in split order (deterministic) and the fused epilogue runs on the sum.
struct TileCfg {
  int bn, S, m_tiles, n_tiles, tiles, total;   // split sp of a tile covers K blocks [sp * num_kb / S, (sp + 1) * num_kb / S)
};
template <int EPI>
__device__ __forceinline__ TileCfg choose_tiles(int M, int n_out, int num_kb, int grid, bool can_split, int ws_tiles,
                                                int min_bn) {
  TileCfg c;
  c.m_tiles = (M + TC_BM - 1) / TC_BM;
  auto ntiles = [&](int bn) {
    const int ob = EPI == EPI_SWIGLU ? bn >> 1 : bn;
    return (n_out + ob - 1) / ob;
  };
  c.bn = 256;
  c.S = 1;
  if (c.m_tiles == 1) {
    // Weight-streaming regime: the widest tiles (most bytes per copy) that, with K split at most four ways and all
    // items in ONE round of the grid, keep at least 0.6 of the SMs streaming.  (Measured on B200: more than four splits
    // or a second round cost more in the hand-over through the workspace than the idle SMs do; narrow tiles without a
    // split are bounded by the ~280 ns one K block takes whatever its size.)
    c.bn = 128 > min_bn ? 128 : min_bn;
    for (int bn = 256; bn >= 128 && bn >= min_bn; bn >>= 1) {
      const int tiles = ntiles(bn);
      int sp = grid / tiles;
      sp = sp < 1 ? 1 : (sp > 4 ? 4 : sp);
      if (sp * 4 > num_kb) sp = num_kb / 4 > 0 ? num_kb / 4 : 1;
      if (!can_split || sp * tiles > ws_tiles) sp = 1;
      c.bn = bn;
      c.S = sp;
      if (5 * tiles * sp >= 3 * grid) break;
    }
  } else if (c.m_tiles > 1 && c.m_tiles * ntiles(256) < grid) {
    // a few row tiles: tile width and K split with the least estimated time, in units of one 256-wide K block:
    // rounds of the grid x (K blocks of an item x relative cost of a block at this width + the cost of meeting in the
    // workspace when K is split).  A narrower tile re-reads the activation tile and uses the tensor pipe less well.
    float best = 3.0e38f;
    for (int bn = 256; bn >= min_bn && bn >= 128; bn >>= 1) {
      const float cbn = bn == 256 ? 1.0f : 0.6f;
      const int tiles = c.m_tiles * ntiles(bn);
      for (int sp = 1; sp <= 8 && sp * 4 <= num_kb; ++sp) {
        if (sp > 1 && (!can_split || sp * tiles > ws_tiles)) break;
        const int rounds = (tiles * sp + grid - 1) / grid;
        const float cost = (float)rounds * ((float)((num_kb + sp - 1) / sp) * cbn + (sp > 1 ? 6.f + 10.f * cbn : 0.f));
        if (cost < best - 1e-6f) {
          best = cost;
          c.bn = bn;
          c.S = sp;
        }
      }
    }
  }
  c.n_tiles = ntiles(c.bn);
  c.tiles = c.m_tiles * c.n_tiles;
  if (c.S > num_kb) c.S = num_kb;
  if (c.S < 1) c.S = 1;
  c.total = c.tiles * c.S;
  return c;
}

// Order of the output tiles.  Row tiles are taken in GROUPS whose activation rows (group rows x K x 2 bytes) stay in L2
// (TILE_GROUP_BYTES, well under the 126 MB); inside a group the row index runs fastest, then the column tile, so a
// weight tile is fetched from DRAM once per group and the activation rows once in all.  With a single group this is
// the plain row-fastest order.  (Before: one group; with M x K x 2 bytes beyond the L2 the activation matrix was
// re-read from DRAM for every few column tiles: 1.28 GB read for the 262 MB of operands of the down projection at
// M = 6587.)
#ifndef TILE_GROUP_MB
#define TILE_GROUP_MB 40
#endif
constexpr long long TILE_GROUP_BYTES = (long long)TILE_GROUP_MB << 20;
__device__ __forceinline__ void tile_of(int w, int m_tiles, int n_tiles, int group, int& mt, int& nt) {
  const int per_group = group * n_tiles;
  const int g = w / per_group, r = w - g * per_group;
  const int m_first = g * group;
  const int g_rows = m_tiles - m_first < group ? m_tiles - m_first : group;   // the last group may be smaller
  nt = r / g_rows;
  mt = m_first + (r - nt * g_rows);
}
__device__ __forceinline__ int tile_group(int tile_rows, int K) {
  const long long g = TILE_GROUP_BYTES / ((long long)tile_rows * K * 2);
  return g < 1 ? 1 : (g > (1 << 20) ? (1 << 20) : (int)g);
}

// ---- CTA-pair path (cta_group::2) for the tensor-pipe-bound regime ---------------------------------------------------
// A cluster of two CTAs owns a 256 x 256 output tile: each CTA loads its own 128 rows of A and HALF of the weight tile
// (128 of its 256 rows), the leader CTA issues tcgen05.mma.cta_group::2 (M = 256) which reads both CTAs' shared memory,
// and each CTA's tensor memory receives the accumulator of its own 128 rows.  Per K block a CTA moves 32 KB instead of
// 48 KB from L2 (the weight half is shared by the pair), which leaves room for six stages.  Barriers: "full" lives in
// the leader (both CTAs' TMA loads count their bytes there), "empty" and "accumulator full" are reached in both CTAs by
// a multicast tcgen05.commit, "accumulator empty" lives in the leader and is reached by the peer's epilogue with a
// remote arrive.  All waits are bounded like in the single-CTA path.
constexpr int TC2_STAGES = 6;

template <int EPI>
__device__ __forceinline__ void run_pair(const CUtensorMap* tmA, const CUtensorMap* tmW0, const CUtensorMap* tmW1,
                                         const CUtensorMap* tmW2, void* __restrict__ Cv, int M, int n_out, int K,
                                         int32_t* status, const QkvArgs& qkv, uint8_t* smem) {
  constexpr int BN = 256;
  constexpr int A_BYTES = TC_BM * TC_BK * 2;              // 16 KB: this CTA's 128 rows of A
  constexpr int B_BYTES = 128 * TC_BK * 2;                // 16 KB: this CTA's half of the weight tile
  constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr int STAGES = TC2_STAGES;
  constexpr uint32_t TMEM_COLS = 512;
  constexpr int OUT_BN = EPI == EPI_SWIGLU ? 128 : 256;

  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto accf_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
  auto acce_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);      // the leader's arrive.expect_tx; transaction bytes of both CTAs
      mbar_init(empty_bar(s), 1);     // one multicast commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accf_bar(a), 1);      // one multicast commit
      mbar_init(acce_bar(a), 8);      // four epilogue warps of each CTA
    }
    *s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) tc_alloc_pair(smem_u32(s_tmem), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                 // the peer's barriers are initialised before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;

  const int m_pairs = (M + 2 * TC_BM - 1) / (2 * TC_BM);
  const int n_tiles = (n_out + OUT_BN - 1) / OUT_BN;
  const int total = m_pairs * n_tiles;
  const int num_kb = (K + TC_BK - 1) / TC_BK;
  const int cid = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  const int group = tile_group(2 * TC_BM, K);

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint64_t keep = l2_policy_evict_last();     // activation tiles: every column tile of the group re-reads them
#ifndef TC2_W_EVICT_FIRST_PAIRS
#define TC2_W_EVICT_FIRST_PAIRS 2
#endif
      // with at most two pair rows a weight tile is read by the pairs that work on it at the same time and never again
      const uint64_t wpol = m_pairs <= TC2_W_EVICT_FIRST_PAIRS ? l2_policy_evict_first() : l2_policy_evict_normal();
      for (int w = cid; w < total && ok; w += n_clusters) {
        int mt, nt;
        tile_of(w, m_pairs, n_tiles, group, mt, nt);
        const int m0 = mt * 2 * TC_BM + (int)rank * TC_BM, n0 = nt * OUT_BN;
        // this CTA's half of the weight tile
        const CUtensorMap* mp = tmW0;
        int brow = n0 + (int)rank * 128;
        if (EPI == EPI_SWIGLU) {                           // leader: gate rows, peer: up rows of the same features
          mp = rank == 0 ? tmW0 : tmW1;
          brow = n0;
        } else if (EPI == EPI_QKV) {
          const int src = n0 / qkv.hd;
          mp = src == 0 ? tmW0 : (src == 1 ? tmW1 : tmW2);
          brow = n0 - src * qkv.hd + (int)rank * 128;
        }
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1, s_abort))) break;
          const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES), sb = sa + A_BYTES;
          const uint32_t fb = mapa_u32(full_bar(stage), 0);
          if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * STAGE_BYTES);
          tma_load_2d_pair_hint(sa, tmA, kb * TC_BK, m0, fb, keep);
          tma_load_2d_pair_hint(sb, mp, kb * TC_BK, brow, fb, wpol);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = idesc_bf16_m128(BN, false, 256);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      for (int w = cid; w < total && ok; w += n_clusters, ++it) {
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
          for (int k = 0; k < TC_BK / 16; ++k)
            tc_mma_bf16_pair(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (kb > 0) | (k != 0));
          tc_commit_pair_mcast(empty_bar(stage), 3);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) tc_commit_pair_mcast(accf_bar(acc), 3);
      }
    }
  } else {
    const int quarter = warp & 3;
    bool ok = true;
    int it = 0;
    // EPI_RESIDUAL: 144-byte staging slot of this thread above the stages and barriers (the odd stride keeps the eight
    // 16-byte stores of a quarter warp on different banks)
    const uint32_t red_slot = EPI == EPI_RESIDUAL
        ? smem_u32(smem + STAGES * STAGE_BYTES + 1024) + (uint32_t)(quarter * 32 + lane) * 144u : 0u;
    static_assert(STAGES * STAGE_BYTES + 1024 + 128 * 144 <= TC_DATA_BYTES, "staging slots must fit the allocation");
    for (int w = cid; w < total && ok; w += n_clusters, ++it) {
      const int acc = it & 1;
      const uint32_t use = (uint32_t)(it >> 1);
      int mt, nt;
      tile_of(w, m_pairs, n_tiles, group, mt, nt);
      const int m0 = mt * 2 * TC_BM + (int)rank * TC_BM, n0 = nt * OUT_BN;
      ok = mbar_wait(accf_bar(acc), use & 1, s_abort);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = m0 + quarter * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
      const int upr = units_per_row<EPI>(BN, n0, qkv);
      if (EPI == EPI_STORE && qkv.lse_part) {
        RowStat rs{-INFINITY, 0.f, 0};
#pragma unroll 1
        for (int u = 0; u < upr; ++u) store_unit_with_stats(TmemSrc{taddr}, row, row < M, u, n0, n_out, Cv, rs);
        if (row < M)
          qkv.lse_part[(size_t)(n0 / BN) * qkv.lse_rows + row] = make_float4(rs.m, rs.s, __int_as_float(rs.am), 0.f);
      } else {
#pragma unroll 1
        for (int u = 0; u < upr; ++u)
          epilogue_unit<EPI, TmemSrc, EPI != EPI_QKV>(TmemSrc{taddr}, BN, row, row < M, u, n0, n_out, Cv, qkv, red_slot);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_u32(acce_bar(acc), 0));
    }
    if (EPI == EPI_RESIDUAL) bulk_wait0();      // every reduction of this thread has been performed before the CTA leaves
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *s_abort) set_status(status, SL_DEV_GEMM_TIMEOUT);
  cluster_sync_all();                 // neither CTA leaves (or frees tensor memory) while the pair may still use it
  if (warp == 1) {
    tc_fence_after();
    tc_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

template <int EPI, int STAGES>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA32,
               const __grid_constant__ CUtensorMap tmA64, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
               const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
               const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmX0,
               const __grid_constant__ CUtensorMap tmX1, const __grid_constant__ CUtensorMap tmX2, void* __restrict__ Cv, const int32_t* __restrict__ n_active,
               int n_out, int K, int32_t* status, const QkvArgs qkv, float* __restrict__ ws, int* __restrict__ counters,
               int ws_tiles, int force_bn, int force_s, int pair_mode, int prefetch_w) {
  // tmA / tmA32 / tmA64: the activation matrix with 128-, 32- and 64-row boxes; tmB*: weight maps with 64-row boxes
  // (any tile width); tmW* / tmX*: the same matrices with 128- and 256-row boxes: a 256-wide tile is one 256-row copy
  // (gate/up: two 128-row copies), the CTA-pair path loads 128-row halves
  constexpr int BN_MAX = 256;
  constexpr int BOX_BYTES = 64 * TC_BK * 2;               // 8 KB
  constexpr uint32_t TMEM_COLS = 2 * BN_MAX;              // two accumulators

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  // prefetch_w: the caller states that neither *n_active nor the weights were written by the kernel launched just
  // before this one (true inside a step): M may then be read, and the first weight copies issued, while that kernel is
  // still draining.  Otherwise nothing is read before it has completed.
  if (!prefetch_w) {
    griddep_wait();
    griddep_launch();
  }
  if (pair_mode) {
    // launched as clusters of two: the CTA-pair path takes the whole launch when 256 x 256 pair tiles fill the grid
    // (large M) and need no more time than single tiles: rounds of pair tiles against rounds of 128 x 256 tiles, which
    // cost about 1.15 x as much per round (more L2 -> SM traffic).  Both CTAs of a pair read the same M and take the
    // same branch.
    const int Mp = *n_active;
    const int obn = EPI == EPI_SWIGLU ? 128 : 256;
    const int nt = (n_out + obn - 1) / obn, half = (int)(gridDim.x >> 1);
    const int pairs = ((Mp + 255) / 256) * nt, singles = ((Mp + 127) / 128) * nt;
    const int rounds_p = (pairs + half - 1) / half, rounds_s = (singles + (int)gridDim.x - 1) / (int)gridDim.x;
    // Also when the pair tiles only partly fill ONE round, if the single tiles are too many to split their K range two
    // ways within a round (more than half the grid): a K block of a pair tile moves 32 instead of 48 KB per SM and takes
    // ~0.8 of a single tile's (measured at 4096 x 4096, 4096 x 12288 and 12288 x 4096 for M = 160 ... 1024: 36-38 vs
    // 42-43 us, 76-78 vs 82-94 us, 45 vs 51 us; with fewer single tiles the K split wins).
    const bool take = (pairs >= half && 20 * rounds_p <= 23 * rounds_s) ||
                      (Mp > TC_BM && pairs < half && 2 * singles > (int)gridDim.x && K >= 24 * TC_BK && force_bn <= 0);
    if (take) {
      if (prefetch_w) {
        griddep_wait();
        griddep_launch();
      }
      if (EPI == EPI_STORE && qkv.lse_valid && blockIdx.x == 0 && threadIdx.x == 0) *qkv.lse_valid = 1;
      run_pair<EPI>(&tmA, &tmW0, &tmW1, &tmW2, Cv, Mp, n_out, K, status, qkv, smem);
      return;
    }
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + TC_DATA_BYTES);
  // bars: full[STAGES], empty[STAGES], acc_full[2], acc_empty[2]
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  volatile int* s_fin = reinterpret_cast<volatile int*>(s_tmem + 2);   // [3] split finishing: role, ticket, claim result

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
  const int num_kb = (K + TC_BK - 1) / TC_BK;
  const int min_bn = EPI == EPI_QKV ? (qkv.dh > 64 ? 128 : 64) : (EPI == EPI_SWIGLU ? 128 : 64);
  TileCfg tc = choose_tiles<EPI>(M, n_out, num_kb, (int)gridDim.x, ws != nullptr, ws_tiles, min_bn);
  if (force_bn > 0) {   // tuning aid (host environment variable): fixed tile width and split
    tc.bn = force_bn < min_bn ? min_bn : force_bn;
    const int ob = EPI == EPI_SWIGLU ? tc.bn >> 1 : tc.bn;
    tc.n_tiles = (n_out + ob - 1) / ob;
    tc.tiles = tc.m_tiles * tc.n_tiles;
    tc.S = ws != nullptr && force_s > 0 && tc.tiles * force_s <= ws_tiles ? force_s : 1;
    if (tc.S > num_kb) tc.S = num_kb;
    tc.total = tc.tiles * tc.S;
  }
  const int bn = tc.bn, S = tc.S, m_tiles = tc.m_tiles, total = tc.total;
  const int group = tile_group(TC_BM, K);
  if (EPI == EPI_STORE && qkv.lse_valid && blockIdx.x == 0 && threadIdx.x == 0) *qkv.lse_valid = (S == 1 && bn == 256) ? 1 : 0;
  const int out_bn = EPI == EPI_SWIGLU ? bn >> 1 : bn;
  // Stage layout, chosen from M like the tiles: with a single row tile of few rows only 32 or 64 activation rows are
  // copied per stage (the MMA still reads 128 rows of shared memory; rows >= M are never stored), which leaves room for
  // more stages: what bounds the weight-streaming regime is the number of weight bytes one SM keeps in flight.
  const int a_rows = m_tiles > 1 || M > 64 ? TC_BM : (M > 32 ? 64 : 32);
  const CUtensorMap* mapA = a_rows == TC_BM ? &tmA : (a_rows == 64 ? &tmA64 : &tmA32);
  const int A_BYTES = a_rows * TC_BK * 2;
  const int STAGE_BYTES = A_BYTES + bn * TC_BK * 2;
  const int nst = TC_DATA_BYTES / STAGE_BYTES < STAGES ? TC_DATA_BYTES / STAGE_BYTES : STAGES;   // 4 .. 16
  const uint32_t stage_tx = (uint32_t)(A_BYTES + bn * TC_BK * 2);

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      // the weight part of stage `st` for K block kb of the tile at column n0
      // with at most four row tiles (M <= 512) a weight tile is read by the few CTAs that work on it at the same time and
      // never again: evict-first, so that the weights do not push the activations, partial tiles and logits out of L2
      // (single-sequence step at 305 rows 8.3 -> 7.8 ms)
#ifndef TC_W_EVICT_FIRST_TILES
#define TC_W_EVICT_FIRST_TILES 4
#endif
      const uint64_t wpol = m_tiles <= TC_W_EVICT_FIRST_TILES ? l2_policy_evict_first() : l2_policy_evict_normal();
      auto load_w = [&](int st, int kb, int n0) {
        const uint32_t sb = smem_u32(smem + st * STAGE_BYTES) + A_BYTES;
        const bool wide = bn == 256;
        if (EPI == EPI_SWIGLU) {
          if (wide) {
            tma_load_2d_hint(sb, &tmW0, kb * TC_BK, n0, full_bar(st), wpol);
            tma_load_2d_hint(sb + 2 * BOX_BYTES, &tmW1, kb * TC_BK, n0, full_bar(st), wpol);
          } else {
            const int hb = bn >> 7;                                  // 64-row boxes per half
            for (int i = 0; i < hb; ++i) {
              tma_load_2d_hint(sb + i * BOX_BYTES, &tmB0, kb * TC_BK, n0 + 64 * i, full_bar(st), wpol);
              tma_load_2d_hint(sb + (hb + i) * BOX_BYTES, &tmB1, kb * TC_BK, n0 + 64 * i, full_bar(st), wpol);
            }
          }
        } else {
          int src = 0, ln0 = n0;
          if (EPI == EPI_QKV) {                                      // a tile never straddles two matrices
            src = n0 / qkv.hd;
            ln0 = n0 - src * qkv.hd;
          }
          if (wide) {
            const CUtensorMap* mp = src == 0 ? &tmX0 : (src == 1 ? &tmX1 : &tmX2);
            tma_load_2d_hint(sb, mp, kb * TC_BK, ln0, full_bar(st), wpol);
          } else {
            const CUtensorMap* mp = src == 0 ? &tmB0 : (src == 1 ? &tmB1 : &tmB2);
            for (int i = 0; i < (bn >> 6); ++i)
              tma_load_2d_hint(sb + i * BOX_BYTES, mp, kb * TC_BK, ln0 + 64 * i, full_bar(st), wpol);
          }
        }
      };
      bool waited = !prefetch_w;
      const uint64_t keep = l2_policy_evict_last();     // activation tiles are re-read by every column tile
      for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
        const int t = w / S, sp = w - t * S;
        int mt, nt;
        tile_of(t, m_tiles, tc.n_tiles, group, mt, nt);
        const int m0 = mt * TC_BM, n0 = nt * out_bn;
        const int kb0 = sp * num_kb / S, kb1 = (sp + 1) * num_kb / S;
        int kb = kb0;
        if (!waited) {
          // first item: the weight halves of the first stages go out now, the activation halves once the previous
          // kernel has completed (the stages are fresh, so there is no "empty" wait)
          const int npre = kb1 - kb0 < nst ? kb1 - kb0 : nst;
          for (int i = 0; i < npre; ++i) {
            mbar_expect_tx(full_bar(i), stage_tx);
            load_w(i, kb0 + i, n0);
          }
          griddep_wait();
          griddep_launch();
          waited = true;
          for (int i = 0; i < npre; ++i)
            tma_load_2d_hint(smem_u32(smem + i * STAGE_BYTES), mapA, (kb0 + i) * TC_BK, m0, full_bar(i), keep);
          stage = npre;
          if (stage == nst) { stage = 0; phase ^= 1; }
          kb = kb0 + npre;
        }
        for (; kb < kb1; ++kb) {
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1, s_abort))) break;
          mbar_expect_tx(full_bar(stage), stage_tx);
          tma_load_2d_hint(smem_u32(smem + stage * STAGE_BYTES), mapA, kb * TC_BK, m0, full_bar(stage), keep);
          load_w(stage, kb, n0);
          if (++stage == nst) { stage = 0; phase ^= 1; }
        }
      }
      if (!waited) {
        griddep_wait();
        griddep_launch();
      }
    } else if (prefetch_w) {
      griddep_wait();
      griddep_launch();
    }
  } else if (warp == 1) {
    if (prefetch_w) {
      griddep_wait();
      griddep_launch();
    }
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_m128(bn);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      for (int w = blockIdx.x; w < total && ok; w += gridDim.x, ++it) {
        const int sp = w % S;
        const int kb0 = sp * num_kb / S, kb1 = (sp + 1) * num_kb / S;
        const int acc = it & 1;
        const uint32_t use = (uint32_t)(it >> 1);
        if (!(ok = mbar_wait(acce_bar(acc), (use & 1) ^ 1, s_abort))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN_MAX);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!(ok = mbar_wait(full_bar(stage), phase, s_abort))) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES), sb = sa + A_BYTES;
          const uint64_t adesc = smem_desc_k_sw128(sa), bdesc = smem_desc_k_sw128(sb);
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k)   // 16 bf16 = 32 bytes along K inside the 128-byte swizzle row
            tc_mma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (kb > kb0) | (k != 0));
          tc_commit(empty_bar(stage));
          if (++stage == nst) { stage = 0; phase ^= 1; }
        }
        if (ok) tc_commit(accf_bar(acc));
      }
    }
  } else {
    if (prefetch_w) {
      griddep_wait();
      griddep_launch();
    }
    const int quarter = warp & 3;             // tensor-memory lanes 32*quarter .. 32*quarter+31
    bool ok = true;
    int it = 0;
    // EPI_RESIDUAL, when the stages leave room below the barriers: this thread's 144-byte staging slot for the
    // residual add as an L2 bulk reduction (see epilogue_unit)
    const uint32_t red_slot = EPI == EPI_RESIDUAL && nst * STAGE_BYTES + 128 * 144 <= TC_DATA_BYTES
        ? smem_u32(smem + nst * STAGE_BYTES) + (uint32_t)((warp - 2) * 32 + lane) * 144u : 0u;
    for (int w = blockIdx.x; w < total && ok; w += gridDim.x, ++it) {
      const int t = w / S, sp = w - t * S;
      const int acc = it & 1;
      const uint32_t use = (uint32_t)(it >> 1);
      int mt, nt;
      tile_of(t, m_tiles, tc.n_tiles, group, mt, nt);
      const int m0 = mt * TC_BM, n0 = nt * out_bn;
      ok = mbar_wait(accf_bar(acc), use & 1, s_abort);
      ok = __all_sync(0xffffffffu, ok);
      if (S > 1) ok = epilogue_warps_agree(ok);           // the splits' meeting below has barriers of all four warps
      if (!ok) break;
      tc_fence_after();
      const int trow = quarter * 32 + lane;
      const int row = m0 + trow;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN_MAX);
      const int upr = units_per_row<EPI>(bn, n0, qkv);
      if (S == 1) {
        if (EPI == EPI_STORE && qkv.lse_part && bn == 256) {
          RowStat rs{-INFINITY, 0.f, 0};
#pragma unroll 1
          for (int u = 0; u < upr; ++u) store_unit_with_stats(TmemSrc{taddr}, row, row < M, u, n0, n_out, Cv, rs);
          if (row < M)
            qkv.lse_part[(size_t)(n0 / 256) * qkv.lse_rows + row] = make_float4(rs.m, rs.s, __int_as_float(rs.am), 0.f);
        } else {
#pragma unroll 1
          for (int u = 0; u < upr; ++u) epilogue_unit<EPI>(TmemSrc{taddr}, bn, row, row < M, u, n0, n_out, Cv, qkv, red_slot);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acce_bar(acc));
      } else {
        // partial tile of this K-split -> workspace, then free the accumulator
        float* ptile = ws + (size_t)(t * S + sp) * TC_BM * bn + (size_t)trow * 4;
#pragma unroll 1
        for (int c0 = 0; c0 < bn; c0 += 32) {
          uint32_t v[32];
          tc_ld32(taddr + c0, v);
          tc_wait_ld();
          if (row < M) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              __stcg(reinterpret_cast<float4*>(ptile + (size_t)((c0 + j) >> 2) * TC_BM * 4),
                     make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]),
                                 __uint_as_float(v[j + 3])));
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acce_bar(acc));
        // The splits of a tile meet here.  Each takes a ticket; the finishing work (sum of the partial tiles in split
        // order + fused epilogue) is cut into S shares of the tile's (row, unit) list.  The last arriver always
        // finishes: its own share, then every share nobody has claimed.  A split that arrives earlier and has no other
        // item to compute waits (bounded) for the rest and finishes the share of its ticket, so that in the usual
        // single-round launch the S CTAs of a tile finish it together.  Shares are claimed with an atomic OR, so each
        // is done exactly once whoever gets there first; the last CTA to leave zeroes the tile's three counters.
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        // With little finishing work per tile (few live rows) the hand-over costs more than it saves: then only
        // the last arriver finishes, as one share, and no share is claimed.
        const int live_rows = M - m0 < TC_BM ? M - m0 : TC_BM;
        const int items = live_rows * upr;
        const bool coop = items >= 384;
        const int shares = coop ? S : 1;
        int* arrived = counters + t;
        unsigned* claimed = reinterpret_cast<unsigned*>(counters + ws_tiles + t);
        int* left = counters + 2 * ws_tiles + t;
        const int e_tid = (warp - 2) * 32 + lane;
        if (e_tid == 0) {
          const int ticket = atomicAdd(arrived, 1);
          int role = 0;                                // 0: leave, 1: finish the share of my ticket, 2: last arriver
          if (ticket == S - 1) {
            role = 2;
          } else if (coop && w + (int)gridDim.x >= total) {
            const unsigned long long t0 = clock64();
            while (clock64() - t0 < SPLIT_HELP_CYCLES) {
              if (*reinterpret_cast<volatile int*>(arrived) >= S) {
                role = 1;
                break;
              }
            }
          }
          s_fin[0] = role;
          s_fin[1] = ticket;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int role = s_fin[0], ticket = s_fin[1];
        if (role) {
          __threadfence();
          auto finish_share = [&](int k) {
            const int lo = (int)((long long)k * items / shares), hi = (int)((long long)(k + 1) * items / shares);
#pragma unroll 1
            for (int i = lo + e_tid; i < hi; i += 128) {   // rows fastest: a warp reads contiguous partials
              const int u = i / live_rows, r = i - u * live_rows;
              WsSrc src{ws + (size_t)(t * S) * TC_BM * bn, r, (size_t)TC_BM * bn, S};
              epilogue_unit<EPI>(src, bn, m0 + r, true, u, n0, n_out, Cv, qkv, red_slot);
            }
          };
          const int nk = role == 2 ? shares : 1;       // the last arriver tries its own share first, then all others
#pragma unroll 1
          for (int q = 0; q < nk; ++q) {
            const int k = role == 2 ? (q == 0 ? shares - 1 : q - 1) : ticket;
            if (coop) {
              asm volatile("bar.sync 1, 128;" ::: "memory");
              if (e_tid == 0) s_fin[2] = (int)((atomicOr(claimed, 1u << k) >> k) & 1u);   // 1: somebody else has it
              asm volatile("bar.sync 1, 128;" ::: "memory");
              if (s_fin[2]) continue;
            }
            finish_share(k);
          }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (e_tid == 0) {
          if (coop) {
            __threadfence();
            if (atomicAdd(left, 1) == S - 1) {
              *arrived = 0;
              *claimed = 0u;
              *left = 0;
            }
          } else if (role == 2) {
            *arrived = 0;                              // every split has arrived and only this CTA is still here
          }
        }
      }
    }
    if (EPI == EPI_RESIDUAL) bulk_wait0();      // every reduction of this thread has been performed before the CTA leaves
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

static int pair_mode() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("SURELOCK_GEMM_PAIR");   // 0 disables the CTA-pair (cta_group::2) path
    v = (e && e[0] == '0') ? 0 : 1;
  }
  return v;
}

static int force_cfg(int which) {
  int v[2] = {0, 0};
  const char* e = getenv("SURELOCK_GEMM_FORCE");   // tuning aid, read at every launch: "bn,S", e.g. "128,3"
  if (e) sscanf(e, "%d,%d", &v[0], &v[1]);
  return v[which];
}

template <int EPI, int STAGES>
static int launch_cfg(const CUtensorMap* a, const CUtensorMap* b, const CUtensorMap* wb, const CUtensorMap* xb, void* C,
                      const int32_t* n_active, int max_rows, int n_out, int K, int32_t* status, const QkvArgs& qkv,
                      const SplitWs& sw, cudaStream_t st) {
  constexpr int SMEM = TC_DATA_BYTES + 1024 + 512;
  static bool attr_set = false;
  if (!attr_set) {
    SL_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<EPI, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM));
    attr_set = true;
  }
  (void)max_rows;
  // persistent: one CTA per SM; the tile shape is chosen on the device from M.  The kernel contains cta_group::2
  // instructions, so it is always launched as clusters of two (an even grid) even when the pair path is switched off.
  const int grid = sm_count() & ~1;
  const int pair = pair_mode();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 2;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  SL_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tc_kernel<EPI, STAGES>, a[0], a[1], a[2], b[0], b[1], b[2], wb[0], wb[1], wb[2], xb[0], xb[1], xb[2], C, n_active,
                                 n_out, K, status, qkv, sw.ws, sw.counters, sw.tiles, force_cfg(0),
                                 force_cfg(1), pair, sw.prefetch_w ? 1 : 0));
  return SL_OK;
}

int launch_gemm_tc(const void* A, const void* W, const void* W2, void* C, const int32_t* n_active, int max_rows,
                   int n_out, int K, int epilogue, int32_t* status, const SplitWs& sw, cudaStream_t st) {
  // TMA needs 16-byte aligned bases and row strides; the epilogue's 128-bit stores need n_out % 8 == 0
  if (K % 8 || n_out % 8 || max_rows < 1) return SL_EUNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(W2) |
       reinterpret_cast<uintptr_t>(C)) & 15)
    return SL_EUNSUPPORTED;
  if (epilogue == EPI_SWIGLU && !W2) return SL_EINVAL;
  CUtensorMap a[3], b[3], wb[3], xb[3];
  int rc = get_tensor_map_2d(A, max_rows, K, TC_BM, &a[0]);
  if (rc == SL_OK) rc = get_tensor_map_2d(A, max_rows, K, 32, &a[1]);
  if (rc == SL_OK) rc = get_tensor_map_2d(A, max_rows, K, 64, &a[2]);
  if (rc == SL_OK) rc = get_tensor_map_2d(W, n_out, K, 64, &b[0]);
  if (rc == SL_OK) rc = get_tensor_map_2d(W, n_out, K, 128, &wb[0]);
  if (rc == SL_OK) rc = get_tensor_map_2d(W, n_out, K, 256, &xb[0]);
  if (rc != SL_OK) return rc;
  b[1] = b[2] = b[0];
  wb[1] = wb[2] = wb[0];
  xb[1] = xb[2] = xb[0];
  if (W2) {
    rc = get_tensor_map_2d(W2, n_out, K, 64, &b[1]);
    if (rc == SL_OK) rc = get_tensor_map_2d(W2, n_out, K, 128, &wb[1]);
    if (rc != SL_OK) return rc;
  }
  switch (epilogue) {
    case EPI_STORE: {
      QkvArgs qa{};
      qa.lse_part = sw.lse_part;
      qa.lse_rows = sw.lse_rows;
      qa.lse_valid = sw.lse_valid;
      return launch_cfg<EPI_STORE, TC_MAX_STAGES>(a, b, wb, xb, C, n_active, max_rows, n_out, K, status, qa, sw, st);
    }
    case EPI_RESIDUAL: return launch_cfg<EPI_RESIDUAL, TC_MAX_STAGES>(a, b, wb, xb, C, n_active, max_rows, n_out, K, status, QkvArgs{}, sw, st);
    case EPI_SWIGLU: return launch_cfg<EPI_SWIGLU, TC_MAX_STAGES>(a, b, wb, xb, C, n_active, max_rows, n_out, K, status, QkvArgs{}, sw, st);
    default: return SL_EINVAL;
  }
}

// Q/K/V projections in one launch with RoPE and the cache scatter in the epilogue (Algorithm 1 lines 10-11).
int launch_gemm_tc_qkv(const void* A, const void* Wq, const void* Wk, const void* Wv, void* q_out, void* k_cache,
                       void* v_cache, const int32_t* idx, const float2* rope, const int32_t* n_active, int max_rows,
                       int n_seq, int hd, int dh, int K, int32_t* status, const SplitWs& sw, cudaStream_t st) {
  if (K % 8 || hd % 256 || (dh != 64 && dh != 128) || max_rows < 1) return SL_EUNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(Wq) | reinterpret_cast<uintptr_t>(Wk) |
       reinterpret_cast<uintptr_t>(Wv) | reinterpret_cast<uintptr_t>(q_out) | reinterpret_cast<uintptr_t>(k_cache) |
       reinterpret_cast<uintptr_t>(v_cache)) & 15)
    return SL_EUNSUPPORTED;
  CUtensorMap a[3], b[3], wb[3], xb[3];
  const void* W[3] = {Wq, Wk, Wv};
  int rc = get_tensor_map_2d(A, max_rows, K, TC_BM, &a[0]);
  if (rc == SL_OK) rc = get_tensor_map_2d(A, max_rows, K, 32, &a[1]);
  if (rc == SL_OK) rc = get_tensor_map_2d(A, max_rows, K, 64, &a[2]);
  for (int i = 0; i < 3 && rc == SL_OK; ++i) {
    rc = get_tensor_map_2d(W[i], hd, K, 64, &b[i]);
    if (rc == SL_OK) rc = get_tensor_map_2d(W[i], hd, K, 128, &wb[i]);
    if (rc == SL_OK) rc = get_tensor_map_2d(W[i], hd, K, 256, &xb[i]);
  }
  if (rc != SL_OK) return rc;
  QkvArgs qa{(bf16*)q_out, (bf16*)k_cache, (bf16*)v_cache, idx, rope, n_seq, hd, dh, nullptr, 0, nullptr};
  return launch_cfg<EPI_QKV, TC_MAX_STAGES>(a, b, wb, xb, nullptr, n_active, max_rows, 3 * hd, K, status, qa, sw, st);
}

}  // namespace sl
