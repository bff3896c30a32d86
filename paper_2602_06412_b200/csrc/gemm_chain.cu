// The contractions of a transformer block for FEW active rows (M <= 64) as ONE persistent kernel per layer:
// output projection -> gate / up (+ SwiGLU) -> down projection -> Q/K/V projections of the NEXT layer (with its
// rotary embedding and K/V cache scatter), i.e. everything of Algorithm 1 lines 10-13 between two attention calls.
//
// Why: with few rows a step is bound by reading every weight once from HBM (the regime in which the paper reports no
// gain, App. "Algorithmic Characteristics on Runtime"), and with one kernel per contraction what is lost is the
// latency chain at every kernel boundary (launch, first bytes, reduction hand-over, exit).  Here the weight stream
// never stops: every CTA (one per SM, cooperative launch) owns, for each contraction, a contiguous range of
// (feature tile, K block) units of equal length, so all SMs stream the same number of bytes; its producer warp walks
// through the ranges of all four contractions back to back, limited only by the shared-memory ring, while the
// dependent work (activation loads, MMAs, reductions) follows behind through the phases.
//
// Per contraction ("phase"):
//   * a CTA's range may cross feature tiles; every (tile, K range) segment accumulates in tensor memory
//     (swapped operands as in gemm_stream.cu: 128 weight rows x 64 K are the 128-row MMA operand, the NP padded
//     activation rows the N operand) and leaves an fp32 partial tile [NP][128] in a workspace;
//   * grid barrier (a counter in global memory; bounded spin);
//   * reduction: the partials of a tile are summed in CTA order (deterministic) and the contraction's epilogue is
//     applied: += into the fp32 residual stream (O, down), silu(gate) * up (gate/up), RoPE + packed q + K/V cache
//     scatter (Q/K/V);
//   * grid barrier; the next phase's activation loads may start.
// RMSNorm is folded in: the reductions of O and down, which produce the final x of a sub-block, also write
// xg = bf16(x * gain) of the norm that follows and per-(row, 32-column chunk) sums of squares; the contraction after
// the norm runs on xg and its reduction scales row r by rsqrt(mean(x_r^2) + eps) (the scale is per row, so it commutes
// with the contraction).
//
// Every wait is bounded (mbarrier waits, grid-barrier spins): on expiry the CTA records SL_DEV_GEMM_TIMEOUT, all
// roles leave, tensor memory is freed.  The grid barrier needs all CTAs resident: the kernel is launched
// cooperatively with one CTA per SM.
#include "tc_common.cuh"

namespace sl {

constexpr int CH_THREADS = 224;          // warp 0 weight producer, 1 activation loader, 2 MMA issue, 3-6 epilogue / reductions
constexpr int CH_BF = 128, CH_BK = 64;
constexpr int CH_W_BYTES = CH_BF * CH_BK * 2;      // 16 KB
constexpr int CH_W_STAGES = 11, CH_X_STAGES = 4;     // at most; with 128 rows (16 KB per activation stage) 10 and 3
__host__ __device__ constexpr int ch_w_stages(int np) { return np <= 64 ? CH_W_STAGES : CH_W_STAGES - 1; }
__host__ __device__ constexpr int ch_x_stages(int np) { return np <= 64 ? CH_X_STAGES : CH_X_STAGES - 1; }
constexpr int CH_MAX_ROWS = 128;         // rows of one pass (the N of the MMA)
constexpr int CH_MAX_SEG = 4;            // (tile, K range) segments of one CTA in one phase
constexpr int CH_MAX_PHASES = 4;
constexpr unsigned long long CH_SPIN_CYCLES = 2000000000ull;   // bound of a grid-barrier wait: ~1 s

enum { CH_O = 0, CH_GATEUP = 1, CH_DOWN = 2, CH_QKV = 3 };

struct ChainPhase {
  int kind, n_tiles, num_kb, w_map0, tiles_per_map, x_map;
  int max_cover;   // bound on the CTAs whose unit ranges meet one tile
};
struct ChainArgs {
  ChainPhase ph[CH_MAX_PHASES];
  int n_phases, np, d, F, hd, dh, n_seq;
  float rms_eps;
  float* x;                    // fp32 residual stream [M][d]
  bf16* xg;                    // [M][d]  bf16(x * gain) of the norm that follows
  bf16* act;                   // [M][F]  SwiGLU output
  const bf16 *gain_ffn, *gain_next;     // gains of the norm after O and after down (nullptr: nothing follows)
  float *ssq_ffn, *ssq_next;   // [rows][d / 32] sums of squares of x per 32-column chunk, written by the O / down reductions
  bf16 *q, *kc, *vc;
  const int32_t* idx;
  const float2* rope;
  float* ws;                   // [grid][CH_MAX_SEG][np][128] partial tiles
  unsigned* bar;               // ONE grid-barrier counter: every barrier of every launch adds `grid` to it, so at a kernel's
                               // start it is a multiple of `grid` (the host zeroes it long before it could wrap)
  const int32_t* n_active;
  int32_t* status;
  int diag_skip;                        // failure-detection diagnostic: this CTA skips its first grid barrier (-1: none)
  float *trace_mid, *trace_out;         // optional copies of x after the O / down reductions
};

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Unit ranges: unit u = tile * num_kb + kb; CTA c owns [c U / G, (c + 1) U / G).  (U * G < 2^31: checked on the host.)
struct ChainRange {
  int begin, end;
};
__device__ __forceinline__ ChainRange chain_range(const ChainPhase& p, int c, int G) {
  const int U = p.n_tiles * p.num_kb;
  return ChainRange{c * U / G, (c + 1) * U / G};
}

// Where a tile's partials lie, looked up instead of derived (the derivation is a dozen integer divisions, which made
// the reductions ALU-bound): per phase and tile, the first CTA whose unit range meets the tile and how many consecutive
// CTAs do (at most CH_MAX_COVER, checked on the host); per phase and CTA, the first tile of its range.  Filled once per
// kernel by all threads.
constexpr int CH_MAX_COVER = 8;
constexpr int CH_TAB_TILES = 512, CH_TAB_CTAS = 160;
struct ChainTables {
  int cover[CH_MAX_PHASES][CH_TAB_TILES];                  // first CTA | count << 16
  short first_tile[CH_MAX_PHASES][CH_TAB_CTAS];
  int2 pos[CH_MAX_ROWS];                                   // per row of the pass: original position, position in its sequence
};
__device__ __forceinline__ void chain_fill_tables(const ChainArgs& a, int G, ChainTables* tb) {
  for (int i = threadIdx.x; i < a.n_phases * CH_TAB_TILES; i += blockDim.x) {
    const int pi = i / CH_TAB_TILES, t = i % CH_TAB_TILES;
    const ChainPhase& p = a.ph[pi];
    if (t >= p.n_tiles) continue;
    const int U = p.n_tiles * p.num_kb, u0 = t * p.num_kb, u1 = u0 + p.num_kb;
    int c0 = u0 * G / U;
    while (c0 > 0 && c0 * U / G > u0) --c0;
    while ((c0 + 1) * U / G <= u0) ++c0;
    int n = 0;
    while (c0 + n < G && (c0 + n) * U / G < u1) ++n;
    tb->cover[pi][t] = c0 | (n << 16);
  }
  for (int i = threadIdx.x; i < a.n_phases * CH_TAB_CTAS; i += blockDim.x) {
    const int pi = i / CH_TAB_CTAS, cc = i % CH_TAB_CTAS;
    const ChainPhase& p = a.ph[pi];
    if (cc < G) tb->first_tile[pi][cc] = (short)((cc * (p.n_tiles * p.num_kb) / G) / p.num_kb);
  }
}

// 32 bytes with one load (L2 only): a thread's eight consecutive features of a partial tile row
struct F8 {
  float v[8];
};
__device__ __forceinline__ F8 ldcg8(const float* p) {
  F8 r;
  asm volatile("ld.global.cg.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
               : "l"(p));
  return r;
}

// Sum of the partial tiles of feature tile t, row r, 8 consecutive features starting at f (inside the tile), in CTA
// order (deterministic); four tiles' loads are issued before the first sum so that the L2 latencies overlap.
__device__ __forceinline__ void sum_partials8(const ChainArgs& a, const int* cover, const short* first_tile, int t, int r,
                                              int f, float* out) {
  const int cv = cover[t], c0 = cv & 0xffff, n = cv >> 16;
#pragma unroll
  for (int j = 0; j < 8; ++j) out[j] = 0.f;
  for (int k0 = 0; k0 < n; k0 += 4) {
    float4 v[4][2];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (k0 + k < n) {
        const int c = c0 + k0 + k, seg = t - first_tile[c];    // which of CTA c's segments this tile is
        const float4* src = reinterpret_cast<const float4*>(a.ws + (unsigned)(((c * CH_MAX_SEG + seg) * a.np + r) * CH_BF + f));
        v[k][0] = __ldcg(src);
        v[k][1] = __ldcg(src + 1);
      }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (k0 + k < n) {
        out[0] += v[k][0].x; out[1] += v[k][0].y; out[2] += v[k][0].z; out[3] += v[k][0].w;
        out[4] += v[k][1].x; out[5] += v[k][1].y; out[6] += v[k][1].z; out[7] += v[k][1].w;
      }
    }
  }
}

// Two such sums at once (same row, two (tile, feature) places): all loads of a round of both are issued before any sum,
// so an item of the gate/up and Q/K/V reductions costs one L2 round trip per two covering CTAs (the usual number there).
__device__ __forceinline__ void sum_partials8x2(const ChainArgs& a, const int* cover, const short* first_tile, int r, int t0,
                                                int f0, int t1, int f1, float* out0, float* out1) {
  const int cv0 = cover[t0], cv1 = cover[t1];
  const int c00 = cv0 & 0xffff, n0 = cv0 >> 16, c10 = cv1 & 0xffff, n1 = cv1 >> 16;
#pragma unroll
  for (int j = 0; j < 8; ++j) out0[j] = out1[j] = 0.f;
  const int nmax = n0 > n1 ? n0 : n1;
  for (int k0 = 0; k0 < nmax; k0 += 2) {
    float4 v[2][2], w[2][2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      if (k0 + k < n0) {
        const int c = c00 + k0 + k, seg = t0 - first_tile[c];
        const float4* src = reinterpret_cast<const float4*>(a.ws + (unsigned)(((c * CH_MAX_SEG + seg) * a.np + r) * CH_BF + f0));
        v[k][0] = __ldcg(src);
        v[k][1] = __ldcg(src + 1);
      }
      if (k0 + k < n1) {
        const int c = c10 + k0 + k, seg = t1 - first_tile[c];
        const float4* src = reinterpret_cast<const float4*>(a.ws + (unsigned)(((c * CH_MAX_SEG + seg) * a.np + r) * CH_BF + f1));
        w[k][0] = __ldcg(src);
        w[k][1] = __ldcg(src + 1);
      }
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      if (k0 + k < n0) {
        out0[0] += v[k][0].x; out0[1] += v[k][0].y; out0[2] += v[k][0].z; out0[3] += v[k][0].w;
        out0[4] += v[k][1].x; out0[5] += v[k][1].y; out0[6] += v[k][1].z; out0[7] += v[k][1].w;
      }
      if (k0 + k < n1) {
        out1[0] += w[k][0].x; out1[1] += w[k][0].y; out1[2] += w[k][0].z; out1[3] += w[k][0].w;
        out1[4] += w[k][1].x; out1[5] += w[k][1].y; out1[6] += w[k][1].z; out1[7] += w[k][1].w;
      }
    }
  }
}

__device__ __forceinline__ uint4 pack8(const float* v) {
  return make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}

// AND of a flag over the 192 threads of named barrier 2 (warps 1-6)
constexpr int CH_RED_THREADS = 192;
__device__ __forceinline__ bool chain_warps_agree(bool ok) {
  int r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 2, 192, q;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"((int)ok) : "memory");
  return r != 0;
}

// rstd of every row from the chunk sums left by the reduction that produced x: s_rstd[r], r < np
__device__ __forceinline__ void row_rstd(const ChainArgs& a, const float* ssq, int e_tid, int M, int row0, float* s_rstd) {
  // four threads per row, each a strided quarter of the chunk sums (fixed order: deterministic)
  const int chunks = a.d >> 5;
  for (int r0 = 0; r0 < a.np; r0 += 32) {
    const int r = r0 + (e_tid >> 2);
    float s = 0.f;
    if (row0 + r < M) {
      const float4* src = reinterpret_cast<const float4*>(ssq + (size_t)(row0 + r) * chunks);
      for (int c = (e_tid & 3); c < (chunks >> 2); c += 32) {          // eight loads in flight
        float4 v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = c + 4 * k < (chunks >> 2) ? __ldcg(src + c + 4 * k) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < 8; ++k) s += (v[k].x + v[k].y) + (v[k].z + v[k].w);
      }
    }
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    if ((e_tid & 3) == 0 && r < a.np) s_rstd[r] = rsqrtf(s / (float)a.d + a.rms_eps);
  }
  asm volatile("bar.sync 1, 128;" ::: "memory");
}

// The reduction + epilogue of one phase, spread over all epilogue threads of the grid.
// Rows: this pass covers packed rows row0 ... row0 + np - 1 (partials and s_rstd are indexed by the row inside the pass).
__device__ __forceinline__ void chain_reduce(const ChainArgs& a, const ChainPhase& p, int G, int c, int r_tid, int M,
                                             int row0, float* s_rstd, const int* cover, const short* first_tile,
                                             const int2* s_pos) {
  const int np = a.np;
  if (p.kind == CH_O || p.kind == CH_DOWN) {
    // x += sum; xg = bf16(x * gain); sums of squares per (row, 32-column chunk).  A CTA takes 32-column chunks, four
    // threads per row.
    const bf16* gain = p.kind == CH_O ? a.gain_ffn : a.gain_next;
    float* ssq = p.kind == CH_O ? a.ssq_ffn : a.ssq_next;
    float* trace = p.kind == CH_O ? a.trace_mid : a.trace_out;
    const int chunks = a.d >> 5;
    for (int ch = c; ch < chunks; ch += G) {
      const int n = ch * 32 + (r_tid & 3) * 8;
      uint4 g4 = make_uint4(0u, 0u, 0u, 0u);
      if (gain) g4 = __ldg(reinterpret_cast<const uint4*>(gain + n));
      for (int r0 = 0; r0 < np; r0 += CH_RED_THREADS / 4) {
        const int r = r0 + (r_tid >> 2);
        float ss = 0.f;
        const int rg = row0 + r;                           // packed row
        if (r < np && rg < M) {
          // the residual row is requested before the partial tiles (independent loads: one round trip, not two)
          float4* xp = reinterpret_cast<float4*>(a.x + (size_t)rg * a.d + n);
          float4 x0 = __ldcg(xp), x1 = __ldcg(xp + 1);
          float s[8];
          sum_partials8(a, cover, first_tile, n >> 7, r, n & 127, s);
          x0.x += s[0]; x0.y += s[1]; x0.z += s[2]; x0.w += s[3];
          x1.x += s[4]; x1.y += s[5]; x1.z += s[6]; x1.w += s[7];
          xp[0] = x0;
          xp[1] = x1;
          if (trace) {
            float4* tp = reinterpret_cast<float4*>(trace + (size_t)rg * a.d + n);
            tp[0] = x0;
            tp[1] = x1;
          }
          const float xv[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
          for (int j = 0; j < 8; ++j) ss += xv[j] * xv[j];
          if (gain) {
            const __nv_bfloat162* gp = reinterpret_cast<const __nv_bfloat162*>(&g4);
            float o[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float2 gf = __bfloat1622float2(gp[j]);
              o[2 * j] = xv[2 * j] * gf.x;
              o[2 * j + 1] = xv[2 * j + 1] * gf.y;
            }
            *reinterpret_cast<uint4*>(a.xg + (size_t)rg * a.d + n) = pack8(o);
          }
        }
        ss += __shfl_xor_sync(0xffffffffu, ss, 1);
        ss += __shfl_xor_sync(0xffffffffu, ss, 2);
        if ((r_tid & 3) == 0 && r < np && rg < M && gain) ssq[(size_t)rg * chunks + ch] = ss;
      }
    }
  } else if (p.kind == CH_GATEUP) {
    // act = silu(rstd * gate) * (rstd * up)
    const int groups = a.F >> 3, half_tiles = p.n_tiles >> 1;
    const int stride = G * CH_RED_THREADS, dr = stride / groups, dg = stride % groups;
    int r = (c * CH_RED_THREADS + r_tid) / groups, fg = (c * CH_RED_THREADS + r_tid) % groups;
    {
      // Software pipeline (a tile is met by at most two CTAs here: checked on the host): the partial tiles of the thread's NEXT item are
      // requested before this item is summed, so the L2 round trips of consecutive items overlap.
      struct Part {
        F8 g[2], u[2];
        int ng, nu;
      };
      auto request = [&](int rr, int f, Part& q) {
        const int tg = f >> 7, tu = half_tiles + tg, cg = cover[tg], cu = cover[tu];
        q.ng = cg >> 16;
        q.nu = cu >> 16;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          if (k < q.ng) {
            const int cc = (cg & 0xffff) + k;
            q.g[k] = ldcg8(a.ws + (unsigned)(((cc * CH_MAX_SEG + (tg - first_tile[cc])) * np + rr) * CH_BF + (f & 127)));
          }
          if (k < q.nu) {
            const int cc = (cu & 0xffff) + k;
            q.u[k] = ldcg8(a.ws + (unsigned)(((cc * CH_MAX_SEG + (tu - first_tile[cc])) * np + rr) * CH_BF + (f & 127)));
          }
        }
      };
      Part cur, nxt;
      bool live = r < np && row0 + r < M;
      if (live) request(r, fg * 8, cur);
      while (live) {
        int r1 = r + dr, fg1 = fg + dg;
        if (fg1 >= groups) {
          fg1 -= groups;
          ++r1;
        }
        const bool live1 = r1 < np && row0 + r1 < M;
        if (live1) request(r1, fg1 * 8, nxt);
        const float rs = s_rstd[r];
        float o[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          float gs = cur.g[0].v[j], us = cur.u[0].v[j];        // CTA order: deterministic
          if (cur.ng > 1) gs += cur.g[1].v[j];
          if (cur.nu > 1) us += cur.u[1].v[j];
          const float gg = gs * rs;
          o[j] = __fdividef(gg, 1.f + __expf(-gg)) * (us * rs);   // silu(g) * u; approximate division (2 ulp)
        }
        *reinterpret_cast<uint4*>(a.act + (size_t)(row0 + r) * a.F + fg * 8) = pack8(o);
        r = r1;
        fg = fg1;
        live = live1;
        cur = nxt;
      }
    }
  } else {
    // Q/K/V: scale by rstd, rotate q and k with the row's ORIGINAL position, q packed, k / v into the cache row
    const int half = a.dh >> 1, per_head = a.dh >> 4;          // 8-feature groups in half a head
    for (int it = c * CH_RED_THREADS + r_tid; it < np * p.n_tiles * 8; it += G * CH_RED_THREADS) {
      const int k = it & 7, t = (it >> 3) % p.n_tiles, r = (it >> 3) / p.n_tiles;
      if (row0 + r >= M) continue;
      const int src = t / p.tiles_per_map;                       // 0 q, 1 k, 2 v
      int f_lo, f_hi;
      if (src == 2) {
        f_lo = 8 * k;
        f_hi = 64 + 8 * k;
      } else {
        f_lo = (k / per_head) * a.dh + (k % per_head) * 8;
        f_hi = f_lo + half;
      }
      // position and rotation factors first: independent of the partial tiles, so one round trip for all
      const int2 ps = s_pos[r];
      float2 cs[8];
      if (src != 2) {
        const float2* tr = a.rope + (size_t)ps.y * half + (f_lo & (a.dh - 1));
#pragma unroll
        for (int j = 0; j < 8; ++j) cs[j] = __ldg(tr + j);
      }
      float lo[8], hi[8];
      sum_partials8x2(a, cover, first_tile, r, t, f_lo, t, f_hi, lo, hi);
      const float rs = s_rstd[r];
      const int ln = (t - src * p.tiles_per_map) * CH_BF;         // first feature of the tile inside its matrix
      bf16* dst = src == 0 ? a.q + (size_t)(row0 + r) * a.hd : (src == 1 ? a.kc : a.vc) + (size_t)ps.x * a.hd;
      float olo[8], ohi[8];
      if (src == 2) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          olo[j] = lo[j] * rs;
          ohi[j] = hi[j] * rs;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float x0 = lo[j] * rs, x1 = hi[j] * rs;
          olo[j] = x0 * cs[j].x - x1 * cs[j].y;
          ohi[j] = x1 * cs[j].x + x0 * cs[j].y;
        }
      }
      *reinterpret_cast<uint4*>(dst + ln + f_lo) = pack8(olo);
      *reinterpret_cast<uint4*>(dst + ln + f_hi) = pack8(ohi);
    }
  }
}

__global__ void __launch_bounds__(CH_THREADS, 1)
gemm_chain_kernel(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
                  const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmW3,
                  const __grid_constant__ CUtensorMap tmW4, const __grid_constant__ CUtensorMap tmW5,
                  const __grid_constant__ CUtensorMap tmW6, const __grid_constant__ CUtensorMap tmX0,
                  const __grid_constant__ CUtensorMap tmX1, const __grid_constant__ CUtensorMap tmX2,
                  const __grid_constant__ ChainArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int np = a.np;
  const int X_BYTES = np * CH_BK * 2;
  const int w_stages = ch_w_stages(np), x_stages = ch_x_stages(np);
  uint8_t* sW = smem;
  uint8_t* sX = sW + w_stages * CH_W_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sX + x_stages * X_BYTES);
  // bars: wfull[W], wempty[W], xfull[X], xempty[X], accfull[2], accempty[2], xready
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * CH_W_STAGES + 2 * CH_X_STAGES + 5);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  float* s_rstd = reinterpret_cast<float*>(s_tmem + 4);                 // [np <= 128]
  ChainTables* tabs = reinterpret_cast<ChainTables*>(reinterpret_cast<uint8_t*>(bars) + 1024);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto wfull = [&](int s) { return bar0 + 8u * s; };
  auto wempty = [&](int s) { return bar0 + 8u * (CH_W_STAGES + s); };
  auto xfull = [&](int s) { return bar0 + 8u * (2 * CH_W_STAGES + s); };
  auto xempty = [&](int s) { return bar0 + 8u * (2 * CH_W_STAGES + CH_X_STAGES + s); };
  const uint32_t accfull0 = bar0 + 8u * (2 * CH_W_STAGES + 2 * CH_X_STAGES), accempty0 = accfull0 + 16u,
                 xready = accfull0 + 32u;
  const int G = (int)gridDim.x, c = (int)blockIdx.x;
  const CUtensorMap* wmaps[7] = {&tmW0, &tmW1, &tmW2, &tmW3, &tmW4, &tmW5, &tmW6};
  const CUtensorMap* xmaps[3] = {&tmX0, &tmX1, &tmX2};

  if (threadIdx.x == 0) {
    for (int s = 0; s < CH_W_STAGES; ++s) {
      mbar_init(wfull(s), 1);
      mbar_init(wempty(s), 1);
    }
    for (int s = 0; s < CH_X_STAGES; ++s) {
      mbar_init(xfull(s), 1);
      mbar_init(xempty(s), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(accfull0 + 8u * i, 1);
      mbar_init(accempty0 + 8u * i, 4);
    }
    mbar_init(xready, 1);
    *s_abort = 0;
    fence_mbar_init();
  }
  chain_fill_tables(a, G, tabs);
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < 2 * np) tmem_cols <<= 1;
  if (warp == 2) tc_alloc(smem_u32(s_tmem), tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  // Rows beyond NP (the host's bound on M was too small) are processed in further passes over the same weights: slow,
  // but every row is computed.  *n_active was written by the compaction at the start of the step.
  const int M = *a.n_active;
  const int n_pass = M > 0 ? (M + np - 1) / np : 0;

  if (warp == 0) {
    // ---- weight producer: walks through the unit ranges of ALL phases; weights depend on nothing
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const int total_pp = n_pass * a.n_phases;
      // the weights are read once: marked evict-first, they do not push the partial tiles and activations out of L2 (the
      // reductions then find them there: step 4-6 % faster)
      const uint64_t w_policy = l2_policy_evict_first();
      for (int pp = 0; pp < total_pp && ok; ++pp) {
        const ChainPhase& p = a.ph[pp % a.n_phases];
        const ChainRange rg = chain_range(p, c, G);
        for (int u = rg.begin; u < rg.end; ++u) {
          const int t = u / p.num_kb, kb = u % p.num_kb;
          if (!(ok = mbar_wait(wempty(stage), phase ^ 1, s_abort))) break;
          mbar_expect_tx(wfull(stage), CH_W_BYTES);
          tma_load_2d_hint(smem_u32(sW + stage * CH_W_BYTES), wmaps[p.w_map0 + t / p.tiles_per_map], kb * CH_BK,
                           (t % p.tiles_per_map) * CH_BF, wfull(stage), w_policy);
          if (++stage == w_stages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else {
    // ---- warps 1-6 walk through the phases together: the activation loader (one thread of warp 1) and the MMA issuer
    // (one thread of warp 2) do their part of a phase, warps 3-6 store the partial tiles and pass the first grid barrier,
    // then ALL SIX warps run the phase's reduction (192 threads: it is bound by dependent L2 round trips per element, so
    // its time falls with the elements per thread), and warps 3-6 pass the second grid barrier.
    const bool is_x = warp == 1, is_mma = warp == 2, is_epi = warp >= 3;
    const int quarter = warp & 3;
    const int f = quarter * 32 + lane;                     // feature inside the tile = tensor-memory lane (warps 3-6)
    const int e_tid = (warp - 3) * 32 + lane;              // warps 3-6: 0..127
    const int r_tid = is_epi ? e_tid : 128 + (warp - 1) * 32 + lane;   // thread of the reduction: 0..191
    griddep_wait();
    bool ok = true;
    int x_stage = 0, ws = 0, xs = 0, mseg = 0, seg = 0;
    uint32_t x_phase = 0, wph = 0, xph = 0;
    const uint32_t idesc = idesc_bf16_m128(np);
    int n_bar = 0;                                         // grid barriers passed so far in this launch
    // The counter's value before this launch: a multiple of the grid size, and no barrier of this launch can complete
    // before every CTA has read it here (each reads before its own first arrival), so what a CTA reads is the base
    // plus fewer than `grid` arrivals.
    unsigned bar_base = 0;
    if (is_epi && e_tid == 0) {
      const unsigned v = ld_acquire_u32(a.bar);
      bar_base = v - v % (unsigned)G;
    }
    auto grid_barrier = [&]() -> bool {                   // warps 3-6 only
      asm volatile("bar.sync 1, 128;" ::: "memory");
      ++n_bar;
      if (e_tid == 0 && c == a.diag_skip && n_bar == 1) {
        // diagnostic: no arrival and no wait, so the other CTAs' bounded wait runs out (and, later, this one's)
      } else if (e_tid == 0) {
        const unsigned target = bar_base + (unsigned)G * (unsigned)n_bar;
        __threadfence();                                  // release: the CTA's stores (ordered before by the bar.sync)
        atomicAdd(a.bar, 1u);
        const unsigned long long t0 = clock64();
        while ((int)(ld_acquire_u32(a.bar) - target) < 0) {
          if (*s_abort || clock64() - t0 > CH_SPIN_CYCLES) {
            *s_abort = 1;
            break;
          }
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      return *s_abort == 0;                               // (the acquire load + bar.sync order the CTA's later loads)
    };
    for (int pp = 0; pp < n_pass * a.n_phases; ++pp) {
      const int pi = pp % a.n_phases;
      const ChainPhase& p = a.ph[pi];
      const int row0 = (pp / a.n_phases) * np;
      const ChainRange rg = chain_range(p, c, G);
      if (is_x) {
        // activation loader: a phase's activations exist once the previous phase's reduction has passed its barrier
        if (lane == 0 && ok) {
          if (pp > 0) ok = mbar_wait(xready, (uint32_t)(pp - 1) & 1, s_abort);
          for (int u = rg.begin; u < rg.end && ok; ++u) {
            const int kb = u % p.num_kb;
            if (!(ok = mbar_wait(xempty(x_stage), x_phase ^ 1, s_abort))) break;
            mbar_expect_tx(xfull(x_stage), (uint32_t)X_BYTES);
            tma_load_2d(smem_u32(sX + x_stage * X_BYTES), xmaps[p.x_map], kb * CH_BK, row0, xfull(x_stage));
            if (++x_stage == x_stages) { x_stage = 0; x_phase ^= 1; }
          }
        }
        __syncwarp();
      } else if (is_mma) {
        if (lane == 0 && ok) {
          int u = rg.begin;
          while (u < rg.end && ok) {
            const int seg_end = min(rg.end, (u / p.num_kb + 1) * p.num_kb);
            const int acc = mseg & 1;
            if (mseg >= 2 && !(ok = mbar_wait(accempty0 + 8u * acc, (uint32_t)((mseg >> 1) - 1) & 1, s_abort))) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(acc * np);
            bool first = true;
            for (; u < seg_end; ++u) {
              if (!(ok = mbar_wait(wfull(ws), wph, s_abort))) break;
              if (!(ok = mbar_wait(xfull(xs), xph, s_abort))) break;
              tc_fence_after();
              const uint64_t wdesc = smem_desc_k_sw128(smem_u32(sW + ws * CH_W_BYTES));
              const uint64_t xdesc = smem_desc_k_sw128(smem_u32(sX + xs * X_BYTES));
#pragma unroll
              for (int k = 0; k < CH_BK / 16; ++k)
                tc_mma_bf16(d_tmem, wdesc + (uint64_t)(2 * k), xdesc + (uint64_t)(2 * k), idesc, (!first) | (k != 0));
              first = false;
              tc_commit(wempty(ws));
              tc_commit(xempty(xs));
              if (++ws == w_stages) { ws = 0; wph ^= 1; }
              if (++xs == x_stages) { xs = 0; xph ^= 1; }
            }
            if (ok) tc_commit(accfull0 + 8u * acc);
            ++mseg;
          }
        }
        __syncwarp();
      } else if (ok) {
        // the row scales this phase's reduction will need: their inputs are complete (the previous phase's second
        // barrier, or the kernel before), and these warps have nothing to do until the first accumulator is full
        if (p.kind == CH_GATEUP) row_rstd(a, a.ssq_ffn, e_tid, M, row0, s_rstd);
        else if (p.kind == CH_QKV) {
          for (int r = e_tid; r < np; r += 128) {          // and the rows' positions (rotary embedding, cache rows)
            const int pos = row0 + r < M ? __ldg(a.idx + row0 + r) : 0;
            tabs->pos[r] = make_int2(pos, pos % a.n_seq);
          }
          row_rstd(a, a.ssq_next, e_tid, M, row0, s_rstd); // (ends with a barrier of these warps)
        }
        int j = 0;
        for (int u = rg.begin; u < rg.end && ok; ++j, ++seg) {
          const int seg_end = min(rg.end, (u / p.num_kb + 1) * p.num_kb);
          const int acc = seg & 1;
          ok = mbar_wait(accfull0 + 8u * acc, (uint32_t)(seg >> 1) & 1, s_abort);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          float* dst = a.ws + ((size_t)c * CH_MAX_SEG + j) * np * CH_BF + f;
          const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * np);
          for (int h = 0; h < np; h += 32) {
            uint32_t v[32];
            tc_ld32(taddr + h, v);
            tc_wait_ld();
#pragma unroll
            for (int r = 0; r < 32; ++r)
              if (h + r < np) __stcg(dst + (size_t)(h + r) * CH_BF, __uint_as_float(v[r]));
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(accempty0 + 8u * acc);
          u = seg_end;
        }
        ok = epilogue_warps_agree(ok);                     // (a warp that gave up must not leave the others at the barrier)
        if (ok) ok = grid_barrier();                       // every partial tile of the phase is in the workspace
      }
      // all six warps: go on together or leave together (a thread that gave up must not strand the others at a barrier)
      if (!chain_warps_agree(ok)) break;
      chain_reduce(a, p, G, c, r_tid, M, row0, s_rstd, tabs->cover[pi], tabs->first_tile[pi], tabs->pos);
      asm volatile("bar.sync 2, 192;" ::: "memory");       // this CTA's share of the reduction is done
      if (is_epi) {
        ok = grid_barrier();                               // the phase's outputs are complete
        if (ok && e_tid == 0) {
          // the next phase's activations were written with ordinary stores (by all CTAs) and are read by bulk tensor copies
          asm volatile("fence.proxy.async.global;" ::: "memory");
          mbar_arrive(xready);
        }
      }
    }
  }

  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *s_abort) set_status(a.status, SL_DEV_GEMM_TIMEOUT);
  if (warp == 2) {
    tc_fence_after();
    tc_dealloc(tmem_base, tmem_cols);
  }
}

// ----------------------------------------------------------------------------------------------- host side
size_t gemm_chain_workspace_bytes(int np_max) { return (size_t)sm_count() * CH_MAX_SEG * np_max * CH_BF * sizeof(float); }

// SL_EUNSUPPORTED when the shapes do not fit (the caller then takes the one-kernel-per-contraction path).
int launch_gemm_chain(const ChainLaunch& L, cudaStream_t st) {
  if (L.m_bound < 1 || L.m_bound > CH_MAX_ROWS || L.max_rows < 1) return SL_EUNSUPPORTED;
  if (L.d % 512 || L.F % 128 || L.hd % 128 || (L.dh != 64 && L.dh != 128)) return SL_EUNSUPPORTED;
  const int np = L.m_bound <= 16 ? 16 : (L.m_bound <= 32 ? 32 : (L.m_bound <= 64 ? 64 : 128));
  const int G = sm_count();
  ChainArgs a = {};
  int n = 0;
  auto add = [&](int kind, int n_tiles, int K, int w0, int tpm, int xm) {
    a.ph[n++] = ChainPhase{kind, n_tiles, K / CH_BK, w0, tpm, xm, 0};
  };
  if (L.wo) {
    add(CH_O, L.d / CH_BF, L.hd, 0, L.d / CH_BF, 0);
    add(CH_GATEUP, 2 * L.F / CH_BF, L.d, 1, L.F / CH_BF, 1);
    add(CH_DOWN, L.d / CH_BF, L.F, 3, L.d / CH_BF, 2);
  }
  if (L.wq) add(CH_QKV, 3 * L.hd / CH_BF, L.d, 4, L.hd / CH_BF, 1);
  if (n == 0) return SL_EINVAL;
  a.n_phases = n;
  for (int i = 0; i < n; ++i) {
    // a CTA's range must not span more than CH_MAX_SEG feature tiles
    const long long U = (long long)a.ph[i].n_tiles * a.ph[i].num_kb;
    if ((U + G - 1) / G > (long long)(CH_MAX_SEG - 1) * a.ph[i].num_kb || U * (G + 1) >= (1ll << 31) || U < G)
      return SL_EUNSUPPORTED;
    a.ph[i].max_cover = (int)(a.ph[i].num_kb / (U / G)) + 2;                       // CTAs that can meet one tile
    if (a.ph[i].max_cover > (a.ph[i].kind == CH_GATEUP ? 2 : CH_MAX_COVER)) return SL_EUNSUPPORTED;
    if (a.ph[i].n_tiles > CH_TAB_TILES || G > CH_TAB_CTAS) return SL_EUNSUPPORTED;   // the lookup tables' extent
  }
  a.np = np; a.d = L.d; a.F = L.F; a.hd = L.hd; a.dh = L.dh; a.n_seq = L.n_seq; a.rms_eps = L.rms_eps;
  a.x = L.x; a.xg = (bf16*)L.xg; a.act = (bf16*)L.act;
  a.gain_ffn = (const bf16*)L.gain_ffn; a.gain_next = (const bf16*)L.gain_next;
  a.ssq_ffn = L.ssq_ffn; a.ssq_next = L.ssq_next;
  a.q = (bf16*)L.q; a.kc = (bf16*)L.kc; a.vc = (bf16*)L.vc; a.idx = L.idx; a.rope = L.rope;
  a.ws = L.ws; a.bar = L.bar; a.n_active = L.n_active; a.status = L.status;
  a.diag_skip = L.diag_skip;
  a.trace_mid = L.trace_mid; a.trace_out = L.trace_out;
  CUtensorMap w[7], x[3];
  const void* wp[7] = {L.wo, L.wg, L.wu, L.wd, L.wq, L.wk, L.wv};
  const int wrows[7] = {L.d, L.F, L.F, L.d, L.hd, L.hd, L.hd}, wk_[7] = {L.hd, L.d, L.d, L.F, L.d, L.d, L.d};
  for (int i = 0; i < 7; ++i) {
    const int src = wp[i] ? i : (L.wo ? 0 : 4);        // unused maps repeat one that is in use
    const int rc = get_tensor_map_2d(wp[src], wrows[src], wk_[src], CH_BF, &w[i]);
    if (rc != SL_OK) return rc;
  }
  int rc = get_tensor_map_2d(L.attn, L.max_rows, L.hd, np, &x[0]);
  if (rc == SL_OK) rc = get_tensor_map_2d(L.xg, L.max_rows, L.d, np, &x[1]);
  if (rc == SL_OK) rc = get_tensor_map_2d(L.act, L.max_rows, L.F, np, &x[2]);
  if (rc != SL_OK) return rc;
  auto smem_for = [](int rows) {
    return ch_w_stages(rows) * CH_W_BYTES + ch_x_stages(rows) * rows * CH_BK * 2 + 1024 + 1024 + (int)sizeof(ChainTables);
  };
  const int smem = smem_for(np);
  static bool attr_set = false;
  if (!attr_set) {
    SL_CUDA_TRY(cudaFuncSetAttribute(gemm_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     smem_for(64) > smem_for(128) ? smem_for(64) : smem_for(128)));
    attr_set = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(G);
  cfg.blockDim = dim3(CH_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeCooperative;          // the grid barrier needs every CTA resident
  at[0].val.cooperative = 1;
  // programmatic dependent launch: the CTAs that find a free SM stream weights while the attention kernel still runs
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  static int with_pdl = -1;                           // -1: not tried yet
  if (with_pdl < 0) with_pdl = pdl_enabled() ? 1 : 0;
  cfg.numAttrs = with_pdl ? 2 : 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, gemm_chain_kernel, w[0], w[1], w[2], w[3], w[4], w[5], w[6], x[0], x[1], x[2], a);
  if (e != cudaSuccess && with_pdl) {                 // the combination of the two attributes is refused: cooperative only
    cudaGetLastError();
    with_pdl = 0;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, gemm_chain_kernel, w[0], w[1], w[2], w[3], w[4], w[5], w[6], x[0], x[1], x[2], a);
  }
  SL_CUDA_TRY(e);
  // the barrier counter only grows: zero it (in stream order, between two launches) long before it could wrap
  if (++*L.bar_base >= (1u << 16)) {
    *L.bar_base = 0;
    SL_CUDA_TRY(cudaMemsetAsync(L.bar, 0, sizeof(unsigned), st));
  }
  return SL_OK;
}

}  // namespace sl
