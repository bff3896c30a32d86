// Weight-streaming GEMM for FEW active rows (M <= 128) on sm_100a: C[r][n] = sum_k X[r][k] W[n][k], bf16 in, fp32
// accumulate; the same contractions as gemm_tc.cu (Algorithm 1 lines 10, 12, 15) in the regime where a step is bound
// by reading the weights once from HBM, not by the tensor pipe (few unlocked rows: the regime in which the paper's own
// implementation gains nothing, App. "Algorithmic Characteristics on Runtime").
//
// Operands are swapped with respect to gemm_tc.cu: a tile of 128 weight rows (output features) x 64 K is the 128-row
// operand of tcgen05.mma, the packed activation rows (padded to NP = 16, 32, 64 or 128) are its N operand, so a K block
// costs NP/256 of the tensor cycles of a 128 x 256 tile and a pipeline stage holds almost only weight bytes.  The
// accumulator in tensor memory is [128 features (lanes)] x [NP rows (columns)].
//
// Work decomposition: one CTA per (feature tile, K split).  The S (1, 2, 4 or 8) K splits of a tile form a thread-block
// CLUSTER and reduce their partial accumulators through distributed shared memory: every CTA sends rows
// [j * 32/S, (j+1) * 32/S) of each 32-row chunk to CTA j of the cluster (plain st.shared::cluster stores, no multicast),
// CTA j adds the S contributions in split order (deterministic) and runs the fused epilogue for its rows.  No global
// workspace, no tickets.  CTAs are small (about 100 KB of shared memory, at most 256 tensor-memory columns when
// NP <= 64), so two fit on an SM: a CTA's set-up and its reduction overlap the other CTA's streaming, and, because
// the kernel lets its successor launch at once (programmatic dependent launch) and touches the activations only after
// griddepcontrol.wait, the next kernel's CTAs move in and start streaming THEIR weights while this kernel drains.
//
// NP and S are chosen by the host from an upper bound of M (the row count itself lives in device memory).  The kernel
// is correct for any M: rows beyond NP are processed in further passes over the same weights (slow, never taken when
// the bound holds).  Every wait is bounded; on expiry the CTA records SL_DEV_GEMM_TIMEOUT, all roles leave their
// loops, the cluster meets once more so that nobody touches a CTA that has left, tensor memory is freed.
#include "tc_common.cuh"

namespace sl {

constexpr int WS_THREADS = 192;          // warp 0 TMA producer, warp 1 MMA issue, warps 2-5 reduction + epilogue
constexpr int WS_BF = 128;               // output features per tile (rows of the weight operand)
constexpr int WS_BK = 64;                // K elements per stage: one 128-byte swizzle row
constexpr int WS_W_BYTES = WS_BF * WS_BK * 2;     // 16 KB
constexpr int WS_EPI_QKV = 3;

struct WsQkv {
  bf16 *q, *kc, *vc;          // q packed [M][hd]; caches [B*N][hd]
  const int32_t* idx;         // [M] flat position of each packed row
  const float2* rope;         // [n_seq][dh/2] (cos, sin)
  int n_seq, hd, dh;
};

__device__ __forceinline__ bool mbar_try_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// bounded wait on a barrier that CTAs of the cluster arrive on (acquire at cluster scope: their remote stores are visible)
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_cluster(bar, parity)) return true;
  const unsigned long long t0 = clock64();
  unsigned spins = 0;
  while (!mbar_try_cluster(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > TC_WAIT_CYCLES) {
        *abort_flag = 1;
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t cluster_addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}
// 16 consecutive fp32 columns of this thread's tensor-memory lane
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

// Shared-memory layout (offsets from the 1024-byte aligned base), the same on host and device.
struct WsLayout {
  int stage_bytes, stages, red_off, red_bytes, bar_off, total;
};
__host__ __device__ inline WsLayout ws_layout(int nacc, int np, int stages, int S) {
  WsLayout l;
  l.stage_bytes = nacc * WS_W_BYTES + np * WS_BK * 2;
  l.stages = stages;
  l.red_off = stages * l.stage_bytes;
  const int cr = np < 32 ? np : 32;
  const int rpo = (cr + S - 1) / S;             // rows of a chunk one CTA finishes (the last CTAs may have fewer)
  l.red_bytes = nacc * S * rpo * WS_BF * 4;     // [nacc][S][rpo][128] floats
  l.bar_off = l.red_off + l.red_bytes;
  l.total = l.bar_off + 512;
  return l;
}

template <int EPI>
__global__ void __launch_bounds__(WS_THREADS, 1)
gemm_stream_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW0,
                   const __grid_constant__ CUtensorMap tmW1, const __grid_constant__ CUtensorMap tmW2,
                   void* __restrict__ Cv, const int32_t* __restrict__ n_active, int n_out, int K, int32_t* status,
                   const WsQkv qkv, int np, int S, int stages, int prefetch_w) {
  constexpr int NACC = EPI == EPI_SWIGLU ? 2 : 1;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const WsLayout L = ws_layout(NACC, np, stages, S);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L.bar_off);
  // bars: full[stages], empty[stages], acc_full, acc_empty, red_full, red_free
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * stages + 4);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (stages + s); };
  const uint32_t accf_bar = bar0 + 8u * (2 * stages), acce_bar = accf_bar + 8u, redf_bar = accf_bar + 16u,
                 rede_bar = accf_bar + 24u;

  // Inside a step neither the weights nor *n_active were written by the kernel launched just before this one
  // (prefetch_w): the weight copies start before the predecessor has completed, and the successor may launch as soon
  // as every CTA of this kernel has its tensor memory.  Otherwise nothing is read before the predecessor has completed.
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW0) : "memory");
    if (EPI == EPI_SWIGLU || EPI == WS_EPI_QKV) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW1) : "memory");
    if (EPI == WS_EPI_QKV) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW2) : "memory");
  }
  if (!prefetch_w) griddep_wait();

  const uint32_t rank = S > 1 ? cluster_ctarank() : 0u;
  const int tile = (int)blockIdx.x / S;
  const int n0 = tile * WS_BF;
  const int num_kb = (K + WS_BK - 1) / WS_BK;
  const int kb0 = (int)rank * num_kb / S, kb1 = ((int)rank + 1) * num_kb / S;
  const int cr = np < 32 ? np : 32;             // rows per reduction chunk
  const int rpo = (cr + S - 1) / S;             // rows of a chunk a CTA finishes: CTA j rows [j * rpo, min(cr, (j + 1) * rpo))
  const int n_chunks = np / cr;
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < NACC * np) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(accf_bar, 1);
    mbar_init(acce_bar, 4);
    mbar_init(redf_bar, 4 * S);                 // one arrival per epilogue warp of every CTA of the cluster
    mbar_init(rede_bar, 4 * S);
    *s_abort = 0;
    fence_mbar_init();
  }
  __syncthreads();
  // the peers' barriers must exist before anything arrives on them: every thread arrives here, and the epilogue warps
  // wait just before their first access to a peer, by which time the phase has long completed
  if (S > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");

  const int M = *n_active;
  const int n_pass = M > 0 ? (M + np - 1) / np : 0;     // 1 when the host's bound on M holds
  uint32_t tmem_base = 0;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      auto load_w = [&](int st, int kb) {
        const uint32_t sw = smem_u32(smem + st * L.stage_bytes);
        if (EPI == EPI_SWIGLU) {
          tma_load_2d(sw, &tmW0, kb * WS_BK, n0, full_bar(st));
          tma_load_2d(sw + WS_W_BYTES, &tmW1, kb * WS_BK, n0, full_bar(st));
        } else if (EPI == WS_EPI_QKV) {
          const int src = n0 / qkv.hd;
          tma_load_2d(sw, src == 0 ? &tmW0 : (src == 1 ? &tmW1 : &tmW2), kb * WS_BK, n0 - src * qkv.hd, full_bar(st));
        } else {
          tma_load_2d(sw, &tmW0, kb * WS_BK, n0, full_bar(st));
        }
      };
      const uint32_t stage_tx = (uint32_t)L.stage_bytes;
      bool waited = !prefetch_w;
      for (int p = 0; p < n_pass && ok; ++p) {
        int kb = kb0;
        if (!waited) {
          // the weight parts of the first stages go out now, the activation parts once the predecessor has completed
          const int npre = kb1 - kb0 < stages ? kb1 - kb0 : stages;
          for (int i = 0; i < npre; ++i) {
            mbar_expect_tx(full_bar(i), stage_tx);
            load_w(i, kb0 + i);
          }
          griddep_wait();
          waited = true;
          for (int i = 0; i < npre; ++i)
            tma_load_2d(smem_u32(smem + i * L.stage_bytes) + NACC * WS_W_BYTES, &tmX, (kb0 + i) * WS_BK, 0, full_bar(i));
          stage = npre;
          if (stage == stages) { stage = 0; phase ^= 1; }
          kb = kb0 + npre;
        }
        for (; kb < kb1; ++kb) {
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1, s_abort))) break;
          mbar_expect_tx(full_bar(stage), stage_tx);
          load_w(stage, kb);
          tma_load_2d(smem_u32(smem + stage * L.stage_bytes) + NACC * WS_W_BYTES, &tmX, kb * WS_BK, p * np, full_bar(stage));
          if (++stage == stages) { stage = 0; phase ^= 1; }
        }
      }
      if (!waited) griddep_wait();
    } else if (prefetch_w) {
      griddep_wait();
    }
  } else if (warp == 1) {
    tc_alloc(smem_u32(s_tmem), tmem_cols);
    // The successor may launch only now that this CTA holds its tensor memory: a successor CTA that shares the SM can
    // then never take the columns this CTA still has to ask for (it would keep them until this kernel completes, and
    // this kernel could not complete).
    griddep_launch();
    tc_fence_before();
    asm volatile("bar.sync 2, 160;" ::: "memory");      // publishes the tensor-memory address to the epilogue warps
    tc_fence_after();
    tmem_base = *s_tmem;
    if (prefetch_w) griddep_wait();
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_m128(np);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int p = 0; p < n_pass && ok; ++p) {
        if (p > 0) {
          if (!(ok = mbar_wait(acce_bar, (uint32_t)(p - 1) & 1, s_abort))) break;
          tc_fence_after();
        }
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!(ok = mbar_wait(full_bar(stage), phase, s_abort))) break;
          tc_fence_after();
          const uint32_t sw = smem_u32(smem + stage * L.stage_bytes), sx = sw + NACC * WS_W_BYTES;
          const uint64_t xdesc = smem_desc_k_sw128(sx);
#pragma unroll
          for (int a = 0; a < NACC; ++a) {
            const uint64_t wdesc = smem_desc_k_sw128(sw + a * WS_W_BYTES);
#pragma unroll
            for (int k = 0; k < WS_BK / 16; ++k)
              tc_mma_bf16(tmem_base + (uint32_t)(a * np), wdesc + (uint64_t)(2 * k), xdesc + (uint64_t)(2 * k), idesc,
                          (kb > kb0) | (k != 0));
          }
          tc_commit(empty_bar(stage));
          if (++stage == stages) { stage = 0; phase ^= 1; }
        }
        if (ok) tc_commit(accf_bar);
      }
    }
  } else {
    asm volatile("bar.sync 2, 160;" ::: "memory");
    tc_fence_after();
    tmem_base = *s_tmem;
    if (prefetch_w) griddep_wait();
    const int quarter = warp & 3;                        // tensor-memory lanes 32 * quarter ... + 31
    const int f = quarter * 32 + lane;                   // feature inside the tile = tensor-memory lane
    float* red = reinterpret_cast<float*>(smem + L.red_off);
    const uint32_t red_u32 = smem_u32(red);
    bool ok = true;
    int ci = 0;                                          // chunks reduced so far (barrier phases)
    if (S > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    for (int p = 0; p < n_pass && ok; ++p) {
      ok = mbar_wait(accf_bar, (uint32_t)p & 1, s_abort);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      for (int c = 0; c < n_chunks && ok; ++c, ++ci) {
        // ---- this CTA's partial sums of chunk c go to their owners: rows [j * rpo, (j + 1) * rpo) to CTA j
        if (ci > 0 && S > 1) {                            // every owner has read the previous chunk out of its buffer
          ok = mbar_wait_cluster(rede_bar, (uint32_t)(ci - 1) & 1, s_abort);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        } else if (ci > 0) {
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
#pragma unroll
        for (int a = 0; a < NACC; ++a) {
          const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * np + c * cr);
          for (int h = 0; h < cr; h += 16) {
            uint32_t v[16];
            tc_ld16(taddr + h, v);
            tc_wait_ld();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int r = h + j, owner = r / rpo, rl = r - owner * rpo;   // owner < S because rpo = ceil(cr / S)
              const uint32_t off = (uint32_t)((((a * S + (int)rank) * rpo + rl) * WS_BF + f) * 4);
              if (S > 1) st_cluster_f32(mapa_u32(red_u32 + off, (uint32_t)owner), __uint_as_float(v[j]));
              else red[off >> 2] = __uint_as_float(v[j]);
            }
          }
        }
        if (c == n_chunks - 1) {                          // the accumulator has been read: the next pass may overwrite it
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(acce_bar);
        }
        if (S > 1) {
          __syncwarp();
          if (lane == 0)
            for (int j = 0; j < S; ++j) mbar_arrive_cluster(mapa_u32(redf_bar, (uint32_t)j));
          ok = mbar_wait_cluster(redf_bar, (uint32_t)ci & 1, s_abort);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        } else {
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        // ---- finish this CTA's rows of the chunk: sum the S contributions in split order, fused epilogue
        const int my_rows = min(rpo, cr - (int)rank * rpo);          // <= 0 for a CTA that owns no row of the chunk
        for (int rl = 0; rl < my_rows; ++rl) {
          const int row = p * np + c * cr + (int)rank * rpo + rl;
          float acc[NACC];
#pragma unroll
          for (int a = 0; a < NACC; ++a) {
            acc[a] = 0.f;
            for (int s = 0; s < S; ++s) acc[a] += red[((a * S + s) * rpo + rl) * WS_BF + f];
          }
          const int n = n0 + f;
          if (EPI == WS_EPI_QKV) {
            const int src = n0 / qkv.hd, ln = n - src * qkv.hd;
            const bool live = row < M;
            const int pos = live ? __ldg(qkv.idx + row) : 0;
            if (src == 2) {
              if (live) qkv.vc[(long long)pos * qkv.hd + ln] = __float2bfloat16_rn(acc[0]);
            } else {
              // rotary embedding: the partner of feature j of a head is j +- dh/2, a lane of another warp: exchange
              // the sums through this thread's own slot of the buffer
              const int half = qkv.dh >> 1, j = f % qkv.dh;
              const bool lo = j < half;
              float2 cs = make_float2(1.f, 0.f);
              if (live) cs = __ldg(qkv.rope + (long long)(pos % qkv.n_seq) * half + (lo ? j : j - half));
              red[rl * WS_BF + f] = acc[0];
              asm volatile("bar.sync 1, 128;" ::: "memory");
              const float other = red[rl * WS_BF + (lo ? f + half : f - half)];
              if (live) {
                const float o = lo ? acc[0] * cs.x - other * cs.y : acc[0] * cs.x + other * cs.y;
                bf16* dst = src == 0 ? qkv.q + (long long)row * qkv.hd : qkv.kc + (long long)pos * qkv.hd;
                dst[ln] = __float2bfloat16_rn(o);
              }
            }
          } else if (row < M && n < n_out) {
            if (EPI == EPI_RESIDUAL) {
              // one add per element and launch, performed by the L2 (no load of x, so no latency chain): deterministic
              atomicAdd(reinterpret_cast<float*>(Cv) + (long long)row * n_out + n, acc[0]);
            } else if (EPI == EPI_SWIGLU) {
              const float g = acc[0];
              reinterpret_cast<bf16*>(Cv)[(long long)row * n_out + n] = __float2bfloat16_rn(g / (1.f + __expf(-g)) * acc[NACC - 1]);
            } else {
              reinterpret_cast<bf16*>(Cv)[(long long)row * n_out + n] = __float2bfloat16_rn(acc[0]);
            }
          }
        }
        // ---- this CTA's buffer may be overwritten with the next chunk
        const bool more = c + 1 < n_chunks || p + 1 < n_pass;
        if (more && S > 1) {
          __syncwarp();
          if (lane == 0)
            for (int j = 0; j < S; ++j) mbar_arrive_cluster(mapa_u32(rede_bar, (uint32_t)j));
        }
      }
    }
  }

  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *s_abort) set_status(status, SL_DEV_GEMM_TIMEOUT);
  // nobody leaves while a peer may still write into its buffer or arrive on its barriers
  if (S > 1) {
    if (warp < 2) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");   // completes the opening phase
    cluster_sync_all();
  }
  if (warp == 1) {                              // the epilogue warps have read the accumulators
    tc_fence_after();
    tc_dealloc(tmem_base, tmem_cols);
  }
}

// ----------------------------------------------------------------------------------------------- host side
struct WsPlan {
  int np, S, stages, smem;
};

// np from the bound on M; S: the most K splits (cluster size, at most 8) that keep at least 8 K blocks per CTA and no
// more than ~2.6 CTAs per SM in the launch; stages: what fits in 112 KB (two CTAs per SM) when np <= 64, else 220 KB.
static WsPlan ws_plan(int epi, int m_bound, int n_out, int K) {
  WsPlan p;
  p.np = m_bound <= 16 ? 16 : (m_bound <= 32 ? 32 : (m_bound <= 64 ? 64 : 128));
  const int nacc = epi == EPI_SWIGLU ? 2 : 1;
  const int tiles = (n_out + WS_BF - 1) / WS_BF, num_kb = (K + WS_BK - 1) / WS_BK;
  // K splits (cluster size): the power of two that brings the launch closest to two CTAs per SM without exceeding the
  // CTAs that can be resident at once (a second wave of clusters costs more than idle SMs), at least four K blocks
  // per CTA.  Measured on B200 at 32 rows: 96 feature tiles (Q/K/V, gate/up) S = 2, 32 tiles (output, down) S = 4 or 8.
  p.S = 1;
  while (p.S < 8 && tiles * p.S * 2 <= 2 * sm_count() && num_kb / (p.S * 2) >= 4) p.S *= 2;
  const WsLayout one = ws_layout(nacc, p.np, 1, p.S);
  const int small_kb = 112;
  int st = p.np <= 64 ? (small_kb * 1024 - one.red_bytes - 512 - 1024) / one.stage_bytes : 0;
  if (st < 2) st = (220 * 1024 - one.red_bytes - 512 - 1024) / one.stage_bytes;      // one CTA per SM
  st = st > 12 ? 12 : st;
  const int need = (num_kb + p.S - 1) / p.S;
  if (st > need) st = need < 2 ? 2 : need;
  p.stages = st;
  p.smem = ws_layout(nacc, p.np, st, p.S).total + 1024;
  return p;
}

template <int EPI>
static int launch_ws(const CUtensorMap& x, const CUtensorMap* w, void* C, const int32_t* n_active, int n_out, int K,
                     int32_t* status, const WsQkv& qkv, const WsPlan& p, bool prefetch_w, cudaStream_t st) {
  static int attr_smem = 0;
  if (p.smem > attr_smem) {
    SL_CUDA_TRY(cudaFuncSetAttribute(gemm_stream_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, p.smem));
    attr_smem = p.smem;
  }
  const int tiles = (n_out + WS_BF - 1) / WS_BF;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tiles * p.S);
  cfg.blockDim = dim3(WS_THREADS);
  cfg.dynamicSmemBytes = p.smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (p.S > 1) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = p.S;
    at[na].val.clusterDim.y = 1;
    at[na].val.clusterDim.z = 1;
    ++na;
  }
  if (pdl_enabled()) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = at;
  cfg.numAttrs = na;
  SL_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_stream_kernel<EPI>, x, w[0], w[1], w[2], C, n_active, n_out, K, status, qkv,
                                 p.np, p.S, p.stages, prefetch_w ? 1 : 0));
  return SL_OK;
}

// Weight-streaming launch for a row bound m_bound <= 128.  SL_EUNSUPPORTED when the shape does not fit (the caller then
// takes the general kernel).
int launch_gemm_stream(const void* A, const void* W, const void* W2, void* C, const int32_t* n_active, int max_rows,
                       int m_bound, int n_out, int K, int epilogue, int32_t* status, bool prefetch_w, cudaStream_t st) {
  if (m_bound < 1 || m_bound > 128 || max_rows < 1 || K % 8 || n_out % 8) return SL_EUNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(W2) |
       reinterpret_cast<uintptr_t>(C)) & 15)
    return SL_EUNSUPPORTED;
  if (epilogue == EPI_SWIGLU && !W2) return SL_EINVAL;
  const WsPlan p = ws_plan(epilogue, m_bound, n_out, K);
  CUtensorMap x, w[3];
  int rc = get_tensor_map_2d(A, max_rows, K, p.np, &x);
  if (rc == SL_OK) rc = get_tensor_map_2d(W, n_out, K, WS_BF, &w[0]);
  if (rc != SL_OK) return rc;
  w[1] = w[2] = w[0];
  if (W2 && (rc = get_tensor_map_2d(W2, n_out, K, WS_BF, &w[1])) != SL_OK) return rc;
  const WsQkv none{};
  switch (epilogue) {
    case EPI_STORE: return launch_ws<EPI_STORE>(x, w, C, n_active, n_out, K, status, none, p, prefetch_w, st);
    case EPI_RESIDUAL: return launch_ws<EPI_RESIDUAL>(x, w, C, n_active, n_out, K, status, none, p, prefetch_w, st);
    case EPI_SWIGLU: return launch_ws<EPI_SWIGLU>(x, w, C, n_active, n_out, K, status, none, p, prefetch_w, st);
    default: return SL_EINVAL;
  }
}

// Q/K/V projections in one launch with the rotary embedding and the cache scatter in the epilogue (Algorithm 1 lines
// 10-11), for a row bound m_bound <= 128.
int launch_gemm_stream_qkv(const void* A, const void* Wq, const void* Wk, const void* Wv, void* q_out, void* k_cache,
                           void* v_cache, const int32_t* idx, const float2* rope, const int32_t* n_active, int max_rows,
                           int m_bound, int n_seq, int hd, int dh, int K, int32_t* status, bool prefetch_w,
                           cudaStream_t st) {
  if (m_bound < 1 || m_bound > 128 || max_rows < 1 || K % 8 || hd % WS_BF || (dh != 64 && dh != 128)) return SL_EUNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(Wq) | reinterpret_cast<uintptr_t>(Wk) |
       reinterpret_cast<uintptr_t>(Wv) | reinterpret_cast<uintptr_t>(q_out) | reinterpret_cast<uintptr_t>(k_cache) |
       reinterpret_cast<uintptr_t>(v_cache)) & 15)
    return SL_EUNSUPPORTED;
  const WsPlan p = ws_plan(WS_EPI_QKV, m_bound, 3 * hd, K);
  CUtensorMap x, w[3];
  const void* W[3] = {Wq, Wk, Wv};
  int rc = get_tensor_map_2d(A, max_rows, K, p.np, &x);
  for (int i = 0; i < 3 && rc == SL_OK; ++i) rc = get_tensor_map_2d(W[i], hd, K, WS_BF, &w[i]);
  if (rc != SL_OK) return rc;
  const WsQkv qa{(bf16*)q_out, (bf16*)k_cache, (bf16*)v_cache, idx, rope, n_seq, hd, dh};
  return launch_ws<WS_EPI_QKV>(x, w, nullptr, n_active, 3 * hd, K, status, qa, p, prefetch_w, st);
}

}  // namespace sl
