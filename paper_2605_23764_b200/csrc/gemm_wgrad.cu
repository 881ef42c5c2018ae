// Weight gradients on CTA pairs, strip by strip, with the strip's A operand resident in shared memory.
//
// dW[e] (M x N) = P_e^T . Q_e with K = the expert's rows: at a few hundred rows per expert a 256 x 256
// tile reads 320 KB of operands for 128 KB of output, and the SM <-> L2 traffic, not the MMAs, sets
// its time.  A pair therefore takes a whole strip (its 256 rows of dW across all column tiles) and
// loads the strip's A operand (this CTA's 128 columns of P_e, all K rows) once: when the expert has at
// most A_RES_KB k-blocks it stays in the five 16 KB A slots for every column tile of the strip, and only
// the B operand streams through the stage ring.  Longer experts stream A through the same slots
// stage by stage, as the per-tile kernel does.
//
// Roles per CTA: warp 0 TMA producer of A (and the stage's byte count), warp 6 TMA producer of B,
// warp 1 MMA issuer (even CTA) and TMEM owner, warps 2..5 epilogue.  An A slot is refilled only after
// the MMAs that read its previous content have completed (a_empty, one commit per content).
#include <stdio.h>
#include <stdlib.h>

#include "gemm_pair.cuh"

namespace moe {

constexpr int WG_STAGES = 5;                 // B stage ring and A slots (16 KB each)
constexpr int A_RES_KB = WG_STAGES;          // k-blocks of A that can stay resident
constexpr int WG_OUT_BUFS = 2;
constexpr int WG_THREADS = GEMM_THREADS + 32;

struct __align__(8) WgradBarriers {
  uint64_t full[WG_STAGES];      // used in the even CTA: bytes of both CTAs' loads of the stage
  uint64_t empty[WG_STAGES];     // in each CTA: the B stage's MMAs are complete
  uint64_t a_empty[WG_STAGES];   // in each CTA: every MMA that reads the A slot's content is complete
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  uint32_t pad;
};

constexpr size_t WGRAD_SMEM_BYTES =
    1024 + (size_t)WG_STAGES * STAGE2_BYTES + 4 * WG_OUT_BUFS * OUT_STAGE_BYTES + sizeof(WgradBarriers);
static_assert(WGRAD_SMEM_BYTES <= 227 * 1024, "shared memory budget");

struct Strip {
  int e, m0, row0, nkb, rows;
  bool resident, idle;
};

__device__ __forceinline__ int wgrad_strips(const GemmArgs& a) { return a.Ep * ((a.n_tiles_m + 1) / 2); }

// Strip s of the launch as CTA `rank` sees it: expert-major, so the pairs working at the same time
// share the expert's B operand in L2.
__device__ __forceinline__ Strip decode_strip(const GemmArgs& a, int s, int rank) {
  Strip st;
  const int tm2 = (a.n_tiles_m + 1) / 2;
  st.e = s / tm2;
  const int mp = s - st.e * tm2;
  st.m0 = (2 * mp + rank) * BLOCK_M;
  st.row0 = a.mb_start[st.e] * BLOCK_M;
  st.rows = a.counts[st.e];
  st.nkb = (st.rows + BK - 1) / BK;
  st.resident = st.nkb <= A_RES_KB;
  st.idle = st.m0 >= a.M;   // the strip's second half lies outside dW: nothing to store
  return st;
}

#ifdef MOE_STATS3
__device__ long long g_stats_wg[160][8];
#define SW_DECL long long sw_t = clock64(), sw_acc[4] = {0, 0, 0, 0}
#define SW_LAP(i) do { const long long n_ = clock64(); sw_acc[i] += n_ - sw_t; sw_t = n_; } while (0)
#define SW_FLUSH(base) do { for (int i_ = 0; i_ < 4; ++i_) g_stats_wg[blockIdx.x][(base) + i_] += sw_acc[i_]; } while (0)
#else
#define SW_DECL
#define SW_LAP(i)
#define SW_FLUSH(base)
#endif

__global__ void __launch_bounds__(WG_THREADS, 1) grouped_wgrad_pair_kernel(const __grid_constant__ GemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;                                   // [WG_STAGES][16 KB] A slots
  uint8_t* sB = smem + WG_STAGES * A_STAGE_BYTES;       // [WG_STAGES][16 KB] B stages
  uint8_t* sOut = smem + WG_STAGES * STAGE2_BYTES;
  WgradBarriers* bars = reinterpret_cast<WgradBarriers*>(sOut + 4 * WG_OUT_BUFS * OUT_STAGE_BYTES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const WaitCtl wc{a.status, a.budget_ns};

  if (threadIdx.x == 0) {
    for (int s = 0; s < WG_STAGES; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
      mbar_init(&bars->a_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->tmem_full[s], 1);
      mbar_init(&bars->tmem_empty[s], 8);
    }
    mbar_init(&bars->drain, 1);
    mbar_fence_init();
    fence_proxy_async();
    tma_prefetch_desc(&a.tmA);
    tma_prefetch_desc(&a.tmB);
    tma_prefetch_desc(&a.tmOut0);
  }
  if (warp == 1) {
    tmem_alloc_pair(&bars->tmem_base, TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;
  const int total = wgrad_strips(a);

  if (warp == 0 || warp == 6) {
    // ------------------------------------------------ TMA producers (both CTAs): warp 0 A, warp 6 B
    uint32_t s = 0, ph = 1;
    uint32_t a_ph = (1u << WG_STAGES) - 1;   // per A slot: parity to wait for before the next refill
    bool ok = true;
    SW_DECL;
    for (int sp = pair; sp < total && ok; sp += npairs) {
      const Strip st = decode_strip(a, sp, rank);
      for (int nb = 0; nb < a.n_tiles_n && ok; ++nb) {
        const bool load_a = !st.resident || nb == 0;
        for (int kb = 0; kb < st.nkb; ++kb) {
          const int slot = st.resident ? kb : (int)s;
          int go = 1;
          SW_LAP(1);
          if (lane == 0) {
            go = mbar_wait(&bars->empty[s], ph, wc, SITE_EMPTY, sp, 50) ? 1 : 0;
            if (go && warp == 0 && load_a) go = mbar_wait(&bars->a_empty[slot], (a_ph >> slot) & 1, wc, SITE_EMPTY, sp, 50) ? 1 : 0;
          }
          go = __shfl_sync(0xffffffffu, go, 0);
          SW_LAP(0);
          if (!go) { ok = false; break; }
          const int k0 = kb * BK;
          if (warp == 0) {
            if (lane == 0 && rank == 0)
              mbar_expect_tx(&bars->full[s], 2 * (HALF_B_BYTES + (load_a ? A_STAGE_BYTES : 0)));
            __syncwarp();
            if (load_a && lane < 2)
              tma_load_2d_pair(sA + slot * A_STAGE_BYTES + lane * MN_BOX_BYTES, &a.tmA, st.m0 + lane * 64, st.row0 + k0,
                               &bars->full[s]);
          } else if (lane < 2) {
            tma_load_2d_pair(sB + s * HALF_B_BYTES + lane * MN_BOX_BYTES, &a.tmB, nb * BN + (2 * rank + lane) * 64,
                             st.row0 + k0, &bars->full[s]);
          }
          if (load_a) a_ph ^= 1u << slot;
          if (++s == WG_STAGES) { s = 0; ph ^= 1; }
        }
      }
    }
    SW_LAP(1);
    if (lane == 0 && warp == 6) SW_FLUSH(4);   // [4] B producer: wait for a free stage, [5] issue
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer (even CTA only)
    if (lane == 0 && rank == 0) {
      uint32_t s = 0, ph = 0, acc_it = 0;
      bool ok = true;
      SW_DECL;
      for (int sp = pair; sp < total && ok; sp += npairs) {
        const Strip st = decode_strip(a, sp, 0);
        if (st.nkb == 0) continue;
        for (int nb = 0; nb < a.n_tiles_n && ok; ++nb) {
          const int as = acc_it & 1;
          SW_LAP(2);
          if (!mbar_wait(&bars->tmem_empty[as], ((acc_it >> 1) & 1) ^ 1, wc, SITE_TMEM_EMPTY, sp)) { ok = false; break; }
          SW_LAP(0);
          tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + as * BN;
          const bool last_use = !st.resident || nb == a.n_tiles_n - 1;
          for (int kb = 0; kb < st.nkb; ++kb) {
            SW_LAP(2);
            if (!mbar_wait(&bars->full[s], ph, wc, SITE_FULL, sp)) { ok = false; break; }
            SW_LAP(1);
            tc_fence_after_sync();
            const int slot = st.resident ? kb : (int)s;
            mma_kblock_pair<GEMM_WGRAD>(d_tmem, smem_u32(sA + slot * A_STAGE_BYTES), smem_u32(sB + s * HALF_B_BYTES),
                                        kb == 0, k16_steps_of(st.rows, kb));
            tc_commit_pair(&bars->empty[s]);
            if (last_use) tc_commit_pair(&bars->a_empty[slot]);
            if (++s == WG_STAGES) { s = 0; ph ^= 1; }
          }
          if (!ok) break;
          tc_commit_pair(&bars->tmem_full[as]);
          ++acc_it;
        }
      }
      SW_LAP(2);
      SW_FLUSH(0);   // [0] wait tmem_empty, [1] wait operands, [2] issue
      if (!ok || *reinterpret_cast<volatile int*>(&a.status->abort)) {
        tc_commit_pair(&bars->drain);
        const WaitCtl shortwc{a.status, 20ull * 1000 * 1000};
        mbar_wait(&bars->drain, 0, shortwc, SITE_DRAIN, 0);
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------ epilogue warps (both CTAs, own rows)
    const int quad = warp & 3;
    Staging stg{sOut + quad * WG_OUT_BUFS * OUT_STAGE_BYTES, WG_OUT_BUFS, 0};
    uint32_t acc_it = 0;
    bool ok = true;
    for (int sp = pair; sp < total && ok; sp += npairs) {
      const Strip st = decode_strip(a, sp, rank);
      Tile tl;
      tl.e = st.e; tl.row0 = st.row0; tl.m0 = st.m0; tl.nkb = st.nkb;
      for (int nb = 0; nb < a.n_tiles_n; ++nb) {
        tl.nb = nb; tl.n0 = nb * BN;
        if (st.nkb == 0) {
          if (!st.idle) epilogue_tile<GEMM_WGRAD>(a, tl, 0, quad, lane, stg);  // an expert without rows: zeros
          continue;
        }
        const int as = acc_it & 1;
        if (!mbar_wait(&bars->tmem_full[as], (acc_it >> 1) & 1, wc, SITE_TMEM_FULL, sp, 200)) { ok = false; break; }
        tc_fence_after_sync();
        if (!st.idle) epilogue_tile<GEMM_WGRAD>(a, tl, tmem_base + as * BN, quad, lane, stg);
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_leader(&bars->tmem_empty[as]);
        ++acc_it;
      }
    }
    if (lane == 0) tma_store_wait_all();
  }

  // ---------------------------------------------------------------- teardown
  if (*reinterpret_cast<volatile int*>(&a.status->abort)) __nanosleep(200000);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

cudaError_t launch_wgrad_strips(const GemmArgs& a, int num_sms, cudaStream_t s, int* launches) {
  ++*launches;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(grouped_wgrad_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)WGRAD_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  static int max_pairs = 0;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3((num_sms / 2) * 2);
  cfg.blockDim = dim3(WG_THREADS);
  cfg.dynamicSmemBytes = WGRAD_SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (max_pairs == 0) {
    int n = 0;
    cudaError_t e = cudaOccupancyMaxActiveClusters(&n, grouped_wgrad_pair_kernel, &cfg);
    if (e != cudaSuccess) return e;
    max_pairs = n > 0 ? n : 1;
  }
  if (2 * max_pairs < (int)cfg.gridDim.x) cfg.gridDim = dim3(2 * max_pairs);
  return cudaLaunchKernelEx(&cfg, grouped_wgrad_pair_kernel, a);
}

#ifdef MOE_STATS3
extern "C" int moe_debug_stats_wg(long long* host, int reset) {
  if (reset) { static long long z[160][8]; return (int)cudaMemcpyToSymbol(g_stats_wg, z, sizeof z); }
  return (int)cudaMemcpyFromSymbol(host, g_stats_wg, sizeof(long long) * 160 * 8);
}
#endif

}  // namespace moe
