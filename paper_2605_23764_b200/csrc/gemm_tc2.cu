// Row-space grouped GEMMs on CTA pairs (tcgen05 cta_group::2) with token-row tiles, one launch per operator:
// the path of shapes whose intermediate size is not a multiple of 16 (the token-column tiles of gemm_tc3.cu
// need F % 16 == 0).
//
// A 128 x 256 tile on one SM asks shared memory for its operands once per MMA (96 B/clk) while
// TMA refills the same stages (another 96 B/clk): the 128 B/clk of one SM's shared memory caps the
// tensor core near two thirds of its rate.  Pairing two SMs on a 256 x 256 tile halves the B traffic
// of each: a CTA holds its own 128 rows of A, half of the B tile (16 KB + 16 KB per 64-deep k-block,
// six stages in flight) and the 128 x 256 accumulator slice of its rows; the even CTA issues the MMAs
// for both, the tensor cores exchange the B halves over the cluster's shared-memory network.
//
// A pair works on two M-blocks of the same expert (same weights) and the same column tile; an expert
// with an odd number of M-blocks leaves the odd CTA of its last pair idle (its rows read as zeros and
// are not stored).  For the weight gradients the pair splits 256 rows of dW.
// Per CTA the roles are those of the single-CTA kernel: warp 0 TMA producer, warp 1 MMA issuer (even
// CTA only) and TMEM owner, warps 2..5 epilogue.  Every barrier the MMA issuer waits on lives in the
// even CTA; the odd CTA's loads and epilogue warps signal it there.
#include <stdio.h>
#include <stdlib.h>

#include "gemm_pair.cuh"
#include "launch_pairs.cuh"

namespace moe {

constexpr int STAGES2 = 5;                                       // 5 x 32 KB operand stages ...
constexpr int OUT_BUFS2 = 2;                                     // ... and double-buffered epilogue staging

struct __align__(8) PairBarriers {
  uint64_t full[STAGES2];     // used in the even CTA: bytes of both CTAs' loads
  uint64_t empty[STAGES2];    // in each CTA: the stage's MMAs are complete
  uint64_t tmem_full[2];      // in each CTA: accumulator ready
  uint64_t tmem_empty[2];     // used in the even CTA: 8 epilogue warps of the pair have drained it
  uint64_t drain;
  uint32_t tmem_base;
  uint32_t pad;
};

constexpr size_t GEMM2_SMEM_BYTES =
    1024 + (size_t)STAGES2 * STAGE2_BYTES + 4 * OUT_BUFS2 * OUT_STAGE_BYTES + sizeof(PairBarriers);
static_assert(GEMM2_SMEM_BYTES <= 227 * 1024, "shared memory budget");

struct PairTile {
  Tile tl;       // this CTA's half, in the terms of the single-CTA epilogues
  bool idle;     // this CTA has no rows in the pair (odd M-block count): no loads of A worth keeping, no stores
};

template <int MODE>
__device__ __forceinline__ int total_pair_tiles(const GemmArgs& a) {
  return a.meta[3] * a.n_tiles_n;
}

// Order as in the single-CTA kernel: expert-major, column tile slow, pair fast.
template <int MODE>
__device__ __forceinline__ PairTile decode_pair_tile(const GemmArgs& a, int t, int rank) {
  PairTile pt;
  Tile& tl = pt.tl;
  pt.idle = false;
  const int e = a.pblk_expert[t / a.n_tiles_n];
  const int ps = a.pair_start[e];
  const int pcount = a.pair_start[e + 1] - ps;
  const int local = t - ps * a.n_tiles_n;
  tl.nb = local / pcount;
  const int pl = local - tl.nb * pcount;
  const int mb = a.mb_start[e] + 2 * pl + rank;
  pt.idle = mb >= a.mb_start[e + 1];
  tl.e = e;
  tl.row0 = pt.idle ? a.cap_rows : mb * BLOCK_M;   // rows beyond the tensor read as zeros
  tl.n0 = tl.nb * (MODE == GEMM_GATE_UP ? BN / 2 : BN);
  tl.m0 = 0;
  tl.nkb = (a.K + BK - 1) / BK;
  return pt;
}

constexpr int GEMM2_THREADS = GEMM_THREADS;

template <int MODE>
__global__ void __launch_bounds__(GEMM2_THREADS, 1) grouped_gemm_pair_kernel(const __grid_constant__ GemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;                                  // [STAGES2][16 KB]
  uint8_t* sB = smem + STAGES2 * A_STAGE_BYTES;        // [STAGES2][16 KB]
  uint8_t* sOut = smem + STAGES2 * STAGE2_BYTES;
  PairBarriers* bars = reinterpret_cast<PairBarriers*>(sOut + 4 * OUT_BUFS2 * OUT_STAGE_BYTES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const WaitCtl wc{a.status, a.budget_ns};

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES2; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
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
  cluster_sync_all();  // both CTAs' barriers exist before anyone signals across the pair
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;
  const int total = total_pair_tiles<MODE>(a);

  if (warp == 0) {
    // ------------------------------------------------ TMA producer (both CTAs, one box per lane)
    uint32_t s = 0, ph = 1;
    bool ok = true;
    for (int t = pair; t < total && ok; t += npairs) {
      const PairTile pt = decode_pair_tile<MODE>(a, t, rank);
      for (int kb = 0; kb < pt.tl.nkb; ++kb) {
        int go = 1;
        if (lane == 0) go = mbar_wait(&bars->empty[s], ph, wc, SITE_EMPTY, t, 50) ? 1 : 0;
        go = __shfl_sync(0xffffffffu, go, 0);
        if (!go) { ok = false; break; }
        load_stage_pair_lanes<MODE>(a, pt.tl, kb, rank, sA + s * A_STAGE_BYTES, sB + s * HALF_B_BYTES, &bars->full[s], lane);
        if (++s == STAGES2) { s = 0; ph ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer (even CTA only)
    if (lane == 0 && rank == 0) {
      uint32_t it = 0, acc_it = 0;
      bool ok = true;
      for (int t = pair; t < total && ok; t += npairs) {
        const PairTile pt = decode_pair_tile<MODE>(a, t, 0);
        const int as = acc_it & 1;
        if (!mbar_wait(&bars->tmem_empty[as], ((acc_it >> 1) & 1) ^ 1, wc, SITE_TMEM_EMPTY, t)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + as * BN;
        for (int kb = 0; kb < pt.tl.nkb; ++kb, ++it) {
          const int s = it % STAGES2;
          if (!mbar_wait(&bars->full[s], (it / STAGES2) & 1, wc, SITE_FULL, t)) { ok = false; break; }
          tc_fence_after_sync();
          mma_kblock_pair<MODE>(d_tmem, smem_u32(sA + s * A_STAGE_BYTES), smem_u32(sB + s * HALF_B_BYTES), kb == 0);
          tc_commit_pair(&bars->empty[s]);   // frees the stage in both CTAs
        }
        if (!ok) break;
        tc_commit_pair(&bars->tmem_full[as]);  // accumulator slices ready in both CTAs
        ++acc_it;
      }
      if (!ok || *reinterpret_cast<volatile int*>(&a.status->abort)) {
        tc_commit_pair(&bars->drain);
        const WaitCtl shortwc{a.status, 20ull * 1000 * 1000};
        mbar_wait(&bars->drain, 0, shortwc, SITE_DRAIN, 0);
      }
    }
  } else {
    // ------------------------------------------------ epilogue warps (both CTAs, own rows)
    const int quad = warp & 3;
    Staging stg{sOut + quad * OUT_BUFS2 * OUT_STAGE_BYTES, OUT_BUFS2, 0};
    uint32_t acc_it = 0;
    for (int t = pair; t < total; t += npairs) {
      const PairTile pt = decode_pair_tile<MODE>(a, t, rank);
      const int as = acc_it & 1;
      if (!mbar_wait(&bars->tmem_full[as], (acc_it >> 1) & 1, wc, SITE_TMEM_FULL, t, 200)) break;  // back off: idle epilogue warps must not take issue slots and power
      tc_fence_after_sync();
      if (!pt.idle) epilogue_tile<MODE>(a, pt.tl, tmem_base + as * BN, quad, lane, stg);
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(&bars->tmem_empty[as]);
      ++acc_it;
    }
    if (lane == 0) tma_store_wait_all();
  }

  // ---------------------------------------------------------------- teardown
  if (*reinterpret_cast<volatile int*>(&a.status->abort)) __nanosleep(200000);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // neither CTA leaves while its partner may still read its shared memory or signal it
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

template <int MODE>
static cudaError_t launch_pair_mode(const GemmArgs& a, int num_sms, cudaStream_t s) {
  static PairLaunchState st;
  return launch_on_pairs(st, grouped_gemm_pair_kernel<MODE>, a, GEMM2_THREADS, GEMM2_SMEM_BYTES, num_sms, false, s);
}

cudaError_t launch_gemm2(GemmMode mode, const GemmArgs& a, int num_sms, cudaStream_t s, int* launches) {
  ++*launches;
  switch (mode) {
    case GEMM_GATE_UP: return launch_pair_mode<GEMM_GATE_UP>(a, num_sms, s);
    case GEMM_DOWN: return launch_pair_mode<GEMM_DOWN>(a, num_sms, s);
    case GEMM_ACT_GRAD: return launch_pair_mode<GEMM_ACT_GRAD>(a, num_sms, s);
    case GEMM_GATE_GRAD: return launch_pair_mode<GEMM_GATE_GRAD>(a, num_sms, s);
    default: break;   // the weight gradients run strip by strip (gemm_wgrad.cu)
  }
  return cudaErrorInvalidValue;
}

}  // namespace moe
