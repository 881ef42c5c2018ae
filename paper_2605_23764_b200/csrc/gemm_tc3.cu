// Row-space grouped GEMMs on CTA pairs with token-column tiles, one launch per operator.
//
// Same roles per CTA as the other CTA-pair kernel (warp 0 TMA producer of the weights, warp 1 MMA issuer
// in the even CTA and TMEM owner, warps 2..5 epilogue) plus warp 6, TMA producer of the tokens; same barriers; what differs is the tile (gemm_swap.cuh):
// the weights are the A operand (256 accumulator rows per pair), an expert's tokens the B operand
// (32..256 accumulator columns), so the bytes a stage expects and the MMA shape vary per tile.
#include <stdio.h>
#include <stdlib.h>

#include "gemm_swap.cuh"

namespace moe {

#ifndef MOE_STAGES3
#define MOE_STAGES3 5
#endif
constexpr int STAGES3 = MOE_STAGES3;   // operand stages: 16 KB of weights + 16 KB of tokens (24 KB in the operators
                                       // that merge token tiles, which keep one staging slot per epilogue warp instead of two)

struct __align__(8) SwapBarriers {
  uint64_t full[STAGES3];     // used in the even CTA: bytes of both CTAs' loads
  uint64_t empty[STAGES3];    // in each CTA: the stage's MMAs are complete
  uint64_t tmem_full[2];      // in each CTA: accumulator ready
  uint64_t tmem_empty[2];     // used in the even CTA: 8 epilogue warps of the pair have drained it
  uint64_t drain;
  uint32_t tmem_base;
  uint32_t pad;
};

// staging per epilogue warp: two slots of 4 KB; the operators that merge store plain 2 KB boxes and keep
// two slots of 2 KB (their operand stages need the room)
template <int MODE>
__host__ __device__ constexpr int staging_slot_bytes3() { return swap_merges<MODE>() ? SW_SLOT_BYTES / 2 : SW_SLOT_BYTES; }
template <int MODE>
__host__ __device__ constexpr size_t gemm3_smem_bytes() {
  return 1024 + (size_t)STAGES3 * (W_STAGE_BYTES + tok_stage_bytes<MODE>()) + 4 * SW_SLOTS * staging_slot_bytes3<MODE>() +
         (MODE == GEMM_ACT_GRAD ? 4 * SW_SCRATCH_BYTES : 0) + sizeof(SwapBarriers);
}
static_assert(gemm3_smem_bytes<GEMM_GATE_UP>() <= 227 * 1024 && gemm3_smem_bytes<GEMM_DOWN>() <= 227 * 1024 &&
                  gemm3_smem_bytes<GEMM_ACT_GRAD>() <= 227 * 1024 && gemm3_smem_bytes<GEMM_GATE_GRAD>() <= 227 * 1024,
              "shared memory budget");

#ifdef MOE_STATS3
__device__ long long g_stats3[5][160][8];
#define S3_DECL long long s3_t = clock64(), s3_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}
#define S3_LAP(i) do { const long long n_ = clock64(); s3_acc[i] += n_ - s3_t; s3_t = n_; } while (0)
#define S3_FLUSH(base) do { for (int i_ = 0; i_ < 4; ++i_) g_stats3[MODE][blockIdx.x][(base) + i_] = s3_acc[i_]; } while (0)
#else
#define S3_DECL
#define S3_LAP(i)
#define S3_FLUSH(base)
#endif

constexpr int GEMM3_THREADS = 224;

template <int MODE>
__global__ void __launch_bounds__(GEMM3_THREADS, 1) grouped_gemm_swap_kernel(const __grid_constant__ GemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int TOKB = tok_stage_bytes<MODE>();
  constexpr int SLOTB = staging_slot_bytes3<MODE>();
  uint8_t* sW = smem;                                   // [STAGES3][16 KB] weights
  uint8_t* sT = smem + STAGES3 * W_STAGE_BYTES;         // [STAGES3][TOKB] tokens (this CTA's half)
  uint8_t* sOut = smem + STAGES3 * (W_STAGE_BYTES + TOKB);
  uint8_t* sScr = sOut + 4 * SW_SLOTS * SLOTB;          // act_grad: per epilogue warp 4 KB for the saved pre-activations
  SwapBarriers* bars = reinterpret_cast<SwapBarriers*>(sScr + (MODE == GEMM_ACT_GRAD ? 4 * SW_SCRATCH_BYTES : 0));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const WaitCtl wc{a.status, a.budget_ns};

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES3; ++s) {
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
    for (int i = 0; i < 3; ++i) tma_prefetch_desc(&a.tmTok[i]);
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
  const int total = total_swap_work<MODE>(a);

  if (warp == 0 || warp == 6) {
    // ------------------------------------------------ TMA producers (both CTAs, one box per lane)
    uint32_t s = 0, ph = 1;
    bool ok = true;
    S3_DECL;
    for (int t = pair; t < total && ok; t += npairs) {
      const SwapWork wk = decode_swap_work<MODE>(a, t);
      const SwapTile& st = wk.a;
      for (int kb = 0; kb < st.nkb; ++kb) {
        int go = 1;
        S3_LAP(1);
        if (lane == 0) go = mbar_wait(&bars->empty[s], ph, wc, SITE_EMPTY, t, 50) ? 1 : 0;
        go = __shfl_sync(0xffffffffu, go, 0);
        S3_LAP(0);
        if (!go) { ok = false; break; }
        if (warp == 0) {
          load_weights_swap<MODE>(a, st, kb, rank, sW + s * W_STAGE_BYTES, &bars->full[s], lane, wk.a.ntok + wk.b.ntok);
        } else {
          load_tokens_swap(a, wk.a, kb, rank, sT + s * TOKB, &bars->full[s], lane);
          if (wk.merged)   // lanes 4..7: the second token tile, behind the first in the stage
            load_tokens_swap(a, wk.b, kb, rank, sT + s * TOKB + (wk.a.ntok >> 1) * (BK * 2), &bars->full[s], lane - 4);
        }
        if (++s == STAGES3) { s = 0; ph ^= 1; }
      }
    }
    S3_LAP(1);
    if (lane == 0 && warp == 0) S3_FLUSH(4);   // [4] wait empty, [5] issue loads
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer (even CTA only)
    if (lane == 0 && rank == 0) {
      // The loop of this one thread bounds the tensor pipe when a k-block's MMAs are short: stage
      // index, phase and descriptor words are carried in registers, nothing is recomputed per k-block.
      uint32_t acc_it = 0;
      uint32_t s = 0, ph = 0;
      const uint32_t w_lo0 = swap_w_desc_lo<MODE>(smem_u32(sW)), t_lo0 = smem_desc_lo(smem_u32(sT), 16);
      uint32_t w_lo = w_lo0, t_lo = t_lo0;
      bool ok = true;
      S3_DECL;
      for (int t = pair; t < total && ok; t += npairs) {
        const SwapWork wk = decode_swap_work<MODE>(a, t);
        const int as = acc_it & 1;
        S3_LAP(2);
        if (!mbar_wait(&bars->tmem_empty[as], ((acc_it >> 1) & 1) ^ 1, wc, SITE_TMEM_EMPTY, t)) { ok = false; break; }
        if (wk.merged &&   // the second token tile accumulates in the other buffer
            !mbar_wait(&bars->tmem_empty[as ^ 1], (((acc_it + 1) >> 1) & 1) ^ 1, wc, SITE_TMEM_EMPTY, t)) { ok = false; break; }
        S3_LAP(0);
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + as * BN, d_tmem_b = tmem_base + (as ^ 1) * BN;
        const uint32_t idesc = swap_idesc<MODE>(wk.a.ntok), idesc_b = swap_idesc<MODE>(wk.merged ? wk.b.ntok : TOK_GRAIN);
        const uint32_t t_off_b = (uint32_t)((wk.a.ntok >> 1) * (BK * 2)) >> 4;
        for (int kb = 0; kb < wk.a.nkb; ++kb) {
          S3_LAP(2);
          if (!mbar_wait(&bars->full[s], ph, wc, SITE_FULL, t)) { ok = false; break; }
          S3_LAP(1);
          tc_fence_after_sync();
          mma_kblock_swap<MODE>(d_tmem, w_lo, t_lo, idesc, kb == 0);
          if (wk.merged) mma_kblock_swap<MODE>(d_tmem_b, w_lo, t_lo + t_off_b, idesc_b, kb == 0);
          tc_commit_pair(&bars->empty[s]);   // frees the stage in both CTAs
          if (++s == STAGES3) {
            s = 0; ph ^= 1; w_lo = w_lo0; t_lo = t_lo0;
          } else {
            w_lo += W_STAGE_BYTES >> 4; t_lo += TOKB >> 4;
          }
        }
        if (!ok) break;
        tc_commit_pair(&bars->tmem_full[as]);  // accumulator slices ready in both CTAs
        ++acc_it;
        if (wk.merged) {
          tc_commit_pair(&bars->tmem_full[as ^ 1]);
          ++acc_it;
        }
      }
      S3_LAP(2);
      S3_FLUSH(0);   // [0] wait tmem_empty, [1] wait operands, [2] issue
      if (!ok || *reinterpret_cast<volatile int*>(&a.status->abort)) {
        tc_commit_pair(&bars->drain);
        const WaitCtl shortwc{a.status, 20ull * 1000 * 1000};
        mbar_wait(&bars->drain, 0, shortwc, SITE_DRAIN, 0);
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------ epilogue warps (both CTAs, own features)
    const int quad = warp & 3;
    SwStaging sg{sOut + quad * SW_SLOTS * SLOTB, 0, sScr + quad * SW_SCRATCH_BYTES, SW_SLOTS, (uint32_t)SLOTB};
    uint32_t acc_it = 0;
    bool ok = true;
    for (int t = pair; t < total && ok; t += npairs) {
      const SwapWork wk = decode_swap_work<MODE>(a, t);
      for (int part = 0; part < (wk.merged ? 2 : 1); ++part) {   // a merged item is two consecutive tiles here
        const int as = acc_it & 1;
        if (!mbar_wait(&bars->tmem_full[as], (acc_it >> 1) & 1, wc, SITE_TMEM_FULL, t, 200)) { ok = false; break; }
        tc_fence_after_sync();
        epilogue_swap<MODE>(a, part ? wk.b : wk.a, tmem_base + as * BN, rank, quad, lane, sg);
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
  cluster_sync_all();  // neither CTA leaves while its partner may still read its shared memory or signal it
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

template <int MODE>
static cudaError_t launch_swap_mode(const GemmArgs& a, int num_sms, cudaStream_t s) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(grouped_gemm_swap_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)gemm3_smem_bytes<MODE>());
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  static int max_pairs = 0;  // CTA pairs that can be resident together (SMs pair up inside a GPC)
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3((num_sms / 2) * 2);
  cfg.blockDim = dim3(GEMM3_THREADS);
  cfg.dynamicSmemBytes = gemm3_smem_bytes<MODE>();
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
    cudaError_t e = cudaOccupancyMaxActiveClusters(&n, grouped_gemm_swap_kernel<MODE>, &cfg);
    if (e != cudaSuccess) return e;
    max_pairs = n > 0 ? n : 1;
  }
  if (2 * max_pairs < (int)cfg.gridDim.x) cfg.gridDim = dim3(2 * max_pairs);
  return cudaLaunchKernelEx(&cfg, grouped_gemm_swap_kernel<MODE>, a);
}

cudaError_t launch_gemm3(GemmMode mode, const GemmArgs& a, int num_sms, cudaStream_t s, int* launches) {
  ++*launches;
  switch (mode) {
    case GEMM_GATE_UP: return launch_swap_mode<GEMM_GATE_UP>(a, num_sms, s);
    case GEMM_DOWN: return launch_swap_mode<GEMM_DOWN>(a, num_sms, s);
    case GEMM_ACT_GRAD: return launch_swap_mode<GEMM_ACT_GRAD>(a, num_sms, s);
    case GEMM_GATE_GRAD: return launch_swap_mode<GEMM_GATE_GRAD>(a, num_sms, s);
    default: break;
  }
  return cudaErrorInvalidValue;
}

#ifdef MOE_STATS3
extern "C" int moe_debug_stats3(long long* host) {
  return (int)cudaMemcpyFromSymbol(host, g_stats3, sizeof(long long) * 5 * 160 * 8);
}
#endif

}  // namespace moe
