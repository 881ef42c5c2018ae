// Weight gradients on CTA pairs, strip by strip (gemm_roles.cuh), one launch per operator.
//
// Roles per CTA: warp 0 TMA producer of A (and the stage's byte count), warp 6 TMA producer of B,
// warp 1 MMA issuer (even CTA) and TMEM owner, warps 2..5 epilogue.
#include "gemm_roles.cuh"
#include "launch_pairs.cuh"

namespace moe {

constexpr int WG_THREADS = GEMM_THREADS + 32;
constexpr size_t WGRAD_SMEM_BYTES = 1024 + WGRAD_LAYOUT_BYTES + sizeof(PipeBarriers);
static_assert(WGRAD_SMEM_BYTES <= 227 * 1024, "shared memory budget");

__global__ void __launch_bounds__(WG_THREADS, 1) grouped_wgrad_pair_kernel(const __grid_constant__ GemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  PipeBarriers* bars = reinterpret_cast<PipeBarriers*>(smem + WGRAD_LAYOUT_BYTES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const WaitCtl wc{a.status, a.budget_ns};
  const NoDeps dep;

  if (threadIdx.x == 0) {
    pipe_init(bars);
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

  // Strips pair, pair + npairs, ..; each role decodes strip i + 1 before it works on strip i.
  const int total = wgrad_strips(a);
  Strip cur, next;
  if (pair < total) cur = decode_strip(a, pair);
  if (warp == 0 || warp == 6) {
    LoaderState ls;
    for (int sp = pair; sp < total; sp += npairs, cur = next) {
      if (sp + npairs < total) next = decode_strip(a, sp + npairs);
      if (!wgrad_load_strip(a, smem, bars, ls, warp == 6, rank, lane, cur, sp, wc, dep)) break;
    }
  } else if (warp == 1) {
    if (rank == 0) {
      IssuerState is;
      bool ok = true;
      for (int sp = pair; sp < total && ok; sp += npairs, cur = next) {
        if (sp + npairs < total) next = decode_strip(a, sp + npairs);
        ok = wgrad_issue_strip(a, smem, bars, tmem_base, is, lane == 0, cur, sp, wc, dep);
      }
      if (lane == 0 && (!ok || *reinterpret_cast<volatile int*>(&a.status->abort))) issuer_drain(bars, a.status);
    }
  } else {
    EpiState es;
    for (int sp = pair; sp < total; sp += npairs, cur = next) {
      if (sp + npairs < total) next = decode_strip(a, sp + npairs);
      if (!wgrad_epilogue_strip(a, smem, bars, tmem_base, es, rank, warp & 3, lane, cur, sp, wc, dep)) break;
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
  static PairLaunchState st;
  return launch_on_pairs(st, grouped_wgrad_pair_kernel, a, WG_THREADS, WGRAD_SMEM_BYTES, num_sms, false, s);
}

}  // namespace moe
