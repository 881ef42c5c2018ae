// Row-space grouped GEMMs (GMM1+SwiGLU, GMM2, act_grad, gate_grad) on CTA pairs with token-column
// tiles, one launch per operator: the roles of gemm_roles.cuh walk the operator's items in a static
// order without event counters -- the kernel boundary orders the operators (the paper's operator-by-operator baseline,
// Section 5.2).
//
// Roles per CTA: warp 0 TMA producer of the weights, warp 1 MMA issuer (even CTA) and TMEM owner,
// warps 2..5 epilogue, warp 6 TMA producer of the tokens.
#include "gemm_roles.cuh"
#include "launch_pairs.cuh"

namespace moe {

template <int MODE>
__host__ __device__ constexpr size_t gemm3_smem_bytes() { return 1024 + swap_layout_bytes<MODE>() + sizeof(PipeBarriers); }
static_assert(gemm3_smem_bytes<GEMM_GATE_UP>() <= 227 * 1024 && gemm3_smem_bytes<GEMM_DOWN>() <= 227 * 1024 &&
                  gemm3_smem_bytes<GEMM_ACT_GRAD>() <= 227 * 1024 && gemm3_smem_bytes<GEMM_GATE_GRAD>() <= 227 * 1024,
              "shared memory budget");

constexpr int GEMM3_THREADS = 224;

template <int MODE>
__global__ void __launch_bounds__(GEMM3_THREADS, 1) grouped_gemm_swap_kernel(const __grid_constant__ GemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  PipeBarriers* bars = reinterpret_cast<PipeBarriers*>(smem + swap_layout_bytes<MODE>());

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
    for (int i = 0; i < 8; ++i) tma_prefetch_desc(&a.tmTok[i]);
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

  // Items pair, pair + npairs, ..; each role decodes item i + 1 before it works on item i (the decode's chain of
  // global loads then completes behind the item's work).
  const int total = total_swap_work<MODE>(a);
  SwapWork cur, next;
  if (pair < total) cur = decode_swap_work<MODE>(a, pair);
  if (warp == 0 || warp == 6) {
    LoaderState ls;
    for (int t = pair; t < total; t += npairs, cur = next) {
      if (t + npairs < total) next = decode_swap_work<MODE>(a, t + npairs);
      if (!swap_load_item<MODE>(a, smem, bars, ls, warp == 6, rank, lane, cur, t, wc, dep)) break;
    }
  } else if (warp == 1) {
    if (rank == 0) {
      IssuerState is;
      bool ok = true;
      for (int t = pair; t < total && ok; t += npairs, cur = next) {
        if (t + npairs < total) next = decode_swap_work<MODE>(a, t + npairs);
        ok = swap_issue_item<MODE>(a, smem, bars, tmem_base, is, lane == 0, cur, t, wc, dep);
      }
      if (lane == 0 && (!ok || *reinterpret_cast<volatile int*>(&a.status->abort))) issuer_drain(bars, a.status);
    }
  } else {
    EpiState es;
    for (int t = pair; t < total; t += npairs, cur = next) {
      if (t + npairs < total) next = decode_swap_work<MODE>(a, t + npairs);
      if (!swap_epilogue_item<MODE>(a, smem, bars, tmem_base, es, rank, warp & 3, lane, cur, t, wc, dep)) break;
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
  static PairLaunchState st;
  return launch_on_pairs(st, grouped_gemm_swap_kernel<MODE>, a, GEMM3_THREADS, gemm3_smem_bytes<MODE>(), num_sms,
                         false, s);
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

}  // namespace moe
