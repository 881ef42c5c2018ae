// Grouped GEMMs of the MoE-FFN layer, one launch per operator (the operator-by-operator mode).
//
// One persistent, warp-specialised kernel body serves the five GEMM-shaped operators of the layer
// (forward GMM1+SwiGLU, GMM2; backward act_grad+SwiGLU_grad, gate_grad, and the two weight
// gradients).  Per CTA: warp 0 = TMA producer (one elected lane), warp 1 = tcgen05.mma issuer (one
// elected lane; the warp also owns the TMEM allocation), warps 2..5 = epilogue.  Operands travel
// global -> shared through TMA into a 4-stage ring of 128-byte-swizzled tiles; accumulators live in
// TMEM, double-buffered (2 x 256 columns) so the epilogue of tile i overlaps the main loop of tile
// i+1.  Tiles are assigned round-robin over the CTAs.
#include "gemm_tile.cuh"

namespace moe {

size_t gemm_smem_bytes() { return GEMM_SMEM_BYTES; }

// ---------------------------------------------------------------- the kernel
template <int MODE>
__global__ void __launch_bounds__(GEMM_THREADS, 1) grouped_gemm_kernel(const __grid_constant__ GemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = smem + STAGES * A_STAGE_BYTES;
  uint8_t* sOut = smem + STAGES * (A_STAGE_BYTES + B_STAGE_BYTES);
  GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(sOut + 4 * OUT_STAGE_BYTES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WaitCtl wc{a.status, a.budget_ns};

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->tmem_full[s], 1);
      mbar_init(&bars->tmem_empty[s], 4);
    }
    mbar_init(&bars->drain, 1);
    mbar_fence_init();
    fence_proxy_async();
    tma_prefetch_desc(&a.tmA);
    tma_prefetch_desc(&a.tmB);
    tma_prefetch_desc(&a.tmOut0);
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;
  const int total = total_tiles<MODE>(a);

  if (warp == 0) {
    // ------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
        const Tile tl = decode_tile<MODE>(a, t);
        for (int kb = 0; kb < tl.nkb; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(&bars->empty[s], ph ^ 1, wc, SITE_EMPTY, t)) { ok = false; break; }
          load_stage<MODE>(a, tl, kb, sA + s * A_STAGE_BYTES, sB + s * B_STAGE_BYTES, &bars->full[s]);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, acc_it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
        const Tile tl = decode_tile<MODE>(a, t);
        if (tl.nkb == 0) continue;
        const int as = acc_it & 1;
        const uint32_t aph = (acc_it >> 1) & 1;
        if (!mbar_wait(&bars->tmem_empty[as], aph ^ 1, wc, SITE_TMEM_EMPTY, t)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + as * BN;
        for (int kb = 0; kb < tl.nkb; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(&bars->full[s], ph, wc, SITE_FULL, t)) { ok = false; break; }
          tc_fence_after_sync();
          mma_kblock<MODE>(d_tmem, smem_u32(sA + s * A_STAGE_BYTES), smem_u32(sB + s * B_STAGE_BYTES), kb == 0);
          tc_commit(&bars->empty[s]);  // frees the smem stage once these MMAs have read it
        }
        if (!ok) break;
        tc_commit(&bars->tmem_full[as]);  // accumulator complete
        ++acc_it;
      }
      if (!ok || *reinterpret_cast<volatile int*>(&a.status->abort)) {
        // leave only after the tensor core has stopped touching shared memory and TMEM
        tc_commit(&bars->drain);
        const WaitCtl shortwc{a.status, 20ull * 1000 * 1000};
        mbar_wait(&bars->drain, 0, shortwc, SITE_DRAIN, 0);
      }
    }
  } else {
    // ------------------------------------------------ epilogue warps
    const int quad = warp & 3;  // TMEM lane quadrant this warp may access
    Staging stg{sOut + quad * OUT_STAGE_BYTES, 1, 0};
    uint32_t acc_it = 0;
    for (int t = blockIdx.x; t < total; t += gridDim.x) {
      const Tile tl = decode_tile<MODE>(a, t);
      if (tl.nkb == 0) {
        epilogue_tile<MODE>(a, tl, 0, quad, lane, stg);  // WGRAD of an expert without rows: zeros
        continue;
      }
      const int as = acc_it & 1;
      const uint32_t aph = (acc_it >> 1) & 1;
      if (!mbar_wait(&bars->tmem_full[as], aph, wc, SITE_TMEM_FULL, t)) break;
      tc_fence_after_sync();
      epilogue_tile<MODE>(a, tl, tmem_base + as * BN, quad, lane, stg);
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->tmem_empty[as]);
      ++acc_it;
    }
    if (lane == 0) tma_store_wait_all();  // this warp's stores are complete before the CTA exits
  }

  // ---------------------------------------------------------------- teardown
  if (*reinterpret_cast<volatile int*>(&a.status->abort)) __nanosleep(200000);  // let in-flight copies land
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

template <int MODE>
static cudaError_t launch_mode(const GemmArgs& a, int num_sms, cudaStream_t s) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(grouped_gemm_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)GEMM_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  grouped_gemm_kernel<MODE><<<num_sms, GEMM_THREADS, GEMM_SMEM_BYTES, s>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_gemm(GemmMode mode, const GemmArgs& a, int num_sms, cudaStream_t s, int* launches) {
  ++*launches;
  switch (mode) {
    case GEMM_GATE_UP: return launch_mode<GEMM_GATE_UP>(a, num_sms, s);
    case GEMM_DOWN: return launch_mode<GEMM_DOWN>(a, num_sms, s);
    case GEMM_ACT_GRAD: return launch_mode<GEMM_ACT_GRAD>(a, num_sms, s);
    case GEMM_GATE_GRAD: return launch_mode<GEMM_GATE_GRAD>(a, num_sms, s);
    case GEMM_WGRAD: return launch_mode<GEMM_WGRAD>(a, num_sms, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace moe
