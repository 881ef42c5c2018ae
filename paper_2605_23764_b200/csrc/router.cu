// Router in the path (Section 2.2, first paragraph: the router scores the experts for every token and keeps the
// top k): logits = x W_r^T on the tensor cores with the softmax top-k of route_layout.cu's router fused into the
// epilogue, and the gradient of the k scores with respect to the logits.
//
// Forward: CTA pairs (tcgen05 cta_group::2) over tiles of 256 tokens.  A = 128 token rows of x per CTA, B = W_r
// (all E experts, each CTA stages half of the rows), K = d in 64-wide blocks through a 6-stage TMA ring; the
// accumulator of a CTA is [128 tokens][E] fp32 in TMEM, two of them so that the epilogue of one tile overlaps the
// MMAs of the next.  Epilogue: TMEM lane = token, so one thread owns one token's E logits and reads them 16 columns
// at a time, twice: once to select (insertion into a sorted list of k, raw logits compared, strict '>' while
// scanning expert ids upward, so ties go to the lower id and slots come out in descending order), once to sum
// exp(l - max) and, if asked, to store the logits.
#include <limits.h>

#include "gemm_pair.cuh"
#include "launch_pairs.cuh"
#include "moe_internal.h"

namespace moe {

constexpr int ROUTER_STAGES = 6;
constexpr int ROUTER_THREADS = 192;   // warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 epilogue
constexpr int ROUTER_TILE_TOKENS = 256;
constexpr int ROUTER_KMAX = 8;
constexpr int ROUTER_ACC_COLS = 256;

struct RouterBarriers {
  uint64_t full[ROUTER_STAGES], empty[ROUTER_STAGES];
  uint64_t tmem_full[2], tmem_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
};
constexpr size_t ROUTER_SMEM_BYTES = 1024 + (size_t)ROUTER_STAGES * STAGE2_BYTES + sizeof(RouterBarriers) + 64;

// One token's logits -> its k experts and scores.  `acc` = TMEM address of the thread's lane, column 0.
__device__ __forceinline__ void router_epilogue_row(const RouterArgs& a, uint32_t acc, int token, bool valid) {
  float val[ROUTER_KMAX];
  int idx[ROUTER_KMAX];
#pragma unroll
  for (int j = 0; j < ROUTER_KMAX; ++j) { val[j] = -INFINITY; idx[j] = INT_MAX; }
  // pass 1: selection (every thread of the warp takes part in the TMEM loads)
  for (int c0 = 0; c0 < a.E; c0 += 16) {
    float v[16];
    tmem_ld16(acc + c0, v);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int e = c0 + i;
      const float x = v[i];
      if (e < a.E && x > val[ROUTER_KMAX - 1]) {
#pragma unroll
        for (int j = ROUTER_KMAX - 1; j > 0; --j) {
          if (x > val[j - 1]) { val[j] = val[j - 1]; idx[j] = idx[j - 1]; }
          else if (x > val[j]) { val[j] = x; idx[j] = e; }
        }
        if (x > val[0]) { val[0] = x; idx[0] = e; }
      }
    }
  }
  // pass 2: softmax denominator over all E (and the logits, if wanted)
  const float mx = val[0];
  float den = 0.f;
  float* lrow = (a.logits && valid) ? a.logits + (size_t)token * a.E : nullptr;
  for (int c0 = 0; c0 < a.E; c0 += 16) {
    float v[16];
    tmem_ld16(acc + c0, v);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 16; ++i)
      if (c0 + i < a.E) den += expf(v[i] - mx);
    if (lrow) {
      if (c0 + 16 <= a.E && (a.E & 3) == 0) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
          reinterpret_cast<float4*>(lrow + c0)[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (c0 + i < a.E) lrow[c0 + i] = v[i];
      }
    }
  }
  if (!valid) return;
  float p[ROUTER_KMAX], wsum = 0.f;
#pragma unroll
  for (int j = 0; j < ROUTER_KMAX; ++j) {
    p[j] = j >= a.k ? 0.f : (a.renorm & GATE_SIGMOID) ? 1.0f / (1.0f + expf(-val[j])) : expf(val[j] - mx) / den;
    wsum += p[j];
  }
#pragma unroll
  for (int j = 0; j < ROUTER_KMAX; ++j)
    if (j < a.k) {
      a.topk_ids[(size_t)token * a.k + j] = idx[j];
      a.topk_w[(size_t)token * a.k + j] = (a.renorm & GATE_RENORM) ? p[j] / wsum : p[j];
      if (a.counts) atomicAdd(&a.counts[idx[j]], 1);
    }
}

__global__ void __launch_bounds__(ROUTER_THREADS, 1) router_fwd_kernel(const __grid_constant__ RouterArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;                                      // [ROUTER_STAGES][16 KB]: this CTA's 128 token rows
  uint8_t* sB = smem + ROUTER_STAGES * A_STAGE_BYTES;      // [ROUTER_STAGES][16 KB]: this CTA's half of W_r's rows
  RouterBarriers* bars = reinterpret_cast<RouterBarriers*>(smem + ROUTER_STAGES * STAGE2_BYTES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const WaitCtl wc{a.status, a.budget_ns};
  const int ntiles = (a.T + ROUTER_TILE_TOKENS - 1) / ROUTER_TILE_TOKENS;
  const int nkb = (a.d + BK - 1) / BK;
  const uint32_t half_b_bytes = (uint32_t)(a.N / 2) * 128u;

  if (threadIdx.x == 0) {
    for (int s = 0; s < ROUTER_STAGES; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->tmem_full[s], 1);
      mbar_init(&bars->tmem_empty[s], 8);   // four epilogue warps in each CTA of the pair
    }
    mbar_init(&bars->drain, 1);
    mbar_fence_init();
    fence_proxy_async();
    tma_prefetch_desc(&a.tmX);
    tma_prefetch_desc(&a.tmW);
  }
  if (warp == 1) {
    tmem_alloc_pair(&bars->tmem_base, 2 * ROUTER_ACC_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();   // both CTAs' barriers exist before anyone signals across the pair
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------ TMA producer (lane 0 of both CTAs)
    if (lane == 0) {
      uint32_t s = 0, ph = 1;
      bool ok = true;
      for (int t = pair; t < ntiles && ok; t += npairs) {
        const int row0 = t * ROUTER_TILE_TOKENS + rank * BLOCK_M;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(&bars->empty[s], ph, wc, SITE_EMPTY, t, 50)) { ok = false; break; }
          if (rank == 0) mbar_expect_tx(&bars->full[s], 2 * (A_STAGE_BYTES + half_b_bytes));
          tma_load_2d_pair(sA + s * A_STAGE_BYTES, &a.tmX, kb * BK, row0, &bars->full[s]);
          tma_load_2d_pair(sB + s * HALF_B_BYTES, &a.tmW, kb * BK, rank * (a.N / 2), &bars->full[s]);
          if (++s == ROUTER_STAGES) { s = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer (even CTA only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = make_idesc_bf16(2 * BLOCK_M, a.N, 0, 0);
      uint32_t it = 0, acc_it = 0;
      bool ok = true;
      for (int t = pair; t < ntiles && ok; t += npairs) {
        const int as = acc_it & 1;
        if (!mbar_wait(&bars->tmem_empty[as], ((acc_it >> 1) & 1) ^ 1, wc, SITE_TMEM_EMPTY, t)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + as * ROUTER_ACC_COLS;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % ROUTER_STAGES;
          if (!mbar_wait(&bars->full[s], (it / ROUTER_STAGES) & 1, wc, SITE_FULL, t)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(sA + s * A_STAGE_BYTES), b_addr = smem_u32(sB + s * HALF_B_BYTES);
#pragma unroll
          for (int k16 = 0; k16 < BK / 16; ++k16)
            tc_mma_bf16_pair(d_tmem, make_smem_desc(a_addr + k16 * 32, 16, 1024), make_smem_desc(b_addr + k16 * 32, 16, 1024),
                             idesc, !(kb == 0 && k16 == 0));
          tc_commit_pair(&bars->empty[s]);   // frees the stage in both CTAs
        }
        if (!ok) break;
        tc_commit_pair(&bars->tmem_full[as]);
        ++acc_it;
      }
      if (!ok || *reinterpret_cast<volatile int*>(&a.status->abort)) {
        tc_commit_pair(&bars->drain);
        const WaitCtl shortwc{a.status, 20ull * 1000 * 1000};
        mbar_wait(&bars->drain, 0, shortwc, SITE_DRAIN, 0);
      }
    }
  } else {
    // ------------------------------------------------ epilogue warps (both CTAs): one thread per token
    const int quad = warp & 3;
    uint32_t acc_it = 0;
    for (int t = pair; t < ntiles; t += npairs) {
      const int as = acc_it & 1;
      if (!mbar_wait(&bars->tmem_full[as], (acc_it >> 1) & 1, wc, SITE_TMEM_FULL, t, 200)) break;
      tc_fence_after_sync();
      const int token = t * ROUTER_TILE_TOKENS + rank * BLOCK_M + quad * 32 + lane;
      router_epilogue_row(a, tmem_base + as * ROUTER_ACC_COLS + ((uint32_t)(quad * 32) << 16), token, token < a.T);
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(&bars->tmem_empty[as]);
      ++acc_it;
    }
  }

  // ---------------------------------------------------------------- teardown
  if (*reinterpret_cast<volatile int*>(&a.status->abort)) __nanosleep(200000);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();   // neither CTA leaves while its partner may still read its shared memory or signal it
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, 2 * ROUTER_ACC_COLS);
  }
}

cudaError_t launch_router_fwd(const RouterArgs& a, int num_sms, cudaStream_t s, int* launches) {
  if (a.T == 0) return cudaSuccess;
  if (a.counts) {
    cudaError_t e = cudaMemsetAsync(a.counts, 0, sizeof(int) * (size_t)a.E, s);
    if (e != cudaSuccess) return e;
  }
  ++*launches;
  static PairLaunchState st;
  return launch_on_pairs(st, router_fwd_kernel, a, ROUTER_THREADS, ROUTER_SMEM_BYTES, num_sms, false, s);
}

// ------------------------------------------------------------------------------------------
// Backward of the scores: one warp per token, expert e on lane e % 32.  p = softmax(logits) over all E.
//   no renormalisation: dl[e] = [e = e_j] g_j p[e] - p[e] * sum_j g_j p[e_j]
//   renormalisation   : w = softmax over the selected experts; dl[e_j] = w_j (g_j - sum_i g_i w_i), 0 elsewhere
// The selection passes no gradient.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) router_bwd_kernel(const float* __restrict__ logits, const int* __restrict__ ids,
                                                          const float* __restrict__ g, int T, int E, int k, int mode,
                                                          float* __restrict__ dlogits) {
  const int lane = threadIdx.x & 31;
  const int t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (t >= T) return;
  const float* l = logits + (size_t)t * E;
  float* dl = dlogits + (size_t)t * E;
  float mx = -INFINITY;
  for (int e = lane; e < E; e += 32) mx = fmaxf(mx, l[e]);
#pragma unroll
  for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  // the k selected experts, one per lane (k <= 32)
  const int my_id = lane < k ? ids[(size_t)t * k + lane] : -1;
  const bool have = my_id >= 0 && my_id < E;
  const float my_g = have ? g[(size_t)t * k + lane] : 0.f;
  const bool renorm = (mode & GATE_RENORM) != 0;
  if (mode & GATE_SIGMOID) {
    // per-expert scores s = sigmoid(l): only the selected experts get a gradient
    const float s = have ? 1.0f / (1.0f + expf(-l[my_id])) : 0.f;
    float Z = s;
#pragma unroll
    for (int off = 16; off; off >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, off);
    float dot = renorm ? my_g * (s / Z) : 0.f;
#pragma unroll
    for (int off = 16; off; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    for (int e = lane; e < E; e += 32) dl[e] = 0.f;
    __syncwarp();
    if (have) dl[my_id] = renorm ? s * (1.0f - s) / Z * (my_g - dot) : my_g * s * (1.0f - s);
    return;
  }
  const float my_ex = have ? expf(l[my_id] - mx) : 0.f;
  float den = 0.f;
  if (renorm) {
    den = my_ex;
  } else {
    for (int e = lane; e < E; e += 32) den += expf(l[e] - mx);
  }
#pragma unroll
  for (int off = 16; off; off >>= 1) den += __shfl_xor_sync(0xffffffffu, den, off);
  const float my_w = my_ex / den;
  float dot = my_g * my_w;
#pragma unroll
  for (int off = 16; off; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
  // dense part
  for (int e = lane; e < E; e += 32) dl[e] = renorm ? 0.f : -(expf(l[e] - mx) / den) * dot;
  __syncwarp();
  // the selected experts are distinct, so each lane corrects its own entry
  if (have) dl[my_id] = renorm ? my_w * (my_g - dot) : my_w * my_g - my_w * dot;
}

cudaError_t launch_router_bwd(const float* logits, const int* ids, const float* g, int T, int E, int k, int gate_mode,
                              float* dlogits, cudaStream_t s, int* launches) {
  if (T == 0) return cudaSuccess;
  const int threads = 256, tokens_per_block = threads / 32;
  router_bwd_kernel<<<(T + tokens_per_block - 1) / tokens_per_block, threads, 0, s>>>(logits, ids, g, T, E, k,
                                                                                      gate_mode, dlogits);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace moe
