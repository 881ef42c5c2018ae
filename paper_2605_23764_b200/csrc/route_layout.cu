// Routing (softmax top-k) and the dispatch layout (per-expert histogram, prefix scan, stable
// permutation, M-block table).  Integer results are bit-exact by construction: every count and
// rank is an integer sum whose value does not depend on evaluation order.
#include <limits.h>

#include "moe_internal.h"

namespace moe {

// ------------------------------------------------------------------------------------------
// Router: one warp per token.  Expert e is held by lane e%32 in register e/32.
// Selection compares raw logits (softmax is monotone), ties go to the lower expert id, slots
// come out in descending logit order.  Scores: fp32 softmax over all E, max-subtracted -- or, in the
// sigmoid gate mode, 1 / (1 + exp(-logit)) per selected expert; `renorm` holds the gate mode bits.
// ------------------------------------------------------------------------------------------
template <int NPL>
__global__ void __launch_bounds__(256) route_kernel(const float* __restrict__ logits, int T, int E, int k,
                                                     int renorm, int* __restrict__ topk_ids,
                                                     float* __restrict__ topk_w, int* __restrict__ counts) {
  const int lane = threadIdx.x & 31;
  const int t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (t >= T) return;
  const float* row = logits + (size_t)t * E;
  float v[NPL];
  float mx = -INFINITY;
#pragma unroll
  for (int i = 0; i < NPL; ++i) {
    int e = i * 32 + lane;
    v[i] = e < E ? row[e] : -INFINITY;
    mx = fmaxf(mx, v[i]);
  }
#pragma unroll
  for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  float den = 0.f;
#pragma unroll
  for (int i = 0; i < NPL; ++i)
    if (i * 32 + lane < E) den += expf(v[i] - mx);
#pragma unroll
  for (int off = 16; off; off >>= 1) den += __shfl_xor_sync(0xffffffffu, den, off);

  uint32_t taken = 0;
  int my_id = 0;
  float my_p = 0.f, wsum = 0.f;
  for (int j = 0; j < k; ++j) {
    float bv = 0.f;
    int bi = INT_MAX;
#pragma unroll
    for (int i = 0; i < NPL; ++i) {
      int e = i * 32 + lane;
      if (e < E && !((taken >> i) & 1u) && (bi == INT_MAX || v[i] > bv)) { bv = v[i]; bi = e; }
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, bv, off);
      int oi = __shfl_xor_sync(0xffffffffu, bi, off);
      if (oi != INT_MAX && (bi == INT_MAX || ov > bv || (ov == bv && oi < bi))) { bv = ov; bi = oi; }
    }
    if ((bi & 31) == lane) taken |= 1u << (bi >> 5);
    float p = (renorm & GATE_SIGMOID) ? 1.0f / (1.0f + expf(-bv)) : expf(bv - mx) / den;
    if (lane == j) { my_id = bi; my_p = p; }
    wsum += p;
  }
  if (lane < k) {
    if (renorm & GATE_RENORM) my_p /= wsum;
    topk_ids[(size_t)t * k + lane] = my_id;
    topk_w[(size_t)t * k + lane] = my_p;
    if (counts) atomicAdd(&counts[my_id], 1);
  }
}

cudaError_t launch_route(const float* logits, int T, int E, int k, int gate_mode, int* topk_ids, float* topk_w,
                         int* counts, cudaStream_t s, int* launches) {
  if (T == 0) return cudaSuccess;
  if (counts) {
    cudaError_t e = cudaMemsetAsync(counts, 0, sizeof(int) * (size_t)E, s);
    if (e != cudaSuccess) return e;
  }
  const int threads = 256, tokens_per_block = threads / 32;
  dim3 grid((T + tokens_per_block - 1) / tokens_per_block);
  const int npl = (E + 31) / 32;
#define MOE_ROUTE_CASE(N) \
  route_kernel<N><<<grid, threads, 0, s>>>(logits, T, E, k, gate_mode, topk_ids, topk_w, counts)
  if (npl <= 1) MOE_ROUTE_CASE(1);
  else if (npl <= 2) MOE_ROUTE_CASE(2);
  else if (npl <= 4) MOE_ROUTE_CASE(4);
  else if (npl <= 8) MOE_ROUTE_CASE(8);
  else if (npl <= 16) MOE_ROUTE_CASE(16);
  else MOE_ROUTE_CASE(32);
#undef MOE_ROUTE_CASE
  ++*launches;
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Dispatch layout.  Flat slot i = t*kp + j; block b owns slots [b*CHUNK, (b+1)*CHUNK), warp w of
// the block owns 256 consecutive slots of it, processed 32 at a time in slot order.
// ------------------------------------------------------------------------------------------
constexpr int LAYOUT_THREADS = 256;
constexpr int LAYOUT_WARPS = LAYOUT_THREADS / 32;
constexpr int SLOTS_PER_WARP = LAYOUT_CHUNK / LAYOUT_WARPS;

__device__ __forceinline__ int slot_expert(const int* __restrict__ ids, int i, int k, int kp, int E) {
  int t = i / kp, j = i - t * kp;
  if (j >= k) return E + (j - k);
  int e = ids[(size_t)t * k + j];
  return (e >= 0 && e < E) ? e : -1;
}

// Per-warp histograms of this block's chunk into shared memory whist[LAYOUT_WARPS][Ep].
__device__ __forceinline__ void chunk_histogram(const int* __restrict__ ids, int n, int k, int kp, int E, int Ep,
                                                int* whist) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int q = threadIdx.x; q < LAYOUT_WARPS * Ep; q += LAYOUT_THREADS) whist[q] = 0;
  __syncthreads();
  int* mine = whist + warp * Ep;
  const int base = blockIdx.x * LAYOUT_CHUNK + warp * SLOTS_PER_WARP;
  for (int g = 0; g < SLOTS_PER_WARP; g += 32) {
    int i = base + g + lane;
    int e = i < n ? slot_expert(ids, i, k, kp, E) : -1;
    uint32_t peers = __match_any_sync(0xffffffffu, e);
    if (e >= 0 && lane == __ffs(peers) - 1) mine[e] += __popc(peers);
    __syncwarp();
  }
  __syncthreads();
}

__global__ void __launch_bounds__(LAYOUT_THREADS) layout_hist_kernel(const int* __restrict__ ids, int n, int k,
                                                                      int kp, int E, int Ep,
                                                                      int* __restrict__ blk_hist, int* __restrict__ tok_last) {
  extern __shared__ int whist[];
  if (tok_last)   // the tokens whose first slot lies in this block's chunk
    for (int i = blockIdx.x * LAYOUT_CHUNK + threadIdx.x; i < min(n, (blockIdx.x + 1) * LAYOUT_CHUNK); i += LAYOUT_THREADS)
      if (i % kp == 0) tok_last[i / kp] = 0;
  chunk_histogram(ids, n, k, kp, E, Ep, whist);
  for (int e = threadIdx.x; e < Ep; e += LAYOUT_THREADS) {
    int tot = 0;
#pragma unroll
    for (int w = 0; w < LAYOUT_WARPS; ++w) tot += whist[w * Ep + e];
    blk_hist[(size_t)blockIdx.x * Ep + e] = tot;
  }
}

// One block.  (1) per expert, exclusive scan of the block histograms over blocks (warp per expert);
// (2) exclusive scans over experts for row offsets and M-block starts; (3) M-block -> expert table.
__global__ void __launch_bounds__(1024) layout_scan_kernel(int nblk, int Ep, LayoutView lv) {
  extern __shared__ int sm[];
  int* s_counts = sm;            // [Ep]
  int* s_mbstart = sm + Ep;      // [Ep+1]
  int* s_pstart = sm + 2 * Ep + 1;  // [Ep+1]
  int* s_wstart = sm + 3 * Ep + 2;  // [Ep+1]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int e = warp; e < Ep; e += 32) {
    int carry = 0;
    for (int b0 = 0; b0 < nblk; b0 += 32) {
      int b = b0 + lane;
      int v = b < nblk ? lv.blk_hist[(size_t)b * Ep + e] : 0;
      int incl = v;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        int o = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += o;
      }
      if (b < nblk) lv.blk_hist[(size_t)b * Ep + e] = carry + incl - v;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) s_counts[e] = carry;
  }
  __syncthreads();
  if (warp == 0) {
    int carry_rows = 0, carry_mb = 0, carry_pr = 0, carry_wi = 0;
    for (int e0 = 0; e0 < Ep; e0 += 32) {
      int e = e0 + lane;
      int c = e < Ep ? s_counts[e] : 0;
      int m = (c + BLOCK_M - 1) / BLOCK_M;
      int pr = (m + 1) >> 1;  // pairs of M-blocks (the tensor-core tile of a CTA pair)
      // work items of the token-column GEMM kernels that merge: the units of the expert, except that an expert
      // that merges (schedule.h) has its last two units (one block; block + tail) share one k-loop
      int wi = pr - (expert_merges(c, m) ? 1 : 0);
      int ic = c, im = m, ip = pr, iw = wi;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        int oc = __shfl_up_sync(0xffffffffu, ic, off);
        int om = __shfl_up_sync(0xffffffffu, im, off);
        int op = __shfl_up_sync(0xffffffffu, ip, off);
        int ow = __shfl_up_sync(0xffffffffu, iw, off);
        if (lane >= off) { ic += oc; im += om; ip += op; iw += ow; }
      }
      if (e < Ep) {
        lv.counts[e] = c;
        lv.offsets[e] = carry_rows + ic - c;
        int ms = carry_mb + im - m;
        s_mbstart[e] = ms;
        lv.mb_start[e] = ms;
        lv.pad_off[e] = ms * BLOCK_M;
        const int ps = carry_pr + ip - pr;
        s_pstart[e] = ps;
        lv.pair_start[e] = ps;
        const int ws = carry_wi + iw - wi;
        s_wstart[e] = ws;
        lv.work_start[e] = ws;
      }
      carry_rows += __shfl_sync(0xffffffffu, ic, 31);
      carry_mb += __shfl_sync(0xffffffffu, im, 31);
      carry_pr += __shfl_sync(0xffffffffu, ip, 31);
      carry_wi += __shfl_sync(0xffffffffu, iw, 31);
    }
    if (lane == 0) {
      lv.offsets[Ep] = carry_rows;
      s_mbstart[Ep] = carry_mb;
      lv.mb_start[Ep] = carry_mb;
      lv.pad_off[Ep] = carry_mb * BLOCK_M;
      lv.meta[0] = carry_mb;
      lv.meta[1] = carry_mb * BLOCK_M;
      lv.meta[2] = carry_rows;
      s_pstart[Ep] = carry_pr;
      lv.pair_start[Ep] = carry_pr;
      lv.meta[3] = carry_pr;
      s_wstart[Ep] = carry_wi;
      lv.work_start[Ep] = carry_wi;
      lv.meta[4] = carry_wi;
    }
  }
  __syncthreads();
  const int num_mb = s_mbstart[Ep];
  for (int mb = threadIdx.x; mb < num_mb; mb += blockDim.x) {
    int lo = 0, hi = Ep - 1;  // last expert whose mb_start <= mb
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (s_mbstart[mid] <= mb) lo = mid; else hi = mid - 1;
    }
    lv.mblk_expert[mb] = lo;
  }
  const int num_pr = s_pstart[Ep];
  for (int pb = threadIdx.x; pb < num_pr; pb += blockDim.x) {
    int lo = 0, hi = Ep - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (s_pstart[mid] <= pb) lo = mid; else hi = mid - 1;
    }
    lv.pblk_expert[pb] = lo;
  }
  const int num_wi = s_wstart[Ep];
  for (int wb = threadIdx.x; wb < num_wi; wb += blockDim.x) {
    int lo = 0, hi = Ep - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (s_wstart[mid] <= wb) lo = mid; else hi = mid - 1;
    }
    lv.wblk_expert[wb] = lo;
  }
}

__global__ void __launch_bounds__(LAYOUT_THREADS) layout_rank_kernel(const int* __restrict__ ids, int n, int k,
                                                                      int kp, int E, int Ep, LayoutView lv,
                                                                      DevStatus* status) {
  extern __shared__ int whist[];
  chunk_histogram(ids, n, k, kp, E, Ep, whist);
  // per expert: running base of each warp inside the block = block prefix + earlier warps
  for (int e = threadIdx.x; e < Ep; e += LAYOUT_THREADS) {
    int run = lv.blk_hist[(size_t)blockIdx.x * Ep + e];
#pragma unroll
    for (int w = 0; w < LAYOUT_WARPS; ++w) {
      int c = whist[w * Ep + e];
      whist[w * Ep + e] = run;
      run += c;
    }
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int* mine = whist + warp * Ep;
  const int base = blockIdx.x * LAYOUT_CHUNK + warp * SLOTS_PER_WARP;
  for (int g = 0; g < SLOTS_PER_WARP; g += 32) {
    int i = base + g + lane;
    int e = i < n ? slot_expert(ids, i, k, kp, E) : -1;
    uint32_t peers = __match_any_sync(0xffffffffu, e);
    int r = 0;
    if (e >= 0) r = mine[e] + __popc(peers & ((1u << lane) - 1u));
    __syncwarp();
    if (e >= 0 && lane == __ffs(peers) - 1) mine[e] += __popc(peers);
    __syncwarp();
    if (i < n) {
      if (e >= 0) {
        int row = lv.offsets[e] + r;
        lv.row_of[i] = row;
        lv.prow_of[i] = lv.pad_off[e] + r;
        lv.src_of[row] = i;
        // the combine order's key: the token's last ROUTED row (shared experts are taken first by the persistent launch)
        if (lv.tok_last && i % kp < k) atomicMax(&lv.tok_last[i / kp], lv.pad_off[e] + r + 1);
      } else {
        lv.row_of[i] = -1;
        lv.prow_of[i] = -1;
        note(status, /*MOE_ERR_BAD_EXPERT_ID*/ 1, i);  // the slot is dropped, the layer carries on
      }
    }
  }
}

// Combine order of the persistent launch: tokens sorted by the M-block of their LAST row in the expert-ordered
// row space (a counting sort; one block).  The operators walk the experts in order, so this is the order in
// which tokens become complete: combine tasks taken in this order find their dependent events met one after
// the other instead of all at the very end.  Tokens without any row come first.
constexpr int ORDER_MAX_BINS = 12000;   // bins (M-blocks + 1) that fit the block's shared memory
__global__ void __launch_bounds__(1024) layout_order_kernel(int T, int kp, LayoutView lv) {
  extern __shared__ int bins[];
  __shared__ int carry_s;
  __shared__ int warp_sums[32];
  const int nb = lv.meta[0] + 1;
  if (nb > ORDER_MAX_BINS) {   // beyond the shared-memory histogram: token order
    for (int t = threadIdx.x; t < T; t += blockDim.x) lv.combine_order[t] = t;
    return;
  }
  for (int i = threadIdx.x; i < nb; i += blockDim.x) bins[i] = 0;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  auto key_of = [&](int t) {   // tok_last[t] = 1 + the token's largest padded row (0: no row), from the rank kernel
    const int last = lv.tok_last[t];
    return last == 0 ? 0 : (last - 1) / BLOCK_M + 1;
  };
  for (int t = threadIdx.x; t < T; t += blockDim.x) atomicAdd(&bins[key_of(t)], 1);
  __syncthreads();
  // exclusive scan of the bins, 1024 at a time
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int base = 0; base < nb; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const int v = i < nb ? bins[i] : 0;
    int incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      int o = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += o;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = warp_sums[lane], wi = w;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        int o = __shfl_up_sync(0xffffffffu, wi, off);
        if (lane >= off) wi += o;
      }
      warp_sums[lane] = wi - w;
    }
    __syncthreads();
    const int excl = carry_s + warp_sums[warp] + incl - v;
    if (i < nb) bins[i] = excl;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry_s = excl + v;
    __syncthreads();
  }
  for (int t = threadIdx.x; t < T; t += blockDim.x) lv.combine_order[atomicAdd(&bins[key_of(t)], 1)] = t;
}

cudaError_t launch_layout_order(const Dims& dm, const LayoutView& lv, int cap_mblocks, cudaStream_t s, int* launches) {
  int nb = cap_mblocks + 2;
  if (nb > ORDER_MAX_BINS) nb = ORDER_MAX_BINS;
  layout_order_kernel<<<1, 1024, sizeof(int) * (size_t)nb, s>>>(dm.T, dm.kp(), lv);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_layout(const int* topk_ids, const Dims& dm, const LayoutView& lv, DevStatus* status,
                          cudaStream_t s, int* launches) {
  const int n = dm.slots(), Ep = dm.Ep();
  const int nblk = n > 0 ? (n + LAYOUT_CHUNK - 1) / LAYOUT_CHUNK : 1;
  const size_t sm_hist = sizeof(int) * (size_t)LAYOUT_WARPS * Ep;
  layout_hist_kernel<<<nblk, LAYOUT_THREADS, sm_hist, s>>>(topk_ids, n, dm.k, dm.kp(), dm.E, Ep, lv.blk_hist, lv.tok_last);
  layout_scan_kernel<<<1, 1024, sizeof(int) * (size_t)(4 * Ep + 3), s>>>(nblk, Ep, lv);
  layout_rank_kernel<<<nblk, LAYOUT_THREADS, sm_hist, s>>>(topk_ids, n, dm.k, dm.kp(), dm.E, Ep, lv, status);
  *launches += 3;
  return cudaGetLastError();
}

}  // namespace moe

// ------------------------------------------------------------------------------------------
// Dispatch layout without any allocation.
//
// Some callers may not allocate device memory at the point where they need the layout: code
// running inside a framework's memory-planned region or a real-time serving loop where cudaMalloc
// (which synchronises the device and may fail under fragmentation) is forbidden, plugins that are
// handed only their input and output buffers, and callers that never created a moe_ctx.  For them
// the scratch of the layout kernels (per-block histograms, M-block table, padded-row indices,
// status word) lives in the fixed-size array below, which every GPU that loads this library holds
// until the process exits (about 1.6 MB).  All calls share it.
// ------------------------------------------------------------------------------------------
#include <mutex>

#include "../../include/moe_b200.h"

namespace {

constexpr int NA_MAX_SLOTS = MOE_NOALLOC_MAX_SLOTS;             // T * (k + S)
constexpr int NA_MAX_EP = MOE_NOALLOC_MAX_EXPERTS;              // E + S
constexpr int NA_MAX_BLOCKS = NA_MAX_SLOTS / moe::LAYOUT_CHUNK; // blocks of the layout kernels
constexpr int NA_MAX_HIST = 1 << 17;                            // ints of per-block histograms (nblk * (E+S))
constexpr int NA_MAX_MBLK = (NA_MAX_SLOTS + NA_MAX_EP * (moe::BLOCK_M - 1)) / moe::BLOCK_M + 2;

struct NoAllocScratch {
  moe::DevStatus status;
  int meta[8];
  int pad_off[NA_MAX_EP + 1];
  int mb_start[NA_MAX_EP + 1];
  int mblk_expert[NA_MAX_MBLK];
  int pair_start[NA_MAX_EP + 1];
  int pblk_expert[NA_MAX_MBLK];
  int work_start[NA_MAX_EP + 1];
  int wblk_expert[NA_MAX_MBLK];
  int blk_hist[NA_MAX_HIST];
  int prow_of[NA_MAX_SLOTS];
};

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

constexpr int NA_MAX_DEVICES = 64;
std::mutex g_na_mutex;
NoAllocScratch* g_na_ptr[NA_MAX_DEVICES] = {};

}  // namespace

extern "C" int moe_layout_noalloc(const int32_t* topk_ids, int32_t T, int32_t E, int32_t k, int32_t n_shared,
                                  int32_t* counts, int32_t* offsets, int32_t* row_of, int32_t* src_of,
                                  int32_t* status2, void* stream) {
  if (!topk_ids || !counts || !offsets || !row_of || !src_of) return MOE_ERR_INVALID_ARG;
  if (T < 1 || E < 1 || E > 1024 || k < 1 || k > E || n_shared < 0) return MOE_ERR_INVALID_ARG;
  const long slots = (long)T * (k + n_shared);
  const int Ep = E + n_shared;
  const long nblk = (slots + moe::LAYOUT_CHUNK - 1) / moe::LAYOUT_CHUNK;
  if (slots > NA_MAX_SLOTS || Ep > NA_MAX_EP || nblk > NA_MAX_BLOCKS || nblk * Ep > NA_MAX_HIST)
    return MOE_ERR_TOO_LARGE;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES) return MOE_ERR_NO_DEVICE;
  NoAllocScratch* sc = nullptr;
  {
    // first call on this device: resolve the device address of the static array (device `dev` is current)
    std::lock_guard<std::mutex> lock(g_na_mutex);
    if (!g_na_ptr[dev]) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
      }
      g_na_ptr[dev] = static_cast<NoAllocScratch*>(p);
    }
    sc = g_na_ptr[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the array keeps the previous call's contents: the status word must start at zero
  if (cudaMemsetAsync(&sc->status, 0, sizeof(moe::DevStatus), st) != cudaSuccess) return MOE_ERR_CUDA;
  moe::Dims dm{T, 8, E, k, n_shared, 8};
  moe::LayoutView lv{};   // (fields not set below stay NULL: no combine order here)
  lv.counts = counts;
  lv.offsets = offsets;
  lv.row_of = row_of;
  lv.src_of = src_of;
  lv.prow_of = sc->prow_of;
  lv.pad_off = sc->pad_off;
  lv.mb_start = sc->mb_start;
  lv.mblk_expert = sc->mblk_expert;
  lv.pair_start = sc->pair_start;
  lv.pblk_expert = sc->pblk_expert;
  lv.work_start = sc->work_start;
  lv.wblk_expert = sc->wblk_expert;
  lv.meta = sc->meta;
  lv.blk_hist = sc->blk_hist;
  int launches = 0;
  if (moe::launch_layout(topk_ids, dm, lv, &sc->status, st, &launches) != cudaSuccess) return MOE_ERR_CUDA;
  if (status2 &&
      cudaMemcpyAsync(status2, &sc->status, 2 * sizeof(int), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return MOE_ERR_CUDA;
  return MOE_OK;
}
