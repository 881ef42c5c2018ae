// Permute-gather (Dispatch / backward Dispatch on one GPU), combine (Combine / backward Combine)
// and the small reduction that finishes the routing-weight gradient.  All three are pure
// HBM-bandwidth work: 16-byte vector accesses, one row handled by one block at a time.
#include <stdlib.h>

#include "launch_pairs.cuh"
#include "moe_internal.h"

namespace moe {

constexpr int PERM_THREADS = 128;

__device__ __forceinline__ uint4 ld_nc_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// dst[p][:] = src[token(p)][:] for every padded row p < R_pad; padding rows are zero-filled so
// that reductions over an expert's rows (weight gradients) may run over whole M-blocks.
__global__ void __launch_bounds__(PERM_THREADS) gather_rows_kernel(const uint16_t* __restrict__ src,
                                                                    const float* __restrict__ topk_w, int d, int k,
                                                                    int kp, LayoutView lv,
                                                                    uint16_t* __restrict__ dst,
                                                                    float* __restrict__ prow_w) {
  const int r_pad = lv.meta[1];
  const int nvec = d >> 3;
  for (int p = blockIdx.x; p < r_pad; p += gridDim.x) {
    const int e = lv.mblk_expert[p / BLOCK_M];
    const int local = p - lv.pad_off[e];
    const bool valid = local < lv.counts[e];
    uint4* out = reinterpret_cast<uint4*>(dst + (size_t)p * d);
    if (valid) {
      const int slot = lv.src_of[lv.offsets[e] + local];
      const int t = slot / kp, j = slot - t * kp;
      const uint4* in = reinterpret_cast<const uint4*>(src + (size_t)t * d);
      for (int v = threadIdx.x; v < nvec; v += PERM_THREADS) out[v] = ld_nc_v4(in + v);
      if (prow_w && threadIdx.x == 0) prow_w[p] = j < k ? topk_w[(size_t)t * k + j] : 1.0f;
    } else {
      for (int v = threadIdx.x; v < nvec; v += PERM_THREADS) out[v] = make_uint4(0, 0, 0, 0);
      if (prow_w && threadIdx.x == 0) prow_w[p] = 0.0f;
    }
  }
}

// Short rows (up to 4 KB): one warp per row, so a block has four rows' index chains in flight.
__global__ void __launch_bounds__(PERM_THREADS) gather_rows_warp_kernel(const uint16_t* __restrict__ src,
                                                                         const float* __restrict__ topk_w, int d, int k,
                                                                         int kp, LayoutView lv,
                                                                         uint16_t* __restrict__ dst,
                                                                         float* __restrict__ prow_w) {
  const int r_pad = lv.meta[1];
  const int nvec = d >> 3;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int WPB = PERM_THREADS / 32;
  for (int p = blockIdx.x * WPB + warp; p < r_pad; p += gridDim.x * WPB) {
    const int e = lv.mblk_expert[p / BLOCK_M];
    const int local = p - lv.pad_off[e];
    const bool valid = local < lv.counts[e];
    uint4* out = reinterpret_cast<uint4*>(dst + (size_t)p * d);
    if (valid) {
      const int slot = lv.src_of[lv.offsets[e] + local];
      const int t = slot / kp, j = slot - t * kp;
      const uint4* in = reinterpret_cast<const uint4*>(src + (size_t)t * d);
      for (int v = lane; v < nvec; v += 32) out[v] = ld_nc_v4(in + v);
      if (prow_w && lane == 0) prow_w[p] = j < k ? topk_w[(size_t)t * k + j] : 1.0f;
    } else {
      for (int v = lane; v < nvec; v += 32) out[v] = make_uint4(0, 0, 0, 0);
      if (prow_w && lane == 0) prow_w[p] = 0.0f;
    }
  }
}

// The same gather with bulk copies: one warp per SM, each of up to eight lanes runs its own
// two-slot pipeline (row i+1 arrives in one shared-memory slot while row i leaves from the other):
// whole rows move as single global -> shared and shared -> global bulk copies, up to 200 KB in
// flight per SM, and no thread touches the data.  Padding rows leave from a zeroed slot.
constexpr int GB_MAX_LANES = 8;
constexpr int GB_SMEM_BUDGET = 216 * 1024;

__global__ void __launch_bounds__(32) gather_rows_bulk_kernel(const uint16_t* __restrict__ src,
                                                              const float* __restrict__ topk_w, int d, int k, int kp,
                                                              LayoutView lv, uint16_t* __restrict__ dst,
                                                              float* __restrict__ prow_w, int lanes, DevStatus* status,
                                                              uint64_t budget_ns) {
  extern __shared__ __align__(128) uint8_t gsm[];
  __shared__ uint64_t full[2 * GB_MAX_LANES];
  const int lane = threadIdx.x;
  const uint32_t row_bytes = (uint32_t)d * 2;
  uint8_t* zero_row = gsm;                                   // [row_bytes]
  uint8_t* slots = gsm + row_bytes;                          // [lanes][2][row_bytes]
  for (uint32_t i = lane; i < row_bytes / 16; i += 32) reinterpret_cast<uint4*>(zero_row)[i] = make_uint4(0, 0, 0, 0);
  if (lane < 2 * GB_MAX_LANES) mbar_init(&full[lane], 1);
  mbar_fence_init();
  fence_proxy_async();
  __syncwarp();
  if (lane >= lanes) return;
  const WaitCtl wc{status, budget_ns};
  const int r_pad = lv.meta[1];
  const int stride = gridDim.x * lanes;
  uint8_t* my = slots + (size_t)lane * 2 * row_bytes;
  // row -> source row (or -1 for a padding row); also writes the row's routing weight
  auto source_of = [&](int p) -> long {
    const int e = lv.mblk_expert[p / BLOCK_M];
    const int local = p - lv.pad_off[e];
    if (local >= lv.counts[e]) {
      if (prow_w) prow_w[p] = 0.0f;
      return -1;
    }
    const int slot = lv.src_of[lv.offsets[e] + local];
    const int t = slot / kp, j = slot - t * kp;
    if (prow_w) prow_w[p] = j < k ? topk_w[(size_t)t * k + j] : 1.0f;
    return t;
  };
  auto load = [&](long t, int b) {
    mbar_expect_tx(&full[2 * lane + b], row_bytes);
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(my + (size_t)b * row_bytes)), "l"(src + (size_t)t * d), "r"(row_bytes),
                   "r"(smem_u32(&full[2 * lane + b]))
                 : "memory");
  };
  int p = blockIdx.x * lanes + lane;
  uint32_t n = 0, ph[2] = {0, 0};
  long t_cur = p < r_pad ? source_of(p) : -1;
  if (p < r_pad && t_cur >= 0) load(t_cur, 0);
  for (; p < r_pad; p += stride, ++n) {
    const int b = n & 1;
    const int pn = p + stride;
    const long t_next = pn < r_pad ? source_of(pn) : -1;
    // the other slot is free once the previous row's store has read it
    tma_store_wait_read();
    if (pn < r_pad && t_next >= 0) load(t_next, b ^ 1);
    const uint8_t* from = zero_row;
    if (t_cur >= 0) {
      if (!mbar_wait(&full[2 * lane + b], ph[b], wc, SITE_FULL, p)) break;
      ph[b] ^= 1;
      from = my + (size_t)b * row_bytes;
    }
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst + (size_t)p * d), "r"(smem_u32(from)), "r"(row_bytes)
                 : "memory");
    tma_store_commit();
    t_cur = t_next;
  }
  tma_store_wait_all();
}

cudaError_t launch_gather(const uint16_t* src, const float* topk_w, const Dims& dm, const LayoutView& lv,
                          uint16_t* dst, float* prow_w, int rows_cap, cudaStream_t s, int* launches,
                          DevStatus* status, uint64_t budget_ns) {
  ++*launches;
  const size_t row_bytes = (size_t)dm.d * 2;
  int lanes = (int)((GB_SMEM_BUDGET - row_bytes) / (2 * row_bytes));
  if (lanes > GB_MAX_LANES) lanes = GB_MAX_LANES;
  // rows of 8 KB and more: below that the per-row latency of the two-slot pipelines outweighs the gain
  if (status && lanes >= 2 && row_bytes >= 8192 && row_bytes % 16 == 0 && ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15) == 0) {
    const size_t smem = row_bytes * (1 + 2 * (size_t)lanes);
    int sms = 148;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    {   // the opt-in shared-memory size is a per-device attribute of the kernel: remember it per device, under a lock
      static std::mutex mu;
      static size_t attr_bytes[MAX_DEVICES] = {};
      std::lock_guard<std::mutex> lock(mu);
      if (smem > attr_bytes[dev]) {
        cudaError_t e = cudaFuncSetAttribute(gather_rows_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_bytes[dev] = smem;
      }
    }
    gather_rows_bulk_kernel<<<sms, 32, smem, s>>>(src, topk_w, dm.d, dm.k, dm.kp(), lv, dst, prow_w, lanes, status,
                                                  budget_ns);
    return cudaGetLastError();
  }
  int grid = rows_cap < 148 * 16 ? rows_cap : 148 * 16;
  if (grid < 1) grid = 1;
  if (row_bytes <= 4096)
    gather_rows_warp_kernel<<<grid, PERM_THREADS, 0, s>>>(src, topk_w, dm.d, dm.k, dm.kp(), lv, dst, prow_w);
  else
    gather_rows_kernel<<<grid, PERM_THREADS, 0, s>>>(src, topk_w, dm.d, dm.k, dm.kp(), lv, dst, prow_w);
  return cudaGetLastError();
}

// out[t][:] = sum_j rows[prow_of[t*kp+j]][:], j ascending, fp32 accumulation, one bf16 rounding.
// Rows already carry their routing weight (it is applied where the activations are produced).
__global__ void __launch_bounds__(PERM_THREADS) combine_rows_kernel(const uint16_t* __restrict__ rows, int t0, int t1,
                                                                     int d, int kp, const int* __restrict__ prow_of,
                                                                     uint16_t* __restrict__ out) {
  const int nvec = d >> 3;
  for (int t = t0 + blockIdx.x; t < t1; t += gridDim.x) {
    for (int v = threadIdx.x; v < nvec; v += PERM_THREADS) {
      float acc[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) acc[q] = 0.f;
      for (int j = 0; j < kp; ++j) {
        int p = prow_of[(size_t)t * kp + j];
        if (p < 0) continue;
        uint4 r = ld_nc_v4(reinterpret_cast<const uint4*>(rows + (size_t)p * d) + v);
        acc[0] += bf16lo(r.x); acc[1] += bf16hi(r.x);
        acc[2] += bf16lo(r.y); acc[3] += bf16hi(r.y);
        acc[4] += bf16lo(r.z); acc[5] += bf16hi(r.z);
        acc[6] += bf16lo(r.w); acc[7] += bf16hi(r.w);
      }
      uint4 o;
      o.x = pack_bf16x2(acc[0], acc[1]);
      o.y = pack_bf16x2(acc[2], acc[3]);
      o.z = pack_bf16x2(acc[4], acc[5]);
      o.w = pack_bf16x2(acc[6], acc[7]);
      reinterpret_cast<uint4*>(out + (size_t)t * d)[v] = o;
    }
  }
}

cudaError_t launch_combine(const uint16_t* rows, const Dims& dm, const LayoutView& lv, uint16_t* out,
                           cudaStream_t s, int* launches, int t0, int t1) {
  if (t1 < 0) t1 = dm.T;
  const int n = t1 - t0;
  int grid = n < 148 * 16 ? n : 148 * 16;
  if (grid < 1) grid = 1;
  combine_rows_kernel<<<grid, PERM_THREADS, 0, s>>>(rows, t0, t1, dm.d, dm.kp(), lv.prow_of, out);
  ++*launches;
  return cudaGetLastError();
}

// d_topk_w[t][j] = sum over the act_grad column tiles of their per-row partial dot products,
// in tile order (deterministic).
__global__ void dw_reduce_kernel(const float* __restrict__ partial, int nparts, int T, int k, int kp,
                                 const int* __restrict__ prow_of, float* __restrict__ d_topk_w) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= T * k) return;
  int t = i / k, j = i - t * k;
  int p = prow_of[(size_t)t * kp + j];
  float s = 0.f;
  if (p >= 0)
    for (int q = 0; q < nparts; ++q) s += partial[(size_t)p * nparts + q];
  d_topk_w[i] = s;
}

cudaError_t launch_dw_reduce(const float* partial, int nparts, const Dims& dm, const LayoutView& lv,
                             float* d_topk_w, cudaStream_t s, int* launches) {
  int n = dm.T * dm.k;
  if (n == 0) return cudaSuccess;
  dw_reduce_kernel<<<(n + 255) / 256, 256, 0, s>>>(partial, nparts, dm.T, dm.k, dm.kp(), lv.prow_of, d_topk_w);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace moe
