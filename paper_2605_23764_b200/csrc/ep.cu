// Expert parallelism over peer memory (Section 4.1: put_mem_signal -- a remote write followed by an update of a
// completion counter on the destination -- and the decomposition of the Dispatch / Combine AllToAll into such tasks;
// Section 4.5: rank-aware task reordering).  Data moves with plain 16-byte stores into the destination rank's buffer
// (a peer mapping when the rank is another GPU), completion is a system-scope release-increment of a counter in the
// destination's memory, and the destination's consumers poll their own counters.  Nothing here loads from a peer
// and nothing uses a multicast.  With one GPU all ranks' buffers live on it and one cooperative launch plays every
// rank, producers and consumers alike.
#include <vector>

#include "../../include/moe_b200.h"
#include "moe_internal.h"

namespace moe {

constexpr int EP_THREADS = 256, EP_WARPS = EP_THREADS / 32;

__device__ __forceinline__ uint4 ep_ld_nc(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
// data that another SM, or another GPU, wrote into this GPU's memory during this launch: read at L2
__device__ __forceinline__ uint4 ep_ld_cg(const void* p) {
  uint4 v;
  asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
// L2 policies: a token row is read once per routed copy (k times, at different moments) while k times as many bytes
// stream out, so the source rows ask to stay in L2 and the stores ask to leave it first.
__device__ __forceinline__ uint64_t ep_policy_keep() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t ep_policy_stream() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint4 ep_ld_hint(const void* p, uint64_t policy) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p), "l"(policy));
  return v;
}
__device__ __forceinline__ void ep_st_hint(void* p, uint4 v, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1,%2,%3,%4}, %5;" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w),
               "l"(policy)
               : "memory");
}
// The put half of put_mem_signal for one row: a warp copies nvec 16-byte vectors, eight loads in flight per lane.
// KEEP_SRC: the source row will be read again soon (Dispatch: the token's other copies).
template <bool KEEP_SRC>
__device__ __forceinline__ void ep_put_row(uint4* dst, const uint4* src, int nvec, int lane) {
  constexpr int U = 8;
  const uint64_t keep = ep_policy_keep(), stream = ep_policy_stream();
  for (int v0 = lane; v0 < nvec; v0 += 32 * U) {
    uint4 t[U];
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (v0 + 32 * u < nvec) t[u] = KEEP_SRC ? ep_ld_hint(src + v0 + 32 * u, keep) : ep_ld_nc(src + v0 + 32 * u);
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (v0 + 32 * u < nvec) ep_st_hint(dst + v0 + 32 * u, t[u], stream);
  }
}
// The signal half of put_mem_signal: after the caller's stores to the destination (ordered before this by a
// barrier among the storing threads), make them visible system-wide, then add to the destination's counter.
__device__ __forceinline__ void ep_signal(int* counter, int inc) {
  __threadfence_system();
  asm volatile("red.release.sys.global.add.s32 [%0], %1;" ::"l"(counter), "r"(inc) : "memory");
}
// Bounded wait of a consumer on one of ITS OWN counters.
__device__ __forceinline__ bool ep_wait(const int* counter, int threshold, const WaitCtl& wc, int what) {
  uint64_t t0 = 0;
  uint32_t sleep_ns = 64;
  for (uint32_t spin = 0;; ++spin) {
    int v;
    asm volatile("ld.acquire.sys.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= threshold) return true;
    if ((spin & 63u) == 63u) {
      if (*reinterpret_cast<volatile int*>(&wc.status->abort)) return false;
      const uint64_t now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > wc.budget_ns) {
        report(wc.status, /*MOE_ERR_TIMEOUT*/ 2, (SITE_DEP << 24) | (what & 0xFFFFFF));
        return false;
      }
    }
    __nanosleep(sleep_ns);
    if (sleep_ns < 1024) sleep_ns <<= 1;
  }
}

struct EpPeers { moe_ep_peer p[MOE_EP_MAX_RANKS]; };

struct EpDispatchArgs {
  EpPeers peers;
  moe_ep_local locals[MOE_EP_MAX_RANKS];
  int n_local, R, k, d;
  int blocks_per_rank, producers_per_rank;
  DevStatus* status;
  uint64_t budget_ns;
};

// Dispatch.  Producer block: one communication task at a time (rows of one expert bound for one rank), a warp per row.
// Consumer block: the receive buffer of its rank, one 128-row block at a time, as soon as the block's rows have arrived.
__global__ void __launch_bounds__(EP_THREADS, 4) ep_dispatch_kernel(const __grid_constant__ EpDispatchArgs a) {
  const WaitCtl wc{a.status, a.budget_ns};
  const int li = blockIdx.x / a.blocks_per_rank, role = blockIdx.x % a.blocks_per_rank;
  const moe_ep_local& me = a.locals[li];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nvec = a.d >> 3;
  __shared__ int task_s, ok_s;
  if (role < a.producers_per_rank || !me.consumed) {   // without a consumer buffer every block of the rank produces
    while (true) {
      if (threadIdx.x == 0) task_s = atomicAdd(me.ticket, 1);
      __syncthreads();
      const int ti = task_s;
      if (ti >= me.n_tasks) break;
      const moe_ep_task tk = me.tasks[ti];
      // a task list that is not this rank's plan must not steer stores: what can be checked here is
      if ((unsigned)tk.dst_rank >= (unsigned)a.R || tk.nrows < 0 || tk.nrows > MOE_EP_TILE_ROWS || tk.src_row0 < 0 ||
          tk.src_row0 + tk.nrows > me.T * a.k || tk.dst_row0 < 0) {
        if (threadIdx.x == 0) report(a.status, MOE_ERR_BAD_EXPERT_ID, ti);
        break;
      }
      const moe_ep_peer& dst = a.peers.p[tk.dst_rank];
      for (int r = warp; r < tk.nrows; r += EP_WARPS) {
        const int slot = me.src_of[tk.src_row0 + r];          // flat slot t*k+j of this expert-ordered row
        const int token = slot / a.k;
        const uint4* src = reinterpret_cast<const uint4*>(me.x + (size_t)token * a.d);
        uint4* out = reinterpret_cast<uint4*>(dst.recv + (size_t)(tk.dst_row0 + r) * a.d);
        ep_put_row<true>(out, src, nvec, lane);
        if (lane == 0)
          reinterpret_cast<int4*>(dst.recv_meta)[tk.dst_row0 + r] =
              make_int4(me.rank, slot, __float_as_int(me.topk_w[slot]), 0);
      }
      __syncthreads();   // every row of the task is stored: one signal per receive block the task touches
      if (threadIdx.x == 0) {
        const int b0 = tk.dst_row0 / MOE_EP_BLOCK_ROWS, b1 = (tk.dst_row0 + tk.nrows - 1) / MOE_EP_BLOCK_ROWS;
        if (b0 == b1) {
          ep_signal(dst.recv_counters + b0, tk.nrows);
        } else {   // a task is at most 32 rows: it touches at most two blocks
          const int first = (b0 + 1) * MOE_EP_BLOCK_ROWS - tk.dst_row0;
          ep_signal(dst.recv_counters + b0, first);
          ep_signal(dst.recv_counters + b1, tk.nrows - first);
        }
      }
    }
  } else {
    const int ci = role - a.producers_per_rank, nc = a.blocks_per_rank - a.producers_per_rank;
    const moe_ep_peer& mine = a.peers.p[me.rank];
    const int nblk = (me.recv_rows + MOE_EP_BLOCK_ROWS - 1) / MOE_EP_BLOCK_ROWS;
    for (int b = ci; b < nblk; b += nc) {
      const int r0 = b * MOE_EP_BLOCK_ROWS, rows = min(MOE_EP_BLOCK_ROWS, me.recv_rows - r0);
      if (threadIdx.x == 0) ok_s = ep_wait(mine.recv_counters + b, rows, wc, b) ? 1 : 0;
      __syncthreads();
      if (!ok_s) break;
      const uint4* src = reinterpret_cast<const uint4*>(mine.recv + (size_t)r0 * a.d);
      uint4* out = reinterpret_cast<uint4*>(me.consumed + (size_t)r0 * a.d);
      for (int i0 = threadIdx.x; i0 < rows * nvec; i0 += 4 * EP_THREADS) {
        uint4 t[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (i0 + u * EP_THREADS < rows * nvec) t[u] = ep_ld_cg(src + i0 + u * EP_THREADS);
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (i0 + u * EP_THREADS < rows * nvec) out[i0 + u * EP_THREADS] = t[u];
      }
      __syncthreads();
    }
  }
}

struct EpCombineArgs {
  EpPeers peers;
  moe_ep_local_combine locals[MOE_EP_MAX_RANKS];
  int n_local, R, k, d;
  int blocks_per_rank, producers_per_rank;
  DevStatus* status;
  uint64_t budget_ns;
};

// Combine.  Producer block: tiles of 32 rows of the rank's expert outputs, each row returned to ret[slot] of its
// source rank (a warp per row); when the tile's rows are stored, one thread per row signals (the fences of a tile run
// side by side instead of one after the other); the tile list starts at a rank-dependent position so that the
// ranks do not all return to the same source at once.  Consumer block: token blocks of its rank; once every row of a
// block has come back, out[t] = sum over the token's k rows in slot order (fp32).
__global__ void __launch_bounds__(EP_THREADS, 4) ep_combine_kernel(const __grid_constant__ EpCombineArgs a) {
  const WaitCtl wc{a.status, a.budget_ns};
  const int li = blockIdx.x / a.blocks_per_rank, role = blockIdx.x % a.blocks_per_rank;
  const moe_ep_local_combine& me = a.locals[li];
  const moe_ep_peer& mine = a.peers.p[me.rank];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nvec = a.d >> 3;
  __shared__ int task_s, ok_s;
  __shared__ int* sig_s[MOE_EP_TILE_ROWS];
  if (role < a.producers_per_rank) {
    const int ntiles = (me.recv_rows + MOE_EP_TILE_ROWS - 1) / MOE_EP_TILE_ROWS;
    const int rot = ntiles ? (int)(((long long)me.rank * ntiles) / a.R) : 0;
    while (true) {
      if (threadIdx.x == 0) task_s = atomicAdd(me.ticket, 1);
      __syncthreads();
      const int ti = task_s;
      __syncthreads();
      if (ti >= ntiles) break;
      const int tile = (ti + rot) % ntiles;
      const int p0 = tile * MOE_EP_TILE_ROWS, n = min(MOE_EP_TILE_ROWS, me.recv_rows - p0);
      for (int r = warp; r < n; r += EP_WARPS) {
        const int4 m = reinterpret_cast<const int4*>(mine.recv_meta)[p0 + r];   // {source rank, source slot, w, 0}
        if ((unsigned)m.x >= (unsigned)a.R || m.y < 0) {   // not what Dispatch writes: refuse to follow it anywhere
          if (lane == 0) { report(a.status, MOE_ERR_BAD_EXPERT_ID, p0 + r); sig_s[r] = nullptr; }
          continue;
        }
        const moe_ep_peer& dst = a.peers.p[m.x];
        const uint4* src = reinterpret_cast<const uint4*>(me.y + (size_t)(p0 + r) * a.d);
        uint4* out = reinterpret_cast<uint4*>(dst.ret + (size_t)m.y * a.d);
        ep_put_row<false>(out, src, nvec, lane);
        if (lane == 0) sig_s[r] = dst.ret_counters + (m.y / a.k) / MOE_EP_TOKEN_BLOCK;
      }
      __syncthreads();   // every row of the tile is stored: one thread per row makes them visible and signals
      if ((int)threadIdx.x < n && sig_s[threadIdx.x]) ep_signal(sig_s[threadIdx.x], 1);
    }
  } else {
    const int ci = role - a.producers_per_rank, nc = a.blocks_per_rank - a.producers_per_rank;
    const int nblk = (me.T + MOE_EP_TOKEN_BLOCK - 1) / MOE_EP_TOKEN_BLOCK;
    for (int b = ci; b < nblk; b += nc) {
      const int t0 = b * MOE_EP_TOKEN_BLOCK, nt = min(MOE_EP_TOKEN_BLOCK, me.T - t0);
      if (threadIdx.x == 0) ok_s = ep_wait(mine.ret_counters + b, nt * a.k, wc, b) ? 1 : 0;
      __syncthreads();
      if (!ok_s) break;
      for (int t = t0 + warp; t < t0 + nt; t += EP_WARPS) {
        for (int v = lane; v < nvec; v += 32) {
          float acc[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) acc[q] = 0.f;
          for (int j0 = 0; j0 < a.k; j0 += 8) {   // eight of the token's rows in flight; summed in slot order
            uint4 rr[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
              if (j0 + u < a.k) rr[u] = ep_ld_cg(reinterpret_cast<const uint4*>(mine.ret + ((size_t)t * a.k + j0 + u) * a.d) + v);
#pragma unroll
            for (int u = 0; u < 8; ++u)
              if (j0 + u < a.k) {
                const uint4 r = rr[u];
                acc[0] += bf16lo(r.x); acc[1] += bf16hi(r.x);
                acc[2] += bf16lo(r.y); acc[3] += bf16hi(r.y);
                acc[4] += bf16lo(r.z); acc[5] += bf16hi(r.z);
                acc[6] += bf16lo(r.w); acc[7] += bf16hi(r.w);
              }
          }
          uint4 o;
          o.x = pack_bf16x2(acc[0], acc[1]); o.y = pack_bf16x2(acc[2], acc[3]);
          o.z = pack_bf16x2(acc[4], acc[5]); o.w = pack_bf16x2(acc[6], acc[7]);
          reinterpret_cast<uint4*>(me.out + (size_t)t * a.d)[v] = o;
        }
      }
      __syncthreads();
    }
  }
}

// resident blocks a cooperative launch may use, split among the local ranks; three of four blocks produce
static int ep_grid(const void* kernel, int n_local, int* blocks_per_rank, int* producers_per_rank) {
  int dev = 0, sms = 0, per_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOE_ERR_NO_DEVICE;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, EP_THREADS, 0) != cudaSuccess || per_sm < 1)
    return MOE_ERR_CUDA;
  int total = sms * (per_sm < 4 ? per_sm : 4);
  int bpr = total / n_local;
  if (bpr < 2) return MOE_ERR_TOO_LARGE;
  *blocks_per_rank = bpr;
  *producers_per_rank = bpr - (bpr + 3) / 4;
  return MOE_OK;
}

}  // namespace moe

using namespace moe;

extern "C" {

int moe_ep_plan(const int32_t* counts, int32_t R, int32_t E, int32_t rank, moe_ep_task* tasks, int32_t task_cap,
                int32_t* n_tasks, int32_t* recv_rows, int32_t* recv_expert_offsets) {
  if (!counts || !n_tasks || R < 1 || R > MOE_EP_MAX_RANKS || E < R || E % R || rank < 0 || rank >= R || task_cap < 0)
    return MOE_ERR_INVALID_ARG;
  const int El = E / R;
  for (int i = 0; i < R * E; ++i) if (counts[i] < 0) return MOE_ERR_INVALID_ARG;
  // first receive row of (expert e, source s) on e's rank: experts in order, inside an expert the sources in rank order
  std::vector<int> seg_start((size_t)E * R), rows(R, 0);
  for (int q = 0; q < R; ++q) {
    int at = 0;
    for (int e = q * El; e < (q + 1) * El; ++e)
      for (int s = 0; s < R; ++s) { seg_start[(size_t)e * R + s] = at; at += counts[(size_t)s * E + e]; }
    rows[q] = at;
  }
  if (recv_rows) for (int q = 0; q < R; ++q) recv_rows[q] = rows[q];
  if (recv_expert_offsets) {
    for (int i = 0; i < El; ++i) recv_expert_offsets[i] = seg_start[(size_t)(rank * El + i) * R];
    recv_expert_offsets[El] = rows[rank];
  }
  // this rank's expert-ordered rows: expert e starts at the prefix sum of its own counts
  std::vector<int> local_off(E + 1, 0);
  for (int e = 0; e < E; ++e) local_off[e + 1] = local_off[e] + counts[(size_t)rank * E + e];
  int n = 0;
  for (int di = 0; di < R; ++di) {
    const int q = (rank + 1 + di) % R;   // rank-rotated destination order: every rank starts with a different peer
    for (int e = q * El; e < (q + 1) * El; ++e) {
      const int cnt = counts[(size_t)rank * E + e];
      for (int r0 = 0; r0 < cnt; r0 += MOE_EP_TILE_ROWS) {
        if (n < task_cap && tasks) {
          const int nr = cnt - r0 < MOE_EP_TILE_ROWS ? cnt - r0 : MOE_EP_TILE_ROWS;
          tasks[n] = moe_ep_task{e, local_off[e] + r0, nr, q, seg_start[(size_t)e * R + rank] + r0};
        }
        ++n;
      }
    }
  }
  *n_tasks = n;
  return (n > task_cap || (n && !tasks)) ? MOE_ERR_WORKSPACE : MOE_OK;
}

static int ep_check_peers(const moe_ep_peer* peers, int R) {
  for (int q = 0; q < R; ++q) {
    const uintptr_t all = reinterpret_cast<uintptr_t>(peers[q].recv) | reinterpret_cast<uintptr_t>(peers[q].recv_meta) |
                          reinterpret_cast<uintptr_t>(peers[q].ret);
    if (!peers[q].recv_counters || !peers[q].ret_counters || (all & 15)) return MOE_ERR_INVALID_ARG;
  }
  return MOE_OK;
}

int moe_ep_dispatch(const moe_ep_peer* peers, const moe_ep_local* locals, int32_t n_local, int32_t R, int32_t k, int32_t d,
                    int32_t* status, void* stream) {
  if (!peers || !locals || !status || n_local < 1 || n_local > R || R < 1 || R > MOE_EP_MAX_RANKS || k < 1 || d < 8 || d % 8)
    return MOE_ERR_INVALID_ARG;
  if (ep_check_peers(peers, R)) return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int major = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOE_ERR_NO_DEVICE;
  cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (major != 10) return MOE_ERR_NO_DEVICE;
  EpDispatchArgs a;
  memset(&a, 0, sizeof a);
  for (int q = 0; q < R; ++q) a.peers.p[q] = peers[q];
  for (int i = 0; i < n_local; ++i) {
    const moe_ep_local& l = locals[i];
    if (l.rank < 0 || l.rank >= R || l.T < 0 || l.n_tasks < 0 || l.recv_rows < 0 || !l.ticket || (l.n_tasks && !l.tasks) ||
        (l.T && (!l.x || !l.topk_w || !l.src_of)) || (l.recv_rows && (!peers[l.rank].recv || !peers[l.rank].recv_meta)))
      return MOE_ERR_INVALID_ARG;
    if (cudaMemsetAsync(l.ticket, 0, 2 * sizeof(int), st) != cudaSuccess) return MOE_ERR_CUDA;
    const int nblk = (l.recv_rows + MOE_EP_BLOCK_ROWS - 1) / MOE_EP_BLOCK_ROWS;
    if (nblk && cudaMemsetAsync(peers[l.rank].recv_counters, 0, sizeof(int) * (size_t)nblk, st) != cudaSuccess) return MOE_ERR_CUDA;
  }
  if (cudaMemsetAsync(status, 0, 4 * sizeof(int), st) != cudaSuccess) return MOE_ERR_CUDA;
  for (int i = 0; i < n_local; ++i) a.locals[i] = locals[i];
  a.n_local = n_local; a.R = R; a.k = k; a.d = d;
  a.status = reinterpret_cast<DevStatus*>(status);
  a.budget_ns = 2000ull * 1000 * 1000;
  const void* fn = reinterpret_cast<const void*>(ep_dispatch_kernel);
  int rc = ep_grid(fn, n_local, &a.blocks_per_rank, &a.producers_per_rank);
  if (rc) return rc;
  void* params[] = {&a};
  // cooperative: consumer blocks wait for producer blocks of the same launch
  cudaError_t e = study_plain_launch().load()   // profiling aid, see moe_debug_set_plain_launch(NULL, ..)
                      ? cudaLaunchKernel(fn, dim3(a.blocks_per_rank * n_local), dim3(EP_THREADS), params, 0, st)
                      : cudaLaunchCooperativeKernel(fn, dim3(a.blocks_per_rank * n_local), dim3(EP_THREADS), params, 0, st);
  return e == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int moe_ep_combine(const moe_ep_peer* peers, const moe_ep_local_combine* locals, int32_t n_local, int32_t R, int32_t k,
                   int32_t d, int32_t* status, void* stream) {
  if (!peers || !locals || !status || n_local < 1 || n_local > R || R < 1 || R > MOE_EP_MAX_RANKS || k < 1 || d < 8 || d % 8)
    return MOE_ERR_INVALID_ARG;
  if (ep_check_peers(peers, R)) return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int major = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOE_ERR_NO_DEVICE;
  cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (major != 10) return MOE_ERR_NO_DEVICE;
  EpCombineArgs a;
  memset(&a, 0, sizeof a);
  for (int q = 0; q < R; ++q) a.peers.p[q] = peers[q];
  for (int i = 0; i < n_local; ++i) {
    const moe_ep_local_combine& l = locals[i];
    if (l.rank < 0 || l.rank >= R || l.T < 0 || l.recv_rows < 0 || !l.ticket || (l.recv_rows && (!l.y || !peers[l.rank].recv_meta)) ||
        (l.T && (!l.out || !peers[l.rank].ret)))
      return MOE_ERR_INVALID_ARG;
    if (cudaMemsetAsync(l.ticket, 0, 2 * sizeof(int), st) != cudaSuccess) return MOE_ERR_CUDA;
    const int nblk = (l.T + MOE_EP_TOKEN_BLOCK - 1) / MOE_EP_TOKEN_BLOCK;
    if (nblk && cudaMemsetAsync(peers[l.rank].ret_counters, 0, sizeof(int) * (size_t)nblk, st) != cudaSuccess) return MOE_ERR_CUDA;
  }
  if (cudaMemsetAsync(status, 0, 4 * sizeof(int), st) != cudaSuccess) return MOE_ERR_CUDA;
  for (int i = 0; i < n_local; ++i) a.locals[i] = locals[i];
  a.n_local = n_local; a.R = R; a.k = k; a.d = d;
  a.status = reinterpret_cast<DevStatus*>(status);
  a.budget_ns = 2000ull * 1000 * 1000;
  const void* fn = reinterpret_cast<const void*>(ep_combine_kernel);
  int rc = ep_grid(fn, n_local, &a.blocks_per_rank, &a.producers_per_rank);
  if (rc) return rc;
  void* params[] = {&a};
  cudaError_t e = study_plain_launch().load()
                      ? cudaLaunchKernel(fn, dim3(a.blocks_per_rank * n_local), dim3(EP_THREADS), params, 0, st)
                      : cudaLaunchCooperativeKernel(fn, dim3(a.blocks_per_rank * n_local), dim3(EP_THREADS), params, 0, st);
  return e == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

}  // extern "C"
