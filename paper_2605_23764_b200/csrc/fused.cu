// The single persistent, dependency-driven launch of the forward (and of the backward) layer.
//
// One cooperative grid of one CTA per SM runs the whole operator chain.  Per CTA:
//   warp 14     scheduler: takes the next ticket of the matrix queue, decodes the tile, polls the
//               tile's dependent counters, then publishes it to the CTA's other roles;
//   warp 0      loader: streams the published tile's operands through TMA (one box per lane);
//   warp 1      tcgen05.mma issuer (and TMEM owner);
//   warps 2-5   epilogue: TMEM -> fused element-wise math -> TMA store, then the tile's trigger
//               counter once the stores are complete;
//   warps 6-13  vector workers: take tickets of the vector queue (permute-gather, zero-fill of
//               weight gradients of experts without rows, routing-weight gradient, combine); the
//               matrix-role warps join them when the matrix queue is exhausted.
// This is the paper's unified runtime (Section 4.4) restated for one SM: matrix and vector work
// progress concurrently inside one launch, ordered only by event counters with static thresholds
// (Section 4.3).  The tile math is the same code the one-launch-per-operator mode runs.
#include <cooperative_groups.h>

#include <vector>

#include "gemm_swap.cuh"
#include "schedule.h"

namespace moe {

// Optional per-CTA wait accounting (diagnostic builds only: -DMOE_STATS).
#ifdef MOE_STATS
#define ST_DECL long long st_t0 = clock64(), st_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}; long long st_mark = st_t0
#define ST_MARK() st_mark = clock64()
#define ST_ADD(i) do { long long _n = clock64(); st_acc[i] += _n - st_mark; st_mark = _n; } while (0)
#define ST_FLUSH(base, n) do { if (fa.stats) { for (int _i = 0; _i < (n); ++_i) fa.stats[blockIdx.x * 32 + (base) + _i] = st_acc[_i]; \
                               fa.stats[blockIdx.x * 32 + (base) + (n)] = clock64() - st_t0; } } while (0)
#else
#define ST_DECL
#define ST_MARK()
#define ST_ADD(i)
#define ST_FLUSH(base, n)
#endif

#ifndef MOE_VEC_WARPS
#define MOE_VEC_WARPS 8
#endif
constexpr int VEC_WARPS = MOE_VEC_WARPS;
constexpr int SCHED_WARP = 6 + VEC_WARPS;         // the last warp
constexpr int TOK_WARP = SCHED_WARP + 1;            // CTA-pair kernel, token-column tiles: TMA producer of the tokens
constexpr int FUSED_THREADS = GEMM_THREADS + 32 * VEC_WARPS + 64;
constexpr int SCHED_AHEAD_KB = 24;                // k-blocks of a ticket left when the next one is fetched
constexpr int RING = 4;                            // published-tile ring depth

struct TileSlot {
  int op, slot, e, row0, n0, m0, nkb, nb;
  int trig_idx;   // counter index to bump per epilogue warp, -1 = none
  int trig_ag;    // also bump the global act_grad counter
  short go_kb;    // k-block at which the loader tells the scheduler to fetch the next ticket (-1: not in this tile)
  short pad;      // CTA-pair kernel: this CTA's half of the tile is idle (no rows / outside the gradient)
  int krows;      // weight gradients: rows of the expert (the reduction length)
                  // token-column tiles (row-space operators): m0 = tokens of the tile, krows = its M-blocks
};

struct __align__(16) FusedShared {
  GemmBarriers bars;
  uint64_t tk_full[RING];
  uint64_t tk_empty[RING];
  uint64_t sched_go;      // loader -> scheduler: fetch the next ticket
  uint64_t vec_ready[2];  // one-shot: the global "all tiles done" conditions the vector tail waits for
  int vec_poller[2];      // which warp polls the global counter on behalf of the CTA
  int pad[2];
  TileSlot ring[RING];
};

constexpr size_t FUSED_SMEM_BYTES = 1024 + (size_t)STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + 4 * OUT_STAGE_BYTES +
                                    sizeof(FusedShared);
static_assert(FUSED_SMEM_BYTES <= 227 * 1024, "shared memory budget");

// ---------------------------------------------------------------- schedule prefix + counter reset
// One block: step_start[i] = tickets before step i (i in [0, Ep+lag]); counters zeroed.
__global__ void __launch_bounds__(1024) build_schedule_kernel(SchedParams sp, LayoutView lv, int* step_start,
                                                              int* ctr, int ctr_count) {
  __shared__ int warp_sums[32];
  __shared__ int carry_s;
  const int n = sp.Ep + sp.lag;
  for (int i = threadIdx.x; i < ctr_count; i += blockDim.x) ctr[i] = 0;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int base = 0; base < n; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const int v = i < n ? step_tiles(sp, i, lv.mb_start) : 0;
    int incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      int o = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += o;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = warp_sums[lane];
      int wi = w;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        int o = __shfl_up_sync(0xffffffffu, wi, off);
        if (lane >= off) wi += o;
      }
      warp_sums[lane] = wi - w;  // exclusive
    }
    __syncthreads();
    const int carry = carry_s;
    const int excl = carry + warp_sums[warp] + incl - v;
    if (i < n) step_start[i] = excl;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry_s = excl + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) step_start[n] = carry_s;
}

// ---------------------------------------------------------------- vector work (one warp per task)
__device__ __forceinline__ uint4 ldg_nc_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void vec_gather(const FusedArgs& fa, int task, int lane) {
  const int mb = task / GATHER_SUB, sub = task - mb * GATHER_SUB;
  const LayoutView& lv = fa.lv;
  const int e = lv.mblk_expert[mb];
  const int cnt = lv.counts[e], pad0 = lv.pad_off[e], off0 = lv.offsets[e];
  const int nvec = fa.d >> 3;
  const int k = fa.sp.k;
  for (int r = 0; r < BLOCK_M / GATHER_SUB; ++r) {
    const int p = mb * BLOCK_M + sub * (BLOCK_M / GATHER_SUB) + r;
    const int local = p - pad0;
    uint4* out = reinterpret_cast<uint4*>(fa.gather_dst + (size_t)p * fa.d);
    if (local < cnt) {
      const int slot = lv.src_of[off0 + local];
      const int t = slot / fa.kp, j = slot - t * fa.kp;
      const uint4* in = reinterpret_cast<const uint4*>(fa.gather_src + (size_t)t * fa.d);
      int v = lane;
      for (; v + 224 < nvec; v += 256) {
        uint4 q[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) q[u] = ldg_nc_v4(in + v + 32 * u);
#pragma unroll
        for (int u = 0; u < 8; ++u) out[v + 32 * u] = q[u];
      }
      for (; v < nvec; v += 32) out[v] = ldg_nc_v4(in + v);
      if (fa.prow_w && lane == 0) fa.prow_w[p] = j < k ? fa.topk_w[(size_t)t * k + j] : 1.0f;
    } else {
      for (int v = lane; v < nvec; v += 32) out[v] = make_uint4(0, 0, 0, 0);
      if (fa.prow_w && lane == 0) fa.prow_w[p] = 0.0f;
    }
  }
}

__device__ __forceinline__ void vec_combine(const FusedArgs& fa, int task, int lane) {
  const int nvec = fa.d >> 3, kp = fa.kp, T = fa.sp.T;
  const int t1 = min(T, (task + 1) * COMBINE_TOKENS);
  for (int t = task * COMBINE_TOKENS; t < t1; ++t) {
    for (int v = lane; v < nvec; v += 32) {
      float acc[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) acc[q] = 0.f;
      for (int j0 = 0; j0 < kp; j0 += 8) {
        uint4 r[8];
        // eight independent row loads in flight; plain (coherent) loads: the rows were written
        // earlier in this same launch
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int j = j0 + u;
          const int p = j < kp ? fa.lv.prow_of[(size_t)t * kp + j] : -1;
          r[u] = p >= 0 ? *(reinterpret_cast<const uint4*>(fa.combine_rows + (size_t)p * fa.d) + v)
                        : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          acc[0] += bf16lo(r[u].x); acc[1] += bf16hi(r[u].x);
          acc[2] += bf16lo(r[u].y); acc[3] += bf16hi(r[u].y);
          acc[4] += bf16lo(r[u].z); acc[5] += bf16hi(r[u].z);
          acc[6] += bf16lo(r[u].w); acc[7] += bf16hi(r[u].w);
        }
      }
      uint4 o;
      o.x = pack_bf16x2(acc[0], acc[1]);
      o.y = pack_bf16x2(acc[2], acc[3]);
      o.z = pack_bf16x2(acc[4], acc[5]);
      o.w = pack_bf16x2(acc[6], acc[7]);
      reinterpret_cast<uint4*>(fa.combine_out + (size_t)t * fa.d)[v] = o;
    }
  }
}

__device__ __forceinline__ void vec_dw(const FusedArgs& fa, int task, int lane) {
  if (!fa.d_topk_w) return;
  const int k = fa.sp.k, n = fa.sp.T * k;
  for (int i = task * DW_SLOTS + lane; i < min(n, (task + 1) * DW_SLOTS); i += 32) {
    const int t = i / k, j = i - t * k;
    const int p = fa.lv.prow_of[(size_t)t * fa.kp + j];
    float s = 0.f;
    if (p >= 0)
      for (int q = 0; q < fa.dw_nparts; ++q) s += fa.dw_partial[(size_t)p * fa.dw_nparts + q];
    fa.d_topk_w[i] = s;
  }
}

__device__ __forceinline__ void vec_zero(const FusedArgs& fa, int task, int lane) {
  const int e = task / ZERO_CHUNKS, ch = task - e * ZERO_CHUNKS;
  if (fa.lv.counts[e] != 0) return;  // only experts without rows: their weight gradients are exact zeros
  uint4* s1 = reinterpret_cast<uint4*>(fa.dW1) + (size_t)e * fa.dW1_slab_vec;
  uint4* s2 = reinterpret_cast<uint4*>(fa.dW2) + (size_t)e * fa.dW2_slab_vec;
  const uint4 z = make_uint4(0, 0, 0, 0);
  for (size_t v = fa.dW1_slab_vec * ch / ZERO_CHUNKS + lane; v < fa.dW1_slab_vec * (ch + 1) / ZERO_CHUNKS; v += 32)
    s1[v] = z;
  for (size_t v = fa.dW2_slab_vec * ch / ZERO_CHUNKS + lane; v < fa.dW2_slab_vec * (ch + 1) / ZERO_CHUNKS; v += 32)
    s2[v] = z;
}

// ---------------------------------------------------------------- matrix-role dispatch on the operator
template <bool BWD>
__device__ __forceinline__ void fused_load_stage(const FusedArgs& fa, const TileSlot& ts, const Tile& tl, int kb,
                                                 uint8_t* sA, uint8_t* sB, uint64_t* bar, int lane) {
  const GemmArgs& g = fa.op[ts.slot];
  if (!BWD) {
    if (ts.op == GEMM_GATE_UP) load_stage_lanes<GEMM_GATE_UP>(g, tl, kb, sA, sB, bar, lane);
    else load_stage_lanes<GEMM_DOWN>(g, tl, kb, sA, sB, bar, lane);
  } else {
    if (ts.op == GEMM_ACT_GRAD) load_stage_lanes<GEMM_ACT_GRAD>(g, tl, kb, sA, sB, bar, lane);
    else if (ts.op == GEMM_GATE_GRAD) load_stage_lanes<GEMM_GATE_GRAD>(g, tl, kb, sA, sB, bar, lane);
    else load_stage_lanes<GEMM_WGRAD>(g, tl, kb, sA, sB, bar, lane);
  }
}
template <bool BWD>
__device__ __forceinline__ void fused_mma(int op, uint32_t d_tmem, uint32_t a_addr, uint32_t b_addr, bool first) {
  if (!BWD) {
    mma_kblock<GEMM_GATE_UP>(d_tmem, a_addr, b_addr, first);  // GATE_UP and DOWN: same operand layouts
  } else {
    if (op == GEMM_WGRAD) mma_kblock<GEMM_WGRAD>(d_tmem, a_addr, b_addr, first);
    else mma_kblock<GEMM_ACT_GRAD>(d_tmem, a_addr, b_addr, first);  // ACT_GRAD and GATE_GRAD alike
  }
}
template <bool BWD>
__device__ __forceinline__ void fused_epilogue(const FusedArgs& fa, const TileSlot& ts, const Tile& tl,
                                               uint32_t tmem_acc, int quad, int lane, Staging& stg) {
  const GemmArgs& g = fa.op[ts.slot];
  if (!BWD) {
    if (ts.op == GEMM_GATE_UP) epilogue_tile<GEMM_GATE_UP>(g, tl, tmem_acc, quad, lane, stg);
    else epilogue_tile<GEMM_DOWN>(g, tl, tmem_acc, quad, lane, stg);
  } else {
    if (ts.op == GEMM_ACT_GRAD) epilogue_tile<GEMM_ACT_GRAD>(g, tl, tmem_acc, quad, lane, stg);
    else if (ts.op == GEMM_GATE_GRAD) epilogue_tile<GEMM_GATE_GRAD>(g, tl, tmem_acc, quad, lane, stg);
    else epilogue_tile<GEMM_WGRAD>(g, tl, tmem_acc, quad, lane, stg);
  }
}

__device__ __forceinline__ Tile slot_tile(const TileSlot& ts) {
  Tile tl;
  tl.e = ts.e; tl.row0 = ts.row0; tl.n0 = ts.n0; tl.m0 = ts.m0; tl.nkb = ts.nkb; tl.nb = ts.nb;
  return tl;
}

// ---------------------------------------------------------------- vector-queue consumer (one warp)
template <bool BWD>
__device__ __forceinline__ void vector_worker_loop(const FusedArgs& fa, uint64_t* vec_ready, int* vec_poller,
                                                   const WaitCtl& wc, int M, int lane) {
  if (!*reinterpret_cast<volatile int*>(&fa.status->abort)) {
    const int vtotal = vec_total(fa.sp, M);
    while (true) {
      int t = 0;
      if (lane == 0) t = atomicAdd(&fa.ctr[CTR_VEC_TICKET], 1);
      t = __shfl_sync(0xffffffffu, t, 0);
      if (t >= vtotal) break;
      const VecTask v = decode_vector_ticket(fa.sp, t, M);
      if (v.dep) {
        // A global completion counter: one warp of the CTA polls it (slowly), the others sleep on a
        // shared-memory barrier -- a thousand warps spinning on one L2 line would slow every load.
        const int kind = v.dep == 2 ? 0 : 1;
        int ok = 1;
        if (lane == 0) {
          if (atomicExch(&vec_poller[kind], 1) == 0) {
            ok = counter_wait(fa.ctr + (kind == 0 ? CTR_DONE : CTR_AG_DONE), v.dep_thr, wc, t, 2000) ? 1 : 0;
            if (ok) mbar_arrive(&vec_ready[kind]);
          } else {
            ok = mbar_wait(&vec_ready[kind], 0, wc, SITE_DEP, t, 4000) ? 1 : 0;
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        __syncwarp();
        if (!ok) break;
      }
      if (v.op == VEC_GATHER) {
        vec_gather(fa, v.idx, lane);
        __syncwarp();
        if (lane == 0) counter_signal(fa.ctr + ctr_gather(v.idx / GATHER_SUB), 1);
      } else if (v.op == VEC_COMBINE) {
        vec_combine(fa, v.idx, lane);
      } else if (BWD && v.op == VEC_DW) {
        vec_dw(fa, v.idx, lane);
      } else if (BWD && v.op == VEC_ZERO) {
        vec_zero(fa, v.idx, lane);
      }
    }
  }

}

// ---------------------------------------------------------------- the kernel
template <bool BWD>
__global__ void __launch_bounds__(FUSED_THREADS, 1) fused_kernel(const __grid_constant__ FusedArgs fa) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = smem + STAGES * A_STAGE_BYTES;
  uint8_t* sOut = smem + STAGES * (A_STAGE_BYTES + B_STAGE_BYTES);
  FusedShared* sh = reinterpret_cast<FusedShared*>(sOut + 4 * OUT_STAGE_BYTES);
  GemmBarriers* bars = &sh->bars;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WaitCtl wc{fa.status, fa.budget_ns};
  const int M = fa.lv.meta[0];

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->tmem_full[s], 1);
      mbar_init(&bars->tmem_empty[s], EPI_WARPS);
    }
    mbar_init(&bars->drain, 1);
    for (int s = 0; s < RING; ++s) {
      mbar_init(&sh->tk_full[s], 1);
      mbar_init(&sh->tk_empty[s], 2 + EPI_WARPS);  // loader, MMA issuer and every epilogue warp release a slot
    }
    mbar_init(&sh->sched_go, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh->vec_ready[s], 1);
      sh->vec_poller[s] = 0;
    }
    mbar_fence_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == SCHED_WARP) {
    // ------------------------------------------------ scheduler: ticket, decode, dependent events
    // It runs ahead of the loader by at most the ring depth inside one ticket, and takes the NEXT
    // ticket only when the loader signals that the current one is about to run out of k-blocks: the
    // atomic, the decode and the counter polls hide behind those last loads, while tiles with
    // adjacent tickets (which share an operand through L2) still start close together in time.
    if (lane == 0) {
      const int total = fa.step_start[fa.sp.Ep + fa.sp.lag];
      uint32_t n = 0, go_n = 0;
      int cursor = 0;  // step of the previous ticket: tickets of one CTA only grow
      bool ok = true;
      ST_DECL;
      while (ok) {
        ST_MARK();
        const int t = atomicAdd(&fa.ctr[CTR_MAT_TICKET], 1);
        TileSlot ts;
        ts.slot = 0; ts.e = 0; ts.row0 = 0; ts.n0 = 0; ts.m0 = 0; ts.nkb = 0; ts.nb = 0;
        ts.trig_idx = -1; ts.trig_ag = 0; ts.go_kb = -1; ts.pad = 0; ts.krows = 0;
        if (t >= total) {
          ts.op = -1;  // end of the queue: tell the other roles
          const int rs = n % RING;
          if (!mbar_wait(&sh->tk_empty[rs], ((n / RING) & 1) ^ 1, wc, SITE_EMPTY, t)) break;
          sh->ring[rs] = ts;
          mbar_arrive(&sh->tk_full[rs]);
          break;
        }
        while (fa.step_start[cursor + 1] <= t) ++cursor;
        const MatTile mt = decode_matrix_ticket_at(fa.sp, t, cursor, fa.step_start, fa.lv.mb_start);
        const GemmArgs& g = fa.op[mt.slot];
        ST_ADD(0);  // ticket + decode
        for (int q = 0; q < mt.dep_count && ok; ++q) {
          const int mbq = mt.dep_first + q;
          const int* c = fa.ctr + (mt.dep_base == 0 ? ctr_gather(mbq) : ctr_act(mbq));
          ok = counter_wait(c, mt.dep_thr, wc, t);
        }
        if (!ok) break;
        ST_ADD(1);  // dependency wait
        ts.op = mt.op; ts.slot = mt.slot; ts.e = mt.e;
        ts.trig_idx = mt.trig_base == 1 ? ctr_act(mt.mb) : (mt.trig_base == 2 ? CTR_DONE : -1);
        ts.trig_ag = mt.trig_also_ag;
        const int nkb = mt.op == GEMM_WGRAD ? (fa.lv.counts[mt.e] + BK - 1) / BK : (g.K + BK - 1) / BK;
        for (int gi = 0; gi < mt.group && ok; ++gi) {
          if (mt.op == GEMM_WGRAD) {
            ts.nb = gi;                       // one 128-row block of the gradient, column tile gi
            ts.m0 = mt.idx * BLOCK_M;
            ts.n0 = gi * BN;
            ts.row0 = fa.lv.mb_start[mt.e] * BLOCK_M;
          } else {
            ts.nb = mt.idx;
            ts.m0 = 0;
            ts.n0 = mt.idx * (mt.op == GEMM_GATE_UP ? BN / 2 : BN);
            ts.row0 = mt.mb * BLOCK_M;
          }
          ts.nkb = nkb;
          ts.krows = mt.op == GEMM_WGRAD ? fa.lv.counts[mt.e] : 0;
          // the k-block of this tile at which SCHED_AHEAD_KB k-blocks of the ticket remain
          const int after = (mt.group - 1 - gi) * nkb;
          ts.go_kb = -1;
          if (after < SCHED_AHEAD_KB && (after + nkb >= SCHED_AHEAD_KB || gi == 0))
            ts.go_kb = max(0, nkb - (SCHED_AHEAD_KB - after));
          const int rs = n % RING;
          if (!mbar_wait(&sh->tk_empty[rs], ((n / RING) & 1) ^ 1, wc, SITE_EMPTY, t)) { ok = false; break; }
          sh->ring[rs] = ts;
          mbar_arrive(&sh->tk_full[rs]);  // release: the slot's contents are visible to the waiters
          ++n;
        }
        ST_ADD(2);  // ring slot waits
        if (!ok || !mbar_wait(&sh->sched_go, go_n & 1, wc, SITE_DEP, t, 200)) break;
        ++go_n;
        ST_ADD(3);  // waiting for the loader's signal (the healthy state)
      }
      ST_FLUSH(0, 4);
    }
  } else if (warp == 0) {
    // ------------------------------------------------ loader: TMA boxes of each k-block, one per lane
    uint32_t it = 0, n = 0;
    bool ok = true;
    while (ok) {
      const int rs = n % RING;
      if (!mbar_wait(&sh->tk_full[rs], (n / RING) & 1, wc, SITE_FULL, -3)) break;
      const TileSlot ts = sh->ring[rs];
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->tk_empty[rs]);
      ++n;
      if (ts.op < 0) break;
      fence_proxy_async();  // the producers' writes (acquired by the scheduler) must be seen by the TMA loads
      const Tile tl = slot_tile(ts);
      for (int kb = 0; kb < ts.nkb; ++kb, ++it) {
        if (kb == ts.go_kb && lane == 0) mbar_arrive(&sh->sched_go);
        const int s = it % STAGES;
        if (!mbar_wait(&bars->empty[s], ((it / STAGES) & 1) ^ 1, wc, SITE_EMPTY, n)) { ok = false; break; }
        fused_load_stage<BWD>(fa, ts, tl, kb, sA + s * A_STAGE_BYTES, sB + s * B_STAGE_BYTES, &bars->full[s], lane);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, acc_it = 0, n = 0;
      bool ok = true;
      ST_DECL;
      while (ok) {
        const int rs = n % RING;
        ST_MARK();
        if (!mbar_wait(&sh->tk_full[rs], (n / RING) & 1, wc, SITE_FULL, -1)) break;
        ST_ADD(0);  // waiting for a published tile
        const int op = sh->ring[rs].op, nkb = sh->ring[rs].nkb;
        mbar_arrive(&sh->tk_empty[rs]);
        ++n;
        if (op < 0) break;
        if (nkb == 0) continue;
        const int as = acc_it & 1;
        if (!mbar_wait(&bars->tmem_empty[as], ((acc_it >> 1) & 1) ^ 1, wc, SITE_TMEM_EMPTY, n)) break;
        ST_ADD(1);  // accumulator not yet drained by the epilogue
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + as * BN;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % STAGES;
          if (!mbar_wait(&bars->full[s], (it / STAGES) & 1, wc, SITE_FULL, n)) { ok = false; break; }
          ST_ADD(2);  // operands not yet in shared memory (starved)
          tc_fence_after_sync();
          fused_mma<BWD>(op, d_tmem, smem_u32(sA + s * A_STAGE_BYTES), smem_u32(sB + s * B_STAGE_BYTES), kb == 0);
          tc_commit(&bars->empty[s]);
          ST_ADD(3);  // issue
        }
        if (!ok) break;
        tc_commit(&bars->tmem_full[as]);
        ++acc_it;
      }
      ST_FLUSH(8, 4);
      if (*reinterpret_cast<volatile int*>(&fa.status->abort)) {
        tc_commit(&bars->drain);
        const WaitCtl shortwc{fa.status, 20ull * 1000 * 1000};
        mbar_wait(&bars->drain, 0, shortwc, SITE_DRAIN, 0);
      }
    }
  } else if (warp < 2 + EPI_WARPS) {
    // ------------------------------------------------ epilogue warps
    const int quad = warp & 3;
    Staging stg{sOut + quad * OUT_STAGE_BYTES, 1, 0};
    uint32_t acc_it = 0, n = 0;
    ST_DECL;
    while (true) {
      const int rs = n % RING;
      ST_MARK();
      if (!mbar_wait(&sh->tk_full[rs], (n / RING) & 1, wc, SITE_FULL, -2, 100)) break;
      ST_ADD(0);
      const TileSlot ts = sh->ring[rs];
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->tk_empty[rs]);
      ++n;
      if (ts.op < 0) break;
      const Tile tl = slot_tile(ts);
      if (ts.nkb == 0) {
        fused_epilogue<BWD>(fa, ts, tl, 0, quad, lane, stg);
      } else {
        const int as = acc_it & 1;
        if (!mbar_wait(&bars->tmem_full[as], (acc_it >> 1) & 1, wc, SITE_TMEM_FULL, n, 100)) break;
        ST_ADD(1);  // waiting for the accumulator
        tc_fence_after_sync();
        fused_epilogue<BWD>(fa, ts, tl, tmem_base + as * BN, quad, lane, stg);
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->tmem_empty[as]);
        ++acc_it;
        ST_ADD(2);  // epilogue work
      }
      if (ts.trig_idx >= 0) {
        // trigger event: only after this warp's part of the tile is readable by everyone
        __syncwarp();
        if (lane == 0) {
          tma_store_wait_all();
          fence_proxy_async();
          counter_signal(fa.ctr + ts.trig_idx, 1);
          if (ts.trig_ag) counter_signal(fa.ctr + CTR_AG_DONE, 1);
        }
        __syncwarp();
        ST_ADD(3);  // trigger (store completion + signal)
      }
    }
    if (quad == 0 && lane == 0) ST_FLUSH(16, 4);
    if (lane == 0) tma_store_wait_all();
  }

  // ------------------------------------------------ vector workers: the dedicated warps from the
  // start, every other warp once its matrix role has reached the end of the matrix queue (the
  // tail of the vector queue -- combine -- then runs on the whole SM)
  __syncwarp();
  vector_worker_loop<BWD>(fa, sh->vec_ready, sh->vec_poller, wc, M, lane);

  // ---------------------------------------------------------------- teardown
  if (*reinterpret_cast<volatile int*>(&fa.status->abort)) __nanosleep(200000);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// =====================================================================================================
// The same persistent launch on CTA pairs: a cluster of two CTAs shares every matrix tile
// (tcgen05 cta_group::2, 256 x 256; see gemm_pair.cuh).  The even CTA owns the scheduler, the MMA
// issuer and every barrier the MMA issuer waits on; it publishes each tile into the tile rings of
// both CTAs (the odd CTA's copy over the cluster's shared-memory network).  Loaders and epilogue
// warps run in both CTAs on their own half of the tile; vector workers are per CTA as before.
// =====================================================================================================
constexpr int STAGESP = 5;  // 5 x 32 KB operand stages per CTA

struct __align__(16) PairShared {
  uint64_t full[STAGESP];      // even CTA: bytes of both CTAs' loads
  uint64_t empty[STAGESP];     // each CTA: the stage's MMAs are complete (multicast commit)
  uint64_t tmem_full[2];       // each CTA: accumulator ready (multicast commit)
  uint64_t tmem_empty[2];      // even CTA: the 8 epilogue warps of the pair have drained it
  uint64_t drain;
  uint64_t tk_full[RING];      // each CTA: a tile has been published into this CTA's ring
  uint64_t tk_empty[RING];     // even CTA: every consumer of both CTAs has read the slot
  uint64_t sched_go;           // even CTA: loader -> scheduler
  uint64_t vec_ready[2];
  int vec_poller[2];
  uint32_t tmem_base;
  uint32_t pad;
  TileSlot ring[RING];
};

constexpr size_t FUSEDP_SMEM_BYTES =
    1024 + (size_t)STAGESP * STAGE2_BYTES + 4 * OUT_STAGE_BYTES + 4 * SW_SCRATCH_BYTES + sizeof(PairShared);
static_assert(FUSEDP_SMEM_BYTES <= 227 * 1024, "shared memory budget");
constexpr int PAIR_TK_EMPTY_COUNT = (3 + EPI_WARPS) + (2 + EPI_WARPS);  // even: 2 loaders, MMA, epilogue; odd: 2 loaders, epilogue

template <bool BWD>
__device__ __forceinline__ void fusedp_load_stage(const FusedArgs& fa, const TileSlot& ts, const Tile& tl, int kb,
                                                  int rank, uint8_t* sA, uint8_t* sB, uint64_t* bar, int lane) {
  const GemmArgs& g = fa.op[ts.slot];
  if (!BWD) {
    if (ts.op == GEMM_GATE_UP) load_stage_pair_lanes<GEMM_GATE_UP>(g, tl, kb, rank, sA, sB, bar, lane);
    else load_stage_pair_lanes<GEMM_DOWN>(g, tl, kb, rank, sA, sB, bar, lane);
  } else {
    if (ts.op == GEMM_ACT_GRAD) load_stage_pair_lanes<GEMM_ACT_GRAD>(g, tl, kb, rank, sA, sB, bar, lane);
    else if (ts.op == GEMM_GATE_GRAD) load_stage_pair_lanes<GEMM_GATE_GRAD>(g, tl, kb, rank, sA, sB, bar, lane);
    else load_stage_pair_lanes<GEMM_WGRAD>(g, tl, kb, rank, sA, sB, bar, lane);
  }
}
template <bool BWD>
__device__ __forceinline__ void fusedp_mma(int op, uint32_t d_tmem, uint32_t a_addr, uint32_t b_addr, bool first,
                                           int k16_steps) {
  if (!BWD) {
    mma_kblock_pair<GEMM_GATE_UP>(d_tmem, a_addr, b_addr, first);
  } else {
    if (op == GEMM_WGRAD) mma_kblock_pair<GEMM_WGRAD>(d_tmem, a_addr, b_addr, first, k16_steps);
    else mma_kblock_pair<GEMM_ACT_GRAD>(d_tmem, a_addr, b_addr, first);
  }
}

// ---- token-column tiles (gemm_swap.cuh) in the persistent launch
__device__ __forceinline__ bool slot_is_tokcol(const FusedArgs& fa, int op) { return fa.sp.tokcol && op != GEMM_WGRAD; }
__device__ __forceinline__ SwapTile slot_swap_tile(const TileSlot& ts) {
  SwapTile st;
  st.e = ts.e; st.row0 = ts.row0; st.ntok = ts.m0; st.n0 = ts.n0; st.nb = ts.nb; st.nkb = ts.nkb;
  return st;
}
template <bool BWD>
__device__ __forceinline__ void fusedp_load_weights_swap(const FusedArgs& fa, const TileSlot& ts, const SwapTile& st,
                                                         int kb, int rank, uint8_t* sW, uint64_t* bar, int lane) {
  const GemmArgs& g = fa.op[ts.slot];
  if (!BWD) {
    if (ts.op == GEMM_GATE_UP) load_weights_swap<GEMM_GATE_UP>(g, st, kb, rank, sW, bar, lane);
    else load_weights_swap<GEMM_DOWN>(g, st, kb, rank, sW, bar, lane);
  } else {
    load_weights_swap<GEMM_ACT_GRAD>(g, st, kb, rank, sW, bar, lane);  // ACT_GRAD and GATE_GRAD alike
  }
}
template <bool BWD>
__device__ __forceinline__ void fusedp_epilogue_swap(const FusedArgs& fa, const TileSlot& ts, const SwapTile& st,
                                                     uint32_t tmem_acc, int rank, int quad, int lane, SwStaging& sg) {
  const GemmArgs& g = fa.op[ts.slot];
  if (!BWD) {
    if (ts.op == GEMM_GATE_UP) epilogue_swap<GEMM_GATE_UP>(g, st, tmem_acc, rank, quad, lane, sg);
    else epilogue_swap<GEMM_DOWN>(g, st, tmem_acc, rank, quad, lane, sg);
  } else {
    if (ts.op == GEMM_ACT_GRAD) epilogue_swap<GEMM_ACT_GRAD>(g, st, tmem_acc, rank, quad, lane, sg);
    else epilogue_swap<GEMM_GATE_GRAD>(g, st, tmem_acc, rank, quad, lane, sg);
  }
}
static_assert(SW_SLOTS * SW_SLOT_BYTES == OUT_STAGE_BYTES, "both epilogue kinds share one staging area per warp");
// Publish one tile into the ring slot `rs` of CTA `rank` (through the cluster address space, also for
// the even CTA itself) and signal that CTA's consumers.
__device__ __forceinline__ void publish_slot(PairShared* sh, int rs, uint32_t rank, const TileSlot& ts) {
  const uint32_t dst = map_to_rank(smem_u32(&sh->ring[rs]), rank);
  const uint4* src = reinterpret_cast<const uint4*>(&ts);
  static_assert(sizeof(TileSlot) == 48, "TileSlot is published as three 16-byte stores");
  st_cluster_v4(dst, src[0]);
  st_cluster_v4(dst + 16, src[1]);
  st_cluster_v4(dst + 32, src[2]);
  mbar_arrive_cluster_addr(map_to_rank(smem_u32(&sh->tk_full[rs]), rank));
}

template <bool BWD>
__global__ void __launch_bounds__(FUSED_THREADS, 1) fused_pair_kernel(const __grid_constant__ FusedArgs fa) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = smem + STAGESP * A_STAGE_BYTES;
  uint8_t* sOut = smem + STAGESP * STAGE2_BYTES;
  uint8_t* sScr = sOut + 4 * OUT_STAGE_BYTES;   // act_grad epilogue: 4 KB per epilogue warp
  PairShared* sh = reinterpret_cast<PairShared*>(sScr + 4 * SW_SCRATCH_BYTES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const WaitCtl wc{fa.status, fa.budget_ns};
  const int M = fa.lv.meta[0];

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGESP; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sh->tmem_full[s], 1);
      mbar_init(&sh->tmem_empty[s], 2 * EPI_WARPS);
      mbar_init(&sh->vec_ready[s], 1);
      sh->vec_poller[s] = 0;
    }
    mbar_init(&sh->drain, 1);
    for (int s = 0; s < RING; ++s) {
      mbar_init(&sh->tk_full[s], 1);
      mbar_init(&sh->tk_empty[s], PAIR_TK_EMPTY_COUNT);
    }
    mbar_init(&sh->sched_go, 1);
    mbar_fence_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc_pair(&sh->tmem_base, TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after_sync();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp == SCHED_WARP && rank == 0) {
    // ------------------------------------------------ scheduler (even CTA): tickets of the pair
    if (lane == 0) {
      const int total = fa.step_start[fa.sp.Ep + fa.sp.lag];
      uint32_t n = 0, go_n = 0;
      int cursor = 0;
      bool ok = true;
      while (ok) {
        const int t = atomicAdd(&fa.ctr[CTR_MAT_TICKET], 1);
        TileSlot ts;
        ts.slot = 0; ts.e = 0; ts.row0 = 0; ts.n0 = 0; ts.m0 = 0; ts.nkb = 0; ts.nb = 0;
        ts.trig_idx = -1; ts.trig_ag = 0; ts.go_kb = -1; ts.pad = 0; ts.krows = 0;
        if (t >= total) {
          ts.op = -1;
          const int rs = n % RING;
          if (!mbar_wait_cluster(&sh->tk_empty[rs], ((n / RING) & 1) ^ 1, wc, SITE_EMPTY, t)) break;
          publish_slot(sh, rs, 0, ts);
          publish_slot(sh, rs, 1, ts);
          break;
        }
        while (fa.step_start[cursor + 1] <= t) ++cursor;
        const MatTile mt = decode_matrix_ticket_at(fa.sp, t, cursor, fa.step_start, fa.lv.mb_start);
        const GemmArgs& g = fa.op[mt.slot];
        for (int q = 0; q < mt.dep_count && ok; ++q) {
          const int mbq = mt.dep_first + q;
          const int* c = fa.ctr + (mt.dep_base == 0 ? ctr_gather(mbq) : ctr_act(mbq));
          ok = counter_wait(c, mt.dep_thr, wc, t);
        }
        if (!ok) break;
        ts.op = mt.op; ts.slot = mt.slot; ts.e = mt.e;
        ts.trig_ag = mt.trig_also_ag;
        const int nkb = mt.op == GEMM_WGRAD ? (fa.lv.counts[mt.e] + BK - 1) / BK : (g.K + BK - 1) / BK;
        ts.nkb = nkb;
        ts.krows = mt.op == GEMM_WGRAD ? fa.lv.counts[mt.e] : 0;
        for (int gi = 0; gi < mt.group && ok; ++gi) {
          const int after = (mt.group - 1 - gi) * nkb;
          ts.go_kb = -1;
          if (after < SCHED_AHEAD_KB && (after + nkb >= SCHED_AHEAD_KB || gi == 0))
            ts.go_kb = max(0, nkb - (SCHED_AHEAD_KB - after));
          const int rs = n % RING;
          if (!mbar_wait_cluster(&sh->tk_empty[rs], ((n / RING) & 1) ^ 1, wc, SITE_EMPTY, t)) { ok = false; break; }
#pragma unroll
          for (int r = 0; r < 2; ++r) {  // the slot as CTA r of the pair sees it
            TileSlot tr = ts;
            if (mt.op == GEMM_WGRAD) {
              tr.nb = gi;
              tr.m0 = (2 * mt.idx + r) * BLOCK_M;  // this CTA's 128 rows of the 256-row strip
              tr.n0 = gi * BN;
              tr.row0 = fa.lv.mb_start[mt.e] * BLOCK_M;
              tr.pad = tr.m0 >= g.M;               // nothing to store: the strip's second half is outside dW
              tr.trig_idx = -1;
            } else if (fa.sp.tokcol) {
              // token-column tile: both CTAs work on all its tokens (each on its half of the features)
              const int n32 = (fa.lv.counts[mt.e] + TOK_GRAIN - 1) & ~(TOK_GRAIN - 1);
              const int first = mt.mb - fa.lv.mb_start[mt.e];
              int end = (first + mt.mb_count) * BLOCK_M;
              if (end > n32) end = n32;
              tr.nb = mt.idx;
              tr.m0 = end - first * BLOCK_M;           // tokens of the tile
              tr.krows = mt.mb_count;
              tr.n0 = mt.idx * (mt.op == GEMM_GATE_UP ? 128 : 256);
              tr.row0 = mt.mb * BLOCK_M;
              tr.pad = 0;
              tr.trig_idx = mt.trig_base == 1 ? ctr_act(mt.mb) : (mt.trig_base == 2 ? CTR_DONE : -1);
            } else {
              const bool idle = r >= mt.mb_count;
              tr.nb = mt.idx;
              tr.m0 = 0;
              tr.n0 = mt.idx * (mt.op == GEMM_GATE_UP ? BN / 2 : BN);
              tr.row0 = idle ? g.cap_rows : (mt.mb + r) * BLOCK_M;  // rows beyond the tensor read as zeros
              tr.pad = idle;
              tr.trig_idx = idle ? -1 : (mt.trig_base == 1 ? ctr_act(mt.mb + r) : (mt.trig_base == 2 ? CTR_DONE : -1));
              if (idle) tr.trig_ag = 0;
            }
            publish_slot(sh, rs, r, tr);
          }
          ++n;
        }
        if (!ok || !mbar_wait(&sh->sched_go, go_n & 1, wc, SITE_DEP, t, 200)) break;
        ++go_n;
      }
    }
  } else if (warp == 0 || warp == TOK_WARP) {
    // ------------------------------------------------ loaders (both CTAs).  Warp 0: own rows of A and own half
    // of B of a token-row tile, or the weights of a token-column tile; TOK_WARP: the tokens of a token-column tile.
    uint32_t s = 0, ph = 1, n = 0;
    bool ok = true;
    ST_DECL;
    while (ok) {
      const int rs = n % RING;
      ST_MARK();
      if (!mbar_wait_cluster(&sh->tk_full[rs], (n / RING) & 1, wc, SITE_FULL, -3)) break;
      ST_ADD(0);  // loader: waiting for a published tile
      const TileSlot ts = sh->ring[rs];
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(&sh->tk_empty[rs]);
      ++n;
      if (ts.op < 0) break;
      fence_proxy_async();
      const bool tokcol = slot_is_tokcol(fa, ts.op);
      const Tile tl = slot_tile(ts);
      const SwapTile st = slot_swap_tile(ts);
      if (warp == TOK_WARP && !fa.sp.tokcol) continue;   // token-row tiles: warp 0 loads everything
      for (int kb = 0; kb < ts.nkb; ++kb) {
        if (warp == 0 && kb == ts.go_kb && lane == 0 && rank == 0) mbar_arrive(&sh->sched_go);
        int go = 1;
        ST_ADD(2);  // loader: issuing loads, loop overhead
        if (lane == 0) go = mbar_wait(&sh->empty[s], ph, wc, SITE_EMPTY, n, 50) ? 1 : 0;
        go = __shfl_sync(0xffffffffu, go, 0);
        ST_ADD(1);  // loader: waiting for a free stage
        if (!go) { ok = false; break; }
        if (!fa.sp.tokcol)
          fusedp_load_stage<BWD>(fa, ts, tl, kb, rank, sA + s * A_STAGE_BYTES, sB + s * HALF_B_BYTES, &sh->full[s], lane);
        else if (!tokcol)   // a weight-gradient tile between token-column tiles
          load_wgrad_part(fa.op[ts.slot], tl, kb, rank, sA + s * A_STAGE_BYTES, sB + s * HALF_B_BYTES, &sh->full[s],
                                 lane, warp == TOK_WARP);
        else if (warp == 0)
          fusedp_load_weights_swap<BWD>(fa, ts, st, kb, rank, sA + s * A_STAGE_BYTES, &sh->full[s], lane);
        else
          load_tokens_swap(fa.op[ts.slot], st, kb, rank, sB + s * HALF_B_BYTES, &sh->full[s], lane);
        if (++s == STAGESP) { s = 0; ph ^= 1; }
      }
      ST_ADD(2);
    }
    if (lane == 0 && rank == 0) ST_FLUSH(warp == 0 ? 16 : 20, 3);
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer (even CTA)
    if (lane == 0 && rank == 0) {
      uint32_t it = 0, acc_it = 0, n = 0;
      bool ok = true;
      ST_DECL;
      while (ok) {
        const int rs = n % RING;
        ST_MARK();
        if (!mbar_wait_cluster(&sh->tk_full[rs], (n / RING) & 1, wc, SITE_FULL, -1)) break;
        ST_ADD(0);  // waiting for a published tile
        const int op = sh->ring[rs].op, nkb = sh->ring[rs].nkb, krows = sh->ring[rs].krows, ntok = sh->ring[rs].m0;
        mbar_arrive(&sh->tk_empty[rs]);
        ++n;
        if (op < 0) break;
        if (nkb == 0) continue;
        const int as = acc_it & 1;
        if (!mbar_wait_cluster(&sh->tmem_empty[as], ((acc_it >> 1) & 1) ^ 1, wc, SITE_TMEM_EMPTY, n)) break;
        ST_ADD(1);  // accumulator not yet drained by the epilogues
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + as * BN;
        const bool tokcol = slot_is_tokcol(fa, op);
        const uint32_t idesc = swap_idesc<BWD ? GEMM_ACT_GRAD : GEMM_GATE_UP>(ntok);
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % STAGESP;
          if (!mbar_wait(&sh->full[s], (it / STAGESP) & 1, wc, SITE_FULL, n)) { ok = false; break; }
          ST_ADD(2);  // operands not yet in shared memory
          tc_fence_after_sync();
          if (tokcol)
            mma_kblock_swap<BWD ? GEMM_ACT_GRAD : GEMM_GATE_UP>(
                d_tmem, swap_w_desc_lo<BWD ? GEMM_ACT_GRAD : GEMM_GATE_UP>(smem_u32(sA + s * A_STAGE_BYTES)),
                smem_desc_lo(smem_u32(sB + s * HALF_B_BYTES), 16), idesc, kb == 0);
          else
            fusedp_mma<BWD>(op, d_tmem, smem_u32(sA + s * A_STAGE_BYTES), smem_u32(sB + s * HALF_B_BYTES), kb == 0,
                            op == GEMM_WGRAD ? k16_steps_of(krows, kb) : BK / 16);
          tc_commit_pair(&sh->empty[s]);
          ST_ADD(op == GEMM_WGRAD ? 4 : 3);  // issue (includes back-pressure of the tensor pipe)
        }
        if (!ok) break;
        tc_commit_pair(&sh->tmem_full[as]);
        ++acc_it;
      }
      ST_FLUSH(8, 5);
      if (*reinterpret_cast<volatile int*>(&fa.status->abort)) {
        tc_commit_pair(&sh->drain);
        const WaitCtl shortwc{fa.status, 20ull * 1000 * 1000};
        mbar_wait(&sh->drain, 0, shortwc, SITE_DRAIN, 0);
      }
    }
  } else if (warp < 2 + EPI_WARPS) {
    // ------------------------------------------------ epilogue warps (both CTAs, own rows)
    const int quad = warp & 3;
    Staging stg{sOut + quad * OUT_STAGE_BYTES, 1, 0};
    uint32_t acc_it = 0, n = 0;
    while (true) {
      const int rs = n % RING;
      if (!mbar_wait_cluster(&sh->tk_full[rs], (n / RING) & 1, wc, SITE_FULL, -2, 100)) break;
      const TileSlot ts = sh->ring[rs];
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(&sh->tk_empty[rs]);
      ++n;
      if (ts.op < 0) break;
      const Tile tl = slot_tile(ts);
      const bool idle = ts.pad != 0;
      const bool tokcol = slot_is_tokcol(fa, ts.op);
      if (ts.nkb != 0) {
        const int as = acc_it & 1;
        if (!mbar_wait(&sh->tmem_full[as], (acc_it >> 1) & 1, wc, SITE_TMEM_FULL, n, 100)) break;
        tc_fence_after_sync();
        if (tokcol) {
          // the staging area changes hands between the two epilogue kinds: let the earlier stores finish reading
          if (lane == 0) tma_store_wait_read();
          __syncwarp();
          SwStaging sg{sOut + quad * OUT_STAGE_BYTES, 0, sScr + quad * SW_SCRATCH_BYTES, SW_SLOTS, SW_SLOT_BYTES};
          fusedp_epilogue_swap<BWD>(fa, ts, slot_swap_tile(ts), tmem_base + as * BN, rank, quad, lane, sg);
        } else if (!idle) {
          fused_epilogue<BWD>(fa, ts, tl, tmem_base + as * BN, quad, lane, stg);
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_leader(&sh->tmem_empty[as]);
        ++acc_it;
      }
      if (ts.trig_idx >= 0) {
        __syncwarp();
        if (lane == 0) {
          tma_store_wait_all();
          fence_proxy_async();
          if (tokcol) {
            // this warp stored its features of every row of the tile's M-blocks (ts.krows of them)
            if (ts.trig_idx == CTR_DONE) counter_signal(fa.ctr + CTR_DONE, ts.krows);
            else for (int q = 0; q < ts.krows; ++q) counter_signal(fa.ctr + ts.trig_idx + 2 * q, 1);
            if (ts.trig_ag) counter_signal(fa.ctr + CTR_AG_DONE, ts.krows);
          } else {
            counter_signal(fa.ctr + ts.trig_idx, 1);
            if (ts.trig_ag) counter_signal(fa.ctr + CTR_AG_DONE, 1);
          }
        }
        __syncwarp();
      }
    }
    if (lane == 0) tma_store_wait_all();
  }

  // ------------------------------------------------ vector workers (per CTA, as in the single-CTA kernel)
  __syncwarp();
  vector_worker_loop<BWD>(fa, sh->vec_ready, sh->vec_poller, wc, M, lane);

  // ---------------------------------------------------------------- teardown
  if (*reinterpret_cast<volatile int*>(&fa.status->abort)) __nanosleep(200000);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // neither CTA leaves while its partner may still read its shared memory or signal it
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

template <bool BWD>
static cudaError_t launch_fused_pair_t(const FusedArgs& fa, int num_sms, cudaStream_t s) {
  static bool attr_set = false;
  static int max_pairs = 0;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(fused_pair_kernel<BWD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)FUSEDP_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3((num_sms / 2) * 2);
  cfg.blockDim = dim3(FUSED_THREADS);
  cfg.dynamicSmemBytes = FUSEDP_SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeCooperative;  // the launch fails rather than run with CTAs that are not all resident
  attr[1].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (max_pairs == 0) {
    int n = 0;
    cudaError_t e = cudaOccupancyMaxActiveClusters(&n, fused_pair_kernel<BWD>, &cfg);
    if (e != cudaSuccess) return e;
    max_pairs = n > 0 ? n : 1;
  }
  if (2 * max_pairs < (int)cfg.gridDim.x) cfg.gridDim = dim3(2 * max_pairs);
  return cudaLaunchKernelEx(&cfg, fused_pair_kernel<BWD>, fa);
}

// ---------------------------------------------------------------- host side
cudaError_t launch_build_schedule(const SchedParams& sp, const LayoutView& lv, int* step_start, int* ctr,
                                  int ctr_count, cudaStream_t s, int* launches) {
  build_schedule_kernel<<<1, 1024, 0, s>>>(sp, lv, step_start, ctr, ctr_count);
  ++*launches;
  return cudaGetLastError();
}

template <bool BWD>
static cudaError_t launch_fused_t(const FusedArgs& fa, int num_sms, cudaStream_t s) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(fused_kernel<BWD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)FUSED_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  void* params[] = {const_cast<FusedArgs*>(&fa)};
  // cooperative: the launch fails rather than run with CTAs that are not all resident
  return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(fused_kernel<BWD>), dim3(num_sms), dim3(FUSED_THREADS),
                                     params, FUSED_SMEM_BYTES, s);
}

cudaError_t launch_fused(bool bwd, const FusedArgs& fa, int num_sms, cudaStream_t s, int* launches) {
  ++*launches;
  if (fa.sp.pair) return bwd ? launch_fused_pair_t<true>(fa, num_sms, s) : launch_fused_pair_t<false>(fa, num_sms, s);
  return bwd ? launch_fused_t<true>(fa, num_sms, s) : launch_fused_t<false>(fa, num_sms, s);
}

}  // namespace moe
