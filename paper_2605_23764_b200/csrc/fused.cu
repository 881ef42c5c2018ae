// The single persistent, dependency-driven launch of the forward (and of the backward) layer.
//
// One cooperative grid of one CTA per SM in clusters of two runs the whole operator chain.  Per CTA:
//   warp 0      TMA producer of the weights (weight gradients: of the A operand)
//   warp 1      tcgen05.mma issuer (even CTA) and TMEM owner
//   warps 2-5   epilogue: TMEM -> fused element-wise math -> TMA store, then the tile's trigger event
//   warp 6      TMA producer of the tokens (weight gradients: of the B operand)
//   warp 7      even CTA: scheduler of the pair -- takes the next ticket of the matrix queue, waits for
//               the item's dependent events, publishes it to the other roles; odd CTA: vector worker
//   warps 8-14  vector workers: tickets of the vector queue (permute-gather, routing-weight
//               gradient, combine); the matrix-role warps join them once the matrix queue is empty.
// The matrix roles are the ones of the one-launch-per-operator kernels (gemm_roles.cuh); here they
// take the items of all operators of the pass from one ticket queue (schedule.h) with the pipeline
// state carried from item to item, so that no SM waits at an operator boundary for the others, the
// permutes run beside the GEMMs, and what orders tiles are event counters with static thresholds --
// the paper's unified runtime (Sections 4.3, 4.4) restated for one SM, where "matrix core" and
// "vector core" are warp roles of the same CTA.
#include "gemm_roles.cuh"
#include "launch_pairs.cuh"
#include "schedule.h"

namespace moe {

constexpr int ROLE_WARPS = 7;
constexpr int SCHED_WARP = 7;   // even CTA: scheduler of the pair; odd CTA: a vector worker
constexpr int VEC_WARPS = 8;
constexpr int FUSED_THREADS = 32 * (ROLE_WARPS + VEC_WARPS);

constexpr size_t cmax(size_t a, size_t b) { return a > b ? a : b; }
constexpr size_t FUSED_LAYOUT_BYTES =
    cmax(cmax(swap_layout_bytes<GEMM_GATE_UP>(), swap_layout_bytes<GEMM_DOWN>()),
         cmax(cmax(swap_layout_bytes<GEMM_ACT_GRAD>(), swap_layout_bytes<GEMM_GATE_GRAD>()), WGRAD_LAYOUT_BYTES));
constexpr size_t FUSED_SMEM_BYTES = 1024 + FUSED_LAYOUT_BYTES + 256 /* PipeBarriers */ + 384 /* TicketRing */;
static_assert(FUSED_SMEM_BYTES <= 227 * 1024, "shared memory budget");

// ---------------------------------------------------------------- vector work (one warp per task)
__device__ __forceinline__ uint4 ldg_nc_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
// data written earlier in this launch by other SMs: read at L2
__device__ __forceinline__ uint4 ldg_cg_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// Dispatch / backward Dispatch: GATHER_ROWS rows of one M-block of the padded expert-ordered row space.  The
// index chains of the rows are resolved first, then the rows are copied together: 16 independent 16-byte
// loads in flight per lane.
constexpr int GATHER_ROWS = BLOCK_M / GATHER_SUB;
__device__ __forceinline__ void vec_gather(const FusedArgs& fa, int task, int lane) {
  const int mb = task / GATHER_SUB, sub = task - mb * GATHER_SUB;
  const LayoutView& lv = fa.lv;
  const int e = lv.mblk_expert[mb];
  const int cnt = lv.counts[e], pad0 = lv.pad_off[e], off0 = lv.offsets[e];
  const int nvec = fa.d >> 3;
  const int k = fa.cp.k;
  const int p0 = mb * BLOCK_M + sub * GATHER_ROWS;
  const uint4* in[GATHER_ROWS];
#pragma unroll
  for (int r = 0; r < GATHER_ROWS; ++r) {
    const int local = p0 + r - pad0;
    in[r] = nullptr;
    float w = 0.0f;
    if (local < cnt) {
      const int slot = lv.src_of[off0 + local];
      const int t = slot / fa.kp, j = slot - t * fa.kp;
      in[r] = reinterpret_cast<const uint4*>(fa.gather_src + (size_t)t * fa.d);
      if (fa.prow_w) w = j < k ? fa.topk_w[(size_t)t * k + j] : 1.0f;
    }
    if (fa.prow_w && lane == 0) fa.prow_w[p0 + r] = w;   // padding rows: weight 0
  }
  uint4* out = reinterpret_cast<uint4*>(fa.gather_dst + (size_t)p0 * fa.d);
  constexpr int U = 16 / GATHER_ROWS;
  for (int v = lane; v < nvec; v += 32 * U) {
    uint4 q[GATHER_ROWS][U];
#pragma unroll
    for (int r = 0; r < GATHER_ROWS; ++r)
#pragma unroll
      for (int u = 0; u < U; ++u)
        q[r][u] = (in[r] && v + 32 * u < nvec) ? ldg_nc_v4(in[r] + v + 32 * u) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int r = 0; r < GATHER_ROWS; ++r)
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (v + 32 * u < nvec) out[(size_t)r * nvec + v + 32 * u] = q[r][u];   // padding rows are zero-filled
  }
}

// Combine / backward Combine of COMBINE_TOKENS tokens.  Dependent events: `done` of every M-block that
// holds one of a token's rows (many-to-many, Section 4.3): each lane polls the counter of one row.
__device__ __forceinline__ bool vec_combine(const FusedArgs& fa, int task, int lane, const WaitCtl& wc) {
  const int nvec = fa.d >> 3, kp = fa.kp, T = fa.cp.T;
  const int i0 = task * COMBINE_TOKENS, i1 = min(T, i0 + COMBINE_TOKENS);
  const int thr = thr_done(fa.cp);
  for (int i = i0; i < i1; ++i) {
    const int t = fa.lv.combine_order ? fa.lv.combine_order[i] : i;   // tokens in the order in which their last row is produced
    const int* prow = fa.lv.prow_of + (size_t)t * kp;
    // dependent events: `done` of every M-block that holds one of the token's rows
    int ok = 1;
    for (int j = lane; j < kp; j += 32) {
      const int p = prow[j];
      if (p >= 0 && !counter_wait(fa.ctr + ctr_index(p / BLOCK_M, CTR_DONE), thr, wc, task, 2048)) ok = 0;
    }
    if (!__all_sync(0xffffffffu, ok)) return false;
    // two vector positions per lane and step: sixteen independent row loads in flight (a warp alone is latency-bound)
    for (int v = lane; v < nvec; v += 64) {
      const bool two = v + 32 < nvec;
      float acc[16];
#pragma unroll
      for (int q = 0; q < 16; ++q) acc[q] = 0.f;
      for (int j0 = 0; j0 < kp; j0 += 8) {
        uint4 r[8], r2[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int j = j0 + u;
          const int p = j < kp ? prow[j] : -1;
          const uint4* row = reinterpret_cast<const uint4*>(fa.combine_rows + (size_t)(p >= 0 ? p : 0) * fa.d);
          r[u] = p >= 0 ? ldg_cg_v4(row + v) : make_uint4(0, 0, 0, 0);
          r2[u] = (p >= 0 && two) ? ldg_cg_v4(row + v + 32) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          acc[0] += bf16lo(r[u].x); acc[1] += bf16hi(r[u].x);
          acc[2] += bf16lo(r[u].y); acc[3] += bf16hi(r[u].y);
          acc[4] += bf16lo(r[u].z); acc[5] += bf16hi(r[u].z);
          acc[6] += bf16lo(r[u].w); acc[7] += bf16hi(r[u].w);
          acc[8] += bf16lo(r2[u].x); acc[9] += bf16hi(r2[u].x);
          acc[10] += bf16lo(r2[u].y); acc[11] += bf16hi(r2[u].y);
          acc[12] += bf16lo(r2[u].z); acc[13] += bf16hi(r2[u].z);
          acc[14] += bf16lo(r2[u].w); acc[15] += bf16hi(r2[u].w);
        }
      }
      uint4 o;
      o.x = pack_bf16x2(acc[0], acc[1]);
      o.y = pack_bf16x2(acc[2], acc[3]);
      o.z = pack_bf16x2(acc[4], acc[5]);
      o.w = pack_bf16x2(acc[6], acc[7]);
      reinterpret_cast<uint4*>(fa.combine_out + (size_t)t * fa.d)[v] = o;
      if (two) {
        o.x = pack_bf16x2(acc[8], acc[9]);
        o.y = pack_bf16x2(acc[10], acc[11]);
        o.z = pack_bf16x2(acc[12], acc[13]);
        o.w = pack_bf16x2(acc[14], acc[15]);
        reinterpret_cast<uint4*>(fa.combine_out + (size_t)t * fa.d)[v + 32] = o;
      }
    }
  }
  return true;
}

// Routing-weight gradient of the rows of one M-block: the act_grad epilogues left partial dot products
// per (row, column tile, CTA, warp); summed here in a fixed order.  Dependent event: `activated`.
__device__ __forceinline__ bool vec_dw(const FusedArgs& fa, int mb, int lane, const WaitCtl& wc) {
  int ok = 1;
  if (lane == 0) ok = counter_wait(fa.ctr + ctr_index(mb, CTR_ACTIVATED), thr_activated(fa.cp), wc, mb, 4096) ? 1 : 0;
  if (!__shfl_sync(0xffffffffu, ok, 0)) return false;
  const LayoutView& lv = fa.lv;
  const int e = lv.mblk_expert[mb];
  const int cnt = lv.counts[e], local0 = mb * BLOCK_M - lv.pad_off[e], off0 = lv.offsets[e];
  const int k = fa.cp.k;
  for (int r = lane; r < BLOCK_M; r += 32) {
    const int local = local0 + r;
    if (local >= cnt) continue;
    const int slot = lv.src_of[off0 + local];
    const int t = slot / fa.kp, j = slot - t * fa.kp;
    if (j >= k) continue;   // a shared expert's row: its weight is the constant 1
    const float* part = fa.dw_partial + (size_t)(mb * BLOCK_M + r) * fa.dw_nparts;
    float s = 0.f;
    for (int q = 0; q < fa.dw_nparts; ++q) s += __ldcg(part + q);
    fa.d_topk_w[(size_t)t * k + j] = s;
  }
  return true;
}

// Vector workers.  The gather of the first GATHER_FAST_MBLOCKS M-blocks -- what the first matrix items of every
// pair wait for -- is taken by every worker; after that only BACKGROUND_GATHERERS warps per CTA keep gathering,
// a few M-blocks' worth of traffic at a time, well ahead of the matrix queue but far below the bandwidth the
// GEMMs need: a gather at full speed takes its bytes from the loads of the matrix tiles and slows them by more
// than it saves.  The other workers go on to the second queue and sleep on its dependent events.
constexpr int BACKGROUND_GATHERERS = 2;
__device__ __forceinline__ void vector_worker_loop(const FusedArgs& fa, const WaitCtl& wc, const TraceCtl& tr, int M,
                                                   int lane, bool background_gatherer) {
  if (*reinterpret_cast<volatile int*>(&fa.status->abort)) return;
  const int ngather = gather_total(M), fast = GATHER_SUB * GATHER_FAST_MBLOCKS;
  // with shared experts the gather starts at their first M-block, like the matrix queue (schedule.h, rotate_index)
  const int S = fa.cp.kp - fa.cp.k;
  const int gather_first = S > 0 ? fa.lv.mb_start[fa.cp.Ep - S] * GATHER_SUB : 0;
  while (true) {
    int t = ngather;
    if (lane == 0) {
      const int seen = *reinterpret_cast<volatile int*>(&fa.ctr[CTR_VEC_TICKET]);
      if (seen < ngather && (background_gatherer || seen < fast)) t = atomicAdd(&fa.ctr[CTR_VEC_TICKET], 1);
    }
    t = __shfl_sync(0xffffffffu, t, 0);
    if (t >= ngather) break;
    t = rotate_index(t, gather_first, ngather);
    uint64_t t0 = 0;
    if (tr.buf && lane == 0) t0 = globaltimer_ns();
    vec_gather(fa, t, lane);
    __syncwarp();
    if (lane == 0) {
      counter_signal(fa.ctr + ctr_index(t / GATHER_SUB, CTR_GATHERED), 1);
      if (tr.buf) trace_put(tr, TR_VEC, VEC_GATHER, t, t0, t0, globaltimer_ns());
    }
  }
  const int npost = post_total(fa.cp, M);
  while (true) {
    int t = 0;
    if (lane == 0) t = atomicAdd(&fa.ctr[CTR_POST_TICKET], 1);
    t = __shfl_sync(0xffffffffu, t, 0);
    if (t >= npost) break;
    VecTask v = decode_post_ticket(fa.cp, t, M);
    if (v.op == VEC_DW) v.idx = rotate_index(v.idx, gather_first / GATHER_SUB, M);   // in the order act_grad produces them
    uint64_t t0 = 0;
    if (tr.buf && lane == 0) t0 = globaltimer_ns();
    const bool ok = v.op == VEC_COMBINE ? vec_combine(fa, v.idx, lane, wc) : vec_dw(fa, v.idx, lane, wc);
    if (tr.buf && lane == 0) trace_put(tr, TR_VEC, v.op, v.idx, t0, t0, globaltimer_ns());
    if (!ok) break;
    if (fa.announce_out && v.op == VEC_COMBINE) {
      // Host-buffer calls: the result may leave for the host as soon as its last row is written, while the
      // launch still computes weight gradients.  The warp's stores, then a device-wide fence, then the count;
      // whoever finishes the last task publishes the word the copy-out stream waits for.
      __syncwarp();
      if (lane == 0) {
        __threadfence();
        const int ncombine = (fa.cp.T + COMBINE_TOKENS - 1) / COMBINE_TOKENS;
        if (atomicAdd(&fa.ctr[CTR_COMBINE_DONE], 1) + 1 == ncombine) {
          __threadfence_system();
          *reinterpret_cast<volatile int*>(&fa.ctr[CTR_OUT_READY]) = 1;
        }
      }
    }
  }
}

// ---------------------------------------------------------------- matrix queue: tickets of a CTA pair
// The matrix queue is the concatenation of the phases' item lists (schedule.h); pairs take tickets with
// one atomic counter.  Tickets are handed out in time order, so the ~74 items in flight are always a
// contiguous window of the queue: items that share an operand (the token tiles of one expert and
// column tile share its weight slab, the strips of one expert share its rows) start within
// microseconds of each other and meet in L2, however the pairs' speeds differ -- a static deal of
// items to pairs loses that as soon as gather or combine traffic makes the pairs drift apart.
// The scheduler warp of the even CTA takes the pair's tickets -- as soon as a ring slot is free, so up to
// TK_RING items ahead of the epilogue -- polls the item's dependent events (one M-block per lane) and
// only then publishes the ticket to every role of both CTAs through a small ring in shared memory:
// ticket, decode and polls hide behind the loads of the items before it.
constexpr int TK_RING = 4;
// A published item: the ticket and the decoded work (decoding takes a chain of dependent global loads; the
// scheduler does it once, ahead of time, for every role of both CTAs).
struct __align__(16) WorkDesc {
  int ticket;                                  // -1: the queue is empty
  int phase, item, merged;
  int e, n0, nb, nkb;                          // strips: nb = 256-row block of dW
  int a_row0, a_ntok, a_mb_first, a_mb_count;  // strips: a_row0 = first padded row, a_ntok = rows of the expert
  int b_row0, b_ntok, b_mb_first, b_mb_count;
};
static_assert(sizeof(WorkDesc) == 64, "published as four 16-byte stores");
struct __align__(16) TicketRing {
  WorkDesc work[TK_RING];
  uint64_t full[TK_RING];    // in each CTA: the slot holds an item
  uint64_t empty[TK_RING];   // used in the even CTA: every consumer of both CTAs has read the slot
};
// consumers: in each CTA both loaders and the 4 epilogue warps, plus the MMA issuer of the even CTA
constexpr int TK_CONSUMERS = 2 * (2 + EPI_WARPS) + 1;

__device__ __forceinline__ void ring_publish(TicketRing* r, uint32_t n, const WorkDesc& wd) {   // one lane; the slot is free
  const int slot = n % TK_RING;
  const uint4* src = reinterpret_cast<const uint4*>(&wd);
#pragma unroll
  for (uint32_t rank = 0; rank < 2; ++rank) {
    const uint32_t dst = map_to_rank(smem_u32(&r->work[slot]), rank);
#pragma unroll
    for (int q = 0; q < 4; ++q) st_cluster_v4(dst + 16 * q, src[q]);
    mbar_arrive_cluster_addr(map_to_rank(smem_u32(&r->full[slot]), rank));   // release: the item is visible
  }
}
// All lanes of a consumer warp; returns false on a failed wait.
__device__ __forceinline__ bool ring_take(TicketRing* r, uint32_t n, WorkDesc* wd, int lane, const WaitCtl& wc) {
  const int slot = n % TK_RING;
  int ok = 1;
  if (lane == 0) ok = mbar_wait_cluster(&r->full[slot], (n / TK_RING) & 1, wc, SITE_FULL, -8, 100) ? 1 : 0;
  if (!__shfl_sync(0xffffffffu, ok, 0)) return false;
  *wd = r->work[slot];
  __syncwarp();
  if (lane == 0) mbar_arrive_leader(&r->empty[slot]);
  return true;
}
__device__ __forceinline__ SwapWork desc_swap_work(const WorkDesc& wd) {
  SwapWork w;
  w.merged = wd.merged != 0;
  w.a.e = w.b.e = wd.e; w.a.n0 = w.b.n0 = wd.n0; w.a.nb = w.b.nb = wd.nb; w.a.nkb = w.b.nkb = wd.nkb;
  w.a.row0 = wd.a_row0; w.a.ntok = wd.a_ntok; w.a.mb_first = wd.a_mb_first; w.a.mb_count = wd.a_mb_count;
  w.b.row0 = wd.b_row0; w.b.ntok = wd.b_ntok; w.b.mb_first = wd.b_mb_first; w.b.mb_count = wd.b_mb_count;
  return w;
}
__device__ __forceinline__ Strip desc_strip(const WorkDesc& wd) {
  Strip st;
  st.e = wd.e; st.mp = wd.nb; st.row0 = wd.a_row0; st.rows = wd.a_ntok; st.nkb = wd.nkb;
  st.resident = st.nkb <= A_RES_KB;
  return st;
}
__device__ __forceinline__ void pack_swap_work(WorkDesc& wd, const SwapWork& w) {
  wd.merged = w.merged ? 1 : 0;
  wd.e = w.a.e; wd.n0 = w.a.n0; wd.nb = w.a.nb; wd.nkb = w.a.nkb;
  wd.a_row0 = w.a.row0; wd.a_ntok = w.a.ntok; wd.a_mb_first = w.a.mb_first; wd.a_mb_count = w.a.mb_count;
  wd.b_row0 = w.b.row0; wd.b_ntok = w.b.ntok; wd.b_mb_first = w.b.mb_first; wd.b_mb_count = w.b.mb_count;
}
// Decode item `item` of phase `phase` (scheduler); *first / *count: the M-blocks whose dependent event it waits for.
template <bool BWD>
__device__ __forceinline__ void decode_item(const FusedArgs& fa, int phase, int item, WorkDesc& wd, int* first, int* count) {
  const bool strip = BWD && (phase == 1 || phase == 3);
  if (strip) {
    const GemmArgs& a = fa.op[phase];
    const Strip st = decode_strip(a, item);
    wd.merged = 0; wd.e = st.e; wd.n0 = 0; wd.nb = st.mp; wd.nkb = st.nkb;
    wd.a_row0 = st.row0; wd.a_ntok = st.rows; wd.a_mb_first = a.mb_start[st.e];
    wd.a_mb_count = a.mb_start[st.e + 1] - a.mb_start[st.e];
    wd.b_row0 = wd.b_ntok = wd.b_mb_first = wd.b_mb_count = 0;
    *first = wd.a_mb_first; *count = st.nkb > 0 ? wd.a_mb_count : 0;   // all rows of the expert
    return;
  }
  SwapWork w;
  if (!BWD) w = phase == 0 ? decode_swap_work<GEMM_GATE_UP>(fa.op[0], item) : decode_swap_work<GEMM_DOWN>(fa.op[1], item);
  else w = phase == 0 ? decode_swap_work<GEMM_ACT_GRAD>(fa.op[0], item) : decode_swap_work<GEMM_GATE_GRAD>(fa.op[2], item);
  pack_swap_work(wd, w);
  *first = w.a.mb_first; *count = w.a.mb_count + w.b.mb_count;
}

// Items of each phase and their prefix sums: ticket t belongs to phase p iff start[p] <= t < start[p + 1].
struct PhaseTable {
  int start[SCHED_MAX_SEG + 1];
};
template <bool BWD>
__device__ __forceinline__ PhaseTable make_phase_table(const FusedArgs& fa) {
  PhaseTable pt;
  pt.start[0] = 0;
  if (!BWD) {
    pt.start[1] = total_swap_work<GEMM_GATE_UP>(fa.op[0]);
    pt.start[2] = pt.start[1] + total_swap_work<GEMM_DOWN>(fa.op[1]);
    pt.start[3] = pt.start[4] = pt.start[2];
  } else {
    pt.start[1] = total_swap_work<GEMM_ACT_GRAD>(fa.op[0]);
    pt.start[2] = pt.start[1] + wgrad_strips(fa.op[1]);
    pt.start[3] = pt.start[2] + total_swap_work<GEMM_GATE_GRAD>(fa.op[2]);
    pt.start[4] = pt.start[3] + wgrad_strips(fa.op[3]);
  }
  return pt;
}
// Where each row-space phase's item list starts when there are shared experts (schedule.h, rotate_index): at the
// first item of the first shared expert.  `first[p]` = 0: no rotation (no shared experts, or a weight-gradient phase).
template <int MODE>
__device__ __forceinline__ int swap_first_item(const GemmArgs& a, int first_shared) {
  return (swap_merges<MODE>() ? a.work_start : a.pair_start)[first_shared] * a.n_tiles_n;
}
template <bool BWD>
__device__ __forceinline__ PhaseTable make_rotation_table(const FusedArgs& fa) {
  PhaseTable r;
  for (int p = 0; p <= SCHED_MAX_SEG; ++p) r.start[p] = 0;
  const int S = fa.cp.kp - fa.cp.k, E = fa.cp.Ep - S;
  if (S == 0) return r;
  if (!BWD) {
    r.start[0] = swap_first_item<GEMM_GATE_UP>(fa.op[0], E);
    r.start[1] = swap_first_item<GEMM_DOWN>(fa.op[1], E);
  } else {
    r.start[0] = swap_first_item<GEMM_ACT_GRAD>(fa.op[0], E);
    r.start[2] = swap_first_item<GEMM_GATE_GRAD>(fa.op[2], E);
  }
  return r;
}
__device__ __forceinline__ int phase_of(const PhaseTable& pt, int t) {
  int p = 0;
  while (p + 1 < SCHED_MAX_SEG && t >= pt.start[p + 1]) ++p;
  return p;
}

__device__ __forceinline__ ChainDeps phase_deps(const FusedArgs& fa, int phase, const WaitCtl& wc, const TraceCtl& tr) {
  ChainDeps d;
  d.ctr = fa.ctr;
  d.wait_kind = phase_wait_kind(fa.cp, phase);
  d.wait_thr = phase_wait_thr(fa.cp, phase);
  d.trig_kind = phase_trigger_kind(fa.cp, phase);
  d.phase = phase;
  d.wc = wc;
  d.tr = tr;
  return d;
}

// ---------------------------------------------------------------- one item, by role
template <bool BWD>
__device__ __forceinline__ bool load_item(const FusedArgs& fa, const WorkDesc& wd, uint8_t* smem, PipeBarriers* bars,
                                          LoaderState& ls, bool second_warp, int rank, int lane, const WaitCtl& wc,
                                          const ChainDeps& dep) {
  const int phase = wd.phase, t = wd.item;
  if (BWD && (phase == 1 || phase == 3))
    return wgrad_load_strip(fa.op[phase], smem, bars, ls, second_warp, rank, lane, desc_strip(wd), t, wc, dep);
  const SwapWork wk = desc_swap_work(wd);
  if (!BWD) {
    if (phase == 0) return swap_load_item<GEMM_GATE_UP>(fa.op[0], smem, bars, ls, second_warp, rank, lane, wk, t, wc, dep);
    return swap_load_item<GEMM_DOWN>(fa.op[1], smem, bars, ls, second_warp, rank, lane, wk, t, wc, dep);
  }
  if (phase == 0) return swap_load_item<GEMM_ACT_GRAD>(fa.op[0], smem, bars, ls, second_warp, rank, lane, wk, t, wc, dep);
  return swap_load_item<GEMM_GATE_GRAD>(fa.op[2], smem, bars, ls, second_warp, rank, lane, wk, t, wc, dep);
}
template <bool BWD>
__device__ __forceinline__ bool issue_item(const FusedArgs& fa, const WorkDesc& wd, uint8_t* smem, PipeBarriers* bars,
                                           uint32_t tmem_base, IssuerState& is, bool issue, const WaitCtl& wc,
                                           const ChainDeps& dep) {
  const int phase = wd.phase, t = wd.item;
  if (BWD && (phase == 1 || phase == 3))
    return wgrad_issue_strip(fa.op[phase], smem, bars, tmem_base, is, issue, desc_strip(wd), t, wc, dep);
  const SwapWork wk = desc_swap_work(wd);
  if (!BWD) {
    if (phase == 0) return swap_issue_item<GEMM_GATE_UP>(fa.op[0], smem, bars, tmem_base, is, issue, wk, t, wc, dep);
    return swap_issue_item<GEMM_DOWN>(fa.op[1], smem, bars, tmem_base, is, issue, wk, t, wc, dep);
  }
  if (phase == 0) return swap_issue_item<GEMM_ACT_GRAD>(fa.op[0], smem, bars, tmem_base, is, issue, wk, t, wc, dep);
  return swap_issue_item<GEMM_GATE_GRAD>(fa.op[2], smem, bars, tmem_base, is, issue, wk, t, wc, dep);
}
template <bool BWD>
__device__ __forceinline__ bool epilogue_item(const FusedArgs& fa, const WorkDesc& wd, uint8_t* smem, PipeBarriers* bars,
                                              uint32_t tmem_base, EpiState& es, int rank, int quad, int lane,
                                              const WaitCtl& wc, const ChainDeps& dep) {
  const int phase = wd.phase, t = wd.item;
  if (BWD && (phase == 1 || phase == 3))
    return wgrad_epilogue_strip(fa.op[phase], smem, bars, tmem_base, es, rank, quad, lane, desc_strip(wd), t, wc, dep);
  const SwapWork wk = desc_swap_work(wd);
  if (!BWD) {
    if (phase == 0)
      return swap_epilogue_item<GEMM_GATE_UP>(fa.op[0], smem, bars, tmem_base, es, rank, quad, lane, wk, t, wc, dep);
    return swap_epilogue_item<GEMM_DOWN>(fa.op[1], smem, bars, tmem_base, es, rank, quad, lane, wk, t, wc, dep);
  }
  if (phase == 0)
    return swap_epilogue_item<GEMM_ACT_GRAD>(fa.op[0], smem, bars, tmem_base, es, rank, quad, lane, wk, t, wc, dep);
  return swap_epilogue_item<GEMM_GATE_GRAD>(fa.op[2], smem, bars, tmem_base, es, rank, quad, lane, wk, t, wc, dep);
}

// ---------------------------------------------------------------- the kernel
template <bool BWD>
__global__ void __launch_bounds__(FUSED_THREADS, 1) fused_chain_kernel(const __grid_constant__ FusedArgs fa) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  PipeBarriers* bars = reinterpret_cast<PipeBarriers*>(smem + FUSED_LAYOUT_BYTES);
  static_assert(sizeof(PipeBarriers) <= 256 && sizeof(TicketRing) <= 384, "shared-memory bookkeeping");
  TicketRing* ring = reinterpret_cast<TicketRing*>(reinterpret_cast<uint8_t*>(bars) + 256);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const WaitCtl wc{fa.status, fa.budget_ns};
  const TraceCtl tr{fa.trace, fa.trace_cap, fa.ctr + CTR_TRACE_CURSOR};
  const int M = fa.lv.meta[0];

  if (threadIdx.x == 0) {
    pipe_init(bars);
    for (int s = 0; s < TK_RING; ++s) {
      mbar_init(&ring->full[s], 1);
      mbar_init(&ring->empty[s], TK_CONSUMERS);
    }
    mbar_fence_init();
    fence_proxy_async();
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

  if (warp == SCHED_WARP && rank == 0) {
    // ------------------------------------------------ scheduler of the pair (even CTA)
    const PhaseTable pt = make_phase_table<BWD>(fa);
    const PhaseTable rot = make_rotation_table<BWD>(fa);   // first item of the first shared expert in each row-space phase
    const int total = pt.start[SCHED_MAX_SEG];
    for (uint32_t n = 0;; ++n) {
      // a free ring slot first, then the ticket: a pair never holds more unstarted items than the ring has slots
      int ok = 1;
      if (lane == 0) ok = mbar_wait_cluster(&ring->empty[n % TK_RING], ((n / TK_RING) & 1) ^ 1, wc, SITE_EMPTY, -7, 100) ? 1 : 0;
      if (!__shfl_sync(0xffffffffu, ok, 0)) break;
      int t = 0;
      if (lane == 0) t = atomicAdd(&fa.ctr[CTR_MAT_TICKET], 1);
      t = __shfl_sync(0xffffffffu, t, 0);
      WorkDesc wd;
      wd.ticket = t;
      if (t >= total) {
        wd.ticket = -1;
        wd.phase = wd.item = wd.merged = wd.e = wd.n0 = wd.nb = wd.nkb = 0;
        wd.a_row0 = wd.a_ntok = wd.a_mb_first = wd.a_mb_count = wd.b_row0 = wd.b_ntok = wd.b_mb_first = wd.b_mb_count = 0;
        if (lane == 0) ring_publish(ring, n, wd);
        break;
      }
      wd.phase = phase_of(pt, t);
      wd.item = t - pt.start[wd.phase];
      if (rot.start[wd.phase]) wd.item = rotate_index(wd.item, rot.start[wd.phase], pt.start[wd.phase + 1] - pt.start[wd.phase]);
      const ChainDeps dep = phase_deps(fa, wd.phase, wc, tr);
      uint64_t t0 = 0;
      if (tr.buf && lane == 0) t0 = globaltimer_ns();
      int first, count;
      decode_item<BWD>(fa, wd.phase, wd.item, wd, &first, &count);
      if (!dep.wait(first, count, lane, t)) break;   // the item's dependent events (Section 4.3)
      if (lane == 0) {
        const uint64_t td = tr.buf ? globaltimer_ns() : 0;
        ring_publish(ring, n, wd);
        if (tr.buf) dep.trace(TR_SCHED, wd.item, t0, td, globaltimer_ns());
      }
    }
  } else if (warp < ROLE_WARPS && !(warp == 1 && rank != 0)) {
    // ------------------------------------------------ matrix roles: the pair's items in ticket order
    LoaderState ls;
    IssuerState is;
    EpiState es;
    int cur_phase = 0;
    bool ok = true;
    for (uint32_t n = 0; ok; ++n) {
      WorkDesc wd;
      ok = ring_take(ring, n, &wd, lane, wc);
      if (!ok || wd.ticket < 0) break;
      const int phase = wd.phase;
      const ChainDeps dep = phase_deps(fa, phase, wc, tr);
      // ---- phase boundary (see phase_wait): staging and operand ring of the new phase overlap the old ones
      if (phase != cur_phase) {
        cur_phase = phase;
        ls.s = ls.a_s = 0;   // every stage has been consumed: the new phase's ring (of its own depth) starts at 0
        is.s = is.a_s = 0;
        if (warp != 1) {
          int go = 1;
          if (lane == 0) {
            if (warp >= 2 && warp < 2 + EPI_WARPS) {
              tma_store_wait_all();
              epi_enter_phase(bars, warp & 3, phase);
            }
            go = phase_wait(bars, phase, wc) ? 1 : 0;
          }
          es.round = 0;
          if (!__shfl_sync(0xffffffffu, go, 0)) break;
        }
      }
      if (warp == 0 || warp == 6)
        ok = load_item<BWD>(fa, wd, smem, bars, ls, warp == 6, rank, lane, wc, dep);
      else if (warp == 1)
        ok = issue_item<BWD>(fa, wd, smem, bars, tmem_base, is, lane == 0, wc, dep);
      else
        ok = epilogue_item<BWD>(fa, wd, smem, bars, tmem_base, es, rank, warp & 3, lane, wc, dep);
    }
    if (warp >= 2 && warp < 2 + EPI_WARPS && lane == 0) {
      tma_store_wait_all();
      epi_enter_phase(bars, warp & 3, SCHED_MAX_SEG);   // nothing of this warp is left in shared memory
    }
    if (warp == 1 && lane == 0 && (!ok || *reinterpret_cast<volatile int*>(&fa.status->abort))) issuer_drain(bars, fa.status);
  }

  // ------------------------------------------------ vector workers: the dedicated warps from the start, the
  // matrix-role warps once the matrix queue is empty (the tail of the vector queue -- combine -- runs on the
  // whole SM)
  __syncwarp();
  vector_worker_loop(fa, wc, tr, M, lane, warp > SCHED_WARP && warp <= SCHED_WARP + BACKGROUND_GATHERERS);

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

cudaError_t launch_fused(bool bwd, const FusedArgs& fa, int num_sms, bool cooperative, cudaStream_t s, int* launches) {
  ++*launches;
  static PairLaunchState st_fwd, st_bwd;
  if (bwd)
    return launch_on_pairs(st_bwd, fused_chain_kernel<true>, fa, FUSED_THREADS, FUSED_SMEM_BYTES, num_sms, cooperative, s);
  return launch_on_pairs(st_fwd, fused_chain_kernel<false>, fa, FUSED_THREADS, FUSED_SMEM_BYTES, num_sms, cooperative, s);
}

}  // namespace moe
