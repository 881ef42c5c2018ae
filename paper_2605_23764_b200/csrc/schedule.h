// The static tile schedule of the single persistent launch: two ticket-ordered queues (matrix
// tiles and vector tasks, the counterparts of the paper's CTQ and VTQ, Section 4.3), the dependent
// and trigger counters of every tile with their static thresholds, and the decode from a ticket to
// a tile.  Plain host/device code without CUDA calls, so the same functions drive the kernels and
// the CPU-side simulation that checks the schedule for deadlock freedom.
//
// Matrix queue.  "Steps" run over the experts in order.  Forward step i holds the gate+up tiles of
// expert i (column tile slow, M-block fast: tiles in flight together share one slab of weights)
// and the down tiles of expert i-lag; the lag keeps a consumer's producers a few hundred tickets
// ahead, so its dependency is normally met when its ticket comes up while the intermediate it reads
// is still L2-resident (the paper's producer/consumer placement, Section 4.4).  Backward step i
// holds the act_grad tiles of expert i and its w2_grad strips (they share the gathered upstream
// gradient: the paper's cache-guided GMM interleaving, Section 4.5), then the gate_grad tiles of
// expert i-lag and its w1_grad strips (they share dH).  A weight-gradient ticket is a strip: one
// 128-row block of the gradient across all its column tiles.
//
// Every tile's producers have smaller tickets in their queue; queues are consumed in ticket
// order by workers that are all resident, hence no deadlock (Section 4.3, correctness argument).
#pragma once

#include <stdint.h>

#ifdef __CUDACC__
#define MOE_HD __host__ __device__ __forceinline__
#else
#define MOE_HD inline
#endif

namespace moe {

constexpr int SCHED_MAX_SEG = 4;
constexpr int GATHER_SUB = 8;          // vector sub-tasks per M-block gather (16 rows each)
constexpr int EPI_WARPS = 4;           // epilogue warps per matrix tile; each signals once
constexpr int COMBINE_TOKENS = 2;      // tokens per combine task
constexpr int ZERO_CHUNKS = 64;        // zero-fill tasks per expert slab pair (only empty experts do work)
constexpr int DW_SLOTS = 1024;         // routing-weight-gradient entries per task

// op codes of matrix tiles (values = GemmMode) and vector tasks
enum VecOp : int { VEC_GATHER = 0, VEC_ZERO = 1, VEC_DW = 2, VEC_COMBINE = 3, VEC_NONE = -1 };

struct SchedParams {
  int is_bwd;
  int pair;                // 1: a row-space ticket covers a PAIR of M-blocks (two CTAs on a 256-row tile)
  int lag;                 // in experts
  int Ep;
  int T, k;
  // tickets per M-block (row-space operators) / per expert (weight-gradient strips), per segment:
  //   forward : seg0 = gate+up (column tiles per M-block), seg1 = down (per M-block, lagged)
  //   backward: seg0 = act_grad (per M-block), seg1 = w2_grad strips (per expert),
  //             seg2 = gate_grad (per M-block, lagged), seg3 = w1_grad strips (per expert, lagged)
  int seg_tiles[SCHED_MAX_SEG];
  int strip_tiles[2];      // column tiles in one w2_grad / w1_grad strip
  int dep_extra;           // test hook: added to the activation-counter thresholds (> 0 = never reached)
  int tokcol;              // 1 (with pair): token-column tiles, balanced units of one or two M-blocks
  int sig;                 // signals one (M-block, column tile) sends to its counters: EPI_WARPS, or
                           // 2 * EPI_WARPS when the epilogue warps of both CTAs of a pair cover every row
};

// Token-column tiles: the ceil(mc / 2) row-space units of an expert with mc M-blocks.  An odd count
// does not leave a lone M-block at the end (a tile of a few tokens still streams the whole weight
// tile): the single block sits before the last unit, which takes the last full block and the tail.
MOE_HD void balanced_unit(int mc, int u, int* first, int* count) {
  const int uc = (mc + 1) >> 1;
  *first = 2 * u;
  *count = 2;
  if ((mc & 1) == 0) return;
  if (u == uc - 1) {
    if (mc == 1) { *first = 0; *count = 1; }
    else *first = 2 * u - 1;
  } else if (u == uc - 2) {
    *count = 1;
  }
}

MOE_HD int expert_mblocks(const int* mb_start, int e) { return mb_start[e + 1] - mb_start[e]; }
// row-space scheduling units of an expert: its M-blocks, or its M-block pairs
MOE_HD int expert_units(const SchedParams& sp, const int* mb_start, int e) {
  const int m = expert_mblocks(mb_start, e);
  return sp.pair ? (m + 1) >> 1 : m;
}

// tickets of step i
MOE_HD int step_tiles(const SchedParams& sp, int i, const int* mb_start) {
  int n = 0;
  const int j = i - sp.lag;
  if (i < sp.Ep) {
    const int m = expert_units(sp, mb_start, i);
    n += m * sp.seg_tiles[0];
    if (sp.is_bwd && m > 0) n += sp.seg_tiles[1];
  }
  if (j >= 0 && j < sp.Ep) {
    const int m = expert_units(sp, mb_start, j);
    if (!sp.is_bwd) {
      n += m * sp.seg_tiles[1];
    } else {
      n += m * sp.seg_tiles[2];
      if (m > 0) n += sp.seg_tiles[3];
    }
  }
  return n;
}

struct MatTile {
  int op;        // GemmMode
  int slot;      // which GemmArgs of the launch (segment index)
  int e;
  int mb;        // first M-block of the tile (row-space operators) or -1
  int mb_count;  // M-blocks of the tile: 1, or 2 for a full pair
  int idx;       // column tile (row-space operators) / strip index = 128-row block of the gradient
  int group;     // tiles processed under this ticket (1, or the strip's column tiles)
  // dependency: every counter dep_ctr[dep_first .. dep_first+dep_count) must reach dep_thr
  int dep_base;  // 0 = gather counters, 1 = activation counters
  int dep_first, dep_count, dep_thr;
  // trigger: counter incremented once per epilogue warp after the tile's stores are complete
  int trig_base; // 1 = activation counter of mb, 2 = global done counter, -1 = none
  int trig_also_ag;  // backward act_grad also bumps the global act_grad counter
};

// Decode ticket t of step i (step_start[i] <= t < step_start[i+1]) into a tile (or strip).
MOE_HD MatTile decode_matrix_ticket_at(const SchedParams& sp, int t, int i, const int* step_start,
                                       const int* mb_start) {
  const int j = i - sp.lag;
  int r = t - step_start[i];
  MatTile m;
  m.trig_also_ag = 0;
  m.group = 1;
  m.mb_count = 0;
  const int stride = sp.pair ? 2 : 1;  // M-blocks per row-space unit
  if (i < sp.Ep) {
    const int uc = expert_units(sp, mb_start, i), mc = expert_mblocks(mb_start, i);
    if (r < uc * sp.seg_tiles[0]) {
      m.slot = 0; m.op = sp.is_bwd ? 2 /*ACT_GRAD*/ : 0 /*GATE_UP*/;
      m.idx = r / uc;
      const int u = r - m.idx * uc;
      m.mb = mb_start[i] + stride * u; m.mb_count = (mc - stride * u) < stride ? (mc - stride * u) : stride; m.e = i;
      if (sp.pair && sp.tokcol) { int f, c; balanced_unit(mc, u, &f, &c); m.mb = mb_start[i] + f; m.mb_count = c; }
      m.dep_base = 0; m.dep_first = m.mb; m.dep_count = m.mb_count; m.dep_thr = GATHER_SUB;
      m.trig_base = 1; m.trig_also_ag = sp.is_bwd;
      return m;
    }
    r -= uc * sp.seg_tiles[0];
    if (sp.is_bwd && mc > 0) {
      if (r < sp.seg_tiles[1]) {
        m.slot = 1; m.op = 4 /*WGRAD*/; m.mb = -1; m.e = i; m.idx = r; m.group = sp.strip_tiles[0];
        m.dep_base = 0; m.dep_first = mb_start[i]; m.dep_count = mc; m.dep_thr = GATHER_SUB;
        m.trig_base = -1;
        return m;
      }
      r -= sp.seg_tiles[1];
    }
  }
  // lagged segments of expert j
  const int uc = expert_units(sp, mb_start, j), mc = expert_mblocks(mb_start, j);
  if (!sp.is_bwd || r < uc * sp.seg_tiles[2]) {
    const int seg = sp.is_bwd ? 2 : 1;
    m.slot = seg; m.op = sp.is_bwd ? 3 /*GATE_GRAD*/ : 1 /*DOWN*/; m.e = j;
    m.idx = r / uc;
    const int u = r - m.idx * uc;
    m.mb = mb_start[j] + stride * u; m.mb_count = (mc - stride * u) < stride ? (mc - stride * u) : stride;
    if (sp.pair && sp.tokcol) { int f, c; balanced_unit(mc, u, &f, &c); m.mb = mb_start[j] + f; m.mb_count = c; }
    m.dep_base = 1; m.dep_first = m.mb; m.dep_count = m.mb_count; m.dep_thr = sp.sig * sp.seg_tiles[0] + sp.dep_extra;
    m.trig_base = 2;
    return m;
  }
  r -= uc * sp.seg_tiles[2];
  m.slot = 3; m.op = 4 /*WGRAD*/; m.mb = -1; m.e = j; m.idx = r; m.group = sp.strip_tiles[1];
  m.dep_base = 1; m.dep_first = mb_start[j]; m.dep_count = mc;
  m.dep_thr = sp.sig * sp.seg_tiles[0] + sp.dep_extra; m.trig_base = -1;
  return m;
}

// Decode ticket t (0 <= t < step_start[Ep+lag]) into a tile (or strip).
MOE_HD MatTile decode_matrix_ticket(const SchedParams& sp, int t, const int* step_start, const int* mb_start) {
  int lo = 0, hi = sp.Ep + sp.lag - 1;  // last step whose start <= t
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (step_start[mid] <= t) lo = mid; else hi = mid - 1;
  }
  return decode_matrix_ticket_at(sp, t, lo, step_start, mb_start);
}

// ---------------------------------------------------------------- vector queue
struct VecTask {
  int op;       // VecOp
  int idx;      // task index inside its kind
  int dep;      // 0 = none, 2 = global done counter, 3 = global act_grad counter
  int dep_thr;
};

MOE_HD int vec_total(const SchedParams& sp, int M) {
  int n = GATHER_SUB * M + (sp.T + COMBINE_TOKENS - 1) / COMBINE_TOKENS;
  if (sp.is_bwd) n += sp.Ep * ZERO_CHUNKS + (sp.T * sp.k + DW_SLOTS - 1) / DW_SLOTS;
  return n;
}

MOE_HD VecTask decode_vector_ticket(const SchedParams& sp, int t, int M) {
  VecTask v;
  v.dep = 0; v.dep_thr = 0;
  if (t < GATHER_SUB * M) { v.op = VEC_GATHER; v.idx = t; return v; }
  t -= GATHER_SUB * M;
  if (sp.is_bwd) {
    if (t < sp.Ep * ZERO_CHUNKS) { v.op = VEC_ZERO; v.idx = t; return v; }
    t -= sp.Ep * ZERO_CHUNKS;
    const int ndw = (sp.T * sp.k + DW_SLOTS - 1) / DW_SLOTS;
    if (t < ndw) {
      v.op = VEC_DW; v.idx = t; v.dep = 3; v.dep_thr = sp.sig * M * sp.seg_tiles[0];
      return v;
    }
    t -= ndw;
  }
  v.op = VEC_COMBINE; v.idx = t; v.dep = 2;
  v.dep_thr = sp.sig * M * (sp.is_bwd ? sp.seg_tiles[2] : sp.seg_tiles[1]);
  return v;
}

// Layout of the counter block in device memory (ints).
constexpr int CTR_MAT_TICKET = 0, CTR_VEC_TICKET = 1, CTR_DONE = 2, CTR_AG_DONE = 3, CTR_PER_MB = 8;
MOE_HD int ctr_gather(int mb) { return CTR_PER_MB + 2 * mb; }
MOE_HD int ctr_act(int mb) { return CTR_PER_MB + 2 * mb + 1; }
MOE_HD int ctr_ints(int cap_mblocks) { return CTR_PER_MB + 2 * cap_mblocks; }

}  // namespace moe
