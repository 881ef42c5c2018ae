// The tile schedule of the single persistent launch: one ticket-ordered matrix queue (the counterpart
// of the paper's matrix-core task queue, Section 4.3), two ticket-ordered vector queues, and the
// dependent / trigger event counters of every tile with their static thresholds.  Plain host/device
// code without CUDA calls, so the same functions drive the kernels and the CPU-side simulation that
// checks the schedule for coverage and deadlock freedom.
//
// Matrix queue.  The operators of a pass are phases in dependency order -- forward: gate+up, down;
// backward: act_grad, w2_grad, gate_grad, w1_grad -- and phase p's work items are numbered
// expert-major (column tile slow, token tile fast).  The queue is the concatenation of the phases'
// item lists, fixed before the launch; CTA pairs take its tickets in order.  The order of the queue
// is static (the paper's statically ordered task lists); which pair runs which item is decided by
// arrival, which keeps the items in flight a contiguous window of the queue: items that share an
// operand (the token tiles of one expert and column tile share its weight slab, the strips of one
// expert share its rows) start within microseconds of each other and meet in L2 however the pairs'
// speeds differ.  A pair that reaches phase p+1 early starts on it while others still finish phase p.
//
// Events (Section 4.3).  Per M-block (128 rows of the padded expert-ordered row space) three
// counters with static thresholds:
//   gathered   += 1 per gather sub-task (4 rows)                  threshold GATHER_SUB
//   activated  += 1 per epilogue warp and column tile of phase 0  threshold SIG * column tiles
//   done       += 1 per epilogue warp and column tile of the last row-space phase (down / gate_grad)
// A phase-0 item depends on `gathered` of its M-blocks, a down / gate_grad item and a w1_grad
// strip on `activated`, a w2_grad strip on `gathered`; a combine task depends on `done` of the
// M-blocks that hold its token's rows (many-to-many: up to k+S counters per token), the
// routing-weight-gradient task of an M-block on its `activated`.
//
// Deadlock freedom: every item's producers have smaller tickets (an earlier phase) or are vector
// tasks that never wait for matrix items of the same or a later phase; tickets are taken in order
// by pairs that are all resident (cooperative launch), so the holder of the smallest unfinished
// ticket always finds its dependent events met in finite time.
#pragma once

#include <stdint.h>

#ifdef __CUDACC__
#define MOE_HD __host__ __device__ __forceinline__
#else
#define MOE_HD inline
#endif

namespace moe {

constexpr int SCHED_MAX_SEG = 4;       // phases of a pass
constexpr int GATHER_SUB = 32;         // vector sub-tasks per M-block gather (4 rows each: the first M-blocks of a
                                       // launch, which every CTA pair waits for, are complete after a few microseconds)
constexpr int EPI_WARPS = 4;           // epilogue warps per CTA
constexpr int SIG = 2 * EPI_WARPS;     // signals per (M-block, column tile): every epilogue warp of the pair
constexpr int COMBINE_TOKENS = 1;      // tokens per combine task

enum VecOp : int { VEC_GATHER = 0, VEC_DW = 2, VEC_COMBINE = 3 };

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

// Which experts merge their last two units in the phases that merge: an odd count of three or more M-blocks whose
// last block is mostly padding (at most MERGE_TAIL_MAX rows).  Then the last unit (block + tail) is small, staging the
// weights once for both units saves the larger half of the shared-memory traffic, and the epilogue that merging
// exposes (both accumulators are in use) is short.  With a full last block (e.g. 384 rows) the exposed epilogue
// costs more than the second weight pass: down was 5 % faster unmerged there and 6 % slower on 257..320-row experts.
constexpr int MERGE_TAIL_MAX = 64;
MOE_HD bool expert_merges(int rows, int mblocks) {
  return (mblocks & 1) && mblocks >= 3 && rows - (mblocks - 1) * 128 <= MERGE_TAIL_MAX;
}

// One work item of a row-space phase: a token tile (unit) of an expert and a column tile, or -- in the
// phases that merge, for an expert that merges (expert_merges) -- its last two units under one k-loop.  `start[e]` = first unit (or first merged item) of expert e, `blk_expert[i]` =
// expert of unit / item i (both from the layout kernels).
struct SwapItem {
  int e, nb;            // expert, column tile
  int unit;             // first unit of the item
  int merged;           // 1: units `unit` and `unit + 1`
  int mb_first;         // first M-block (absolute) of the item
  int mb_count;         // M-blocks of the item (both units): 1..3, contiguous
  int mb_count_a;       // M-blocks of the first unit
};
MOE_HD SwapItem decode_swap_item(int t, int n_tiles_n, bool merges, const int* start, const int* blk_expert,
                                 const int* mb_start) {
  SwapItem it;
  const int e = blk_expert[t / n_tiles_n];
  const int ws = start[e];
  const int wcount = start[e + 1] - ws;
  const int local = t - ws * n_tiles_n;
  it.nb = local / wcount;
  const int wi = local - it.nb * wcount;
  const int mc = mb_start[e + 1] - mb_start[e];
  it.e = e;
  it.unit = wi;
  // the item table has one entry fewer than the expert has units exactly when the expert merges
  it.merged = (merges && wcount == ((mc + 1) >> 1) - 1 && wi == wcount - 1) ? 1 : 0;
  int f, c;
  balanced_unit(mc, wi, &f, &c);
  it.mb_first = mb_start[e] + f;
  it.mb_count_a = c;
  it.mb_count = c;
  if (it.merged) {
    int f2, c2;
    balanced_unit(mc, wi + 1, &f2, &c2);
    it.mb_count += c2;
  }
  return it;
}

// What a pass consists of (filled on the host from the layer's shape).
struct ChainParams {
  int is_bwd;
  int Ep, T, k, kp;
  int n_phases;                 // 2 (forward) or 4 (backward)
  int ntn[SCHED_MAX_SEG];       // column tiles per item (row-space phases) / per strip (weight gradients)
  int strips[SCHED_MAX_SEG];    // weight-gradient phases: strips (256 rows of dW) per expert; else 0
  int merges[SCHED_MAX_SEG];    // row-space phases: 1 if the phase merges the last two units of odd experts
  int dep_extra;                // test hook: added to the `activated` threshold (> 0 = never reached)
  int want_dw;                  // backward: routing-weight-gradient tasks are part of the vector queue
};
MOE_HD int thr_gathered() { return GATHER_SUB; }
MOE_HD int thr_activated(const ChainParams& cp) { return SIG * cp.ntn[0] + cp.dep_extra; }
MOE_HD int thr_done(const ChainParams& cp) { return SIG * cp.ntn[cp.is_bwd ? 2 : 1]; }

// Queue order with shared experts: every queue of the persistent launch (gather tasks, the items of the row-space
// phases) starts at the first shared expert and wraps around.  Every token has a row in every shared expert, and those
// experts come last in expert order: taken in expert order, no token would be complete before the very end and the
// whole combine would be a tail.  Started first, the shared rows are done early and a token is complete with its last
// ROUTED row, as without shared experts.  Dependencies are unchanged (an item still follows its producers in every
// queue, all queues being rotated alike); only the order among independent tasks changes (Section 4.5).
MOE_HD int rotate_index(int i, int first, int n) {
  const int j = i + first;
  return j >= n ? j - n : j;
}

// ---------------------------------------------------------------- counters (ints in device memory)
constexpr int CTR_VEC_TICKET = 0, CTR_TRACE_CURSOR = 1, CTR_MAT_TICKET = 2, CTR_POST_TICKET = 3, CTR_PER_MB = 8, CTR_STRIDE = 4;
// combine tasks finished, and the word that turns 1 when all of them are (a copy-out stream may wait on it)
constexpr int CTR_COMBINE_DONE = 4, CTR_OUT_READY = 5;
enum CtrKind : int { CTR_GATHERED = 0, CTR_ACTIVATED = 1, CTR_DONE = 2, CTR_NONE = -1 };
MOE_HD int ctr_index(int mb, int kind) { return CTR_PER_MB + CTR_STRIDE * mb + kind; }
MOE_HD int ctr_ints(int cap_mblocks) { return CTR_PER_MB + CTR_STRIDE * cap_mblocks; }

// dependent / trigger counter kind of each phase
MOE_HD int phase_wait_kind(const ChainParams& cp, int phase) {
  if (!cp.is_bwd) return phase == 0 ? CTR_GATHERED : CTR_ACTIVATED;
  return (phase == 0 || phase == 1) ? CTR_GATHERED : CTR_ACTIVATED;
}
MOE_HD int phase_wait_thr(const ChainParams& cp, int phase) {
  return phase_wait_kind(cp, phase) == CTR_GATHERED ? thr_gathered() : thr_activated(cp);
}
MOE_HD int phase_trigger_kind(const ChainParams& cp, int phase) {
  if (!cp.is_bwd) return phase == 0 ? CTR_ACTIVATED : CTR_DONE;
  return phase == 0 ? CTR_ACTIVATED : (phase == 2 ? CTR_DONE : CTR_NONE);
}

// ---------------------------------------------------------------- vector queues (ticket order)
// Two queues: the gather sub-tasks in M-block order, and behind them the tasks that consume matrix tiles
// (backward: the routing-weight gradient per M-block; then the combine tasks).  A worker leaves the first
// queue for the second only when the first is empty -- or earlier, when it is not one of the few workers
// that keep gathering in the background (see fused.cu).
constexpr int GATHER_FAST_MBLOCKS = 32;   // M-blocks every vector worker helps to gather at the start of a launch
struct VecTask {
  int op;       // VecOp
  int idx;      // gather: M-block * GATHER_SUB + sub-task; dw: M-block; combine: task (COMBINE_TOKENS tokens)
};
MOE_HD int gather_total(int M) { return GATHER_SUB * M; }
MOE_HD int post_total(const ChainParams& cp, int M) {
  int n = (cp.T + COMBINE_TOKENS - 1) / COMBINE_TOKENS;
  if (cp.is_bwd && cp.want_dw) n += M;
  return n;
}
MOE_HD VecTask decode_post_ticket(const ChainParams& cp, int t, int M) {
  VecTask v;
  if (cp.is_bwd && cp.want_dw) {
    if (t < M) { v.op = VEC_DW; v.idx = t; return v; }
    t -= M;
  }
  v.op = VEC_COMBINE; v.idx = t;
  return v;
}

}  // namespace moe
