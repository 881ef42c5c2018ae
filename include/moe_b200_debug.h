/*
 * moe_b200 -- test and diagnostic entry points of the library (not needed to run the layer):
 * views of workspace tensors, failure injection for the bounded waits, the host-only schedule
 * simulation and the per-tile trace.
 */
#ifndef MOE_B200_DEBUG_H
#define MOE_B200_DEBUG_H

#include "moe_b200.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Test/diagnostic access to workspace tensors of the last forward/backward.  `which` is a
 * MOE_BUF_* id; *ptr receives a device pointer into the workspace (valid until the next call on
 * the context), *elems its element count.  Rows of expert-ordered tensors live in a padded row
 * space: expert e starts at row pad_off[e] (a multiple of 128) and holds counts[e] rows. */
enum {
  MOE_BUF_COUNTS = 0,    /* int32 [E+S] */
  MOE_BUF_OFFSETS = 1,   /* int32 [E+S+1] */
  MOE_BUF_ROW_OF = 2,    /* int32 [T*(k+S)] unpadded rows */
  MOE_BUF_SRC_OF = 3,    /* int32 [T*(k+S)] */
  MOE_BUF_PROW_OF = 4,   /* int32 [T*(k+S)] padded rows */
  MOE_BUF_PAD_OFF = 5,   /* int32 [E+S+1] */
  MOE_BUF_XP = 6,        /* bf16 [R_pad][d]   gathered x */
  MOE_BUF_H = 7,         /* bf16 [R_pad][2F]  gate|up pre-activations */
  MOE_BUF_A = 8,         /* bf16 [R_pad][F]   w * silu(g) * u */
  MOE_BUF_Y = 9,         /* bf16 [R_pad][d]   expert outputs (already weighted) */
  MOE_BUF_DOUTP = 10,    /* bf16 [R_pad][d]   gathered dout */
  MOE_BUF_DH = 11,       /* bf16 [R_pad][2F]  gradient of the pre-activations */
  MOE_BUF_DXP = 12,      /* bf16 [R_pad][d]   per-row input gradient */
  MOE_BUF_META = 13,     /* int32 [8]: {num_mblocks, R_pad, rows, ...} */
  MOE_BUF_TRACE = 14,    /* int32 [8 * records]: raw trace records (MOE_FLAG_TRACE contexts) */
  MOE_BUF_EVENT_COUNTERS = 15, /* int32: event counters of the last persistent launch: [1] = trace
                            records written, from [8] on four ints per M-block {gathered, activated,
                            done, unused} */
};
int moe_debug_buffer(moe_ctx* ctx, int which, void** ptr, size_t* elems);

/* Failure-handling test hook: with on != 0 the persistent launches of this context wait for one more
 * producer signal than will ever arrive (a threshold nothing reaches).  The bounded waits then run
 * out after the wait budget, the kernel records MOE_ERR_TIMEOUT and returns normally (no trap, no
 * hang); moe_get_status reports it and the context stays usable once the hook is switched off. */
int moe_debug_set_unreachable_dependency(moe_ctx* ctx, int32_t on);

/* Profiling aid: with on != 0 the persistent launches of this context are made without the cooperative
 * launch attribute (some profilers reject cooperative launches of thread-block clusters).  The grid is
 * sized to what can be resident either way; what is lost is the driver's guarantee of co-residency when
 * other work shares the GPU -- every device-side wait stays bounded.  ctx == NULL switches the persistent
 * launches of the context-free entry points (moe_sched_study, moe_taskflow_run, moe_ep_dispatch, moe_ep_combine;
 * process-wide) instead. */
int moe_debug_set_plain_launch(moe_ctx* ctx, int32_t on);

/* Host-only check of the static tile schedule of the single persistent launch (Section 4.3: tasks
 * in statically ordered queues, dependent/trigger event counters with static thresholds).  For the
 * given per-expert row counts[Ep] and layer shape it builds the layout tables, the matrix queue of
 * each of `pairs` CTA pairs (the operators of the pass as consecutive phases, items dealt round-robin)
 * and the vector queue, verifies that every M-block is covered exactly once by every column tile of
 * every row-space phase, lets the pairs and `vec_workers` vector workers run -- each blocking on the
 * dependent counters of its current item -- and verifies that every counter ends at its threshold.
 * Returns 0, or a positive code naming the violated property (10 = malformed item, 13 = coverage,
 * 20 = deadlock, 30 = counter off its threshold).  stats[4] (may be NULL) = {matrix items, vector
 * tasks, scheduler rounds, stalled polls}.  Needs no GPU. */
int moe_debug_simulate_schedule(const int32_t* counts, int32_t Ep, int32_t T, int32_t k, int32_t n_shared,
                                int32_t d, int32_t F, int32_t is_bwd, int32_t pairs, int32_t vec_workers,
                                int64_t* stats);

/* Per-tile trace of the context's last persistent launch (contexts created with MOE_FLAG_TRACE).
 * Synchronises the stream of the last call, copies up to max_records records to `records` (host) and
 * sets *n_written to the number of records the launch produced (records beyond the buffer's 262144
 * are dropped but counted).  A record covers one interval of one role:
 *   role 0 = token loader of a matrix item (t0 = before its dependent event, dep_ns = time until it
 *            was met, t1 = last load issued), 1 = MMA issuer (first operands present .. last MMA
 *            issued), 2 = epilogue warp 0 of a CTA (accumulator ready .. trigger event signalled),
 *            3 = vector task (phase = 0 gather, 2 routing-weight gradient, 3 combine);
 *   phase  = operator index inside the pass (forward: 0 gate+up, 1 down; backward: 0 act_grad,
 *            1 w2_grad, 2 gate_grad, 3 w1_grad);  item = index in the phase's item list (or task). */
typedef struct {
  uint64_t t0_ns, t1_ns;   /* globaltimer */
  uint8_t role, phase;
  uint16_t pad;
  int32_t item;
  uint32_t cta;
  uint32_t dep_ns;
} moe_trace_record;
int moe_debug_trace(moe_ctx* ctx, moe_trace_record* records, size_t max_records, size_t* n_written);

#ifdef __cplusplus
}
#endif
#endif /* MOE_B200_DEBUG_H */
